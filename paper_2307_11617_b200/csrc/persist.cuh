// Persistent multi-round kernel for problems whose whole state sits in L2.
//
// With a few kilobytes to a few megabytes of state a round is three short dependent phases
// (mix | per-row scalars of the gradient | per-coordinate gradient + tracking) and the run is
// bound by launch and drain latency, not by bandwidth.  This kernel runs a whole span of rounds
// in ONE cooperative launch: CTAs pick work items of the current phase round-robin and meet at
// a grid barrier between phases.  The phases call the same device functions as the
// one-kernel-per-phase path, so the results are bit-identical.
//
// Grid barrier: one monotone counter in global memory; CTA leaders add 1 and spin until it
// reaches (number of barriers so far) x (number of CTAs).  Every spin is bounded in time: when
// it runs out (or another CTA has already given up) the CTA records a code in the status word
// and returns; the host reports RFAST_ETIMEOUT.  The launch is cooperative, so all CTAs are
// co-resident and the barrier cannot starve.  State written by other CTAs earlier in the same
// launch is read with L2 (cg) loads.
#pragma once

#include "kernels.cuh"

namespace rfast {

struct PersistArgs {
    RoundArgs a;                 // a.ev = descriptors of ALL events of the schedule
    GradArgs  g;                 // g.ev = same
    const int*   act_ptr;        // device [K+1]
    const float* alpha_round;    // device [K] or null (constant a.alpha)
    int r0, r1;
    const float* feat;  const float* target;  const int* label;
    float* scratch;              // residuals [events in round][B] / logits [events in round][B][C]
    int use_all;                 // least squares: the whole shard is the batch
    unsigned int* bar;           // barrier counter, zero at launch
    int* status;                 // 0, or kPersistTimeout once a wait ran out
};

constexpr int kPersistTimeout = 9;
constexpr unsigned long long kBarrierLimitNs = 2000000000ull;

// false: give up (status is set)
__device__ __forceinline__ bool grid_barrier(unsigned int* bar, unsigned int& target, int* status) {
    __syncthreads();
    int ok = 1;
    if (threadIdx.x == 0) {
        target += gridDim.x;
        __threadfence();                                   // publish this CTA's writes
        atomicAdd(bar, 1u);
        unsigned long long t0, now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        while (true) {
            unsigned int seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(bar) : "memory");
            if (seen >= target) break;
            int st;
            asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(st) : "l"(status) : "memory");
            if (st != 0) { ok = 0; break; }
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (now - t0 > kBarrierLimitNs) { atomicExch(status, kPersistTimeout); ok = 0; break; }
        }
        __threadfence();                                   // and see everybody else's
    }
    return __syncthreads_and(ok) != 0;
}

// MODEL: RFAST_MODEL_LEAST_SQUARES or RFAST_MODEL_SOFTMAX.  Launched cooperatively with
// gridDim.x <= number of co-resident CTAs; dynamic shared memory: B*C floats + B ints (softmax).
template <int MODEL, bool COMP>
__global__ void __launch_bounds__(kThreads)
k_persist_rounds(PersistArgs P) {
    extern __shared__ float sm[];
    RoundArgs a = P.a;
    GradArgs g = P.g;
    const int tiles = (a.n4 + kThreads - 1) / kThreads;
    unsigned int target = 0;
    for (int r = P.r0; r < P.r1; ++r) {
        const int ev0 = P.act_ptr[r], nev = P.act_ptr[r + 1] - ev0;
        if (nev == 0) continue;                              // the same decision in every CTA
        if (P.alpha_round) a.alpha = P.alpha_round[r];
        // ---- phase 1: S1 + S2a ----------------------------------------------------------------
        for (int item = blockIdx.x; item < nev * tiles; item += gridDim.x) {
            const EvDesc e = a.ev[ev0 + item / tiles];
            mix_tile<1, false, false, true>(a, e, item % tiles, nullptr, nullptr, 0, 0.f);
        }
        if (!grid_barrier(P.bar, target, P.status)) return;
        // ---- phase 2: per-row scalars of the sample gradient --------------------------------------
        if (MODEL == RFAST_MODEL_LEAST_SQUARES) {
            const int groups = (g.B + 7) / 8;
            for (int item = blockIdx.x; item < nev * groups; item += gridDim.x) {
                const int el = item / groups, k = (item % groups) * 8 + (threadIdx.x >> 5);
                if (k < g.B)
                    ls_residual_row<true>(g, a.ev[ev0 + el], el, k, threadIdx.x & 31, P.feat, P.target, P.scratch, P.use_all);
            }
        } else {
            for (int item = blockIdx.x; item < nev * g.B; item += gridDim.x) {
                const int el = item / g.B;
                softmax_logits_row<true>(g, a.ev[ev0 + el], el, item % g.B, P.feat, P.scratch);
            }
        }
        if (!grid_barrier(P.bar, target, P.status)) return;
        // ---- phase 3: gradient per coordinate, then S2b + S2c on the same coordinates ---------------
        for (int item = blockIdx.x; item < nev * tiles; item += gridDim.x) {
            const int el = item / tiles, tile = item % tiles;
            const EvDesc e = a.ev[ev0 + el];
            float* delta = sm;
            int* rowid = reinterpret_cast<int*>(sm + g.B * g.C);
            if (MODEL == RFAST_MODEL_SOFTMAX) {
                __syncthreads();                             // the previous item's readers are done
                softmax_delta_block<true>(g, e, el, P.label, P.scratch, delta, rowid);
            }
            const int i4 = tile * kThreads + threadIdx.x;
            const int64_t row = (int64_t)e.node * a.stride;
            float4 gnv[1], gov[1], zh[1];
            gnv[0] = gov[0] = zh[0] = make_float4(0, 0, 0, 0);
            if (i4 < a.n4) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t q = (int64_t)i4 * 4 + j;
                    float v = 0.f;
                    if (q < g.p)
                        v = MODEL == RFAST_MODEL_SOFTMAX ? softmax_grad_coord<true>(g, e, q, P.feat, delta, rowid)
                                                         : ls_grad_coord<true>(g, e, el, (int)q, P.feat, P.scratch, P.use_all);
                    comp(gnv[0], j) = v;
                }
                reinterpret_cast<float4*>(g.gbuf + (int64_t)(e.g_par ^ 1) * g.gplane + row)[i4] = gnv[0];
                zh[0] = ld_sel<true>(a.z + row, i4);
                gov[0] = ld_sel<true>(g.gbuf + (int64_t)e.g_par * g.gplane + row, i4);
            }
            track_and_push<1, COMP, true>(a, e, i4, a.z + row, zh, gnv, gov);
        }
        if (!grid_barrier(P.bar, target, P.status)) return;
    }
}

}  // namespace rfast
