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
// reaches (number of barriers so far) x (number of CTAs).  Every spin is bounded in time (2 s by
// default, RFAST_OPT_WAIT_LIMIT_MS): when
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
    int xs_off;                  // offset (floats) of the x staging area in dynamic shared memory
    int rows_per_item;           // softmax: sampled rows handled per work item of phase 2
    unsigned int phantom;        // arrivals the barrier expects beyond the launched CTAs (0 in normal
                                 // use; a host-side failure-injection hook: nobody makes them, so the
                                 // bounded wait runs out and the kernel returns with the status set)
    unsigned long long limit_ns; // bound of every barrier wait
    unsigned int* bar;           // barrier counter, zero at launch
    int* status;                 // 0, or kPersistTimeout once a wait ran out
};

constexpr int kPersistTimeout = 9;

// false: give up (status is set)
__device__ __forceinline__ bool grid_barrier(unsigned int* bar, unsigned int& target, int* status,
                                             unsigned int arrivals, unsigned long long limit_ns) {
    __syncthreads();
    int ok = 1;
    if (threadIdx.x == 0) {
        target += arrivals;
        __threadfence();                                   // publish this CTA's writes
        atomicAdd(bar, 1u);
        unsigned long long t0 = 0, now;
        for (unsigned int spins = 0;; ++spins) {
            unsigned int seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(bar) : "memory");
            if (seen >= target) break;
            if ((spins & 255u) == 255u) {                    // the clock and the status word are slow to read
                int st;
                asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(st) : "l"(status) : "memory");
                if (st != 0) { ok = 0; break; }
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
                if (t0 == 0) t0 = now;
                else if (now - t0 > limit_ns) { atomicExch(status, kPersistTimeout); ok = 0; break; }
            }
        }
        __threadfence();                                   // and see everybody else's
    }
    return __syncthreads_and(ok) != 0;
}

// Phase 3 of a round for one tile of kThreads float4: the sample gradient of the tile's
// coordinates from the per-row scalars of phase 2 (softmax: delta in shared memory; least
// squares: the residuals, staged in shared memory), stored as the new remembered gradient, then
// S2b + S2c on the same coordinates.  sm: B*C floats + B ints (softmax) or B floats.
template <int MODEL, bool COMP, bool CG>
__device__ __forceinline__ void grad_track_tile(const RoundArgs& a, const GradArgs& g, const EvDesc& e, int el, int tile,
                                                const float* feat, const int* label, const float* scratch,
                                                int use_all, float* sm) {
    float* delta = sm;
    int* rowid = reinterpret_cast<int*>(sm + g.B * g.C);
    __syncthreads();                                         // the previous item's readers are done
    if (MODEL == RFAST_MODEL_SOFTMAX) {
        softmax_delta_block<CG>(g, e, el, label, scratch, delta, rowid);
    } else {
        for (int k = threadIdx.x; k < g.B; k += kThreads) delta[k] = ld_sel1<CG>(scratch + (int64_t)el * g.B + k);
        __syncthreads();
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
            if (q < g.p) {
                if (MODEL == RFAST_MODEL_SOFTMAX) {
                    v = softmax_grad_coord<CG>(g, e, q, feat, delta, rowid);
                } else {                                     // same order of operations as ls_grad_coord
                    const float* abase = feat + (int64_t)e.node * g.rows * g.F;
                    float s = 0.f;
                    for (int k = 0; k < g.B; ++k) {
                        const int rrow = use_all ? k : g.batch_idx[(int64_t)e.sample * g.B + k];
                        s = fmaf(abase[(int64_t)rrow * g.F + q], delta[k], s);
                    }
                    v = s / (float)g.B + g.l2 * ld_sel1<CG>(g.x + row + q);
                }
            }
            comp(gnv[0], j) = v;
        }
        reinterpret_cast<float4*>(g.gbuf + (int64_t)(e.g_par ^ 1) * g.gplane + row)[i4] = gnv[0];
        zh[0] = ld_sel<CG>(a.z + row, i4);
        gov[0] = ld_sel<CG>(g.gbuf + (int64_t)e.g_par * g.gplane + row, i4);
    }
    track_and_push<1, COMP, CG>(a, e, i4, a.z + row, zh, gnv, gov);
}

// MODEL: RFAST_MODEL_LEAST_SQUARES or RFAST_MODEL_SOFTMAX.  Launched cooperatively with
// gridDim.x <= number of co-resident CTAs; dynamic shared memory: B*C floats + B ints (softmax) or
// B floats (least squares: the residuals of the item's event), then stride floats for x.
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
            mix_tile<1, false, true>(a, e, item % tiles, nullptr);
        }
        if (!grid_barrier(P.bar, target, P.status, gridDim.x + P.phantom, P.limit_ns)) return;
        // ---- phase 2: per-row scalars of the sample gradient --------------------------------------
        // The new x of the item's node is first copied into shared memory with wide L2 loads that
        // are all in flight together; the dot products then run out of shared memory.  (Reading x
        // element by element through L2 inside the reduction loops would serialise on L2 latency.)
        {
            float* xs = sm + P.xs_off;                       // [stride] floats
            const int per_ev = MODEL == RFAST_MODEL_LEAST_SQUARES ? (g.B + 7) / 8 : (g.B + P.rows_per_item - 1) / P.rows_per_item;
            int have = -1;                                   // event whose x is in shared memory
            for (int item = blockIdx.x; item < nev * per_ev; item += gridDim.x) {
                const int el = item / per_ev, sub = item % per_ev;
                const EvDesc e = a.ev[ev0 + el];
                if (have != el) {
                    __syncthreads();
                    const float* xr = g.x + (int64_t)e.node * g.stride;
                    for (int i4 = threadIdx.x; i4 < a.n4; i4 += kThreads)
                        reinterpret_cast<float4*>(xs)[i4] = __ldcg(reinterpret_cast<const float4*>(xr) + i4);
                    __syncthreads();
                    have = el;
                }
                if (MODEL == RFAST_MODEL_LEAST_SQUARES) {
                    const int k = sub * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
                    if (k < g.B) {
                        const int rrow = P.use_all ? k : g.batch_idx[(int64_t)e.sample * g.B + k];
                        const float* arow = P.feat + ((int64_t)e.node * g.rows + rrow) * g.F;
                        float s = 0.f;
                        for (int c = lane; c < g.F; c += 32) s = fmaf(arow[c], xs[c], s);
                        s = warp_sum(s);
                        if (lane == 0) P.scratch[(int64_t)el * g.B + k] = s - P.target[(int64_t)e.node * g.rows + rrow];
                    }
                } else {
                    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
                    for (int k = sub * P.rows_per_item; k < min(g.B, (sub + 1) * P.rows_per_item); ++k) {
                        const int rrow = g.batch_idx[(int64_t)e.sample * g.B + k];
                        const float* arow = P.feat + ((int64_t)e.node * g.rows + rrow) * g.F;
                        for (int c = warp; c < g.C; c += 8) {
                            const float* w = xs + (int64_t)c * g.F;
                            float s = 0.f;
                            if ((g.F & 3) == 0) {            // same order of operations as softmax_logits_row
                                for (int f4 = lane; f4 < g.F / 4; f4 += 32) {
                                    const float4 av = reinterpret_cast<const float4*>(arow)[f4];
                                    const float4 wv = reinterpret_cast<const float4*>(w)[f4];
                                    s = fmaf(av.w, wv.w, fmaf(av.z, wv.z, fmaf(av.y, wv.y, fmaf(av.x, wv.x, s))));
                                }
                            } else {
                                for (int f = lane; f < g.F; f += 32) s = fmaf(arow[f], w[f], s);
                            }
                            s = warp_sum(s);
                            if (lane == 0) P.scratch[((int64_t)el * g.B + k) * g.C + c] = s + xs[(int64_t)g.C * g.F + c];
                        }
                    }
                }
            }
        }
        if (!grid_barrier(P.bar, target, P.status, gridDim.x + P.phantom, P.limit_ns)) return;
        // ---- phase 3: gradient per coordinate, then S2b + S2c on the same coordinates ---------------
        for (int item = blockIdx.x; item < nev * tiles; item += gridDim.x) {
            const int el = item / tiles;
            grad_track_tile<MODEL, COMP, true>(a, g, a.ev[ev0 + el], el, item % tiles, P.feat, P.label, P.scratch,
                                               P.use_all, sm);
        }
        if (!grid_barrier(P.bar, target, P.status, gridDim.x + P.phantom, P.limit_ns)) return;
    }
}

}  // namespace rfast
