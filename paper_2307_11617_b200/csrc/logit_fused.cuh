// Sparse-logistic activation in ONE pass over HBM: a thread-block cluster per activation.
//
// The sample gradient needs the whole freshly mixed x (sparse dot products a_k . x) before the
// tracking update can run, which is why the plain path is three kernels and reads x and z
// twice.  Here the CTAs of a cluster split the coordinates of one activation among them and
// each keeps its slice of the new x and of z in shared memory (p = 100k in a cluster of eight:
// 12.5k coordinates, 2 x 50 KB per CTA, two CTAs of different activations per SM):
//   A  the slices of x and z come in by two bulk asynchronous copies straight into shared
//      memory while the threads fetch the first in-neighbour's v; then S1 + S2a: v out (if a
//      packet leaves), x out, the new x kept on chip
//   B  partial dot products of the sampled rows over the slice, out of shared memory, one warp
//      per row; the entries read on the way are kept in shared memory (as many as fit); the
//      cluster's partial sums are exchanged through distributed shared memory and added in CTA
//      order (the same bits on every run); coef_k = -y_k / (1 + exp(y_k s_k)) / B
//   C  the slice of the gradient in place: l2 x, then row after row (the oracle's order) the
//      sampled rows' entries added in, all threads on one row at a time: columns are distinct
//      inside a row, so nothing collides and the sum is the same on every run
//   D  S2b + S2c on the slice: the remembered gradient, the news rows and the running sums
//      stream through once (requested into L2 while B and C leave the memory system idle);
//      g, z and the running sums go out
// so every vector is read and written exactly once per activation: the method's own byte count.
// Waits: the hardware cluster barrier, and one mbarrier for the bulk copies whose wait is
// bounded in time (on expiry the CTA records a code in the status word and goes on without
// computing, so that its peers are never left waiting at a cluster barrier).
#pragma once

#include <cooperative_groups.h>

#include "kernels.cuh"

namespace rfast {

constexpr int kFusedMaxBatch = 64;                         // sampled rows per activation this kernel takes
constexpr int kFusedTimeout = 12;                          // status code: the bulk copies did not land in time
constexpr int kFusedPerThread = 8;                         // float4 of a slice per thread, at most

struct LogitFusedArgs {
    RoundArgs a;                       // a.ev = descriptors of this round's events
    GradArgs  g;
    const int64_t* range_ptr;          // [shard rows][nranges + 1] first entry of a row in each 512-coordinate range
    int nranges;
    const int* sp_col;  const float* sp_val;  const int* label;
    int ranges_per_cta;                // R: a CTA owns ranges [rank R, (rank + 1) R)
    int stash_cap;                     // entries of the sampled rows a CTA can keep in shared memory
    int* status;                       // 0, or kFusedTimeout
    unsigned long long limit_ns;       // bound of the wait for the bulk copies
    unsigned int phantom_bytes;        // bytes the mbarrier expects beyond what is copied (0 in normal use; a
                                       // host-side failure-injection hook: nobody delivers them, so the bounded
                                       // wait runs out and the timeout path is exercised)
};

__device__ __forceinline__ uint32_t fused_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// false when the limit ran out
__device__ __forceinline__ bool fused_mbar_wait(uint64_t* bar, uint32_t parity, unsigned long long limit_ns) {
    const uint32_t addr = fused_smem_u32(bar);
    unsigned long long t0 = 0, now;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (it == 0) t0 = now;
        else if (now - t0 > limit_ns) return false;
    }
}

// grid = (cluster size, events of the round), cluster = (cluster size, 1, 1), kFusedThreads threads
// (a slice has at most kFusedPerThread float4 per thread); dynamic shared memory: 2 * R * 512
// floats (x slice, z slice) + stash_cap * 6 bytes
template <bool COMP, int kFusedThreads>
__global__ void __launch_bounds__(kFusedThreads, 1024 / kFusedThreads)
k_logit_fused(LogitFusedArgs P) {
    namespace cg = cooperative_groups;
    extern __shared__ __align__(128) float fsm[];
    __shared__ float s_part[kFusedMaxBatch], s_coef[kFusedMaxBatch];   // partial dot products, coefficients
    __shared__ long long s_base[kFusedMaxBatch];                       // first entry of sampled row k in the slice
    __shared__ int s_cnt[kFusedMaxBatch], s_pos[kFusedMaxBatch + 1];   // its entries in the slice; their place in the stash
    __shared__ __align__(8) uint64_t s_bar;
    __shared__ int s_ok;
    cg::cluster_group cluster = cg::this_cluster();
    const RoundArgs& a = P.a;
    const GradArgs& g = P.g;
    const int rank = (int)blockIdx.x, csize = (int)gridDim.x;
    const EvDesc e = a.ev[blockIdx.y];
    const int span = P.ranges_per_cta * kLogitRange;       // coordinates of a slice
    float* xs = fsm;                                        // [span] x, then the new x, then the gradient
    float* zs = fsm + span;                                 // [span] z
    float* stash_val = fsm + 2 * span;                      // [stash_cap]
    unsigned short* stash_col = reinterpret_cast<unsigned short*>(stash_val + P.stash_cap);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rg0 = min(rank * P.ranges_per_cta, P.nranges);
    const int rg1 = min(P.nranges, rg0 + P.ranges_per_cta);
    const int lo4 = rg0 * (kLogitRange / 4);                // first float4 of the slice
    const int hi4 = max(lo4, min(a.n4, rg1 * (kLogitRange / 4)));   // a CTA beyond the vector has an empty slice
    const int c0 = rg0 * kLogitRange;
    const int64_t row = (int64_t)e.node * a.stride;
    float* xr = a.x + row;
    float* zr = a.z + row;

    // ---- A: x and z slices by bulk copy into shared memory
    const uint32_t slice_bytes = (uint32_t)(hi4 - lo4) * 16u;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(fused_smem_u32(&s_bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s_ok = 1;
        if (slice_bytes) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(fused_smem_u32(&s_bar)), "r"(2u * slice_bytes + P.phantom_bytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(fused_smem_u32(xs)), "l"(xr + (int64_t)lo4 * 4), "r"(slice_bytes), "r"(fused_smem_u32(&s_bar)) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(fused_smem_u32(zs)), "l"(zr + (int64_t)lo4 * 4), "r"(slice_bytes), "r"(fused_smem_u32(&s_bar)) : "memory");
        }
    }
    // the first in-neighbour's v, all of this thread's float4 in flight together
    float4 nb[kFusedPerThread];
    const bool has_nb = e.mix_cnt > 0;
    {
        const float* nr = a.vbuf + (int64_t)(has_nb ? a.mix_slot[e.mix_beg] : 0) * a.stride;
#pragma unroll
        for (int u = 0; u < kFusedPerThread; ++u) {
            const int i4 = lo4 + u * kFusedThreads + (int)threadIdx.x;
            nb[u] = make_float4(0, 0, 0, 0);
            if (has_nb && i4 < hi4) nb[u] = ld_stream(nr, i4);
        }
    }
    // where the sampled rows' entries of this slice are: batch index -> shard row -> range offsets
    if (threadIdx.x < g.B) {
        const int k = threadIdx.x;
        const int rrow = g.batch_idx[(int64_t)e.sample * g.B + k];
        const int64_t* rp = P.range_ptr + ((int64_t)e.node * g.rows + rrow) * (P.nranges + 1);
        const int64_t qa = rp[rg0], qb = rp[rg1];
        s_base[k] = qa;
        s_cnt[k] = (int)(qb - qa);
        for (int64_t q = qa; q < qb; q += 32) { prefetch_l2(P.sp_col + q); prefetch_l2(P.sp_val + q); }
    }
    __syncthreads();                                        // the barrier is initialised, the row table is there
    if (threadIdx.x == 0) {
        int pos = 0;
        for (int k = 0; k < g.B; ++k) { s_pos[k] = pos; pos += s_cnt[k]; }
        s_pos[g.B] = pos;
        if (slice_bytes && !fused_mbar_wait(&s_bar, 0, P.limit_ns)) { atomicExch(P.status, kFusedTimeout); s_ok = 0; }
    }
    __syncthreads();
    const bool ok = s_ok != 0;                              // false: go through the barriers, compute nothing
    if (ok) {                                               // S1 + S2a
        float* vr = e.v_out >= 0 ? a.vbuf + (int64_t)e.v_out * a.stride : nullptr;
        const float w0 = has_nb ? a.mix_w[e.mix_beg] : 0.f;
#pragma unroll
        for (int u = 0; u < kFusedPerThread; ++u) {
            const int i4 = lo4 + u * kFusedThreads + (int)threadIdx.x;
            if (i4 < hi4) {
                const float4 xv = reinterpret_cast<const float4*>(xs)[i4 - lo4];
                const float4 zv = reinterpret_cast<const float4*>(zs)[i4 - lo4];
                const float4 v = f4_axpy(-a.alpha, zv, xv);                        // S1
                float4 acc = f4_scale(e.w_self, v);                                  // S2a, own term first
                if (vr) st_stream(vr, i4, v);
                if (has_nb) acc = f4_axpy(w0, nb[u], acc);
                for (int m = 1; m < e.mix_cnt; ++m)                                  // further in-neighbours, ascending
                    acc = f4_axpy(a.mix_w[e.mix_beg + m], ld_stream(a.vbuf + (int64_t)a.mix_slot[e.mix_beg + m] * a.stride, i4), acc);
                st_stream(xr, i4, acc);
                reinterpret_cast<float4*>(xs)[i4 - lo4] = acc;
            }
        }
    }
    // the operands of part D are requested into L2 now, so that they arrive while parts B and C
    // leave the memory system idle: one request per 128-byte line
    const float* gold = g.gbuf + (int64_t)e.g_par * g.gplane + row;
    if (ok && (lane & 7) == 0) {
        for (int b0 = lo4 + (int)threadIdx.x; b0 < hi4; b0 += kFusedThreads) {
            const int64_t off = (int64_t)b0 * 4;
            prefetch_l2(gold + off);
            for (int m = 0; m < e.news_cnt; ++m) {
                prefetch_l2(a.rbuf + (int64_t)a.news_new[e.news_beg + m] * a.stride + off);
                const int prev = a.news_prev[e.news_beg + m];
                if (prev >= 0) prefetch_l2(a.rbuf + (int64_t)prev * a.stride + off);
            }
            for (int m = 0; m < e.out_cnt; ++m) {
                const int cur = a.out_cur[e.out_beg + m];
                if (cur >= 0) prefetch_l2(a.rbuf + (int64_t)cur * a.stride + off);
            }
        }
    }
    __syncthreads();

    // ---- B: partial dot products over the slice, one warp per sampled row; entries kept
    for (int k = warp; k < g.B; k += kFusedThreads / 32) {
        float s = 0.f;
        if (ok) {
            const long long qa = s_base[k];
            const int cnt = s_cnt[k], pos = s_pos[k];
            for (int t = lane; t < cnt; t += 32) {
                const int col = P.sp_col[qa + t] - c0;
                const float val = P.sp_val[qa + t];
                s = fmaf(val, xs[col], s);
                if (pos + t < P.stash_cap) { stash_val[pos + t] = val; stash_col[pos + t] = (unsigned short)col; }
            }
        }
        s = warp_sum(s);
        if (lane == 0) s_part[k] = s;
    }
    cluster.sync();                                         // every CTA's partial sums are in place
    for (int k = threadIdx.x; k < g.B; k += kFusedThreads) {
        float s = 0.f;
        for (int c = 0; c < csize; ++c) s += cluster.map_shared_rank(s_part, c)[k];       // CTA order
        const int rrow = g.batch_idx[(int64_t)e.sample * g.B + k];
        const float y = (float)P.label[(int64_t)e.node * g.rows + rrow];
        s_coef[k] = -y / (1.f + expf(y * s)) / (float)g.B;
    }
    cluster.barrier_arrive();                               // done with the peers' shared memory (waited for at the end)

    // ---- C: the slice of the new gradient, in place: l2 x, then the sampled rows in batch order
    if (ok) {
        for (int i = threadIdx.x; i < (hi4 - lo4); i += kFusedThreads) {
            const float4 v = reinterpret_cast<float4*>(xs)[i];
            reinterpret_cast<float4*>(xs)[i] = f4_scale(g.l2, v);
        }
        __syncthreads();
        for (int k = 0; k < g.B; ++k) {
            const float ck = s_coef[k];
            const long long qa = s_base[k];
            const int cnt = s_cnt[k], pos = s_pos[k];
            for (int t = threadIdx.x; t < cnt; t += kFusedThreads) {
                const bool kept = pos + t < P.stash_cap;      // what did not fit is read again
                const int col = kept ? (int)stash_col[pos + t] : P.sp_col[qa + t] - c0;
                const float val = kept ? stash_val[pos + t] : P.sp_val[qa + t];
                xs[col] += ck * val;                         // columns are distinct inside a row
            }
            __syncthreads();
        }
    }

    // ---- D: S2b + S2c on the slice
    float* gnew = g.gbuf + (int64_t)(e.g_par ^ 1) * g.gplane + row;
    if (ok) {
        RoundArgs as = a;
        as.n4 = hi4;                                        // the slice's end bounds every access
        const int grp = threadIdx.x / kThreads, l256 = threadIdx.x % kThreads;
        for (int c = lo4 + grp * 2 * kThreads; c < hi4; c += (kFusedThreads / kThreads) * 2 * kThreads) {
            const int base = c + l256;
            float4 zh[2], gnv[2], gov[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int i4 = base + u * kThreads;
                zh[u] = gnv[u] = gov[u] = make_float4(0, 0, 0, 0);
                if (i4 < hi4) {
                    gnv[u] = reinterpret_cast<const float4*>(xs)[i4 - lo4];
                    zh[u] = reinterpret_cast<const float4*>(zs)[i4 - lo4];
                    gov[u] = ld_stream(gold, i4);
                    st_stream(gnew, i4, gnv[u]);
                }
            }
            track_and_push<2, COMP>(as, e, base, zr, zh, gnv, gov);
        }
    }
    cluster.barrier_wait();                                 // no peer reads this CTA's shared memory any more
    // after a timed-out wait the copies may still be on their way: they must land (or the second
    // limit run out) before the shared memory goes away
    if (!ok && threadIdx.x == 0 && slice_bytes) fused_mbar_wait(&s_bar, 0, P.limit_ns);
}

}  // namespace rfast
