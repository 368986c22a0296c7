// Device kernels of the R-FAST activation step (sm_100a).
//
// State layout: every per-node / per-version vector is one row of `stride` floats
// (stride = p rounded up to 32 floats, so rows start on 128-byte boundaries and can be
// walked with 128-bit accesses); the padding stays zero.  All passes over coordinates are
// pure streaming: each byte is touched once per activation, so loads and stores carry the
// streaming (evict-first) hint.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rfast_internal.h"

namespace rfast {

struct RoundArgs {
    const EvDesc* ev;            // events of this round
    const int*    mix_slot;  const float* mix_w;
    const int*    news_new;  const int*   news_prev;
    const int*    out_cur;   const int*   out_new;   const float* out_a;
    float* x;  float* z;         // [n][stride]
    float* zc;                   // [n][stride] low-order part of the tracker (compensated mode), else null
    float* vbuf;                 // [v rows][stride]   published v versions
    float* rbuf;                 // [rho rows][stride] running-sum versions
    int64_t rlo_off;             // > 0: the running sums are two floats; low parts live this many
                                 // floats after the high parts (compensation level 2)
    int64_t stride;              // floats per row
    int     n4;                  // float4 per row (stride / 4)
    float   alpha;
};

// one request brings the 128-byte line into L2; issued by one lane in eight (8 x 16 bytes)
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ float4 ld_stream(const float* row, int i4) {
    return __ldcs(reinterpret_cast<const float4*>(row) + i4);
}
// CG = true: go to L2 (ld.global.cg).  Used inside the persistent multi-round kernel, where rows
// written by other CTAs earlier in the same launch must never be served from a stale L1 line.
template <bool CG>
__device__ __forceinline__ float4 ld_sel(const float* row, int i4) {
    return CG ? __ldcg(reinterpret_cast<const float4*>(row) + i4) : __ldcs(reinterpret_cast<const float4*>(row) + i4);
}
template <bool CG>
__device__ __forceinline__ float ld_sel1(const float* p) { return CG ? __ldcg(p) : *p; }
__device__ __forceinline__ void st_stream(float* row, int i4, float4 v) {
    __stcs(reinterpret_cast<float4*>(row) + i4, v);
}
__device__ __forceinline__ float4 f4_axpy(float a, float4 x, float4 y) {   // a*x + y
    return make_float4(fmaf(a, x.x, y.x), fmaf(a, x.y, y.y), fmaf(a, x.z, y.z), fmaf(a, x.w, y.w));
}
__device__ __forceinline__ float4 f4_add(float4 a, float4 b) {
    return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
}
__device__ __forceinline__ float4 f4_sub(float4 a, float4 b) {
    return make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w);
}
__device__ __forceinline__ float4 f4_scale(float a, float4 x) {
    return make_float4(a * x.x, a * x.y, a * x.z, a * x.w);
}


// Error-free addition (Knuth): s + err == a + b exactly.
__device__ __forceinline__ void two_sum(float a, float b, float& s, float& err) {
    s = __fadd_rn(a, b);
    const float bb = __fsub_rn(s, a);
    err = __fadd_rn(__fsub_rn(a, __fsub_rn(s, bb)), __fsub_rn(b, bb));
}
__device__ __forceinline__ float& comp(float4& v, int c) { return reinterpret_cast<float*>(&v)[c]; }
__device__ __forceinline__ float comp(const float4& v, int c) { return reinterpret_cast<const float*>(&v)[c]; }

constexpr int kThreads = 256;


// ---------------------------------------------------------------------------------------------
// S2b + S2c on U float4 per thread, shared by the fused and the split kernels.
//   z^ = z + sum over in-edges with news (rho[tau'] - rho[tau_prev]) + g_new - g_old
//   z' = a_ii z^ ;  rho'_ji = rho_ji + a_ji z^  for every out-edge
// COMP = false: plain fp32, in the order written above.
// COMP = true: the tracker is carried as an unevaluated sum of two floats (z + zc) and every
// rounding error of the mass-moving operations (the additions into z^, the products with the
// weights, the additions into the running sums) is captured with error-free transformations
// and kept in the node's own low-order part, so that the tracked mass of Lemma 3 is conserved
// to second order instead of drifting with every fp32 rounding.  The running sums stay fp32,
// unless a.rlo_off > 0: then they are two floats as well, which removes the last fp32-sized
// quantity from the tracking path (a receiver otherwise sees its in-neighbours' mass at the
// resolution of an fp32 sum that keeps growing).
// ---------------------------------------------------------------------------------------------
template <int U, bool COMP, bool CG = false>
__device__ __forceinline__ void track_and_push(const RoundArgs& a, const EvDesc& e, int base, float* zr,
                                               const float4 (&zv)[U], const float4 (&gn)[U],
                                               const float4 (&go)[U]) {
    if (!COMP) {
        float4 zh[U];
#pragma unroll
        for (int u = 0; u < U; ++u) zh[u] = zv[u];
        for (int m = 0; m < e.news_cnt; ++m) {                          // ascending sender id
            const float* nr = a.rbuf + (int64_t)a.news_new[e.news_beg + m] * a.stride;
            const int prev = a.news_prev[e.news_beg + m];
            const float* pr = a.rbuf + (int64_t)(prev < 0 ? 0 : prev) * a.stride;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i4 = base + u * kThreads;
                if (i4 < a.n4) {
                    float4 dl = ld_sel<CG>(nr, i4);
                    if (prev >= 0) dl = f4_sub(dl, ld_sel<CG>(pr, i4));
                    zh[u] = f4_add(zh[u], dl);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            zh[u] = f4_sub(f4_add(zh[u], gn[u]), go[u]);
            const int i4 = base + u * kThreads;
            if (i4 < a.n4) st_stream(zr, i4, f4_scale(e.a_self, zh[u]));   // S2c keep
        }
        for (int m = 0; m < e.out_cnt; ++m) {                           // S2c accumulate
            const int cur = a.out_cur[e.out_beg + m];
            const float* cr = a.rbuf + (int64_t)(cur < 0 ? 0 : cur) * a.stride;
            float* wr = a.rbuf + (int64_t)a.out_new[e.out_beg + m] * a.stride;
            const float aw = a.out_a[e.out_beg + m];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i4 = base + u * kThreads;
                if (i4 < a.n4) {
                    float4 r = f4_scale(aw, zh[u]);
                    if (cur >= 0) r = f4_add(ld_sel<CG>(cr, i4), r);
                    st_stream(wr, i4, r);
                }
            }
        }
    } else {
        float* cr_ = a.zc + (zr - a.z);
        float4 hi[U], lo[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i4 = base + u * kThreads;
            hi[u] = zv[u];
            lo[u] = make_float4(0, 0, 0, 0);
            if (i4 < a.n4) lo[u] = ld_sel<CG>(cr_, i4);
        }
        for (int m = 0; m < e.news_cnt; ++m) {
            const float* nr = a.rbuf + (int64_t)a.news_new[e.news_beg + m] * a.stride;
            const int prev = a.news_prev[e.news_beg + m];
            const float* pr = a.rbuf + (int64_t)(prev < 0 ? 0 : prev) * a.stride;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i4 = base + u * kThreads;
                if (i4 < a.n4) {
                    const float4 nv = ld_sel<CG>(nr, i4);
                    const float4 pv = prev >= 0 ? ld_sel<CG>(pr, i4) : make_float4(0, 0, 0, 0);
                    float4 nl = make_float4(0, 0, 0, 0), pl = nl;
                    if (a.rlo_off > 0) {
                        nl = ld_sel<CG>(nr + a.rlo_off, i4);
                        if (prev >= 0) pl = ld_sel<CG>(pr + a.rlo_off, i4);
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float d, de, s, se;
                        two_sum(comp(nv, c), -comp(pv, c), d, de);
                        two_sum(comp(hi[u], c), d, s, se);
                        comp(hi[u], c) = s;
                        comp(lo[u], c) += se + de + (comp(nl, c) - comp(pl, c));
                    }
                }
            }
        }
        float4 zh_hi[U], zh_lo[U], k_hi[U], k_lo[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float s, se, t, te;
                two_sum(comp(hi[u], c), comp(gn[u], c), s, se);
                two_sum(s, -comp(go[u], c), t, te);
                const float l = comp(lo[u], c) + (se + te);
                float zh, zl;
                two_sum(t, l, zh, zl);
                comp(zh_hi[u], c) = zh;
                comp(zh_lo[u], c) = zl;
                const float kh = __fmul_rn(e.a_self, zh);
                comp(k_hi[u], c) = kh;
                comp(k_lo[u], c) = __fmaf_rn(e.a_self, zh, -kh) + e.a_self * zl;
            }
        }
        for (int m = 0; m < e.out_cnt; ++m) {
            const int cur = a.out_cur[e.out_beg + m];
            const float* cr = a.rbuf + (int64_t)(cur < 0 ? 0 : cur) * a.stride;
            float* wr = a.rbuf + (int64_t)a.out_new[e.out_beg + m] * a.stride;
            const float aw = a.out_a[e.out_beg + m];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i4 = base + u * kThreads;
                if (i4 < a.n4) {
                    const float4 cv = cur >= 0 ? ld_sel<CG>(cr, i4) : make_float4(0, 0, 0, 0);
                    float4 r;
                    if (a.rlo_off > 0) {                     // two-float running sum: nothing is left over
                        const float4 cl = cur >= 0 ? ld_sel<CG>(cr + a.rlo_off, i4) : make_float4(0, 0, 0, 0);
                        float4 rl;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float inc = __fmul_rn(aw, comp(zh_hi[u], c));
                            const float ierr = __fmaf_rn(aw, comp(zh_hi[u], c), -inc) + aw * comp(zh_lo[u], c);
                            float s, se;
                            two_sum(comp(cv, c), inc, s, se);
                            two_sum(s, comp(cl, c) + se + ierr, comp(r, c), comp(rl, c));
                        }
                        st_stream(wr + a.rlo_off, i4, rl);
                    } else {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float inc = __fmul_rn(aw, comp(zh_hi[u], c));
                            const float ierr = __fmaf_rn(aw, comp(zh_hi[u], c), -inc) + aw * comp(zh_lo[u], c);
                            float s, se;
                            two_sum(comp(cv, c), inc, s, se);
                            comp(r, c) = s;
                            comp(k_lo[u], c) += se + ierr;   // what did not fit stays with the sender
                        }
                    }
                    st_stream(wr, i4, r);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i4 = base + u * kThreads;
            if (i4 < a.n4) {
                float4 zf, cf;
#pragma unroll
                for (int c = 0; c < 4; ++c) two_sum(comp(k_hi[u], c), comp(k_lo[u], c), comp(zf, c), comp(cf, c));
                st_stream(zr, i4, zf);
                st_stream(cr_, i4, cf);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Fused activation for the element-wise objective f_i(x) = 0.5 || d_i .* (x - b_i) ||^2:
// S1 v = x - alpha z;  S2a x' = w_ii v + sum_j w_ij v_j[tau];  g' = d^2 (x' - b), g = d^2 (x - b)
// (the remembered gradient is recomputed from the unchanged x instead of being stored);
// S2b z^ = z + sum_news (rho[tau'] - rho[tau_prev]) + g' - g;  S2c z' = a_ii z^, rho' = rho + a_ji z^.
// The buffer update S4 is a change of row id done by the host compiler (rho~ is the version
// last consumed, kept alive instead of copied).  One HBM pass per activation.
// grid = (tiles, events of the round)
// ---------------------------------------------------------------------------------------------
// (at most 42 registers per thread: six CTAs per SM keep enough loads in flight; measured +4 %
// over five, +9 % over the two-float4-per-thread variant at three)
template <int U, bool COMP>
__global__ void __launch_bounds__(kThreads, 6)
k_fused_quad(RoundArgs a, const float* __restrict__ qd, const float* __restrict__ qb) {
    const EvDesc e = a.ev[blockIdx.y];
    const int64_t row = (int64_t)e.node * a.stride;
    float* xr = a.x + row;
    float* zr = a.z + row;
    const float* dr = qd + row;
    const float* br = qb + row;
    const int base = blockIdx.x * (kThreads * U) + threadIdx.x;

    float4 xv[U], zv[U], dv[U], bv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int i4 = base + u * kThreads;
        xv[u] = zv[u] = dv[u] = bv[u] = make_float4(0, 0, 0, 0);
        if (i4 < a.n4) {
            xv[u] = ld_stream(xr, i4);
            zv[u] = ld_stream(zr, i4);
            dv[u] = ld_stream(dr, i4);
            bv[u] = ld_stream(br, i4);
        }
    }
    float4 acc[U], v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        v[u] = f4_axpy(-a.alpha, zv[u], xv[u]);                    // S1
        acc[u] = f4_scale(e.w_self, v[u]);                          // S2a, own term first
    }
    if (e.v_out >= 0) {
        float* vr = a.vbuf + (int64_t)e.v_out * a.stride;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i4 = base + u * kThreads;
            if (i4 < a.n4) st_stream(vr, i4, v[u]);
        }
    }
    for (int m = 0; m < e.mix_cnt; ++m) {                           // ascending sender id
        const float* nr = a.vbuf + (int64_t)a.mix_slot[e.mix_beg + m] * a.stride;
        const float w = a.mix_w[e.mix_beg + m];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i4 = base + u * kThreads;
            if (i4 < a.n4) acc[u] = f4_axpy(w, ld_stream(nr, i4), acc[u]);
        }
    }
    float4 gn[U], go[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int i4 = base + u * kThreads;
        if (i4 < a.n4) st_stream(xr, i4, acc[u]);
        const float4 d2 = make_float4(dv[u].x * dv[u].x, dv[u].y * dv[u].y, dv[u].z * dv[u].z, dv[u].w * dv[u].w);
        gn[u] = make_float4(d2.x * (acc[u].x - bv[u].x), d2.y * (acc[u].y - bv[u].y),
                            d2.z * (acc[u].z - bv[u].z), d2.w * (acc[u].w - bv[u].w));
        go[u] = make_float4(d2.x * (xv[u].x - bv[u].x), d2.y * (xv[u].y - bv[u].y),
                            d2.z * (xv[u].z - bv[u].z), d2.w * (xv[u].w - bv[u].w));
    }
    track_and_push<U, COMP>(a, e, base, zr, zv, gn, go);
}

// z_i^0 = grad f_i(x_i^0) for the element-wise objective.  grid = (tiles, n)
__global__ void __launch_bounds__(kThreads)
k_quad_grad(const float* __restrict__ x, const float* __restrict__ qd, const float* __restrict__ qb,
            float* __restrict__ out, int64_t stride, int n4) {
    const int64_t row = (int64_t)blockIdx.y * stride;
    const int i4 = blockIdx.x * kThreads + threadIdx.x;
    if (i4 >= n4) return;
    const float4 xv = ld_stream(x + row, i4), d = ld_stream(qd + row, i4), b = ld_stream(qb + row, i4);
    st_stream(out + row, i4, make_float4(d.x * d.x * (xv.x - b.x), d.y * d.y * (xv.y - b.y),
                                         d.z * d.z * (xv.z - b.z), d.w * d.w * (xv.w - b.w)));
}

// ---------------------------------------------------------------------------------------------
// S1 + S2a for objectives whose gradient needs the whole new x first.  Optionally leaves a
// bf16 copy of the new x (operand of the MLP's matrix products).  grid = (tiles, events)
// ---------------------------------------------------------------------------------------------
template <int U, bool BF16, bool CG>
__device__ __forceinline__ void mix_tile(const RoundArgs& a, const EvDesc& e, int tile, __nv_bfloat16* xb) {
    const int64_t row = (int64_t)e.node * a.stride;
    float* xr = a.x + row;
    const float* zr = a.z + row;
    const int base = tile * (kThreads * U) + threadIdx.x;
    float4 acc[U], v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int i4 = base + u * kThreads;
        float4 xv = make_float4(0, 0, 0, 0), zv = xv;
        if (i4 < a.n4) { xv = ld_sel<CG>(xr, i4); zv = ld_sel<CG>(zr, i4); }
        v[u] = f4_axpy(-a.alpha, zv, xv);
        acc[u] = f4_scale(e.w_self, v[u]);
    }
    if (e.v_out >= 0) {
        float* vr = a.vbuf + (int64_t)e.v_out * a.stride;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i4 = base + u * kThreads;
            if (i4 < a.n4) st_stream(vr, i4, v[u]);
        }
    }
    for (int m = 0; m < e.mix_cnt; ++m) {
        const float* nr = a.vbuf + (int64_t)a.mix_slot[e.mix_beg + m] * a.stride;
        const float w = a.mix_w[e.mix_beg + m];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i4 = base + u * kThreads;
            if (i4 < a.n4) acc[u] = f4_axpy(w, ld_sel<CG>(nr, i4), acc[u]);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int i4 = base + u * kThreads;
        if (i4 < a.n4) {
            // the gradient kernels re-read x soon: keep it cacheable
            reinterpret_cast<float4*>(xr)[i4] = acc[u];
            if (BF16) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(acc[u].x, acc[u].y);
                __nv_bfloat162 hi = __floats2bfloat162_rn(acc[u].z, acc[u].w);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&lo);
                pk.y = *reinterpret_cast<uint32_t*>(&hi);
                reinterpret_cast<uint2*>(xb + row)[i4] = pk;
            }
        }
    }
}

// PF: the state does not fit L2; the rows read behind an edge-list entry are requested into L2 first
template <int U, bool BF16, bool PF = false>
__global__ void __launch_bounds__(kThreads)
k_mix(RoundArgs a, __nv_bfloat16* __restrict__ xb) {
    const EvDesc e = a.ev[blockIdx.y];
    const int base = blockIdx.x * (kThreads * U) + threadIdx.x;
    if (PF && U == 1 && (threadIdx.x & 7) == 0 && base < a.n4)
        for (int m = 0; m < e.mix_cnt; ++m)
            prefetch_l2(a.vbuf + (int64_t)a.mix_slot[e.mix_beg + m] * a.stride + (int64_t)base * 4);
    mix_tile<U, BF16, false>(a, e, blockIdx.x, xb);
}

// ---------------------------------------------------------------------------------------------
// S2b + S2c (+ S4 by row id) with the gradients taken from the two gradient buffers:
// g_old = gbuf[par][node], g_new = gbuf[par^1][node].  grid = (tiles, events)
// ---------------------------------------------------------------------------------------------
template <int U, bool COMP, bool PF = false>
__global__ void __launch_bounds__(kThreads)
k_track(RoundArgs a, const float* __restrict__ gbuf, int64_t gplane) {
    const EvDesc e = a.ev[blockIdx.y];
    const int64_t row = (int64_t)e.node * a.stride;
    float* zr = a.z + row;
    const float* go = gbuf + (int64_t)e.g_par * gplane + row;
    const float* gn = gbuf + (int64_t)(e.g_par ^ 1) * gplane + row;
    const int base = blockIdx.x * (kThreads * U) + threadIdx.x;
    float4 zh[U], gnv[U], gov[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int i4 = base + u * kThreads;
        zh[u] = gnv[u] = gov[u] = make_float4(0, 0, 0, 0);
        if (i4 < a.n4) { zh[u] = ld_stream(zr, i4); gnv[u] = ld_stream(gn, i4); gov[u] = ld_stream(go, i4); }
    }
    // the news and running-sum rows are read behind the list entries that name them
    if (PF && U == 1 && (threadIdx.x & 7) == 0 && base < a.n4) {
        const int64_t off = (int64_t)base * 4;
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
    track_and_push<U, COMP>(a, e, base, zr, zh, gnv, gov);
}

// ---------------------------------------------------------------------------------------------
// Sample gradients.  Every kernel takes the round's events; x_i is the freshly mixed row and
// the result goes to gbuf[par^1][node].  Reductions run in a fixed order (run-to-run identical).
// ---------------------------------------------------------------------------------------------

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// The per-row and per-coordinate pieces below are shared by the one-kernel-per-phase path and
// by the persistent multi-round kernel, so that both produce the same bits.  ev_local is the
// event's index inside its round (the scratch arrays are laid out per round).

// Least squares, phase 1: residual r_k = a_k . x - y_k, one warp per sampled row.
template <bool CG>
__device__ __forceinline__ void ls_residual_row(const GradArgs& g, const EvDesc& e, int ev_local, int k, int lane,
                                                const float* feat, const float* target, float* res, int use_all) {
    const int rrow = use_all ? k : g.batch_idx[(int64_t)e.sample * g.B + k];
    const float* a = feat + ((int64_t)e.node * g.rows + rrow) * g.F;
    const float* x = g.x + (int64_t)e.node * g.stride;
    float s = 0.f;
    for (int c = lane; c < g.F; c += 32) s = fmaf(a[c], ld_sel1<CG>(x + c), s);
    s = warp_sum(s);
    if (lane == 0) res[(int64_t)ev_local * g.B + k] = s - target[(int64_t)e.node * g.rows + rrow];
}
// grid = (ceil(B / 8), events), 256 threads.  res: [events][B]
__global__ void __launch_bounds__(256)
k_ls_residual(GradArgs g, const float* __restrict__ feat, const float* __restrict__ target,
              float* __restrict__ res, int use_all) {
    const int k = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (k >= g.B) return;
    ls_residual_row<false>(g, g.ev[blockIdx.y], blockIdx.y, k, threadIdx.x & 31, feat, target, res, use_all);
}

// Least squares, phase 2: g_c = (1/B) sum_k a_k[c] r_k + l2 x_c.
template <bool CG>
__device__ __forceinline__ float ls_grad_coord(const GradArgs& g, const EvDesc& e, int ev_local, int c,
                                               const float* feat, const float* res, int use_all) {
    const float* abase = feat + (int64_t)e.node * g.rows * g.F;
    float s = 0.f;
    for (int k = 0; k < g.B; ++k) {
        const int rrow = use_all ? k : g.batch_idx[(int64_t)e.sample * g.B + k];
        s = fmaf(abase[(int64_t)rrow * g.F + c], ld_sel1<CG>(res + (int64_t)ev_local * g.B + k), s);
    }
    return s / (float)g.B + g.l2 * ld_sel1<CG>(g.x + (int64_t)e.node * g.stride + c);
}
// grid = (ceil(p/256), events)
__global__ void __launch_bounds__(256)
k_ls_grad(GradArgs g, const float* __restrict__ feat, const float* __restrict__ res, int use_all) {
    const EvDesc e = g.ev[blockIdx.y];
    const int c = blockIdx.x * 256 + threadIdx.x;
    if (c >= g.F) return;
    g.gbuf[(int64_t)(e.g_par ^ 1) * g.gplane + (int64_t)e.node * g.stride + c] =
        ls_grad_coord<false>(g, e, blockIdx.y, c, feat, res, use_all);
}

// Softmax regression, phase 1: logits[k][c] = W_c . a_k + bias_c for one sampled row k by one
// block, one warp per class (round-robin).  logit: [events][B][C]
template <bool CG>
__device__ __forceinline__ void softmax_logits_row(const GradArgs& g, const EvDesc& e, int ev_local, int k,
                                                   const float* feat, float* logit) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rrow = g.batch_idx[(int64_t)e.sample * g.B + k];
    const float* a = feat + ((int64_t)e.node * g.rows + rrow) * g.F;
    const float* x = g.x + (int64_t)e.node * g.stride;
    for (int c = warp; c < g.C; c += 8) {
        const float* w = x + (int64_t)c * g.F;
        float s = 0.f;
        if ((g.F & 3) == 0) {                                // rows are 16-byte aligned: 128-bit loads
            for (int f4 = lane; f4 < g.F / 4; f4 += 32) {
                const float4 av = reinterpret_cast<const float4*>(a)[f4];
                const float4 wv = CG ? __ldcg(reinterpret_cast<const float4*>(w) + f4)
                                     : reinterpret_cast<const float4*>(w)[f4];
                s = fmaf(av.w, wv.w, fmaf(av.z, wv.z, fmaf(av.y, wv.y, fmaf(av.x, wv.x, s))));
            }
        } else {
            for (int f = lane; f < g.F; f += 32) s = fmaf(a[f], ld_sel1<CG>(w + f), s);
        }
        s = warp_sum(s);
        if (lane == 0) logit[((int64_t)ev_local * g.B + k) * g.C + c] = s + ld_sel1<CG>(x + (int64_t)g.C * g.F + c);
    }
}
// grid = (B, events)
__global__ void __launch_bounds__(256)
k_softmax_logits(GradArgs g, const float* __restrict__ feat, float* __restrict__ logit) {
    softmax_logits_row<false>(g, g.ev[blockIdx.y], blockIdx.y, blockIdx.x, feat, logit);
}

// Softmax regression, phase 2: delta = (softmax(logits) - onehot) / B for all sampled rows of
// one event into shared memory (block-wide, ends with a barrier) ...
template <bool CG>
__device__ __forceinline__ void softmax_delta_block(const GradArgs& g, const EvDesc& e, int ev_local,
                                                    const int* label, const float* logit, float* delta, int* rowid) {
    // one thread per (row, class): every thread forms the row's maximum and denominator itself
    // (same order of operations for all classes of a row), so nothing waits for a reduction
    for (int t = threadIdx.x; t < g.B * g.C; t += 256) {
        const int k = t / g.C, c = t - k * g.C;
        const int rrow = g.batch_idx[(int64_t)e.sample * g.B + k];
        if (c == 0) rowid[k] = rrow;
        const int lab = label[(int64_t)e.node * g.rows + rrow];
        const float* lg = logit + ((int64_t)ev_local * g.B + k) * g.C;
        float m = ld_sel1<CG>(lg);
        for (int cc = 1; cc < g.C; ++cc) m = fmaxf(m, ld_sel1<CG>(lg + cc));
        float den = 0.f;
        for (int cc = 0; cc < g.C; ++cc) den += expf(ld_sel1<CG>(lg + cc) - m);
        delta[t] = (expf(ld_sel1<CG>(lg + c) - m) / den - (c == lab ? 1.f : 0.f)) / (float)g.B;
    }
    __syncthreads();
}
// ... then g[c][f] = sum_k delta[k][c] a_k[f] + l2 W[c][f], and the bias gradient, per coordinate q.
template <bool CG>
__device__ __forceinline__ float softmax_grad_coord(const GradArgs& g, const EvDesc& e, int64_t q,
                                                    const float* feat, const float* delta, const int* rowid) {
    float s = 0.f;
    if (q < (int64_t)g.C * g.F) {
        const int c = (int)(q / g.F), f = (int)(q % g.F);
        const float* abase = feat + (int64_t)e.node * g.rows * g.F;
        int k = 0;
        for (; k + 16 <= g.B; k += 16) {                   // sixteen feature loads in flight, summed in order
            float av[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) av[u] = abase[(int64_t)rowid[k + u] * g.F + f];
#pragma unroll
            for (int u = 0; u < 16; ++u) s = fmaf(delta[(k + u) * g.C + c], av[u], s);
        }
        for (; k < g.B; ++k) s = fmaf(delta[k * g.C + c], abase[(int64_t)rowid[k] * g.F + f], s);
    } else {
        const int c = (int)(q - (int64_t)g.C * g.F);
        for (int k = 0; k < g.B; ++k) s += delta[k * g.C + c];
    }
    return s + g.l2 * ld_sel1<CG>(g.x + (int64_t)e.node * g.stride + q);
}
// grid = (ceil(p / 256), events); dynamic shared memory: B*C floats + B ints
__global__ void __launch_bounds__(256)
k_softmax_grad(GradArgs g, const float* __restrict__ feat, const int* __restrict__ label,
               const float* __restrict__ logit) {
    extern __shared__ float sm[];
    float* delta = sm;                                   // [B][C]
    int* rowid = reinterpret_cast<int*>(sm + g.B * g.C); // [B]
    const EvDesc e = g.ev[blockIdx.y];
    softmax_delta_block<false>(g, e, blockIdx.y, label, logit, delta, rowid);
    const int64_t q = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (q >= g.p) return;
    g.gbuf[(int64_t)(e.g_par ^ 1) * g.gplane + (int64_t)e.node * g.stride + q] =
        softmax_grad_coord<false>(g, e, q, feat, delta, rowid);
}

// Sparse logistic regression, phase 1: coef_k = -y_k / (1 + exp(y_k a_k.x)) / B, one warp per
// sampled row.  grid = (ceil(B / 8), events).  coef: [events][B]
__global__ void __launch_bounds__(256)
k_logit_coef(GradArgs g, const int64_t* __restrict__ sp_ptr, const int* __restrict__ sp_col,
             const float* __restrict__ sp_val, const int* __restrict__ label, float* __restrict__ coef) {
    const EvDesc e = g.ev[blockIdx.y];
    const int k = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (k >= g.B) return;
    const int rrow = g.batch_idx[(int64_t)e.sample * g.B + k];
    const int64_t r = (int64_t)e.node * g.rows + rrow;
    const float* x = g.x + (int64_t)e.node * g.stride;
    float s = 0.f;
    for (int64_t q = sp_ptr[r] + lane; q < sp_ptr[r + 1]; q += 32) s = fmaf(sp_val[q], x[sp_col[q]], s);
    s = warp_sum(s);
    if (lane == 0) {
        const float y = (float)label[r];
        coef[(int64_t)blockIdx.y * g.B + k] = -y / (1.f + expf(y * s)) / (float)g.B;
    }
}

// Sparse logistic regression, phase 2, fused with S2b/S2c.  A CTA owns a tile of kLogitTile
// coordinates of one activation: it forms g = l2 x + sum_k coef_k a_k for the tile in shared
// memory, stores it as the new remembered gradient and, unless init_only, runs the tracking
// update on the tile, 1024 coordinates at a time.
// Assembly: warp w owns the coordinates [512 w, 512 (w+1)) of the tile and fetches, for every
// sampled row, exactly the entries that fall there: range_ptr[r][j] = index of the first entry of
// shard row r with column >= 512 j (computed once per problem on the host), so nothing is
// searched and the warps never wait for one another.  The entries are taken 32 at a time in
// row-major order; entries of different rows that hit the same coordinate (rare) are found with
// a warp match and added in row order, so the sum is the same on every run.
// grid = (tiles, events), 256 threads

constexpr int kLogitSub = 4;                               // passes of kThreads float4 per tile
constexpr int kLogitTile = kLogitSub * 4 * kThreads;
constexpr int kLogitRange = kLogitTile / (kThreads / 32);  // coordinates a warp assembles
template <bool COMP>
__global__ void __launch_bounds__(kThreads)
k_logit_track(RoundArgs a, GradArgs g, const int64_t* __restrict__ range_ptr, int nranges,
              const int* __restrict__ sp_col, const float* __restrict__ sp_val,
              const float* __restrict__ coef, int init_only) {
    __shared__ float tile[kLogitTile];
    const EvDesc e = g.ev[blockIdx.y];
    const int64_t row = (int64_t)e.node * g.stride;
    const int64_t c0 = (int64_t)blockIdx.x * kLogitTile;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr unsigned kFull = 0xffffffffu;
    // The tracking part at the end is a chain of dependent loads per sub-pass (edge lists -> row
    // ids -> rows); its operands are requested into L2 now, while the tile is assembled: the
    // lists into shared memory (the later reads then hit L1), the rows by prefetch, one request
    // per 128-byte line.
    constexpr int kPre = 16;
    __shared__ int pre_row[3 * kPre];
    const float* gold = g.gbuf + (int64_t)e.g_par * g.gplane + row;
    if (!init_only) {
        if (threadIdx.x < 3 * kPre) {
            const int m = threadIdx.x % kPre, what = threadIdx.x / kPre;
            int id = -1;
            if (what == 0 && m < e.news_cnt) id = a.news_new[e.news_beg + m];
            if (what == 1 && m < e.news_cnt) id = a.news_prev[e.news_beg + m];
            if (what == 2 && m < e.out_cnt) id = a.out_cur[e.out_beg + m];
            pre_row[threadIdx.x] = id;
        }
        if ((lane & 7) == 0) {
#pragma unroll
            for (int sub = 0; sub < kLogitSub; ++sub) {
                const int i4 = (blockIdx.x * kLogitSub + sub) * kThreads + threadIdx.x;
                if (i4 < a.n4) {
                    prefetch_l2(a.z + row + (int64_t)i4 * 4);
                    prefetch_l2(gold + (int64_t)i4 * 4);
                }
            }
        }
    }
    // the warp's first batch of rows: batch index -> entry range, started before the x tile is stored
    const int rg = blockIdx.x * (kThreads / 32) + warp;      // this warp's coordinate range inside a row
    const bool mine = rg < nranges;
    int64_t lo = 0;
    int cnt = 0;
    float ck = 0.f;
    if (mine && lane < min(32, g.B)) {
        const int rrow = g.batch_idx[(int64_t)e.sample * g.B + lane];
        const int64_t r = (int64_t)e.node * g.rows + rrow;
        lo = range_ptr[r * (nranges + 1) + rg];
        cnt = (int)(range_ptr[r * (nranges + 1) + rg + 1] - lo);
        ck = coef[(int64_t)blockIdx.y * g.B + lane];
    }
#pragma unroll
    for (int sub = 0; sub < kLogitSub; ++sub) {
        const int i4 = (blockIdx.x * kLogitSub + sub) * kThreads + threadIdx.x;
        float4 xv = make_float4(0, 0, 0, 0);
        if (i4 < a.n4) xv = reinterpret_cast<const float4*>(g.x + row)[i4];
        reinterpret_cast<float4*>(tile)[sub * kThreads + threadIdx.x] = f4_scale(g.l2, xv);
    }
    __syncthreads();                                        // tile = l2 x; pre_row is visible
    if (!init_only && (lane & 7) == 0) {
        for (int m = 0; m < 3 * kPre; ++m) {
            const int id = pre_row[m];
            if (id < 0) continue;
            const float* rr = a.rbuf + (int64_t)id * a.stride;
#pragma unroll
            for (int sub = 0; sub < kLogitSub; ++sub) {
                const int i4 = (blockIdx.x * kLogitSub + sub) * kThreads + threadIdx.x;
                if (i4 < a.n4) prefetch_l2(rr + (int64_t)i4 * 4);
            }
        }
    }
    if (mine) {
        for (int k0 = 0; k0 < g.B; k0 += 32) {              // up to 32 sampled rows per pass, one per lane
            const int nb = min(32, g.B - k0);
            if (k0 > 0) {
                lo = 0; cnt = 0; ck = 0.f;
                if (lane < nb) {
                    const int rrow = g.batch_idx[(int64_t)e.sample * g.B + k0 + lane];
                    const int64_t r = (int64_t)e.node * g.rows + rrow;
                    lo = range_ptr[r * (nranges + 1) + rg];
                    cnt = (int)(range_ptr[r * (nranges + 1) + rg + 1] - lo);
                    ck = coef[(int64_t)blockIdx.y * g.B + k0 + lane];
                }
            }
            int incl = cnt;                                 // entries of rows 0 .. lane (this pass, this range)
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += v;
            }
            const int total = __shfl_sync(kFull, incl, 31);
            for (int t0 = 0; t0 < total; t0 += 32) {        // entry t of the row-major list
                const int t = t0 + lane;
                const bool act = t < total;
                int k = 0;
                for (int j = 0; j < nb; ++j) k += (__shfl_sync(kFull, incl, j) <= t) ? 1 : 0;
                k = min(k, nb - 1);
                const int64_t lo_k = __shfl_sync(kFull, lo, k);
                const int excl_k = __shfl_sync(kFull, incl - cnt, k);
                const float ck_k = __shfl_sync(kFull, ck, k);
                int col = -1 - lane;                        // inactive lanes: distinct dummies
                float val = 0.f;
                if (act) {
                    const int64_t q = lo_k + (t - excl_k);
                    col = sp_col[q] - (int)c0;
                    val = ck_k * sp_val[q];
                }
                const unsigned same = __match_any_sync(kFull, col);
                const int rank = __popc(same & ((1u << lane) - 1u));   // earlier rows on the same coordinate
                int maxr = rank;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) maxr = max(maxr, __shfl_xor_sync(kFull, maxr, o));
                for (int rr = 0; rr <= maxr; ++rr) {        // almost always one turn
                    if (act && rank == rr) tile[col] += val;
                    __syncwarp();
                }
            }
        }
    }
    __syncthreads();
    float* zr = a.z + row;
    float* gnew = g.gbuf + (int64_t)(e.g_par ^ 1) * g.gplane + row;
    for (int sub = 0; sub < kLogitSub; ++sub) {
        const int base = (blockIdx.x * kLogitSub + sub) * kThreads + threadIdx.x;
        if (base >= a.n4) break;
        float4 zh[1], gnv[1], gov[1];
        gnv[0] = reinterpret_cast<const float4*>(tile)[sub * kThreads + threadIdx.x];
        reinterpret_cast<float4*>(gnew)[base] = gnv[0];
        if (init_only) continue;
        zh[0] = ld_stream(zr, base);
        gov[0] = ld_stream(gold, base);
        track_and_push<1, COMP>(a, e, base, zr, zh, gnv, gov);
    }
}

// Diagnostics: per coordinate, sums over nodes and edges; per block, partial results.
//   part[block][0] = sum_c (sum_i x_ic^2 - n xbar_c^2)    (consensus error squared)
//   part[block][1] = sum_c xbar_c^2
//   part[block][2] = max_c | sum_i z_ic + sum_e (rho_ec - rho~_ec) - sum_i g_ic |
//   part[block][3] = max_c | sum_i g_ic |
//   part[block][4] = sum_c sum_i z_ic^2
//   part[block][5] = sum_c (grad F(xbar))_c^2 for the element-wise objective, where the full gradient
//                    sum_i d_ic^2 (xbar_c - b_ic) is coordinate-wise; 0 otherwise
//   part[block][6] = this block's share of F(xbar) = sum_i f_i(xbar) for the element-wise objective:
//                    sum_c sum_i (d_ic (xbar_c - b_ic))^2 / 2; 0 otherwise
// g_i is row gsel[i] of gpool (or recomputed for the element-wise objective when gpool is null).
// xbar_out (may be null) receives the mean iterate in fp32.
// grid = tiles of kThreads coordinates (scalar: diagnostics favour clarity over speed)
constexpr int kDiagSlots = 7;
__global__ void __launch_bounds__(kThreads)
k_diagnostics(const float* __restrict__ x, const float* __restrict__ z, const float* __restrict__ zc,
              const float* __restrict__ gpool, const int* __restrict__ gsel,
              const float* __restrict__ qd, const float* __restrict__ qb,
              const float* __restrict__ rbuf, int64_t rlo_off, const int* __restrict__ rho_latest,
              const int* __restrict__ rho_buf, int n, int n_edges, int64_t stride, int64_t p,
              float* __restrict__ xbar_out, double* __restrict__ part) {
    __shared__ double red[kDiagSlots][kThreads];
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    double cons = 0, xb2 = 0, res = 0, gs = 0, z2 = 0, gf2 = 0, fl = 0;
    if (c < p) {
        double sx = 0, sx2 = 0, sz = 0, sg = 0;
#pragma unroll 8
        for (int i = 0; i < n; ++i) {
            const double xv = x[(int64_t)i * stride + c];
            double zv = z[(int64_t)i * stride + c];
            if (zc) zv += (double)zc[(int64_t)i * stride + c];
            double gv;
            if (gpool) gv = gpool[(int64_t)gsel[i] * stride + c];
            else { const float d = qd[(int64_t)i * stride + c]; gv = d * d * ((float)xv - qb[(int64_t)i * stride + c]); }
            sx += xv; sx2 += xv * xv; sz += zv; sg += gv; z2 += zv * zv;
        }
        double mass = 0;
        for (int e = 0; e < n_edges; ++e) {
            if (rho_latest[e] >= 0) {
                mass += (double)rbuf[(int64_t)rho_latest[e] * stride + c];
                if (rlo_off > 0) mass += (double)rbuf[(int64_t)rho_latest[e] * stride + rlo_off + c];
            }
            if (rho_buf[e] >= 0) {
                mass -= (double)rbuf[(int64_t)rho_buf[e] * stride + c];
                if (rlo_off > 0) mass -= (double)rbuf[(int64_t)rho_buf[e] * stride + rlo_off + c];
            }
        }
        const double xbar = sx / n;
        cons = sx2 - n * xbar * xbar;
        xb2 = xbar * xbar;
        res = fabs(sz + mass - sg);
        gs = fabs(sg);
        if (xbar_out) xbar_out[c] = (float)xbar;
        if (!gpool) {
            double gf = 0;
#pragma unroll 8
            for (int i = 0; i < n; ++i) {
                const double d = qd[(int64_t)i * stride + c];
                const double r = d * (xbar - (double)qb[(int64_t)i * stride + c]);
                gf += d * r;
                fl += 0.5 * r * r;
            }
            gf2 = gf * gf;
        }
    }
    red[0][threadIdx.x] = cons; red[1][threadIdx.x] = xb2; red[2][threadIdx.x] = res;
    red[3][threadIdx.x] = gs; red[4][threadIdx.x] = z2; red[5][threadIdx.x] = gf2; red[6][threadIdx.x] = fl;
    __syncthreads();
    for (int s = kThreads / 2; s > 0; s >>= 1) {
        if (threadIdx.x < s) {
            red[0][threadIdx.x] += red[0][threadIdx.x + s];
            red[1][threadIdx.x] += red[1][threadIdx.x + s];
            red[2][threadIdx.x] = fmax(red[2][threadIdx.x], red[2][threadIdx.x + s]);
            red[3][threadIdx.x] = fmax(red[3][threadIdx.x], red[3][threadIdx.x + s]);
            red[4][threadIdx.x] += red[4][threadIdx.x + s];
            red[5][threadIdx.x] += red[5][threadIdx.x + s];
            red[6][threadIdx.x] += red[6][threadIdx.x + s];
        }
        __syncthreads();
    }
    if (threadIdx.x < kDiagSlots) part[(int64_t)blockIdx.x * kDiagSlots + threadIdx.x] = red[threadIdx.x][0];
}

// Full least-squares gradient at the mean iterate, for the merit function:
// residuals of every row of every shard, r_ik = a_ik . xbar - y_ik.  grid = (ceil(rows / 8), n)
__global__ void __launch_bounds__(256)
k_diag_ls_residual(const float* __restrict__ feat, const float* __restrict__ target,
                   const float* __restrict__ xbar, float* __restrict__ res, int rows, int F) {
    const int k = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (k >= rows) return;
    const int64_t r = (int64_t)blockIdx.y * rows + k;
    const float* a = feat + r * F;
    float s = 0.f;
    for (int c = lane; c < F; c += 32) s = fmaf(a[c], xbar[c], s);
    s = warp_sum(s);
    if (lane == 0) res[r] = s - target[r];
}
// ... then (grad F(xbar))_c = sum_i [ (1/rows) sum_k a_ik[c] r_ik + l2 xbar_c ], squared and summed
// per block into part[block][5]; the block's share of F(xbar) = sum_i [ sum_k r_ik^2 / (2 rows) +
// l2 |xbar|^2 / 2 ] into part[block][6].  grid = tiles of kThreads coordinates
__global__ void __launch_bounds__(kThreads)
k_diag_ls_grad(const float* __restrict__ feat, const float* __restrict__ xbar, const float* __restrict__ res,
               int n, int rows, int F, float l2, double* __restrict__ part) {
    __shared__ double red[kThreads], redf[kThreads];
    const int c = blockIdx.x * kThreads + threadIdx.x;
    double gf = 0, fl = 0;
    for (int64_t r = c; r < (int64_t)n * rows; r += (int64_t)gridDim.x * kThreads) fl += 0.5 * (double)res[r] * (double)res[r] / rows;
    if (c < F) {
        fl += 0.5 * n * (double)l2 * (double)xbar[c] * (double)xbar[c];
        for (int i = 0; i < n; ++i) {
            double s = 0;
            for (int k = 0; k < rows; ++k) {
                const int64_t r = (int64_t)i * rows + k;
                s += (double)feat[r * F + c] * (double)res[r];
            }
            gf += s / rows + (double)l2 * (double)xbar[c];
        }
    }
    red[threadIdx.x] = gf * gf;
    redf[threadIdx.x] = fl;
    __syncthreads();
    for (int s = kThreads / 2; s > 0; s >>= 1) {
        if (threadIdx.x < s) { red[threadIdx.x] += red[threadIdx.x + s]; redf[threadIdx.x] += redf[threadIdx.x + s]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        part[(int64_t)blockIdx.x * kDiagSlots + 5] = red[0];
        part[(int64_t)blockIdx.x * kDiagSlots + 6] = redf[0];
    }
}

// Full gradient at the mean iterate for the sampled objectives, out of the minibatch kernels:
// every row of the state := xbar (grid = (tiles, n)) ...
__global__ void __launch_bounds__(kThreads)
k_diag_fill_rows(float* __restrict__ x, const float* __restrict__ xbar, int64_t stride, int n4) {
    const int i4 = blockIdx.x * kThreads + threadIdx.x;
    if (i4 >= n4) return;
    reinterpret_cast<float4*>(x + (int64_t)blockIdx.y * stride)[i4] = reinterpret_cast<const float4*>(xbar)[i4];
}
// ... acc_c += sum_i (row sel[i] of the gradient pool)_c after each chunk of shard rows ...
__global__ void __launch_bounds__(kThreads)
k_diag_accumulate(const float* __restrict__ gpool, const int* __restrict__ sel, int n, int64_t stride, int64_t p,
                  double* __restrict__ acc) {
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= p) return;
    double s = 0;
    for (int i = 0; i < n; ++i) s += (double)gpool[(int64_t)sel[i] * stride + c];
    acc[c] += s;
}
// ... and part[block][5] = sum_c (acc_c / chunks)^2 (the mean over the chunks is the full-shard gradient)
__global__ void __launch_bounds__(kThreads)
k_diag_norm2(const double* __restrict__ acc, int64_t p, double inv_chunks, double* __restrict__ part) {
    __shared__ double red[kThreads];
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const double v = c < p ? acc[c] * inv_chunks : 0.0;
    red[threadIdx.x] = v * v;
    __syncthreads();
    for (int s = kThreads / 2; s > 0; s >>= 1) {
        if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) part[(int64_t)blockIdx.x * kDiagSlots + 5] = red[0];
}

// Objective of eq. (1) at the mean iterate for the sampled objectives: one warp per shard row, the
// row's loss (without the L2 term) in double into rowloss[node * rows + k].  Plain and slow on
// purpose (diagnostics).  grid = (ceil(rows / 8), n), 256 threads.
//   softmax: x = [W (C x F) | bias (C)], loss = logsumexp(W a + bias) - (W a + bias)[label]
__global__ void __launch_bounds__(256)
k_diag_loss_softmax(const float* __restrict__ feat, const int* __restrict__ label, const float* __restrict__ xbar,
                    double* __restrict__ rowloss, int rows, int F, int C) {
    const int k = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (k >= rows) return;
    const int64_t r = (int64_t)blockIdx.y * rows + k;
    const float* a = feat + r * F;
    const int lab = label[r];
    double mx = -1e300, own = 0, se = 0;
    double lg[32];                                        // C <= 32 classes here
    for (int c = 0; c < C; ++c) {
        double s = 0;
        for (int f = lane; f < F; f += 32) s += (double)xbar[(int64_t)c * F + f] * (double)a[f];
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s += (double)xbar[(int64_t)C * F + c];
        lg[c] = s;
        mx = fmax(mx, s);
        if (c == lab) own = s;
    }
    for (int c = 0; c < C; ++c) se += exp(lg[c] - mx);
    if (lane == 0) rowloss[r] = mx + log(se) - own;
}
//   sparse logistic: loss = log(1 + exp(-y a.x))
__global__ void __launch_bounds__(256)
k_diag_loss_logistic(const int64_t* __restrict__ sp_ptr, const int* __restrict__ sp_col, const float* __restrict__ sp_val,
                     const int* __restrict__ label, const float* __restrict__ xbar, double* __restrict__ rowloss, int rows) {
    const int k = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (k >= rows) return;
    const int64_t r = (int64_t)blockIdx.y * rows + k;
    double s = 0;
    for (int64_t q = sp_ptr[r] + lane; q < sp_ptr[r + 1]; q += 32) s += (double)sp_val[q] * (double)xbar[sp_col[q]];
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const double m = (double)label[r] * s;
    if (lane == 0) rowloss[r] = m > 0 ? log1p(exp(-m)) : -m + log1p(exp(m));
}
//   MLP: x = [W1 (H x F) | b1 (H) | W2 (C x H) | b2 (C)]; the operands of A W1^T rounded to bf16 (the
//   matrix product the tensor cores take), everything else as it is; dynamic shared memory: 8 * H doubles
__global__ void __launch_bounds__(256)
k_diag_loss_mlp(const float* __restrict__ feat, const int* __restrict__ label, const float* __restrict__ xbar,
                double* __restrict__ rowloss, int rows, int F, int H, int C) {
    extern __shared__ double hs_all[];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k = blockIdx.x * 8 + w;
    if (k >= rows) return;
    double* hs = hs_all + (size_t)w * H;
    const int64_t r = (int64_t)blockIdx.y * rows + k;
    const float* a = feat + r * F;
    const float *W1 = xbar, *b1 = xbar + (int64_t)H * F, *W2 = b1 + H, *b2 = W2 + (int64_t)C * H;
    for (int j = 0; j < H; ++j) {
        double s = 0;
        for (int f = lane; f < F; f += 32)
            s += (double)__bfloat162float(__float2bfloat16_rn(W1[(int64_t)j * F + f])) * (double)__bfloat162float(__float2bfloat16_rn(a[f]));
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) hs[j] = fmax(s + (double)b1[j], 0.0);
    }
    __syncwarp();
    const int lab = label[r];
    double mx = -1e300, own = 0, se = 0;
    double lg[32];
    for (int c = 0; c < C; ++c) {
        double s = 0;
        for (int j = lane; j < H; j += 32) s += (double)W2[(int64_t)c * H + j] * hs[j];
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s += (double)b2[c];
        lg[c] = s;
        mx = fmax(mx, s);
        if (c == lab) own = s;
    }
    for (int c = 0; c < C; ++c) se += exp(lg[c] - mx);
    if (lane == 0) rowloss[r] = mx + log(se) - own;
}

// bf16 copy (round-to-nearest-even) of every row.  grid = (tiles, rows)
__global__ void __launch_bounds__(kThreads)
k_rows_to_bf16(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int64_t stride, int n4) {
    const int i4 = blockIdx.x * kThreads + threadIdx.x;
    if (i4 >= n4) return;
    const int64_t row = (int64_t)blockIdx.y * stride;
    const float4 v = reinterpret_cast<const float4*>(src + row)[i4];
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(dst + row)[i4] = pk;
}

}  // namespace rfast
