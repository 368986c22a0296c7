// Sample gradient of the one-hidden-layer MLP (softmax cross-entropy), sm_100a.
//
// Per activation (batch of B = 64 sampled rows A, parameters W1 [H x F], b1, W2 [C x H], b2):
//   pre = q(A) q(W1)^T + b1,  h = relu(pre),  logits = h W2^T + b2,  dlog = (softmax - onehot) / B
//   gW2 = dlog^T h,  gb2 = sum_k dlog,  dh = dlog W2,  dpre = dh .* (pre > 0)
//   gW1 = q(dpre)^T q(A),  gb1 = sum_k dpre                      (q = round to bf16)
// The two products that carry the work, pre (H x B x F) and gW1 (H x F x B), are dense
// contractions and run on the 5th-generation tensor cores: operands are brought into shared
// memory by TMA (128-byte swizzle), tcgen05.mma (kind::f16, bf16 x bf16 -> fp32) accumulates in
// tensor memory, and the epilogue reads the accumulator back with tcgen05.ld.  Both are
// computed transposed (M = a 128-row slab of hidden units) so that M is the tensor core's
// native 128.  The C <= 16 wide products in between are far too thin for an MMA tile and run
// in fp32 on the CUDA cores: the logits as per-slab shares in the forward kernel's epilogue,
// while h is still in shared memory, the rest in the backward kernel.
//
// Every wait on an mbarrier is bounded: when it runs out the CTA records a code in a status
// word, leaves its loops, frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <string>

#include "rfast_internal.h"

namespace rfast {

namespace {

constexpr int kBatch = 64;          // rows per minibatch the tensor-core path is built for
constexpr int kMTile = 128;         // hidden units per CTA (UMMA M)
constexpr int kKBlock = 64;         // bf16 elements per 128-byte swizzle row
constexpr int kStagesFwd = 4;
constexpr int kFwdWorkers = 256;    // warps 2..9 of the forward kernel
constexpr int kFwdThreads = 64 + kFwdWorkers;   // warp 0: TMA, warp 1: MMA + tensor memory
constexpr int kHsPitch = 132;       // floats per staged row of 128 hidden activations (rows fall on different banks)
constexpr int kGemmThreads = 192;   // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..5: epilogue
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // every mbarrier wait gives up after 2 s

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait; false when the limit ran out (the caller records it and bails out).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
        uint64_t now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (it == 0) t0 = now;
        else if (now - t0 > kWaitLimitNs) return false;
    }
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// Tile store shared -> global; completion is tracked by the thread's bulk async-group.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, const void* src, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
        ::"l"(map), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// until the stores of all committed groups have read their shared-memory source
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// the same, the most recent group excepted
__device__ __forceinline__ void tma_store_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
// makes this thread's shared-memory writes visible to the async (TMA) proxy
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {     // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {         // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, both operands K-major bf16, fp32 accumulate; one thread issues.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The barrier gets one arrival when all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread t of the warp gets lane (base lane + t).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory operand descriptor: K-major tile of rows x 64 bf16 as written by TMA with the
// 128-byte swizzle (row pitch 128 B, groups of 8 rows = 1024 B), tile base 1024-byte aligned.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);        // start address
    d |= (uint64_t)1 << 16;                          // leading-dimension byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride between 8-row groups
    d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                          // 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, shape M x N.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

enum { kErrNone = 0, kErrProducer = 1, kErrMma = 2, kErrEpilogue = 3 };

}  // namespace

struct MlpPlan;
void mlp_plan_destroy(MlpPlan* p);

struct MlpPlan {
    int n = 0, rows = 0, F = 0, H = 0, C = 0, B = 0, Fp = 0, NT = 0, maxev = 0;
    int64_t stride = 0;
    __nv_bfloat16 *featb = nullptr, *Ab = nullptr, *AbT = nullptr, *dpqT = nullptr;
    float* hf = nullptr;               // [ev][B][H] hidden activations
    float* share = nullptr;            // [ev][H / 128][B][16] logit shares of the slabs, zero beyond C
    int* status = nullptr;
    CUtensorMap tmW1, tmA, tmD, tmAT, tmX, tmG;
};

// ---------------------------------------------------------------------------------------------
// kernels
// ---------------------------------------------------------------------------------------------

// fp32 -> bf16 (nearest even), flat
__global__ void k_to_bf16(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int64_t count) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) dst[i] = __float2bfloat16_rn(src[i]);
}

// Sampled rows of one activation, as the two GEMMs want them:
//   Ab  [ev][B][Fp]  row k = features of sample k, zero beyond F (K-major operand of pre)
//   AbT [ev][F][B]   the transpose                      (K-major operand of gW1, K = batch)
// One CTA moves a 64 x 64 tile with 16-byte accesses and transposes it through shared memory
// (F is a multiple of 16, so a group of 8 features never straddles F).  grid = (Fp / 64, events)
__global__ void __launch_bounds__(256)
k_mlp_gather(const EvDesc* __restrict__ evs, const int* __restrict__ batch_idx,
             const __nv_bfloat16* __restrict__ featb, __nv_bfloat16* __restrict__ Ab,
             __nv_bfloat16* __restrict__ AbT, int rows, int F, int Fp) {
    __shared__ __align__(16) __nv_bfloat16 tile[kBatch][kKBlock + 8];   // row pitch 144 B: 16-byte aligned rows
    const int ev = blockIdx.y, f0 = blockIdx.x * kKBlock;
    const EvDesc e = evs[ev];
    const __nv_bfloat16* shard = featb + (int64_t)e.node * rows * F;
    __nv_bfloat16* ab = Ab + (int64_t)ev * kBatch * Fp;
    __nv_bfloat16* abt = AbT + (int64_t)ev * F * kBatch;
#pragma unroll
    for (int u = 0; u < 2; ++u) {                          // 64 rows x 8 groups of 8 features
        const int q = threadIdx.x + u * 256;
        const int k = q >> 3, f = (q & 7) * 8;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (f0 + f < F) {
            const int r = batch_idx[(int64_t)e.sample * kBatch + k];
            v = *reinterpret_cast<const uint4*>(shard + (int64_t)r * F + f0 + f);
        }
        *reinterpret_cast<uint4*>(ab + (int64_t)k * Fp + f0 + f) = v;
        *reinterpret_cast<uint4*>(&tile[k][f]) = v;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < 2; ++u) {                          // 64 features x 8 groups of 8 samples
        const int q = threadIdx.x + u * 256;
        const int f = q & 63, k0 = (q >> 6) * 8;
        if (f0 + f < F) {
            uint32_t pk[4];
#pragma unroll
            for (int kk = 0; kk < 8; kk += 2)
                pk[kk >> 1] = (uint32_t)__bfloat16_as_ushort(tile[k0 + kk][f]) |
                              ((uint32_t)__bfloat16_as_ushort(tile[k0 + kk + 1][f]) << 16);
            *reinterpret_cast<uint4*>(abt + (int64_t)(f0 + f) * kBatch + k0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
    }
}

// pre^T slab = W1[h0 .. h0+128) x A^T, then h = relu(pre + b1), stored in hf[ev][k][j], and the
// slab's share of the logits, share[ev][slab][k][c] = sum over the slab's 128 hidden units of
// h[k][j] W2[c][j]: h is still on chip when the product ends (it is staged in the operand
// stages, which are free by then), so the output layer costs no second pass over h.  The shares
// of the H / 128 slabs are added, in slab order, by the backward kernel.
// grid = (H / 128, events), 320 threads; dynamic shared memory kFwdSmem
template <int CQ>
__global__ void __launch_bounds__(kFwdThreads, 2)
k_mlp_fwd(const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmA,
          const EvDesc* __restrict__ evs, const float* __restrict__ x, int64_t stride,
          float* __restrict__ hf, float* __restrict__ share, int F, int H, int C, int kblocks, int* status) {
    constexpr int CP = CQ * 4;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int kABytes = kMTile * kKBlock * 2, kBBytes = kBatch * kKBlock * 2;
    uint8_t* sA = smem;                                   // [stages][128][64] bf16
    uint8_t* sB = smem + kStagesFwd * kABytes;            // [stages][64][64] bf16
    float* hs = reinterpret_cast<float*>(smem);           // after the product: h [64][kHsPitch]
    float* w2s = reinterpret_cast<float*>(smem + kStagesFwd * (kABytes + kBBytes));   // [16][kHsPitch]
    __shared__ uint64_t full[kStagesFwd], empty[kStagesFwd], acc_full;
    __shared__ uint32_t tmem_base;
    __shared__ volatile int bad;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ev = blockIdx.y, h0 = blockIdx.x * kMTile;
    const EvDesc e = evs[ev];
    const int64_t row = (int64_t)e.node * stride;
    const int64_t ob1 = (int64_t)H * F, oW2 = ob1 + H;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStagesFwd; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(&acc_full, 1);
        bad = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(&tmem_base, 64);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tacc = tmem_base;
    const int wt = threadIdx.x - 64;                       // worker thread id, 0..255 in warps 2..9

    if (warp == 0 && lane == 0) {                          // ---- TMA producer
        int issued = 0;
        bool ok = true;
        for (int kb = 0; kb < kblocks && ok; ++kb) {
            const int s = kb % kStagesFwd;
            if (kb >= kStagesFwd) ok = mbar_wait(&empty[s], ((kb / kStagesFwd) - 1) & 1);
            if (!ok) break;
            mbar_expect_tx(&full[s], kABytes + kBBytes);
            tma_load_3d(sA + s * kABytes, &tmW1, &full[s], kb * kKBlock, h0, e.node);
            tma_load_2d(sB + s * kBBytes, &tmA, &full[s], kb * kKBlock, ev * kBatch);
            ++issued;
        }
        if (!ok) {
            atomicExch(status, kErrProducer);
            bad = 1;
            // let the copies already issued land before the CTA's shared memory goes away
            for (int q = (issued > kStagesFwd ? issued - kStagesFwd : 0); q < issued; ++q)
                mbar_wait(&full[q % kStagesFwd], (q / kStagesFwd) & 1);
        }
    } else if (warp == 1 && lane == 0) {                   // ---- MMA issuer
        const uint32_t idesc = umma_idesc_bf16(kMTile, kBatch);
        bool ok = true;
        for (int kb = 0; kb < kblocks; ++kb) {
            const int s = kb % kStagesFwd;
            ok = mbar_wait(&full[s], (kb / kStagesFwd) & 1);
            if (!ok) break;
            tc_fence_after();
            const uint64_t ad = umma_desc_sw128(smem_u32(sA + s * kABytes));
            const uint64_t bd = umma_desc_sw128(smem_u32(sB + s * kBBytes));
#pragma unroll
            for (int k = 0; k < kKBlock / 16; ++k)          // 16 bf16 = 32 bytes per step inside the swizzle row
                umma_bf16(tacc, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc, (kb | k) ? 1u : 0u);
            umma_commit(&empty[s]);
        }
        if (ok) umma_commit(&acc_full);
        else { atomicExch(status, kErrMma); bad = 1; __threadfence_block(); mbar_arrive(&acc_full); }
    } else if (warp >= 2) {                                // ---- epilogue: TMEM -> relu -> hf and shared memory
        // while the product runs: the W2 columns of the slab (rows C .. CP-1 zero) and the bias
        for (int o = wt; o < CP * kMTile; o += kFwdWorkers) {
            const int c = o >> 7, j = o & (kMTile - 1);
            w2s[c * kHsPitch + j] = c < C ? x[row + oW2 + (int64_t)c * H + h0 + j] : 0.f;
        }
        const int q = warp & 3;                             // this warp owns tensor-memory lanes 32q .. 32q+31
        const int colh = (warp - 2) >> 2;                   // and columns 32 colh .. 32 colh + 31
        const int jl = q * 32 + lane;                       // hidden unit inside the slab
        const float b1 = x[row + ob1 + h0 + jl];
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&acc_full, 0));   // one decision per warp
        tc_fence_after();
        if (!ok) { if (lane == 0) { atomicExch(status, kErrEpilogue); bad = 1; } }
        else if (!bad) {
            float* out = hf + (int64_t)ev * kBatch * H + h0 + jl;
#pragma unroll
            for (int c0 = 0; c0 < 32; c0 += 16) {
                float v[16];
                tmem_ld16(tacc + ((uint32_t)(q * 32) << 16) + colh * 32 + c0, v);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float hval = fmaxf(v[i] + b1, 0.f);
                    out[(int64_t)(colh * 32 + c0 + i) * H] = hval;
                    hs[(colh * 32 + c0 + i) * kHsPitch + jl] = hval;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();                                       // h and the W2 columns are in shared memory
    if (warp >= 2 && bad == 0) {                           // ---- the slab's share of the logits
        // Register tile of 4 rows x CQ classes per thread over a quarter of the hidden units: every
        // value read from shared memory feeds 4 (W2) or CQ (h) products, a third of the reads of
        // one row per thread.  Lane bits: jq = quarter of the units (interleaved: float4 4t + jq),
        // kg = rows kg, kg + 16, kg + 32, kg + 48; cgp = classes cgp, cgp + 4, ...  The four
        // quarters sit in adjacent lanes and are added in a fixed tree.
        const int jq = wt & 3, kg = (wt >> 2) & 15, cgp = wt >> 6;
        float acc[4][CQ];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int i = 0; i < CQ; ++i) acc[r][i] = 0.f;
#pragma unroll 2
        for (int t = 0; t < kMTile / 16; ++t) {
            const int j4 = 4 * t + jq;
            float4 hv[4], wv[CQ];
#pragma unroll
            for (int r = 0; r < 4; ++r) hv[r] = reinterpret_cast<const float4*>(hs + (kg + 16 * r) * kHsPitch)[j4];
#pragma unroll
            for (int i = 0; i < CQ; ++i) wv[i] = reinterpret_cast<const float4*>(w2s + (cgp + 4 * i) * kHsPitch)[j4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int i = 0; i < CQ; ++i)
                    acc[r][i] = fmaf(hv[r].w, wv[i].w, fmaf(hv[r].z, wv[i].z, fmaf(hv[r].y, wv[i].y, fmaf(hv[r].x, wv[i].x, acc[r][i]))));
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int i = 0; i < CQ; ++i) {
                float v = acc[r][i];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                acc[r][i] = v;
            }
        if (jq == 0) {
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                float* dst = share + (((int64_t)ev * gridDim.x + blockIdx.x) * kBatch + kg + 16 * r) * 16;
#pragma unroll
                for (int i = 0; i < 4; ++i) dst[cgp + 4 * i] = i < CQ ? acc[r][i < CQ ? i : 0] : 0.f;
            }
        }
    }
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tacc, 64); }
}

// Backward through the output layer for a slab of 64 hidden units.  Every CTA first finishes
// the output layer for the whole batch (64 x C values: the logit shares of the forward kernel
// added in slab order, bias, softmax, dlog = (softmax - onehot) / B; the four class quads of a
// row sit in adjacent lanes and combine maximum and denominator by shuffles), then forms gW2,
// gb1, dpre and its bf16 transpose for the second big product; the first slab also sums gb2.
// A thread owns one hidden unit and a quarter of the batch; the four partial sums are added in
// a fixed order.  CQ = ceil(C / 4): the class dimension is processed in quads, zero beyond C.
// grid = (H / 64, events), 256 threads
template <int CQ>
__global__ void __launch_bounds__(256)
k_mlp_back(const EvDesc* __restrict__ evs, const int* __restrict__ batch_idx, const int* __restrict__ label,
           const float* __restrict__ x, int64_t stride, const float* __restrict__ hf,
           const float* __restrict__ share, int R, __nv_bfloat16* __restrict__ dpqT,
           float* __restrict__ gbuf, int64_t gplane, int rows, int F, int H, int C, float l2) {
    constexpr int CP = CQ * 4, kSlab = 64, kQuarter = kBatch / 4;
    __shared__ float4 dl[kBatch][4];                       // [B][16]
    __shared__ float part[4][kSlab][CP + 1];               // gw2[0..CP), gb1
    const int ev = blockIdx.y;
    const EvDesc e = evs[ev];
    const int64_t row = (int64_t)e.node * stride;
    const int64_t oW2 = (int64_t)H * F + H, ob2 = oW2 + (int64_t)C * H;
    const float* W2 = x + row + oW2;
    float* g = gbuf + (int64_t)(e.g_par ^ 1) * gplane + row;
    const int jl = threadIdx.x & (kSlab - 1), kq = threadIdx.x >> 6;
    const int j = blockIdx.x * kSlab + jl;
    // everything this thread needs from global memory, all in flight together
    const int ks = threadIdx.x >> 2, quad = threadIdx.x & 3;   // output layer: sampled row, class quad
    const int lab = label[(int64_t)e.node * rows + batch_idx[(int64_t)e.sample * kBatch + ks]];
    float4 lg = make_float4(0, 0, 0, 0);
    if (quad < CQ) {
        const float4* sh = reinterpret_cast<const float4*>(share + ((int64_t)ev * R * kBatch + ks) * 16) + quad;
        lg = sh[0];
        for (int r = 1; r < R; ++r) {                       // slab order
            const float4 t = sh[(int64_t)r * kBatch * 4];
            lg.x += t.x; lg.y += t.y; lg.z += t.z; lg.w += t.w;
        }
    }
    float b2[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) b2[i] = 4 * quad + i < C ? x[row + ob2 + 4 * quad + i] : 0.f;
    const float* h = hf + (int64_t)ev * kBatch * H + j;
    float hv[kQuarter];
#pragma unroll
    for (int kk = 0; kk < kQuarter; ++kk) hv[kk] = h[(int64_t)(kq * kQuarter + kk) * H];
    float w2[CP], gw2[CP];
#pragma unroll
    for (int c = 0; c < CP; ++c) { w2[c] = c < C ? W2[(int64_t)c * H + j] : 0.f; gw2[c] = 0.f; }
    {
        float l4[4] = {lg.x + b2[0], lg.y + b2[1], lg.z + b2[2], lg.w + b2[3]};
        float m = -3.0e38f;
#pragma unroll
        for (int i = 0; i < 4; ++i) if (4 * quad + i < C) m = fmaxf(m, l4[i]);
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
        float ex[4], den = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) { ex[i] = 4 * quad + i < C ? expf(l4[i] - m) : 0.f; den += ex[i]; }
        den += __shfl_xor_sync(0xffffffffu, den, 1);       // the same tree in all four lanes
        den += __shfl_xor_sync(0xffffffffu, den, 2);
        float d[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            d[i] = 4 * quad + i < C ? (ex[i] / den - (4 * quad + i == lab ? 1.f : 0.f)) / (float)kBatch : 0.f;
        dl[ks][quad] = make_float4(d[0], d[1], d[2], d[3]);
    }
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x < 32) {             // gb2: two halves of the batch, lower half first
        const int c = threadIdx.x & 15, half = threadIdx.x >> 4;
        const float* dlf = reinterpret_cast<const float*>(&dl[0][0]);
        float s = 0.f;
        for (int k = half * (kBatch / 2); k < (half + 1) * (kBatch / 2); ++k) s += dlf[k * 16 + c];
        const float o = __shfl_down_sync(0xffffffffu, s, 16);
        if (threadIdx.x < C) g[ob2 + c] = l2 != 0.f ? (s + o) + l2 * x[row + ob2 + c] : (s + o);   // no load without a regulariser
    }
    float gb1 = 0.f;
    __nv_bfloat16* drow = dpqT + ((int64_t)ev * H + j) * kBatch + kq * kQuarter;
#pragma unroll
    for (int k0 = 0; k0 < kQuarter; k0 += 8) {
        uint32_t pk[4];
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const int k = kq * kQuarter + k0 + kk;
            float d[CP];
#pragma unroll
            for (int cq = 0; cq < CQ; ++cq) {
                const float4 t = dl[k][cq];
                d[cq * 4] = t.x; d[cq * 4 + 1] = t.y; d[cq * 4 + 2] = t.z; d[cq * 4 + 3] = t.w;
            }
            float dh = 0.f;
#pragma unroll
            for (int c = 0; c < CP; ++c) dh = fmaf(d[c], w2[c], dh);
            const float dp = hv[k0 + kk] > 0.f ? dh : 0.f;
            gb1 += dp;
            const uint32_t b = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(dp));
            if (kk & 1) pk[kk >> 1] |= b << 16; else pk[kk >> 1] = b;
#pragma unroll
            for (int c = 0; c < CP; ++c) gw2[c] = fmaf(d[c], hv[k0 + kk], gw2[c]);
        }
        *reinterpret_cast<uint4*>(drow + k0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
#pragma unroll
    for (int c = 0; c < CP; ++c) part[kq][jl][c] = gw2[c];
    part[kq][jl][CP] = gb1;
    __syncthreads();
    // (C + 1) x 64 outputs, consecutive threads on consecutive hidden units
    for (int o = threadIdx.x; o < (C + 1) * kSlab; o += 256) {
        const int c = o >> 6, jj = o & (kSlab - 1);        // c == C: gb1
        const int pc = c < C ? c : CP;
        const float tot = ((part[0][jj][pc] + part[1][jj][pc]) + part[2][jj][pc]) + part[3][jj][pc];
        const int64_t at = c < C ? oW2 + (int64_t)c * H + blockIdx.x * kSlab + jj : (int64_t)H * F + blockIdx.x * kSlab + jj;
        g[at] = l2 != 0.f ? tot + l2 * x[row + at] : tot;
    }
}

// One tile of gW1: hidden units [h0, h0+128) x features [f0, f0+NT) = q(dpre)^T (K = batch) x q(A),
// plus l2 * W1.  The fp32 side of the epilogue also goes through TMA, in pieces of 32 rows x 16
// floats (64-byte swizzle): a thread owns a whole row of the accumulator, so plain stores would
// touch 32 different cache lines per instruction.  Each epilogue warp has a ring of two pieces
// in shared memory: it adds its accumulator rows to the W1 piece loaded there (or just writes
// them when there is no regulariser), stores the piece with a TMA tile store, and reuses the
// slot once that store has read it.  The small footprint lets four CTAs share an SM.
// grid = (H / 128, F / NT, events); dynamic shared memory kDw1Smem
__global__ void __launch_bounds__(kGemmThreads, 1)
k_mlp_dw1(const __grid_constant__ CUtensorMap tmD, const __grid_constant__ CUtensorMap tmAT,
          const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmG,
          const EvDesc* __restrict__ evs, int n, int F, int H, int NT, float l2, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int kABytes = kMTile * kKBlock * 2;          // q(dpre)^T slab
    constexpr int kPiece = 32 * 16 * 4;                    // 32 rows x 16 floats
    uint8_t* sA = smem;
    uint8_t* sB = smem + kABytes;                          // [NT][64] bf16 tile of A^T (at most 16 KB)
    uint8_t* ring = smem + 2 * kABytes;                    // [4 warps][2 slots] pieces
    __shared__ uint64_t ab_full, acc_full, x_full[4][2];
    __shared__ uint32_t tmem_base;
    __shared__ volatile int aborted;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ev = blockIdx.z, h0 = blockIdx.x * kMTile, f0 = blockIdx.y * NT;
    const EvDesc e = evs[ev];
    const bool reg = l2 != 0.f;
    const int np = NT / 16;
    if (threadIdx.x == 0) {
        mbar_init(&ab_full, 1);
        mbar_init(&acc_full, 1);
        for (int q = 0; q < 4; ++q) { mbar_init(&x_full[q][0], 1); mbar_init(&x_full[q][1], 1); }
        aborted = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(&tmem_base, 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tacc = tmem_base;

    if (warp == 0 && lane == 0) {                          // ---- TMA producer
        mbar_expect_tx(&ab_full, kABytes + NT * kKBlock * 2);
        tma_load_2d(sA, &tmD, &ab_full, 0, ev * H + h0);
        tma_load_2d(sB, &tmAT, &ab_full, 0, ev * F + f0);
    } else if (warp == 1 && lane == 0) {                   // ---- MMA issuer
        const uint32_t idesc = umma_idesc_bf16(kMTile, NT);
        const bool ok = mbar_wait(&ab_full, 0);
        if (ok) {
            tc_fence_after();
            const uint64_t ad = umma_desc_sw128(smem_u32(sA));
            const uint64_t bd = umma_desc_sw128(smem_u32(sB));
#pragma unroll
            for (int k = 0; k < kKBlock / 16; ++k)
                umma_bf16(tacc, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc, k ? 1u : 0u);
            umma_commit(&acc_full);
        } else {
            atomicExch(status, kErrMma);
            aborted = 1;
            __threadfence_block();
            mbar_arrive(&acc_full);
        }
    } else if (warp >= 2) {                                // ---- epilogue: TMEM (+ l2 x) -> shared -> TMA store
        const int q = warp & 3;                             // rows 32q .. 32q+31 of the tile = tensor-memory lanes
        uint8_t* slot0 = ring + q * 2 * kPiece;
        const int sw = (lane >> 1) & 3;                     // 64-byte swizzle: 16-byte chunk index ^ address bits 7..8
        // W1 pieces are requested two ahead: pieces 0 and 1 here, piece pc + 2 when piece pc is stored
        if (reg && lane == 0)
            for (int pc = 0; pc < 2 && pc < np; ++pc) {
                mbar_expect_tx(&x_full[q][pc], kPiece);
                tma_load_3d(slot0 + pc * kPiece, &tmX, &x_full[q][pc], f0 + pc * 16, h0 + q * 32, e.node);
            }
        bool ok = __all_sync(0xffffffffu, mbar_wait(&acc_full, 0));         // one decision per warp
        tc_fence_after();
        const bool run = ok && !aborted;
        const int plane = (e.g_par ^ 1) * n + e.node;
        int pc = 0;
        for (; pc < np; ++pc) {
            const int s = pc & 1;
            uint8_t* slot = slot0 + s * kPiece;
            if (reg) ok = __all_sync(0xffffffffu, mbar_wait(&x_full[q][s], (pc >> 1) & 1)) && ok;
            if (!run || !ok) break;
            if (!reg && pc >= 2) {                          // the store of piece pc - 2 has read this slot
                if (lane == 0) tma_store_wait_read_1();
                __syncwarp();
            }
            float v[16];
            tmem_ld16(tacc + ((uint32_t)(q * 32) << 16) + pc * 16, v);
            float4* rowp = reinterpret_cast<float4*>(slot + lane * 64);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float4 o = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                float4* at = rowp + (c ^ sw);
                if (reg) {
                    const float4 xv = *at;
                    o.x = fmaf(l2, xv.x, o.x); o.y = fmaf(l2, xv.y, o.y); o.z = fmaf(l2, xv.z, o.z); o.w = fmaf(l2, xv.w, o.w);
                }
                *at = o;
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                tma_store_3d(&tmG, slot, f0 + pc * 16, h0 + q * 32, plane);
                tma_store_commit();
                if (reg && pc + 2 < np) {                   // next W1 piece into this slot, once the store has read it
                    tma_store_wait_read();
                    mbar_expect_tx(&x_full[q][s], kPiece);
                    tma_load_3d(slot, &tmX, &x_full[q][s], f0 + (pc + 2) * 16, h0 + q * 32, e.node);
                }
            }
        }
        // left early: the one piece requested beyond the last one awaited must land before the CTA ends
        if (reg && pc < np && pc + 1 < np) mbar_wait(&x_full[q][(pc + 1) & 1], ((pc + 1) >> 1) & 1);
        if (!ok && lane == 0) atomicExch(status, kErrEpilogue);
        if (lane == 0) tma_store_wait_read();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tacc, 128); }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// innermost dimension first; strides in bytes for dimensions 1.. ; bf16 with the 128-byte swizzle
// (GEMM operands) or fp32 with the 64-byte swizzle (epilogue tiles of 16 floats per row)
bool make_map(CUtensorMap* m, void* base, int rank, const uint64_t* dims, const uint64_t* strides,
              const uint32_t* box, bool f32 = false) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t d[3], s[2];
    cuuint32_t b[3], es[3] = {1, 1, 1};
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) s[i] = strides[i];
    return fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, base, d, s, b, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, f32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr size_t kFwdSmem = kStagesFwd * (kMTile * kKBlock * 2 + kBatch * kKBlock * 2) + 16 * kHsPitch * 4 + 1024;
constexpr size_t kDw1Smem = 2 * (size_t)kMTile * kKBlock * 2 + 4 * 2 * (32 * 16 * 4) + 1024;

}  // namespace

int mlp_plan_create(int n, int rows, int F, int H, int C, int B, int64_t stride, int max_events,
                    const float* d_feat, const __nv_bfloat16* xb, const float* x, float* gbuf, cudaStream_t st,
                    MlpPlan** out, size_t* dev_bytes, std::string& err) {
    *out = nullptr;
    *dev_bytes = 0;
    if (B != kBatch || H % kMTile != 0 || H <= 0 || F % 16 != 0 || F <= 0 || C < 2 || C > 16) {
        err = "MLP: the tensor-core path needs batch = 64, n_hidden a multiple of 128, n_features a multiple of 16, 2 <= n_classes <= 16";
        return RFAST_EINVAL;
    }
    MlpPlan* p = new MlpPlan();
    p->n = n; p->rows = rows; p->F = F; p->H = H; p->C = C; p->B = B; p->stride = stride; p->maxev = max_events;
    p->Fp = (F + kKBlock - 1) / kKBlock * kKBlock;
    p->NT = 16;
    for (int nt = 128; nt >= 16; nt -= 16) if (F % nt == 0) { p->NT = nt; break; }
    size_t total = 0;
    auto alloc = [&](__nv_bfloat16** q, size_t cnt) {
        cudaError_t e = cudaMalloc((void**)q, cnt * sizeof(__nv_bfloat16));
        if (e == cudaSuccess) total += cnt * sizeof(__nv_bfloat16);
        return e == cudaSuccess;
    };
    const size_t nfeat = (size_t)n * rows * F;
    bool ok = alloc(&p->featb, nfeat) && alloc(&p->Ab, (size_t)max_events * kBatch * p->Fp) &&
              alloc(&p->AbT, (size_t)max_events * F * kBatch) &&
              alloc(&p->dpqT, (size_t)max_events * H * kBatch) &&
              cudaMalloc((void**)&p->hf, (size_t)max_events * kBatch * H * sizeof(float)) == cudaSuccess &&
              cudaMalloc((void**)&p->share, (size_t)max_events * (H / kMTile) * kBatch * 16 * sizeof(float)) == cudaSuccess &&
              cudaMalloc((void**)&p->status, sizeof(int)) == cudaSuccess;
    if (!ok) { mlp_plan_destroy(p); err = "MLP: device allocation failed"; return RFAST_ENOMEM; }
    cudaMemsetAsync(p->status, 0, sizeof(int), st);
    k_to_bf16<<<(unsigned)((nfeat + 255) / 256), 256, 0, st>>>(d_feat, p->featb, (int64_t)nfeat);
    {
        const uint64_t dW[3] = {(uint64_t)F, (uint64_t)H, (uint64_t)n};
        const uint64_t sW[2] = {(uint64_t)F * 2, (uint64_t)stride * 2};
        const uint32_t bW[3] = {kKBlock, kMTile, 1};
        const uint64_t dA[2] = {(uint64_t)p->Fp, (uint64_t)max_events * kBatch};
        const uint64_t sA[1] = {(uint64_t)p->Fp * 2};
        const uint32_t bA[2] = {kKBlock, kBatch};
        const uint64_t dD[2] = {(uint64_t)kBatch, (uint64_t)max_events * H};
        const uint64_t sD[1] = {(uint64_t)kBatch * 2};
        const uint32_t bD[2] = {kKBlock, kMTile};
        const uint64_t dT[2] = {(uint64_t)kBatch, (uint64_t)max_events * F};
        const uint32_t bT[2] = {kKBlock, (uint32_t)p->NT};
        // fp32 views of the W1 block: x [n][H][F] and the two gradient planes [2n][H][F]
        const uint64_t dX[3] = {(uint64_t)F, (uint64_t)H, (uint64_t)n}, dG[3] = {(uint64_t)F, (uint64_t)H, (uint64_t)2 * n};
        const uint64_t sX[2] = {(uint64_t)F * 4, (uint64_t)stride * 4};
        const uint32_t bX[3] = {16, 32, 1}, bG[3] = {16, 32, 1};
        if (!make_map(&p->tmW1, (void*)xb, 3, dW, sW, bW) || !make_map(&p->tmA, p->Ab, 2, dA, sA, bA) ||
            !make_map(&p->tmD, p->dpqT, 2, dD, sD, bD) || !make_map(&p->tmAT, p->AbT, 2, dT, sD, bT) ||
            !make_map(&p->tmX, (void*)x, 3, dX, sX, bX, true) || !make_map(&p->tmG, gbuf, 3, dG, sX, bG, true)) {
            mlp_plan_destroy(p);
            err = "MLP: cuTensorMapEncodeTiled failed";
            return RFAST_ECUDA;
        }
    }
    if (cudaFuncSetAttribute(k_mlp_fwd<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFwdSmem) != cudaSuccess ||
        cudaFuncSetAttribute(k_mlp_fwd<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFwdSmem) != cudaSuccess ||
        cudaFuncSetAttribute(k_mlp_fwd<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFwdSmem) != cudaSuccess ||
        cudaFuncSetAttribute(k_mlp_fwd<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFwdSmem) != cudaSuccess ||
        cudaFuncSetAttribute(k_mlp_dw1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDw1Smem) != cudaSuccess) {
        mlp_plan_destroy(p);
        err = "MLP: cannot reserve shared memory";
        return RFAST_ECUDA;
    }
    *out = p;
    *dev_bytes = total + sizeof(int) + (size_t)max_events * kBatch * H * sizeof(float) +
                 (size_t)max_events * (H / kMTile) * kBatch * 16 * sizeof(float);
    return RFAST_OK;
}

void mlp_plan_destroy(MlpPlan* p) {
    if (!p) return;
    void* ptrs[] = {p->featb, p->Ab, p->AbT, p->hf, p->share, p->dpqT, p->status};
    for (void* q : ptrs) if (q) cudaFree(q);
    delete p;
}

int mlp_grad_launch(MlpPlan* p, const GradArgs& g, const __nv_bfloat16* xb, const int* label,
                    int n_events, cudaStream_t st, int64_t* launches, std::string& err) {
    if (!p || n_events > p->maxev) { err = "MLP: too many events for the plan"; return RFAST_EINVAL; }
    k_mlp_gather<<<dim3(p->Fp / kKBlock, n_events), 256, 0, st>>>(g.ev, g.batch_idx, p->featb, p->Ab, p->AbT, p->rows, p->F, p->Fp);
    {
        const int R = p->H / kMTile;
        const dim3 gf(R, n_events), gb(p->H / 64, n_events);
#define RFAST_MID(CQ)                                                                                              \
    k_mlp_fwd<CQ><<<gf, kFwdThreads, kFwdSmem, st>>>(p->tmW1, p->tmA, g.ev, g.x, g.stride, p->hf, p->share, p->F, \
                                                     p->H, p->C, p->Fp / kKBlock, p->status);                      \
    k_mlp_back<CQ><<<gb, 256, 0, st>>>(g.ev, g.batch_idx, label, g.x, g.stride, p->hf, p->share, R, p->dpqT,      \
                                       g.gbuf, g.gplane, p->rows, p->F, p->H, p->C, g.l2)
        switch ((p->C + 3) / 4) {
            case 1: RFAST_MID(1); break;
            case 2: RFAST_MID(2); break;
            case 3: RFAST_MID(3); break;
            default: RFAST_MID(4); break;
        }
#undef RFAST_MID
    }
    k_mlp_dw1<<<dim3(p->H / kMTile, p->F / p->NT, n_events), kGemmThreads, kDw1Smem, st>>>(
        p->tmD, p->tmAT, p->tmX, p->tmG, g.ev, p->n, p->F, p->H, p->NT, g.l2, p->status);
    *launches += 4;
    return RFAST_OK;
}

void mlp_plan_clear_status(MlpPlan* p, cudaStream_t st) {
    if (p) cudaMemsetAsync(p->status, 0, sizeof(int), st);
}

// 0 when no bounded wait ran out so far (synchronises the stream)
int mlp_plan_status(MlpPlan* p, cudaStream_t st) {
    int h = 0;
    if (!p) return 0;
    if (cudaMemcpyAsync(&h, p->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return -1;
    if (cudaStreamSynchronize(st) != cudaSuccess) return -1;
    return h;
}

}  // namespace rfast
