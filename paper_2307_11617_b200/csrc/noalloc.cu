// Full-shard least-squares gradient that allocates nothing (see rfast_ls_gradient_static in
// rfast.h).  The per-row residuals, which the handle-based path keeps in a cudaMalloc'ed
// buffer, live here in a fixed array inside the library image.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "rfast.h"

namespace {

constexpr int kMaxDevices = 64;

// Residual scratch: one float per shard row.  Lives in every GPU that loads the library until
// the process exits (RFAST_STATIC_MAX_ROWS * 4 bytes = 256 KiB per GPU).
static __device__ __align__(256) float g_residual_scratch[RFAST_STATIC_MAX_ROWS];

// Device address of the array, per device; filled on the first call made with that device current.
float*     g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// r_k = a_k . x - y_k, one warp per row.  grid = ceil(rows / 8), 256 threads
__global__ void __launch_bounds__(256)
k_static_residual(const float* __restrict__ feat, const float* __restrict__ target,
                  const float* __restrict__ x, float* __restrict__ res, int rows, int F) {
    const int k = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (k >= rows) return;
    const float* a = feat + (int64_t)k * F;
    float s = 0.f;
    for (int c = lane; c < F; c += 32) s = fmaf(a[c], x[c], s);
    s = warp_sum(s);
    if (lane == 0) res[k] = s - target[k];
}

// g_c = (1/rows) sum_k a_k[c] r_k + l2 x_c, rows in ascending order.  grid = ceil(F / 256)
__global__ void __launch_bounds__(256)
k_static_grad(const float* __restrict__ feat, const float* __restrict__ x,
              const float* __restrict__ res, float* __restrict__ grad, int rows, int F, float l2) {
    const int c = blockIdx.x * 256 + threadIdx.x;
    if (c >= F) return;
    float s = 0.f;
    for (int k = 0; k < rows; ++k) s = fmaf(feat[(int64_t)k * F + c], res[k], s);
    grad[c] = s / (float)rows + l2 * x[c];
}

int fail(char* err, size_t err_len, int code, const char* what, const char* detail = "") {
    if (err && err_len) std::snprintf(err, err_len, "%s%s", what, detail);
    return code;
}

}  // namespace

extern "C" int rfast_ls_gradient_static(const float* d_feat, const float* d_target, const float* d_x,
                                        float* d_grad, int32_t rows, int32_t n_features, float l2,
                                        void* cuda_stream, char* err, size_t err_len) {
    if (!d_feat || !d_target || !d_x || !d_grad)
        return fail(err, err_len, RFAST_EINVAL, "rfast_ls_gradient_static: null device pointer");
    if (rows <= 0 || n_features <= 0)
        return fail(err, err_len, RFAST_EINVAL, "rfast_ls_gradient_static: rows and n_features must be positive");
    if (rows > RFAST_STATIC_MAX_ROWS) {
        if (err && err_len)
            std::snprintf(err, err_len, "rfast_ls_gradient_static: %d rows exceed the built-in scratch of %d rows",
                          rows, RFAST_STATIC_MAX_ROWS);
        return RFAST_EINVAL;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(err, err_len, RFAST_ECUDA, "cudaGetDevice: ", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(err, err_len, RFAST_EINVAL, "rfast_ls_gradient_static: device index beyond the supported 64");
    float* scratch = nullptr;
    {
        // one-time set-up per device, with that device current: in host code the array's name
        // is only a stand-in, the kernels need the address the runtime reports for this device
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_addr[dev]) {
            float* ptr = nullptr;
            e = cudaGetSymbolAddress((void**)&ptr, g_residual_scratch);
            if (e != cudaSuccess || !ptr)
                return fail(err, err_len, RFAST_ECUDA, "cudaGetSymbolAddress: ", cudaGetErrorString(e));
            g_scratch_addr[dev] = ptr;
        }
        scratch = g_scratch_addr[dev];
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // the array keeps whatever the previous call left: start the used part from zero
    e = cudaMemsetAsync(scratch, 0, (size_t)rows * sizeof(float), st);
    if (e != cudaSuccess) return fail(err, err_len, RFAST_ECUDA, "cudaMemsetAsync: ", cudaGetErrorString(e));
    k_static_residual<<<(rows + 7) / 8, 256, 0, st>>>(d_feat, d_target, d_x, scratch, rows, n_features);
    k_static_grad<<<(n_features + 255) / 256, 256, 0, st>>>(d_feat, d_x, scratch, d_grad, rows, n_features, l2);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(err, err_len, RFAST_ECUDA, "kernel launch: ", cudaGetErrorString(e));
    return RFAST_OK;
}
