// Loss of Algorithm 3's parameter search when no model is at hand: how far a budgeted cache moves
// the attention outputs away from the dense cache's.  For rows o_i, ref_i (bf16 [rows, D]):
//     loss = mean_i ||o_i - ref_i||^2 / max(||ref_i||^2, 1e-30)
// Kernel 1: one warp per row, fp32 sums in a fixed lane order, one ratio per row.
// Kernel 2: a single CTA adds the ratios in double precision in a fixed order (deterministic).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "baklava.h"
#include "common.h"

namespace {

constexpr int kRowThreads = 256;          // eight rows per CTA
constexpr int kSumThreads = 1024;

__global__ void __launch_bounds__(kRowThreads) row_error_kernel(const __nv_bfloat16* __restrict__ out,
                                                                const __nv_bfloat16* __restrict__ ref,
                                                                int64_t rows, int D, float* __restrict__ ratio) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (kRowThreads / 32) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const __nv_bfloat162* a = reinterpret_cast<const __nv_bfloat162*>(out + row * D);
    const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(ref + row * D);
    float num = 0.0f, den = 0.0f;
    for (int i = lane; i < D / 2; i += 32) {
        const float2 x = __bfloat1622float2(a[i]), y = __bfloat1622float2(b[i]);
        const float d0 = x.x - y.x, d1 = x.y - y.y;
        num = fmaf(d0, d0, num); num = fmaf(d1, d1, num);
        den = fmaf(y.x, y.x, den); den = fmaf(y.y, y.y, den);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        num += __shfl_xor_sync(0xffffffffu, num, off);
        den += __shfl_xor_sync(0xffffffffu, den, off);
    }
    if (lane == 0) ratio[row] = num / fmaxf(den, 1e-30f);
}

__global__ void __launch_bounds__(kSumThreads) mean_ratio_kernel(const float* __restrict__ ratio, int64_t rows,
                                                                 double* __restrict__ loss) {
    __shared__ double part[kSumThreads];
    double acc = 0.0;
    for (int64_t i = threadIdx.x; i < rows; i += kSumThreads) acc += (double)ratio[i];
    part[threadIdx.x] = acc;
    __syncthreads();
    for (int s = kSumThreads / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) part[threadIdx.x] += part[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) loss[0] = rows > 0 ? part[0] / (double)rows : 0.0;
}

}  // namespace

extern "C" __attribute__((visibility("default"))) size_t baklava_output_error_workspace_size(int64_t rows) {
    return rows > 0 ? (size_t)rows * sizeof(float) : 0;
}

extern "C" __attribute__((visibility("default"))) int baklava_output_error(
        const void* out, const void* ref, int64_t rows, int32_t D, double* loss, void* ws, size_t ws_bytes,
        void* stream) {
    if (!loss || rows < 0 || (rows > 0 && (!out || !ref))) return BAKLAVA_ERR_INVALID_ARG;
    if (D <= 0 || (D & 1)) return BAKLAVA_ERR_SHAPE;
    if (((uintptr_t)out & 3u) || ((uintptr_t)ref & 3u) || ((uintptr_t)loss & 7u)) return BAKLAVA_ERR_INVALID_ARG;
    if (rows > 0 && (!ws || ((uintptr_t)ws & 3u))) return BAKLAVA_ERR_INVALID_ARG;
    if (ws_bytes < baklava_output_error_workspace_size(rows)) return BAKLAVA_ERR_WORKSPACE;
    const int64_t blocks = (rows + kRowThreads / 32 - 1) / (kRowThreads / 32);
    if (blocks > INT32_MAX) return BAKLAVA_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float* ratio = static_cast<float*>(ws);
    if (rows > 0) {
        row_error_kernel<<<(unsigned)blocks, kRowThreads, 0, s>>>(static_cast<const __nv_bfloat16*>(out),
                                                                  static_cast<const __nv_bfloat16*>(ref), rows, D, ratio);
        if (cudaGetLastError() != cudaSuccess) return BAKLAVA_ERR_CUDA;
    }
    mean_ratio_kernel<<<1, kSumThreads, 0, s>>>(ratio, rows, loss);
    return cudaGetLastError() == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
}
