// Helpers of the two-sided path: tiled out-of-place matrix transpose.
#include "harp_internal.h"

namespace {

constexpr int kTile = 64;

// dst[c][r] = src[r][c]; 64x64 tiles through padded shared memory, 256 threads.
template <typename T>
__global__ void __launch_bounds__(256)
transpose_kernel(const T *__restrict__ src, T *__restrict__ dst, int64_t rows, int64_t cols) {
    __shared__ T tile[kTile][kTile + 2];
    const int64_t r0 = (int64_t)blockIdx.y * kTile, c0 = (int64_t)blockIdx.x * kTile;
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;           // 64 x 4
    for (int i = ty; i < kTile; i += 4) {
        const int64_t r = r0 + i, c = c0 + tx;
        if (r < rows && c < cols) tile[i][tx] = src[r * cols + c];
    }
    __syncthreads();
    for (int i = ty; i < kTile; i += 4) {
        const int64_t c = c0 + i, r = r0 + tx;
        if (r < rows && c < cols) dst[c * rows + r] = tile[tx][i];
    }
}

}  // namespace

harp_status_t harp_transpose_matrix(const void *src, void *dst, int64_t rows, int64_t cols, harp_dtype_t dtype,
                                    cudaStream_t stream) {
    const int64_t gx = (cols + kTile - 1) / kTile, gy = (rows + kTile - 1) / kTile;
    if (gy > 65535 || gx > 0x7fffffffLL) return HARP_ERR_BAD_DIM;
    dim3 grid((unsigned)gx, (unsigned)gy);
    if (dtype == HARP_F32)
        transpose_kernel<float><<<grid, 256, 0, stream>>>((const float *)src, (float *)dst, rows, cols);
    else
        transpose_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>((const __nv_bfloat16 *)src, (__nv_bfloat16 *)dst, rows, cols);
    g_harp_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}
