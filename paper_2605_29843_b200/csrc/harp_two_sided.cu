// Helpers of the two-sided path: tiled out-of-place matrix transpose.
#include <mutex>

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

// ---------------------------------------------------------------------------
// Two-sided processing for callers that must not allocate.
//
// Some users of this library run where device allocation is off the table: inside a
// serving loop whose memory pool is fixed at start-up, under a memory budget owned by
// another framework, or in a process that has handed the whole device to an allocator
// the library cannot see.  For them the transposed copy of W that the column side needs
// lives in the fixed array below instead of in a buffer obtained at call time.  The
// array is part of the loaded module: every device that loads the library holds these
// 32 MiB until the process exits.
// ---------------------------------------------------------------------------
#define HARP_STATIC_SCRATCH_BYTES (32ll << 20)
static __device__ __align__(256) unsigned char g_two_sided_scratch[HARP_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
void *g_scratch_addr[kMaxDevices] = {};     // device address of the array, per device

// The array's name is only a host-side handle; the address a kernel may use has to be
// asked for, once per device, with that device current.
harp_status_t static_scratch_address(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HARP_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_two_sided_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return HARP_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return HARP_OK;
}
}  // namespace

extern "C" int64_t harp_two_sided_static_capacity_bytes(void) { return HARP_STATIC_SCRATCH_BYTES; }

extern "C" harp_status_t harp_apply_two_sided_static(void *W, harp_dtype_t dtype, const harp_plan_t *plan_out,
                                                     const harp_plan_t *plan_in, void *stream) {
    if (!W || !plan_out || !plan_in) return HARP_ERR_NULL;
    if (dtype != HARP_F32 && dtype != HARP_BF16) return HARP_ERR_BAD_DTYPE;
    if ((reinterpret_cast<uintptr_t>(W) & (harp_dtype_size(dtype) - 1)) != 0) return HARP_ERR_BAD_DIM;
    const int64_t d_out = plan_out->d, d_in = plan_in->d;
    if (d_out * d_in * (int64_t)harp_dtype_size(dtype) > HARP_STATIC_SCRATCH_BYTES) return HARP_ERR_TOO_LARGE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return HARP_ERR_CUDA;
    if (dev != plan_out->device || dev != plan_in->device) return HARP_ERR_DIM_MISMATCH;
    void *scratch = nullptr;
    harp_status_t st = static_scratch_address(&scratch);
    if (st != HARP_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Every byte of the scratch region that is read below is written first by the
    // transpose, so nothing needs clearing between calls.
    st = harp_apply(plan_in, W, d_out, dtype, 0, s);
    if (st == HARP_OK) st = harp_transpose_matrix(W, scratch, d_out, d_in, dtype, s);
    if (st == HARP_OK) st = harp_apply(plan_out, scratch, d_in, dtype, 0, s);
    if (st == HARP_OK) st = harp_transpose_matrix(scratch, W, d_in, d_out, dtype, s);
    return st;
}
