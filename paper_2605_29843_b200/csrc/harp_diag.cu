// Diagnostics of a processed layer: weight incoherence (Eq. 4), off-block energy of the
// rotated curvature proxy (Eq. 15) and the diagonal Hessian-weighted reconstruction proxy
// (Eq. 14).  Each is one pass over a row-major matrix: a thread owns V neighbouring columns
// (one 16-byte vector where the layout allows it), walks down the rows of its CTA's row
// class and accumulates in fp64; CTAs combine with one atomic per quantity, and a one-thread
// kernel forms the final scalar.  Nothing is allocated: the caller's four doubles are the
// accumulators.
#include "harp_internal.h"

namespace {

constexpr int kThreads = 256;

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// V values of a row starting at column c (V * sizeof(T) == 16 and 16-byte aligned, or V == 1)
template <typename T, int V>
__device__ __forceinline__ void load_vec(const T *p, float (&out)[V]) {
    if (V == 1) {
        out[0] = to_f32<T>(p[0]);
    } else {
        const uint4 raw = *reinterpret_cast<const uint4 *>(p);
        const T *e = reinterpret_cast<const T *>(&raw);
#pragma unroll
        for (int v = 0; v < V; ++v) out[v] = to_f32<T>(e[v]);
    }
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
// CTA-wide sum (or max) of one double per thread, then one atomic into *dst by thread 0
__device__ void cta_accumulate(double v, double *dst, bool is_max) {
    __shared__ double part[kThreads / 32];
    __syncthreads();                         // part may still be read from the previous call
    v = is_max ? warp_max(v) : warp_sum(v);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        double r = part[0];
        for (int w = 1; w < kThreads / 32; ++w) r = is_max ? fmax(r, part[w]) : r + part[w];
        if (is_max) {
            // non-negative doubles order like their bit patterns
            atomicMax(reinterpret_cast<unsigned long long *>(dst), (unsigned long long)__double_as_longlong(r));
        } else {
            atomicAdd(dst, r);
        }
    }
}

// acc[1] = max |a|, acc[2] = sum a^2, acc[3] = sum of a^2 over the diagonal blocks (block > 0)
// BLOCKS: also sum the squares inside the diagonal blocks (off-block energy); without it the loop
// spends one conversion and one fp64 multiply-add per element (the maximum is taken in fp32,
// which is exact for fp32 and bf16 inputs) -- fp64 issue is what bounds this kernel.
template <typename T, int V, bool BLOCKS>
__global__ void __launch_bounds__(kThreads)
stats_kernel(const T *__restrict__ A, int64_t m, int64_t n, int64_t block, double *acc) {
    const int64_t c0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * V;
    float mxf = 0.f;
    double ss = 0.0, sd = 0.0;
    if (c0 < n) {
        int64_t lo[V];                                    // first row of the diagonal block of column c0 + v
#pragma unroll
        for (int v = 0; v < V; ++v) lo[v] = BLOCKS ? (c0 + v) / block * block : 0;
        // c0 is a multiple of V: when V divides the block size the thread's V columns share a block
        // and one comparison per row decides whether the row's partial sum is inside it
        const bool one_block = BLOCKS && block % V == 0;
#pragma unroll 4
        for (int64_t r = blockIdx.y; r < m; r += gridDim.y) {
            float a[V];
            load_vec<T, V>(A + r * n + c0, a);
            double row_ss = 0.0, row_sd = 0.0;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const double x = (double)a[v];
                mxf = fmaxf(mxf, fabsf(a[v]));
                row_ss += x * x;
                if (BLOCKS && !one_block && r >= lo[v] && r < lo[v] + block) row_sd += x * x;
            }
            ss += row_ss;
            if (BLOCKS) sd += one_block ? ((r >= lo[0] && r < lo[0] + block) ? row_ss : 0.0) : row_sd;
        }
    }
    cta_accumulate((double)mxf, acc + 1, true);
    cta_accumulate(ss, acc + 2, false);
    if (BLOCKS) cta_accumulate(sd, acc + 3, false);
}

// acc[1] = sum_ij (Wt_ij - Wq_ij)^2 |H_jj|, acc[2] = sum_j |H_jj| (added by the CTAs of row class 0 only)
template <typename T, typename TH, int V>
__global__ void __launch_bounds__(kThreads)
diag_error_kernel(const T *__restrict__ Wt, const T *__restrict__ Wq, int64_t d_out, int64_t d_in,
                  const TH *__restrict__ H, double *acc) {
    const int64_t c0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * V;
    double s = 0.0, wsum = 0.0;
    if (c0 < d_in) {
        double w[V];
#pragma unroll
        for (int v = 0; v < V; ++v) {
            w[v] = fabs((double)to_f32<TH>(H[(c0 + v) * d_in + (c0 + v)]));
            wsum += w[v];
        }
#pragma unroll 4
        for (int64_t r = blockIdx.y; r < d_out; r += gridDim.y) {
            float a[V], b[V];
            load_vec<T, V>(Wt + r * d_in + c0, a);
            load_vec<T, V>(Wq + r * d_in + c0, b);
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const double dlt = (double)a[v] - (double)b[v];
                s += dlt * dlt * w[v];
            }
        }
    }
    cta_accumulate(s, acc + 1, false);
    if (blockIdx.y == 0) cta_accumulate(wsum, acc + 2, false);
}

enum FinalKind { FINAL_INCOHERENCE, FINAL_OFFBLOCK, FINAL_DIAG_ERROR };
__global__ void finalize_kernel(double *acc, int kind, double m, double n) {
    if (kind == FINAL_INCOHERENCE) {
        acc[0] = acc[2] > 0.0 ? sqrt(m * n) * acc[1] / sqrt(acc[2]) : 0.0;       // Eq. 4
    } else if (kind == FINAL_OFFBLOCK) {
        acc[0] = (acc[2] - acc[3]) / (n * n);                                     // Eq. 15
    } else {
        // Eq. 14 with w-bar = w / mean(w): sum / (d_out * d_in * mean(w)) = sum / (d_out * sum_j w_j)
        acc[0] = acc[2] > 0.0 ? acc[1] / (m * acc[2]) : 0.0;
    }
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

dim3 grid_for(int64_t rows, int64_t cols, int V) {
    const int64_t gx = (cols + (int64_t)kThreads * V - 1) / ((int64_t)kThreads * V);
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int64_t gy = std::max<int64_t>(1, ((int64_t)sms * 8 + gx - 1) / gx);
    gy = std::min<int64_t>(std::min<int64_t>(gy, rows), 65535);
    return dim3((unsigned)gx, (unsigned)gy);
}

harp_status_t check_common(const void *A, int64_t m, int64_t n, harp_dtype_t dtype, double *out) {
    if (!A || !out) return HARP_ERR_NULL;
    if (m <= 0 || n <= 0 || m > (1ll << 31) || n > (1ll << 31)) return HARP_ERR_BAD_DIM;
    if (dtype != HARP_F32 && dtype != HARP_BF16) return HARP_ERR_BAD_DTYPE;
    if (reinterpret_cast<uintptr_t>(A) % harp_dtype_size(dtype) != 0 || reinterpret_cast<uintptr_t>(out) % 8 != 0)
        return HARP_ERR_BAD_DIM;
    return HARP_OK;
}

template <typename T, int V>
void launch_stats(bool vec, const T *A, int64_t m, int64_t n, int64_t block, double *out, cudaStream_t stream) {
    if (vec && block > 0) stats_kernel<T, V, true><<<grid_for(m, n, V), kThreads, 0, stream>>>(A, m, n, block, out);
    else if (vec) stats_kernel<T, V, false><<<grid_for(m, n, V), kThreads, 0, stream>>>(A, m, n, block, out);
    else if (block > 0) stats_kernel<T, 1, true><<<grid_for(m, n, 1), kThreads, 0, stream>>>(A, m, n, block, out);
    else stats_kernel<T, 1, false><<<grid_for(m, n, 1), kThreads, 0, stream>>>(A, m, n, block, out);
}

harp_status_t run_stats(const void *A, int64_t m, int64_t n, int64_t block, harp_dtype_t dtype, double *out,
                        int final_kind, cudaStream_t stream) {
    if (cudaMemsetAsync(out, 0, 4 * sizeof(double), stream) != cudaSuccess) return HARP_ERR_CUDA;
    const int V = dtype == HARP_F32 ? 4 : 8;
    const bool vec = aligned16(A) && n % V == 0;
    if (dtype == HARP_F32) {
        launch_stats<float, 4>(vec, (const float *)A, m, n, block, out, stream);
    } else {
        launch_stats<__nv_bfloat16, 8>(vec, (const __nv_bfloat16 *)A, m, n, block, out, stream);
    }
    finalize_kernel<<<1, 1, 0, stream>>>(out, final_kind, (double)m, (double)n);
    g_harp_launches.fetch_add(2, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}

template <typename T, int V>
void launch_diag_error(const void *Wt, const void *Wq, int64_t d_out, int64_t d_in, const void *H, harp_dtype_t h_dtype,
                       double *out, cudaStream_t stream) {
    const dim3 grid = grid_for(d_out, d_in, V);
    if (h_dtype == HARP_F32)
        diag_error_kernel<T, float, V><<<grid, kThreads, 0, stream>>>((const T *)Wt, (const T *)Wq, d_out, d_in, (const float *)H, out);
    else
        diag_error_kernel<T, __nv_bfloat16, V><<<grid, kThreads, 0, stream>>>((const T *)Wt, (const T *)Wq, d_out, d_in,
                                                                              (const __nv_bfloat16 *)H, out);
}

}  // namespace

extern "C" {

harp_status_t harp_weight_incoherence(const void *A, int64_t m, int64_t n, harp_dtype_t dtype, double *out, void *stream) {
    const harp_status_t st = check_common(A, m, n, dtype, out);
    if (st != HARP_OK) return st;
    return run_stats(A, m, n, 0, dtype, out, FINAL_INCOHERENCE, static_cast<cudaStream_t>(stream));
}

harp_status_t harp_offblock_energy(const void *H, int64_t n, int64_t block, harp_dtype_t dtype, double *out, void *stream) {
    const harp_status_t st = check_common(H, n, n, dtype, out);
    if (st != HARP_OK) return st;
    if (block <= 0 || block > n) return HARP_ERR_BAD_DIM;
    return run_stats(H, n, n, block, dtype, out, FINAL_OFFBLOCK, static_cast<cudaStream_t>(stream));
}

harp_status_t harp_diag_weighted_error(const void *Wt, const void *Wq, int64_t d_out, int64_t d_in, harp_dtype_t dtype,
                                       const void *H, harp_dtype_t h_dtype, double *out, void *stream) {
    harp_status_t st = check_common(Wt, d_out, d_in, dtype, out);
    if (st != HARP_OK) return st;
    st = check_common(Wq, d_out, d_in, dtype, out);
    if (st != HARP_OK) return st;
    st = check_common(H, d_in, d_in, h_dtype, out);
    if (st != HARP_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(out, 0, 4 * sizeof(double), s) != cudaSuccess) return HARP_ERR_CUDA;
    const int V = dtype == HARP_F32 ? 4 : 8;
    const bool vec = aligned16(Wt) && aligned16(Wq) && d_in % V == 0;
    if (dtype == HARP_F32) {
        if (vec) launch_diag_error<float, 4>(Wt, Wq, d_out, d_in, H, h_dtype, out, s);
        else launch_diag_error<float, 1>(Wt, Wq, d_out, d_in, H, h_dtype, out, s);
    } else {
        if (vec) launch_diag_error<__nv_bfloat16, 8>(Wt, Wq, d_out, d_in, H, h_dtype, out, s);
        else launch_diag_error<__nv_bfloat16, 1>(Wt, Wq, d_out, d_in, H, h_dtype, out, s);
    }
    finalize_kernel<<<1, 1, 0, s>>>(out, FINAL_DIAG_ERROR, (double)d_out, (double)d_in);
    g_harp_launches.fetch_add(2, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}

}  // extern "C"
