// Gradient of a scalar loss with respect to the block kernels of a processor (what a fitting
// loop such as Algorithm 3 needs from the apply; the gradient with respect to the rows is the
// transpose apply and needs nothing new).
//
// Forward, rows as row vectors (Algorithm 1):  v_0[i] = s[perm[i]] x[perm[i]],  v_{t+1} = v_t M_t,
// y = v_m.  With G = dL/dy:   g_m = G,   g_t = g_{t+1} M_t^T,
//     dL/dK_t[c][i][j] = sum over rows of  v_t[base_c + i s_t] * g_{t+1}[base_c + j s_t].
//
// This first version favours clarity over speed: the rows are processed in chunks; for a chunk
// all forward states v_0..v_{m-1} are kept in global scratch (fp32), the gradient state is walked
// back stage by stage, and every entry of the result is owned by one thread that sums over the
// chunk's rows in fp64 in a fixed order -- no atomics, so the result does not depend on scheduling.
#include <algorithm>

#include "harp_internal.h"

namespace {

constexpr int kThreads = 256;

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// v0[r][i] = s[perm[i]] * x[r][perm[i]],  g[r][i] = gy[r][i]   (both fp32)
template <typename T>
__global__ void __launch_bounds__(kThreads)
load_kernel(const T *__restrict__ x, const T *__restrict__ gy, int64_t rows, int64_t d, const int32_t *__restrict__ perm,
            const int8_t *__restrict__ signs, float *__restrict__ v0, float *__restrict__ g) {
    const int64_t total = rows * d;
    for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < total; e += (int64_t)gridDim.x * kThreads) {
        const int64_t r = e / d, i = e - r * d;
        const int64_t src = perm ? perm[i] : i;
        const float sg = (signs && signs[src] < 0) ? -1.f : 1.f;
        v0[e] = sg * to_f32<T>(x[r * d + src]);
        g[e] = to_f32<T>(gy[e]);
    }
}

// one stage on a chunk: out[r][base + j s] = sum_i in[r][base + i s] * K[c][i][j]   (transpose: K[c][j][i])
__global__ void __launch_bounds__(kThreads)
stage_kernel(const float *__restrict__ in, float *__restrict__ out, int64_t rows, int64_t d, int b, int64_t s,
             const float *__restrict__ K, int transpose) {
    const int64_t total = rows * d;
    for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < total; e += (int64_t)gridDim.x * kThreads) {
        const int64_t r = e / d, pos = e - r * d;
        const int64_t alpha = pos / (b * s), rem = pos - alpha * b * s;
        const int64_t j = rem / s, beta = rem - j * s;
        const int64_t base = alpha * b * s + beta;
        const float *Kc = K + (alpha * s + beta) * b * b;
        const float *row = in + r * d + base;
        float acc = 0.f;
        for (int i = 0; i < b; ++i) acc = fmaf(row[(int64_t)i * s], Kc[transpose ? j * b + i : (int64_t)i * b + j], acc);
        out[e] = acc;
    }
}

// grad[c][i][j] (+)= sum_r v[r][base_c + i s] * g[r][base_c + j s].  A CTA owns 32 neighbouring
// entries (one per lane); its eight warps take the rows r = w, w + 8, ... and their partial sums
// are added in a fixed order, so the result does not depend on scheduling.
__global__ void __launch_bounds__(kThreads)
outer_kernel(const float *__restrict__ v, const float *__restrict__ g, int64_t rows, int64_t d, int b, int64_t s,
             float *__restrict__ grad, int accumulate) {
    __shared__ double part[kThreads / 32][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t total = d * b;                       // (d / b) blocks of b*b entries
    for (int64_t e0 = (int64_t)blockIdx.x * 32; e0 < total; e0 += (int64_t)gridDim.x * 32) {
        const int64_t e = e0 + lane;
        double acc = 0.0;
        if (e < total) {
            const int64_t c = e / (b * b), ij = e - c * b * b;
            const int64_t i = ij / b, j = ij - i * b;
            const int64_t alpha = c / s, beta = c - alpha * s;
            const int64_t base = alpha * b * s + beta;
            const float *pv = v + base + i * s, *pg = g + base + j * s;
            for (int64_t r = w; r < rows; r += kThreads / 32) acc += (double)pv[r * d] * (double)pg[r * d];
        }
        part[w][lane] = acc;
        __syncthreads();
        if (w == 0 && e < total) {
            double sum = part[0][lane];
            for (int k = 1; k < kThreads / 32; ++k) sum += part[k][lane];
            grad[e] = accumulate ? grad[e] + (float)sum : (float)sum;
        }
        __syncthreads();
    }
}

unsigned grid_for(int64_t work) {
    return (unsigned)std::max<int64_t>(1, std::min<int64_t>((work + kThreads - 1) / kThreads, 148 * 16));
}

}  // namespace

extern "C" int64_t harp_plan_n_params(const harp_plan_t *plan) { return plan ? plan->n_params : -1; }

extern "C" harp_status_t harp_grad_blocks(const harp_plan_t *plan, const void *x, const void *gy, int64_t n_rows,
                                          harp_dtype_t dtype, float *grad, int accumulate, void *stream) {
    if (!plan || !grad) return HARP_ERR_NULL;
    if (dtype != HARP_F32 && dtype != HARP_BF16) return HARP_ERR_BAD_DTYPE;
    if (n_rows < 0) return HARP_ERR_BAD_DIM;
    if (n_rows > 0 && (!x || !gy)) return HARP_ERR_NULL;
    const size_t es = harp_dtype_size(dtype);
    if (reinterpret_cast<uintptr_t>(x) % es || reinterpret_cast<uintptr_t>(gy) % es || reinterpret_cast<uintptr_t>(grad) % 4)
        return HARP_ERR_BAD_DIM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t d = plan->d;
    const int m = plan->st.m;
    if (n_rows == 0) {
        if (!accumulate && cudaMemsetAsync(grad, 0, sizeof(float) * (size_t)plan->n_params, st) != cudaSuccess) return HARP_ERR_CUDA;
        return HARP_OK;
    }
    // chunk of rows whose m forward states and one gradient state (+ one spare) fit ~256 MB
    const int64_t per_row = (int64_t)(m + 2) * d * (int64_t)sizeof(float);
    const int64_t chunk = std::max<int64_t>(1, std::min<int64_t>(n_rows, (256ll << 20) / per_row));
    float *scratch = nullptr;
    if (cudaMallocAsync(reinterpret_cast<void **>(&scratch), (size_t)(chunk * per_row), st) != cudaSuccess) {
        cudaGetLastError();
        return HARP_ERR_ALLOC;
    }
    const int64_t plane = chunk * d;                  // floats per state
    float *ga = scratch + (int64_t)m * plane, *gb = ga + plane;
    harp_status_t rc = HARP_OK;
    for (int64_t r0 = 0; r0 < n_rows && rc == HARP_OK; r0 += chunk) {
        const int64_t rows = std::min(chunk, n_rows - r0);
        const unsigned grid = grid_for(rows * d);
        if (dtype == HARP_F32)
            load_kernel<float><<<grid, kThreads, 0, st>>>((const float *)x + r0 * d, (const float *)gy + r0 * d, rows, d,
                                                          plan->d_perm, plan->d_signs, scratch, ga);
        else
            load_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>((const __nv_bfloat16 *)x + r0 * d, (const __nv_bfloat16 *)gy + r0 * d,
                                                                  rows, d, plan->d_perm, plan->d_signs, scratch, ga);
        // forward states v_1 .. v_{m-1} (v_t in plane t)
        for (int t = 0; t + 1 < m; ++t)
            stage_kernel<<<grid, kThreads, 0, st>>>(scratch + t * plane, scratch + (t + 1) * plane, rows, d, plan->st.b[t],
                                                    plan->st.s[t], plan->d_blocks + plan->st.off[t], 0);
        // backward: entry sums, then the gradient state one stage back
        float *g_cur = ga, *g_nxt = gb;
        for (int t = m - 1; t >= 0; --t) {
            outer_kernel<<<(unsigned)std::min<int64_t>((d * plan->st.b[t] + 31) / 32, 148 * 64), kThreads, 0, st>>>(scratch + t * plane, g_cur, rows, d, plan->st.b[t], plan->st.s[t],
                                                                      grad + plan->st.off[t], (accumulate || r0 > 0) ? 1 : 0);
            if (t > 0) {
                stage_kernel<<<grid, kThreads, 0, st>>>(g_cur, g_nxt, rows, d, plan->st.b[t], plan->st.s[t],
                                                        plan->d_blocks + plan->st.off[t], 1);
                std::swap(g_cur, g_nxt);
            }
        }
        g_harp_launches.fetch_add(1 + (m - 1) + m + (m - 1), std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) rc = HARP_ERR_CUDA;
    }
    cudaFreeAsync(scratch, st);
    return rc;
}
