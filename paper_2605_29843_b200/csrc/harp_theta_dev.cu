// Block kernels from stored parameters, on the device (Eq. 9-11; appendix "Int8 storage of HARP
// parameters"): B_c = Q(theta_c) G_b with Q the Givens rotation (b = 2) or the Cayley map
// (I + A)^{-1} (I - A) of the skew-symmetric A whose strict upper triangle is theta_c, from fp32
// values or from int8 values with one scale per block.  This is the step a deployment runs right
// before the apply path: parameters stay in their stored form (b(b-1)/2 bytes + one scale per
// block as int8) and the b x b kernels are rebuilt where they are used.
//
// One thread block per matrix block: [I + A | I - A] in shared memory in fp64, Gauss-Jordan
// elimination with partial pivoting, then the product with the mixer, one rounding to fp32.
#include <cmath>

#include "harp_internal.h"

namespace {

constexpr int kThetaThreads = 128;
constexpr int kThetaMaxB = 54;       // 2 * 54 * 54 doubles + the factor column fit the default 48 KB

__device__ __forceinline__ double mixer_entry(const float *mixer, int b, int i, int j) {
    if (mixer) return (double)mixer[i * b + j];
    // normalised Sylvester Hadamard matrix: (-1)^popcount(i & j) / sqrt(b)
    return ((__popc((unsigned)(i & j)) & 1) ? -1.0 : 1.0) * rsqrt((double)b);
}

__global__ void givens_kernel(int64_t n_blocks, const float *theta, const int8_t *theta_q, const float *scales,
                              const float *mixer, float *out) {
    const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= n_blocks) return;
    const double th = theta ? (double)theta[c] : (double)scales[c] * (double)theta_q[c];
    double sn, cs;
    sincos(th, &sn, &cs);
    const double q[4] = {cs, -sn, sn, cs};
    for (int i = 0; i < 2; ++i)
        for (int j = 0; j < 2; ++j)
            out[c * 4 + i * 2 + j] = (float)(q[i * 2] * mixer_entry(mixer, 2, 0, j) + q[i * 2 + 1] * mixer_entry(mixer, 2, 1, j));
}

__global__ void __launch_bounds__(kThetaThreads)
cayley_kernel(int b, const float *theta, const int8_t *theta_q, const float *scales, const float *mixer, float *out) {
    extern __shared__ double sm[];
    const int w = 2 * b;
    double *m = sm;                      // [b][2b] = [I + A | I - A]
    double *fcol = sm + (size_t)b * w;   // column of elimination factors
    __shared__ int piv_s;
    const int64_t c = blockIdx.x;
    const int np = b * (b - 1) / 2;
    const int tid = threadIdx.x;
    for (int idx = tid; idx < b * b; idx += kThetaThreads) {
        const int i = idx / b, j = idx - i * b;
        if (i == j) {
            m[i * w + i] = 1.0;
            m[i * w + b + i] = 1.0;
        } else if (i < j) {
            const int k = i * b - i * (i + 1) / 2 + (j - i - 1);
            const double a = theta ? (double)theta[c * np + k] : (double)scales[c] * (double)theta_q[c * np + k];
            m[i * w + j] = a;
            m[j * w + i] = -a;
            m[i * w + b + j] = -a;
            m[j * w + b + i] = a;
        }
    }
    __syncthreads();
    for (int col = 0; col < b; ++col) {
        if (tid < 32) {                  // pivot: largest magnitude in the column, rows col..b-1, lowest row on ties
            double best = -1.0;
            int row = col;
            for (int r = col + tid; r < b; r += 32) {
                const double v = fabs(m[r * w + col]);
                if (v > best) { best = v; row = r; }
            }
            for (int off = 16; off > 0; off >>= 1) {
                const double ob = __shfl_down_sync(0xffffffffu, best, off);
                const int orow = __shfl_down_sync(0xffffffffu, row, off);
                if (ob > best || (ob == best && orow < row)) { best = ob; row = orow; }
            }
            if (tid == 0) piv_s = row;
        }
        __syncthreads();
        const int piv = piv_s;
        if (piv != col)
            for (int j = tid; j < w; j += kThetaThreads) {
                const double t = m[piv * w + j];
                m[piv * w + j] = m[col * w + j];
                m[col * w + j] = t;
            }
        __syncthreads();
        const double inv = 1.0 / m[col * w + col];
        for (int r = tid; r < b; r += kThetaThreads) fcol[r] = m[r * w + col];
        __syncthreads();
        for (int j = col + tid; j < w; j += kThetaThreads) m[col * w + j] *= inv;
        __syncthreads();
        const int span = w - col;
        for (int idx = tid; idx < b * span; idx += kThetaThreads) {
            const int r = idx / span, j = col + (idx - r * span);
            if (r != col) m[r * w + j] -= fcol[r] * m[col * w + j];
        }
        __syncthreads();
    }
    // B = Q G, Q = right half of m
    for (int idx = tid; idx < b * b; idx += kThetaThreads) {
        const int i = idx / b, j = idx - i * b;
        double acc = 0.0;
        for (int k = 0; k < b; ++k) acc += m[i * w + b + k] * mixer_entry(mixer, b, k, j);
        out[c * (int64_t)b * b + idx] = (float)acc;
    }
}

}  // namespace

extern "C" int32_t harp_theta_device_max_radix(void) { return kThetaMaxB; }

extern "C" harp_status_t harp_blocks_from_theta_device(int32_t b, int64_t n_blocks, const float *theta,
                                                       const int8_t *theta_q, const float *scales, const float *mixer,
                                                       float *out_blocks, void *stream) {
    if (!out_blocks || (!theta && !theta_q) || (theta_q && !theta && !scales)) return HARP_ERR_NULL;
    if (b < 2 || n_blocks < 0) return HARP_ERR_BAD_SCHEDULE;
    if (b > kThetaMaxB) return HARP_ERR_UNSUPPORTED;
    if (!mixer && (b & (b - 1)) != 0) return HARP_ERR_NULL;     // no default mixer for a radix that is not a power of two
    if (n_blocks == 0) return HARP_OK;
    if (n_blocks > 0x7fffffffLL) return HARP_ERR_BAD_DIM;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (b == 2) {
        givens_kernel<<<(unsigned)((n_blocks + 255) / 256), 256, 0, s>>>(n_blocks, theta, theta_q, scales, mixer, out_blocks);
    } else {
        const size_t smem = ((size_t)b * 2 * b + (size_t)b) * sizeof(double);
        cayley_kernel<<<(unsigned)n_blocks, kThetaThreads, smem, s>>>(b, theta, theta_q, scales, mixer, out_blocks);
    }
    g_harp_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}
