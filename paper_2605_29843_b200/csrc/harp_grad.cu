// Gradient of a scalar loss with respect to the block kernels of a processor (what a fitting
// loop such as Algorithm 3 needs from the apply; the gradient with respect to the rows is the
// transpose apply and needs nothing new).
//
// Forward, rows as row vectors (Algorithm 1):  v_0[i] = s[perm[i]] x[perm[i]],  v_{t+1} = v_t M_t,
// y = v_m.  With G = dL/dy:   g_m = G,   g_t = g_{t+1} M_t^T,
//     dL/dK_t[c][i][j] = sum over rows of  v_t[base_c + i s_t] * g_{t+1}[base_c + j s_t].
//
// The rows are processed in chunks; for a chunk all forward states v_0..v_{m-1} are kept in global
// scratch (fp32) and the gradient state is walked back stage by stage.  Every sum over rows is
// taken in fp64 in a fixed order -- no atomics, so the result does not depend on scheduling.
//
// Stages of radix 2 to 8 run in "block owner" kernels: a thread owns one block c of the stage,
// keeps K_t[c] in registers and walks the rows of its slice of the chunk, so neighbouring lanes
// read neighbouring coordinates (or one vector when s_t = 1) and K is read once.  The backward
// kernel of such a stage does both jobs in one sweep over v_t and g_{t+1}: it writes g_t and adds
// v_t[i] g_{t+1}[j] into its B x B fp64 accumulators; the per-slice sums are then added slice by
// slice.  Other radices use the plain one-thread-per-element kernels below them.
#include <algorithm>
#include <map>
#include <mutex>

#include "harp_internal.h"

namespace {

constexpr int kThreads = 256;

// The kernels of one call form a chain, each reading what the one before wrote, and most last
// 5-30 us; they are launched with the programmatic stream-serialisation attribute so that the
// launch of the next one overlaps the tail of the current one.  Each kernel calls
// prior_kernel_done() before it touches anything a kernel before it wrote (griddepcontrol.wait
// returns when that kernel has completed and its writes are visible), and only then lets the
// kernel after it start, so at most one later kernel is resident early.
__device__ __forceinline__ void prior_kernel_done() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
void launch_dep(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);     // errors are read with cudaGetLastError by the caller
}

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

constexpr int kOwnThreads = 128;   // block-owner kernels: blocks per CTA
constexpr int kFwdSliceRows = 8;   //                      rows per CTA, forward
constexpr int kBwdSliceRows = 32;  //                      rows per CTA (one set of partial sums), backward
constexpr int kRowBatch = 4;       //                      rows whose loads are issued together

template <int B> __device__ __forceinline__ void load_block(const float *p, int64_t s, float (&v)[B]) {
    if (s == 1 && (B == 2 || B % 4 == 0)) {
        if constexpr (B == 2) {
            const float2 a = *reinterpret_cast<const float2 *>(p);
            v[0] = a.x; v[1] = a.y;
        } else {
#pragma unroll
            for (int q = 0; q < B / 4; ++q) {
                const float4 a = reinterpret_cast<const float4 *>(p)[q];
                v[4 * q] = a.x; v[4 * q + 1] = a.y; v[4 * q + 2] = a.z; v[4 * q + 3] = a.w;
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < B; ++i) v[i] = p[(int64_t)i * s];
    }
}

template <int B> __device__ __forceinline__ void store_block(float *p, int64_t s, const float (&v)[B]) {
    if (s == 1 && (B == 2 || B % 4 == 0)) {
        if constexpr (B == 2) {
            *reinterpret_cast<float2 *>(p) = make_float2(v[0], v[1]);
        } else {
#pragma unroll
            for (int q = 0; q < B / 4; ++q)
                reinterpret_cast<float4 *>(p)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < B; ++i) p[(int64_t)i * s] = v[i];
    }
}

// forward stage, block owner: out[r][base_c + j s] = sum_i in[r][base_c + i s] K[c][i][j]
template <int B>
__global__ void __launch_bounds__(kOwnThreads)
fwd_owner_kernel(const float *__restrict__ in, float *__restrict__ out, int64_t rows, int64_t d, int64_t s,
                 const float *__restrict__ K) {
    const int64_t c = (int64_t)blockIdx.x * kOwnThreads + threadIdx.x;
    if (c >= d / B) return;
    float k[B][B];
#pragma unroll
    for (int i = 0; i < B; ++i)
#pragma unroll
        for (int j = 0; j < B; ++j) k[i][j] = K[c * (B * B) + i * B + j];
    prior_kernel_done();
    const int64_t alpha = c / s, base = alpha * B * s + (c - alpha * s);
    const int64_t r0 = (int64_t)blockIdx.y * kFwdSliceRows, r1 = min(rows, r0 + kFwdSliceRows);
    for (int64_t r = r0; r < r1; r += kRowBatch) {
        float v[kRowBatch][B];
#pragma unroll
        for (int u = 0; u < kRowBatch; ++u)
            if (r + u < r1) load_block<B>(in + (r + u) * d + base, s, v[u]);
#pragma unroll
        for (int u = 0; u < kRowBatch; ++u) {
            if (r + u >= r1) break;
            float o[B];
#pragma unroll
            for (int j = 0; j < B; ++j) {
                float acc = 0.f;
#pragma unroll
                for (int i = 0; i < B; ++i) acc = fmaf(v[u][i], k[i][j], acc);
                o[j] = acc;
            }
            store_block<B>(out + (r + u) * d + base, s, o);
        }
    }
}

// backward stage, block owner: g_out[r][base_c + i s] = sum_j g[r][base_c + j s] K[c][i][j] (when
// g_out is given) and part[slice][i B + j][c] = sum over the slice's rows of v[..i..] g[..j..].
template <int B>
__global__ void __launch_bounds__(kOwnThreads)
bwd_owner_kernel(const float *__restrict__ v, const float *__restrict__ g, float *__restrict__ g_out, int64_t rows,
                 int64_t d, int64_t s, const float *__restrict__ K, double *__restrict__ part) {
    const int64_t nblk = d / B;
    const int64_t c = (int64_t)blockIdx.x * kOwnThreads + threadIdx.x;
    if (c >= nblk) return;
    float k[B][B];
    double acc[B][B];
#pragma unroll
    for (int i = 0; i < B; ++i)
#pragma unroll
        for (int j = 0; j < B; ++j) {
            k[i][j] = K[c * (B * B) + i * B + j];
            acc[i][j] = 0.0;
        }
    prior_kernel_done();
    const int64_t alpha = c / s, base = alpha * B * s + (c - alpha * s);
    constexpr int U = B >= 7 ? 2 : kRowBatch;         // radices 7 and 8 already fill the register file
    const int64_t r0 = (int64_t)blockIdx.y * kBwdSliceRows, r1 = min(rows, r0 + kBwdSliceRows);
    for (int64_t r = r0; r < r1; r += U) {
        float vv[U][B], gg[U][B];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (r + u < r1) {
                load_block<B>(v + (r + u) * d + base, s, vv[u]);
                load_block<B>(g + (r + u) * d + base, s, gg[u]);
            }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (r + u >= r1) break;
#pragma unroll
            for (int i = 0; i < B; ++i)
#pragma unroll
                for (int j = 0; j < B; ++j) acc[i][j] += (double)vv[u][i] * (double)gg[u][j];
            if (g_out) {
                float o[B];
#pragma unroll
                for (int i = 0; i < B; ++i) {
                    float a = 0.f;
#pragma unroll
                    for (int j = 0; j < B; ++j) a = fmaf(gg[u][j], k[i][j], a);
                    o[i] = a;
                }
                store_block<B>(g_out + (r + u) * d + base, s, o);
            }
        }
    }
    double *dst = part + (int64_t)blockIdx.y * (B * B) * nblk + c;
#pragma unroll
    for (int i = 0; i < B; ++i)
#pragma unroll
        for (int j = 0; j < B; ++j) dst[(int64_t)(i * B + j) * nblk] = acc[i][j];
}

// Radix 16: a block kernel does not fit one thread's registers, so a thread owns block c and four
// of its sixteen outputs (forward: columns j0..j0+3 of K[c]; backward: rows i0..i0+3, i.e. the
// transposed product), with the four threads of a block in the same CTA so that they share the
// sixteen inputs through L1.
constexpr int kTileRows16 = 32;    // rows per CTA of the radix-16 kernels (one set of partial sums)

__global__ void __launch_bounds__(128)
stage16_kernel(const float *__restrict__ in, float *__restrict__ out, int64_t rows, int64_t d, int64_t s,
               const float *__restrict__ K, int transpose) {
    const int64_t c = (int64_t)blockIdx.x * 32 + (threadIdx.x & 31);
    const int t0 = 4 * (threadIdx.x >> 5);
    if (c >= d / 16) return;
    float k[16][4];
#pragma unroll
    for (int q = 0; q < 16; ++q)
#pragma unroll
        for (int t = 0; t < 4; ++t) k[q][t] = K[c * 256 + (transpose ? (t0 + t) * 16 + q : q * 16 + t0 + t)];
    prior_kernel_done();
    const int64_t alpha = c / s, base = alpha * 16 * s + (c - alpha * s);
    const int64_t r0 = (int64_t)blockIdx.y * kFwdSliceRows, r1 = min(rows, r0 + kFwdSliceRows);
#pragma unroll 2
    for (int64_t r = r0; r < r1; ++r) {
        float v[16];
        load_block<16>(in + r * d + base, s, v);
        float o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int q = 0; q < 16; ++q)
#pragma unroll
            for (int t = 0; t < 4; ++t) o[t] = fmaf(v[q], k[q][t], o[t]);
        float *dst = out + r * d + base + (int64_t)t0 * s;
        if (s == 1) {
            *reinterpret_cast<float4 *>(dst) = make_float4(o[0], o[1], o[2], o[3]);
        } else {
#pragma unroll
            for (int t = 0; t < 4; ++t) dst[(int64_t)t * s] = o[t];
        }
    }
}

// part[slice][i 16 + j][c] = sum over the slice's rows of v[base_c + i s] g[base_c + j s]; a thread
// owns block c and a 4 x 4 tile of (i, j); the sixteen tiles of a block sit in the same CTA.
__global__ void __launch_bounds__(512)
outer16_kernel(const float *__restrict__ v, const float *__restrict__ g, int64_t rows, int64_t d, int64_t s,
               double *__restrict__ part) {
    const int64_t nblk = d / 16;
    const int64_t c = (int64_t)blockIdx.x * 32 + (threadIdx.x & 31);
    const int tile = threadIdx.x >> 5, i0 = 4 * (tile >> 2), j0 = 4 * (tile & 3);
    if (c >= nblk) return;
    double acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
    prior_kernel_done();
    const int64_t alpha = c / s, base = alpha * 16 * s + (c - alpha * s);
    const int64_t r0 = (int64_t)blockIdx.y * kTileRows16, r1 = min(rows, r0 + kTileRows16);
    for (int64_t r = r0; r < r1; r += 2) {
        float vv[2][4], gg[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u)
            if (r + u < r1) {
                load_block<4>(v + (r + u) * d + base + (int64_t)i0 * s, s, vv[u]);
                load_block<4>(g + (r + u) * d + base + (int64_t)j0 * s, s, gg[u]);
            }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (r + u >= r1) break;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] += (double)vv[u][i] * (double)gg[u][j];
        }
    }
    double *dst = part + (int64_t)blockIdx.y * 256 * nblk + c;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[(int64_t)((i0 + i) * 16 + j0 + j) * nblk] = acc[i][j];
}

// grad[c][i][j] (+)= sum over slices of part[slice][i b + j][c].  A CTA owns 32 neighbouring
// entries (one per lane); warp w adds the slices w, w + 8, ... and the eight sums are added in
// the order of w, so the result does not depend on scheduling.
__global__ void __launch_bounds__(kThreads)
reduce_slices_kernel(const double *__restrict__ part, int64_t n_slices, int64_t nblk, int bb, float *__restrict__ grad,
                     int accumulate) {
    prior_kernel_done();
    __shared__ double warp_sum[kThreads / 32][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t total = nblk * bb;
    for (int64_t q0 = (int64_t)blockIdx.x * 32; q0 < total; q0 += (int64_t)gridDim.x * 32) {
        const int64_t q = q0 + lane;
        double sum = 0.0;
        if (q < total) {
#pragma unroll 4
            for (int64_t sl = w; sl < n_slices; sl += kThreads / 32) sum += part[sl * total + q];
        }
        warp_sum[w][lane] = sum;
        __syncthreads();
        if (w == 0 && q < total) {
            double all = warp_sum[0][lane];
            for (int k = 1; k < kThreads / 32; ++k) all += warp_sum[k][lane];
            const int64_t ij = q / nblk, c = q - ij * nblk;
            float *dst = grad + c * bb + ij;
            *dst = accumulate ? *dst + (float)all : (float)all;
        }
        __syncthreads();
    }
}

// position of element i in the staged row of load_rows_kernel: two elements of padding per 64,
// so that a digit-reversal gather (strides of 64 elements and more) spreads over the banks
__device__ __forceinline__ int64_t staged_pos(int64_t i) { return i + 2 * (i >> 6); }

// as load_kernel, one CTA per row: the row of x is read in order into shared memory and gathered
// from there, so the permutation costs no scattered global reads
template <typename T>
__global__ void __launch_bounds__(kThreads)
load_rows_kernel(const T *__restrict__ x, const T *__restrict__ gy, int64_t rows, int64_t d, const int32_t *__restrict__ perm,
                 const int8_t *__restrict__ signs, float *__restrict__ v0, float *__restrict__ g) {
    prior_kernel_done();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T *row = reinterpret_cast<T *>(smem_raw);
    constexpr int V = 16 / (int)sizeof(T);                 // elements per 16-byte access
    // 16-byte accesses when every row starts on a 16-byte boundary; V divides 64, so the V elements
    // of one access stay next to each other in the staged row
    const bool vec = d % V == 0 && ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(gy)) & 15) == 0;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        if (vec) {
            for (int64_t i = (int64_t)threadIdx.x * V; i < d; i += (int64_t)kThreads * V) {
                const uint4 raw = *reinterpret_cast<const uint4 *>(x + r * d + i);
                const uint32_t *w = reinterpret_cast<const uint32_t *>(&raw);
                uint32_t *dst = reinterpret_cast<uint32_t *>(row + staged_pos(i));   // 4-byte aligned: staged_pos(i) is even
#pragma unroll
                for (int k = 0; k < 4; ++k) dst[k] = w[k];
                const uint4 rg = *reinterpret_cast<const uint4 *>(gy + r * d + i);
                const T *tg = reinterpret_cast<const T *>(&rg);
                float *gd = g + r * d + i;
#pragma unroll
                for (int k = 0; k < V; k += 4)
                    *reinterpret_cast<float4 *>(gd + k) =
                        make_float4(to_f32<T>(tg[k]), to_f32<T>(tg[k + 1]), to_f32<T>(tg[k + 2]), to_f32<T>(tg[k + 3]));
            }
        } else {
            for (int64_t i = threadIdx.x; i < d; i += kThreads) {
                row[staged_pos(i)] = x[r * d + i];
                g[r * d + i] = to_f32<T>(gy[r * d + i]);
            }
        }
        __syncthreads();
        if (d % 4 == 0) {
            for (int64_t i = (int64_t)threadIdx.x * 4; i < d; i += (int64_t)kThreads * 4) {
                const int4 src = *reinterpret_cast<const int4 *>(perm + i);
                const int sidx[4] = {src.x, src.y, src.z, src.w};
                float o[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float sg = (signs && signs[sidx[k]] < 0) ? -1.f : 1.f;
                    o[k] = sg * to_f32<T>(row[staged_pos(sidx[k])]);
                }
                *reinterpret_cast<float4 *>(v0 + r * d + i) = make_float4(o[0], o[1], o[2], o[3]);
            }
        } else {
            for (int64_t i = threadIdx.x; i < d; i += kThreads) {
                const int64_t src = perm[i];
                const float sg = (signs && signs[src] < 0) ? -1.f : 1.f;
                v0[r * d + i] = sg * to_f32<T>(row[staged_pos(src)]);
            }
        }
        __syncthreads();
    }
}

// v0[r][i] = s[perm[i]] * x[r][perm[i]],  g[r][i] = gy[r][i]   (both fp32)
template <typename T>
__global__ void __launch_bounds__(kThreads)
load_kernel(const T *__restrict__ x, const T *__restrict__ gy, int64_t rows, int64_t d, const int32_t *__restrict__ perm,
            const int8_t *__restrict__ signs, float *__restrict__ v0, float *__restrict__ g) {
    prior_kernel_done();
    // a thread keeps its coordinate and walks over rows (blockIdx.y, then in steps of gridDim.y)
    const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (i >= d) return;
    const int64_t src = perm ? perm[i] : i;
    const float sg = (signs && signs[src] < 0) ? -1.f : 1.f;
    for (int64_t r = blockIdx.y; r < rows; r += gridDim.y) {
        v0[r * d + i] = sg * to_f32<T>(x[r * d + src]);
        g[r * d + i] = to_f32<T>(gy[r * d + i]);
    }
}

// one stage on a chunk: out[r][base + j s] = sum_i in[r][base + i s] * K[c][i][j]   (transpose: K[c][j][i]).
// Neighbouring lanes hold neighbouring positions: inside one block when s is small, in neighbouring
// blocks otherwise -- so K is read block-major (entry k of block c at c b^2 + k) for s < 8 and
// element-major (at k D + c) from s = 8 on; kc_step / kk_step are the two strides of that choice.
__global__ void __launch_bounds__(kThreads)
stage_kernel(const float *__restrict__ in, float *__restrict__ out, int64_t rows, int64_t d, int b, int64_t s,
             const float *__restrict__ K, int64_t kc_step, int64_t kk_step, int transpose) {
    prior_kernel_done();
    // a thread keeps its position (the index arithmetic is done once) and walks over rows
    const int64_t pos = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (pos >= d) return;
    const int64_t alpha = pos / (b * s), rem = pos - alpha * b * s;
    const int64_t j = rem / s, beta = rem - j * s;
    const int64_t base = alpha * b * s + beta;
    const float *Kc = K + (alpha * s + beta) * kc_step + (transpose ? j * b : j) * kk_step;
    const int64_t k_step = (transpose ? 1 : (int64_t)b) * kk_step;     // from K[..][i][j] to K[..][i+1][j] (or [j][i+1])
    for (int64_t r = blockIdx.y; r < rows; r += gridDim.y) {
        const float *row = in + r * d + base;
        float acc = 0.f;
        for (int i = 0; i < b; ++i) acc = fmaf(row[(int64_t)i * s], Kc[(int64_t)i * k_step], acc);
        out[r * d + pos] = acc;
    }
}

// grad[c][i][j] (+)= sum_r v[r][base_c + i s] * g[r][base_c + j s].  A CTA owns 32 neighbouring
// entries (one per lane); its eight warps take the rows r = w, w + 8, ... and their partial sums
// are added in a fixed order, so the result does not depend on scheduling.
// The 32 entries are neighbours within a block for s < 8 and the same entry of 32 neighbouring
// blocks from s = 8 on (by_block = 0), so that the lanes read neighbouring coordinates either way.
__global__ void __launch_bounds__(kThreads)
outer_kernel(const float *__restrict__ v, const float *__restrict__ g, int64_t rows, int64_t d, int b, int64_t s,
             float *__restrict__ grad, int accumulate, int by_block) {
    prior_kernel_done();
    __shared__ double part[kThreads / 32][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t total = d * b;                       // (d / b) blocks of b*b entries
    const int64_t nblk = d / b;
    for (int64_t e0 = (int64_t)blockIdx.x * 32; e0 < total; e0 += (int64_t)gridDim.x * 32) {
        const int64_t q = e0 + lane;
        int64_t e = q;
        double acc = 0.0;
        if (q < total) {
            const int64_t c = by_block ? q / (b * b) : q % nblk, ij = by_block ? q - c * b * b : q / nblk;
            e = c * b * b + ij;
            const int64_t i = ij / b, j = ij - i * b;
            const int64_t alpha = c / s, beta = c - alpha * s;
            const int64_t base = alpha * b * s + beta;
            const float *pv = v + base + i * s, *pg = g + base + j * s;
            for (int64_t r = w; r < rows; r += kThreads / 32) acc += (double)pv[r * d] * (double)pg[r * d];
        }
        part[w][lane] = acc;
        __syncthreads();
        if (w == 0 && q < total) {
            double sum = part[0][lane];
            for (int k = 1; k < kThreads / 32; ++k) sum += part[k][lane];
            grad[e] = accumulate ? grad[e] + (float)sum : (float)sum;
        }
        __syncthreads();
    }
}

// Scratch comes from a memory pool of the library's own (one per device, created on first use)
// whose release threshold is unlimited: the default pool hands its memory back at every
// synchronisation, and mapping 256 MB anew costs more than the kernels of a call.  Returns null
// if the pool cannot be created; the caller then allocates from the device's default pool.
cudaMemPool_t scratch_pool(int device) {
    static std::mutex mu;
    static std::map<int, cudaMemPool_t> pools;
    std::lock_guard<std::mutex> lock(mu);
    auto it = pools.find(device);
    if (it != pools.end()) return it->second;
    cudaMemPoolProps props = {};
    props.allocType = cudaMemAllocationTypePinned;
    props.handleTypes = cudaMemHandleTypeNone;
    props.location.type = cudaMemLocationTypeDevice;
    props.location.id = device;
    cudaMemPool_t pool = nullptr;
    if (cudaMemPoolCreate(&pool, &props) != cudaSuccess) {
        cudaGetLastError();
        pool = nullptr;
    } else {
        uint64_t keep = ~0ull;
        cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
    }
    pools[device] = pool;
    return pool;
}

// grid of the kernels in which a thread keeps its coordinate and walks over rows
dim3 column_grid(int64_t d, int64_t rows) {
    const int64_t gx = (d + kThreads - 1) / kThreads;
    const int64_t gy = std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(rows, 65535), (148 * 16 + gx - 1) / gx));
    return dim3((unsigned)gx, (unsigned)gy);
}

bool owner_radix(int b) { return b >= 2 && b <= 8; }

dim3 owner_grid16(int64_t d, int64_t rows, int slice_rows) {
    return dim3((unsigned)((d / 16 + 31) / 32), (unsigned)((rows + slice_rows - 1) / slice_rows));
}

dim3 owner_grid(int64_t d, int b, int64_t rows, int slice_rows) {
    return dim3((unsigned)((d / b + kOwnThreads - 1) / kOwnThreads), (unsigned)((rows + slice_rows - 1) / slice_rows));
}

void launch_fwd_owner(int b, const float *in, float *out, int64_t rows, int64_t d, int64_t s, const float *K, cudaStream_t st) {
    const dim3 grid = owner_grid(d, b, rows, kFwdSliceRows);
    switch (b) {
        case 2: launch_dep(fwd_owner_kernel<2>, dim3(grid), dim3(kOwnThreads), 0, st, in, out, rows, d, s, K); break;
        case 3: launch_dep(fwd_owner_kernel<3>, dim3(grid), dim3(kOwnThreads), 0, st, in, out, rows, d, s, K); break;
        case 4: launch_dep(fwd_owner_kernel<4>, dim3(grid), dim3(kOwnThreads), 0, st, in, out, rows, d, s, K); break;
        case 5: launch_dep(fwd_owner_kernel<5>, dim3(grid), dim3(kOwnThreads), 0, st, in, out, rows, d, s, K); break;
        case 6: launch_dep(fwd_owner_kernel<6>, dim3(grid), dim3(kOwnThreads), 0, st, in, out, rows, d, s, K); break;
        case 7: launch_dep(fwd_owner_kernel<7>, dim3(grid), dim3(kOwnThreads), 0, st, in, out, rows, d, s, K); break;
        default: launch_dep(fwd_owner_kernel<8>, dim3(grid), dim3(kOwnThreads), 0, st, in, out, rows, d, s, K); break;
    }
}

void launch_bwd_owner(int b, const float *v, const float *g, float *g_out, int64_t rows, int64_t d, int64_t s, const float *K,
                      double *part, cudaStream_t st) {
    const dim3 grid = owner_grid(d, b, rows, kBwdSliceRows);
    switch (b) {
        case 2: launch_dep(bwd_owner_kernel<2>, dim3(grid), dim3(kOwnThreads), 0, st, v, g, g_out, rows, d, s, K, part); break;
        case 3: launch_dep(bwd_owner_kernel<3>, dim3(grid), dim3(kOwnThreads), 0, st, v, g, g_out, rows, d, s, K, part); break;
        case 4: launch_dep(bwd_owner_kernel<4>, dim3(grid), dim3(kOwnThreads), 0, st, v, g, g_out, rows, d, s, K, part); break;
        case 5: launch_dep(bwd_owner_kernel<5>, dim3(grid), dim3(kOwnThreads), 0, st, v, g, g_out, rows, d, s, K, part); break;
        case 6: launch_dep(bwd_owner_kernel<6>, dim3(grid), dim3(kOwnThreads), 0, st, v, g, g_out, rows, d, s, K, part); break;
        case 7: launch_dep(bwd_owner_kernel<7>, dim3(grid), dim3(kOwnThreads), 0, st, v, g, g_out, rows, d, s, K, part); break;
        default: launch_dep(bwd_owner_kernel<8>, dim3(grid), dim3(kOwnThreads), 0, st, v, g, g_out, rows, d, s, K, part); break;
    }
}

template <typename T>
void launch_load(const T *x, const T *gy, int64_t rows, int64_t d, const harp_plan_t *plan, float *v0, float *g, cudaStream_t st) {
    const size_t smem = (size_t)(d + 2 * (d >> 6) + 2) * sizeof(T);
    // per call: the attribute belongs to the current device's copy of the kernel
    const bool big_ok = smem > 48 * 1024 &&
        cudaFuncSetAttribute(load_rows_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) == cudaSuccess;
    if (plan->d_perm && (smem <= 48 * 1024 || (big_ok && smem <= 200 * 1024)))
        launch_dep(load_rows_kernel<T>, dim3((unsigned)std::min<int64_t>(rows, 148 * 8)), dim3(kThreads), smem, st, x, gy, rows, d,
                   plan->d_perm, plan->d_signs, v0, g);
    else
        launch_dep(load_kernel<T>, column_grid(d, rows), dim3(kThreads), 0, st, x, gy, rows, d, plan->d_perm, plan->d_signs, v0, g);
}

}  // namespace

extern "C" int64_t harp_plan_n_params(const harp_plan_t *plan) { return plan ? plan->n_params : -1; }

extern "C" harp_status_t harp_grad_blocks(const harp_plan_t *plan, const void *x, const void *gy, int64_t n_rows,
                                          harp_dtype_t dtype, float *grad, int accumulate, void *stream) {
    if (!plan || !grad) return HARP_ERR_NULL;
    if (dtype != HARP_F32 && dtype != HARP_BF16) return HARP_ERR_BAD_DTYPE;
    {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) return HARP_ERR_CUDA;
        if (dev != plan->device) return HARP_ERR_DIM_MISMATCH;      // the scratch pool and the plan's tables live on plan->device
    }
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
    // chunk of rows whose m forward states, two gradient states and the per-slice sums of the
    // block-owner stages (at most one state: 8 bytes x d b / 32 per row, b <= 16) fit ~256 MB
    const int64_t per_row = (int64_t)(m + 3) * d * (int64_t)sizeof(float);
    const int64_t chunk = std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(n_rows, 1 << 18), (256ll << 20) / per_row));
    int64_t part_bytes = 0;                          // per-slice sums of the stage that needs most
    for (int t = 0; t < m; ++t) {
        const int b = plan->st.b[t];
        const int slice = owner_radix(b) ? kBwdSliceRows : (b == 16 ? kTileRows16 : 0);
        if (slice) part_bytes = std::max<int64_t>(part_bytes, ((chunk + slice - 1) / slice) * d * b * (int64_t)sizeof(double));
    }
    const int64_t state_bytes = (int64_t)(m + 2) * chunk * d * (int64_t)sizeof(float);
    float *scratch = nullptr;
    const size_t scratch_bytes = (size_t)(state_bytes + 256 + part_bytes);
    cudaMemPool_t pool = scratch_pool(plan->device);
    const cudaError_t alloc_err = pool ? cudaMallocFromPoolAsync(reinterpret_cast<void **>(&scratch), scratch_bytes, pool, st)
                                       : cudaMallocAsync(reinterpret_cast<void **>(&scratch), scratch_bytes, st);
    if (alloc_err != cudaSuccess) {
        cudaGetLastError();
        return HARP_ERR_ALLOC;
    }
    const int64_t plane = chunk * d;                  // floats per state
    float *ga = scratch + (int64_t)m * plane, *gb = ga + plane;
    // fp64 per-slice sums of the block-owner stages, behind the states, on the next 256-byte boundary
    double *part = reinterpret_cast<double *>((reinterpret_cast<uintptr_t>(gb + plane) + 255) & ~(uintptr_t)255);
    harp_status_t rc = HARP_OK;
    for (int64_t r0 = 0; r0 < n_rows && rc == HARP_OK; r0 += chunk) {
        const int64_t rows = std::min(chunk, n_rows - r0);
        if (dtype == HARP_F32)
            launch_load<float>((const float *)x + r0 * d, (const float *)gy + r0 * d, rows, d, plan, scratch, ga, st);
        else
            launch_load<__nv_bfloat16>((const __nv_bfloat16 *)x + r0 * d, (const __nv_bfloat16 *)gy + r0 * d, rows, d, plan, scratch,
                                       ga, st);
        int launches = 1;
        // forward states v_1 .. v_{m-1} (v_t in plane t)
        for (int t = 0; t + 1 < m; ++t, ++launches) {
            const int b = plan->st.b[t];
            const float *K = plan->d_blocks + plan->st.off[t];
            const int64_t s = plan->st.s[t];
            const bool em = s >= 8;                          // see stage_kernel
            const float *v_in = scratch + t * plane;
            float *v_out = scratch + (t + 1) * plane;
            if (owner_radix(b))
                launch_fwd_owner(b, v_in, v_out, rows, d, s, K, st);
            else if (b == 16)
                launch_dep(stage16_kernel, owner_grid16(d, rows, kFwdSliceRows), dim3(128), 0, st, v_in, v_out, rows, d, s, K, 0);
            else
                launch_dep(stage_kernel, column_grid(d, rows), dim3(kThreads), 0, st, v_in, v_out, rows, d, b, s,
                           em ? plan->d_blocks_em + plan->st.off[t] : K, em ? 1 : (int64_t)b * b, em ? d / b : 1, 0);
        }
        // backward: entry sums, and the gradient state one stage back
        float *g_cur = ga, *g_nxt = gb;
        const int acc = (accumulate || r0 > 0) ? 1 : 0;
        for (int t = m - 1; t >= 0; --t) {
            const int b = plan->st.b[t];
            const int64_t s = plan->st.s[t];
            const float *K = plan->d_blocks + plan->st.off[t];
            const float *v_t = scratch + t * plane;
            float *grad_t = grad + plan->st.off[t];
            const dim3 reduce_grid((unsigned)std::min<int64_t>((d * b + 31) / 32, 148 * 16));
            if (owner_radix(b)) {
                launch_bwd_owner(b, v_t, g_cur, t > 0 ? g_nxt : nullptr, rows, d, s, K, part, st);
                launch_dep(reduce_slices_kernel, reduce_grid, dim3(kThreads), 0, st, part, (rows + kBwdSliceRows - 1) / kBwdSliceRows,
                           d / b, b * b, grad_t, acc);
                launches += 2;
            } else if (b == 16) {
                launch_dep(outer16_kernel, owner_grid16(d, rows, kTileRows16), dim3(512), 0, st, v_t, g_cur, rows, d, s, part);
                launch_dep(reduce_slices_kernel, reduce_grid, dim3(kThreads), 0, st, part, (rows + kTileRows16 - 1) / kTileRows16,
                           d / b, b * b, grad_t, acc);
                if (t > 0)
                    launch_dep(stage16_kernel, owner_grid16(d, rows, kFwdSliceRows), dim3(128), 0, st, g_cur, g_nxt, rows, d, s, K, 1);
                launches += t > 0 ? 3 : 2;
            } else {
                const bool em = s >= 8;
                launch_dep(outer_kernel, dim3((unsigned)std::min<int64_t>((d * b + 31) / 32, 148 * 64)), dim3(kThreads), 0, st, v_t,
                           g_cur, rows, d, b, s, grad_t, acc, em ? 0 : 1);
                if (t > 0)
                    launch_dep(stage_kernel, column_grid(d, rows), dim3(kThreads), 0, st, g_cur, g_nxt, rows, d, b, s,
                               em ? plan->d_blocks_em + plan->st.off[t] : K, em ? 1 : (int64_t)b * b, em ? d / b : 1, 1);
                launches += t > 0 ? 2 : 1;
            }
            if (t > 0) std::swap(g_cur, g_nxt);
        }
        g_harp_launches.fetch_add(launches, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) rc = HARP_ERR_CUDA;
    }
    cudaFreeAsync(scratch, st);
    return rc;
}
