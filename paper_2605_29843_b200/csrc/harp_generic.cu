// Generic CUDA-core kernel: any schedule, any radix, fp32 arithmetic.
//
// One CTA owns a tile of R whole rows in shared memory (fp32) for all stages, so a
// row is read from HBM once and written once.  A work item is one output
// coordinate of one row; every thread computes its items of a stage into
// registers, the CTA synchronises, the items are written back in place, and the
// next stage starts.  Block kernels are read through the read-only path from L2.
// This path defines correct behaviour for every plan the ABI accepts (up to the
// shared-memory capacity); the tensor-core path in harp_fast.cu is faster where
// it applies.
#include <algorithm>

#include <cstdlib>

#include "harp_internal.h"
#include "harp_fuse.h"

namespace {

constexpr int kThreads = 1024;
constexpr int kMaxItems = 32;   // R*d <= kThreads*kMaxItems

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
// four neighbouring elements, p aligned to 4 * sizeof(T)
template <typename T> __device__ __forceinline__ void load4(const T *p, float (&e)[4]);
template <> __device__ __forceinline__ void load4<float>(const float *p, float (&e)[4]) {
    const float4 q = *reinterpret_cast<const float4 *>(p);
    e[0] = q.x; e[1] = q.y; e[2] = q.z; e[3] = q.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16 *p, float (&e)[4]) {
    const uint2 q = *reinterpret_cast<const uint2 *>(p);
    e[0] = __uint_as_float(q.x << 16); e[1] = __uint_as_float(q.x & 0xffff0000u);
    e[2] = __uint_as_float(q.y << 16); e[3] = __uint_as_float(q.y & 0xffff0000u);
}
template <typename T> __device__ __forceinline__ void store4(T *p, const float (&e)[4]);
template <> __device__ __forceinline__ void store4<float>(float *p, const float (&e)[4]) {
    *reinterpret_cast<float4 *>(p) = make_float4(e[0], e[1], e[2], e[3]);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16 *p, const float (&e)[4]) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(e[0], e[1]), hi = __floats2bfloat162_rn(e[2], e[3]);
    uint2 q;
    q.x = *reinterpret_cast<const uint32_t *>(&lo);
    q.y = *reinterpret_cast<const uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(p) = q;
}
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T, int ITEMS>
__global__ void __launch_bounds__(kThreads, 1)
harp_generic_kernel(T *__restrict__ x, int64_t n_rows, int d, int rows_per_cta, StageTable st,
                    const float *__restrict__ blocks, const int32_t *__restrict__ perm,
                    const int8_t *__restrict__ signs, int transpose) {
    extern __shared__ float v[];                     // [rows_per_cta][d]
    const int64_t row0 = (int64_t)blockIdx.x * rows_per_cta;
    const int rows = (int)min((int64_t)rows_per_cta, n_rows - row0);
    const int total = rows * d;
    T *xt = x + row0 * d;

    // a1-a3: load, sign, gather (forward) -- or plain load (transpose)
    for (int idx = threadIdx.x; idx < total; idx += kThreads) {
        const int r = idx / d, i = idx - r * d;
        if (!transpose) {
            const int src = perm ? perm[i] : i;
            float val = to_f32<T>(xt[(int64_t)r * d + src]);
            if (signs && signs[src] < 0) val = -val;
            v[idx] = val;
        } else {
            v[idx] = to_f32<T>(xt[idx]);
        }
    }
    __syncthreads();

    // a4 / a6: stages 0..m-1 (forward) or m-1..0 with transposed kernels
    for (int k = 0; k < st.m; ++k) {
        const int t = transpose ? st.m - 1 - k : k;
        const int b = st.b[t], s = st.s[t];
        const int bs = b * s;
        const float *Kt = blocks + st.off[t];
        float acc[ITEMS];
#pragma unroll
        for (int it = 0; it < ITEMS; ++it) {
            const int idx = threadIdx.x + it * kThreads;
            acc[it] = 0.f;
            if (idx < total) {
                const int r = idx / d, p = idx - r * d;
                const int alpha = p / bs, rem = p - alpha * bs;
                const int j = rem / s, beta = rem - j * s;
                const int c = alpha * s + beta;
                const float *Kc = Kt + (int64_t)c * b * b;
                const float *vin = v + r * d + alpha * bs + beta;
                float a = 0.f;
                if (!transpose) {
                    for (int i = 0; i < b; ++i) a = fmaf(vin[i * s], __ldg(Kc + i * b + j), a);
                } else {
                    for (int i = 0; i < b; ++i) a = fmaf(vin[i * s], __ldg(Kc + j * b + i), a);
                }
                acc[it] = a;
            }
        }
        __syncthreads();
#pragma unroll
        for (int it = 0; it < ITEMS; ++it) {
            const int idx = threadIdx.x + it * kThreads;
            if (idx < total) v[idx] = acc[it];
        }
        __syncthreads();
    }

    // a5: store -- or scatter and sign (transpose)
    for (int idx = threadIdx.x; idx < total; idx += kThreads) {
        const int r = idx / d, i = idx - r * d;
        if (!transpose) {
            xt[idx] = from_f32<T>(v[idx]);
        } else {
            const int dst = perm ? perm[i] : i;
            float val = v[idx];
            if (signs && signs[dst] < 0) val = -val;
            xt[(int64_t)r * d + dst] = from_f32<T>(val);
        }
    }
}

// ---------------------------------------------------------------------------------------
// Block-owner kernel (radices up to 8): a thread owns one block of the current stage, keeps its
// b x b kernel in registers and walks over the rows of the tile, so a block kernel is fetched
// once per tile instead of once per output coordinate, all index arithmetic is done once per
// block, and (a block being updated in place by its only owner) one barrier per stage suffices.
// Position of coordinate i of a row in shared memory.  With SWZ the index bits 2-4 are XORed with
// bits 5-6 (inside aligned runs of 128 coordinates, so d must be a multiple of 128): the lanes
// of a warp, which own neighbouring blocks, then read and write 32 different banks also in the
// stages of stride 4 and 16, where the plain layout gives 4- and 2-way conflicts; aligned
// groups of four coordinates stay together.
template <bool SWZ>
__device__ __forceinline__ int row_pos(int i) {
    return SWZ ? (i ^ (((i >> 5) & 3) << 2) ^ (((i >> 6) & 1) << 4)) : i;
}

template <int B, bool SWZ>
__device__ __forceinline__ void stage_blocks(float *v, int rows, int d, int s, const float *__restrict__ Kt, int transpose) {
    const int nblk = d / B;
    for (int c = threadIdx.x; c < nblk; c += blockDim.x) {
        const int alpha = c / s, beta = c - alpha * s;
        const int base = alpha * B * s + beta;
        int pos[B];
#pragma unroll
        for (int i = 0; i < B; ++i) pos[i] = row_pos<SWZ>(base + i * s);
        float *p = v;
        float K[B][B];
        const float *Kc = Kt + c;                // element-major: entry k of block c at Kt[k * nblk + c]
#pragma unroll
        for (int i = 0; i < B; ++i)
#pragma unroll
            for (int j = 0; j < B; ++j) K[i][j] = __ldg(Kc + (size_t)(transpose ? j * B + i : i * B + j) * nblk);
#pragma unroll 2
        for (int r = 0; r < rows; ++r, p += d) {
            float in[B];
            if (B == 4 && s == 1) {              // the block is one aligned 16-byte group
                const float4 q4 = *reinterpret_cast<const float4 *>(p + pos[0]);
                in[0] = q4.x; in[1] = q4.y; in[2 % B] = q4.z; in[3 % B] = q4.w;
            } else {
#pragma unroll
                for (int i = 0; i < B; ++i) in[i] = p[pos[i]];
            }
            float out[B];
#pragma unroll
            for (int j = 0; j < B; ++j) {
                float a = in[0] * K[0][j];
#pragma unroll
                for (int i = 1; i < B; ++i) a = fmaf(in[i], K[i][j], a);
                out[j] = a;
            }
            if (B == 4 && s == 1) {
                *reinterpret_cast<float4 *>(p + pos[0]) = make_float4(out[0], out[1], out[2 % B], out[3 % B]);
            } else {
#pragma unroll
                for (int j = 0; j < B; ++j) p[pos[j]] = out[j];
            }
        }
    }
}

template <typename T, int NT, bool BIG, bool SWZ>
__global__ void __launch_bounds__(NT, 1)
harp_blockowner_kernel(T *__restrict__ x, int64_t n_rows, int d, int rows_per_cta, StageTable st,
                       const float *__restrict__ blocks, const int32_t *__restrict__ perm,
                       const int8_t *__restrict__ signs, int transpose) {
    extern __shared__ float v[];                     // [rows_per_cta][d]
    const int64_t row0 = (int64_t)blockIdx.x * rows_per_cta;
    const int rows = (int)min((int64_t)rows_per_cta, n_rows - row0);
    T *xt = x + row0 * d;
    // without a permutation a thread moves aligned groups of four coordinates (one vector access in
    // global and one in shared memory; the swizzle keeps such groups together)
    const bool vec4 = !perm && d % 4 == 0 && (reinterpret_cast<uintptr_t>(x) % (4 * sizeof(T))) == 0;
    // a1-a3: load, sign, gather (forward) -- or plain load (transpose); a thread keeps its columns
    if (vec4) {
        for (int i = 4 * threadIdx.x; i < d; i += 4 * NT) {
            float sg[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) sg[k] = (!transpose && signs && signs[i + k] < 0) ? -1.f : 1.f;
            const T *col = xt + i;
            float *dst = v + row_pos<SWZ>(i);
#pragma unroll 4
            for (int r = 0; r < rows; ++r) {
                float e[4];
                load4<T>(col + (int64_t)r * d, e);
                *reinterpret_cast<float4 *>(dst + r * d) = make_float4(sg[0] * e[0], sg[1] * e[1], sg[2] * e[2], sg[3] * e[3]);
            }
        }
    } else {
        for (int i = threadIdx.x; i < d; i += NT) {
            const int src = (!transpose && perm) ? perm[i] : i;
            const float sg = (!transpose && signs && signs[src] < 0) ? -1.f : 1.f;
            const T *col = xt + src;
#pragma unroll 4
            for (int r = 0; r < rows; ++r) v[r * d + row_pos<SWZ>(i)] = sg * to_f32<T>(col[(int64_t)r * d]);
        }
    }
    __syncthreads();
    for (int k = 0; k < st.m; ++k) {
        const int t = transpose ? st.m - 1 - k : k;
        const float *Kt = blocks + st.off[t];
        const int b = st.b[t];
        if (b == 2) stage_blocks<2, SWZ>(v, rows, d, st.s[t], Kt, transpose);
        else if (b == 3) stage_blocks<3, SWZ>(v, rows, d, st.s[t], Kt, transpose);
        else if (b == 4) stage_blocks<4, SWZ>(v, rows, d, st.s[t], Kt, transpose);
        else if (BIG) {
            if (b == 5) stage_blocks<5, SWZ>(v, rows, d, st.s[t], Kt, transpose);
            else if (b == 6) stage_blocks<6, SWZ>(v, rows, d, st.s[t], Kt, transpose);
            else if (b == 7) stage_blocks<7, SWZ>(v, rows, d, st.s[t], Kt, transpose);
            else stage_blocks<8, SWZ>(v, rows, d, st.s[t], Kt, transpose);
        }
        __syncthreads();
    }
    // a5: store -- or scatter and sign (transpose)
    if (vec4) {
        for (int i = 4 * threadIdx.x; i < d; i += 4 * NT) {
            float sg[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) sg[k] = (transpose && signs && signs[i + k] < 0) ? -1.f : 1.f;
            T *col = xt + i;
            const float *src = v + row_pos<SWZ>(i);
#pragma unroll 4
            for (int r = 0; r < rows; ++r) {
                const float4 q4 = *reinterpret_cast<const float4 *>(src + r * d);
                const float e[4] = {sg[0] * q4.x, sg[1] * q4.y, sg[2] * q4.z, sg[3] * q4.w};
                store4<T>(col + (int64_t)r * d, e);
            }
        }
    } else {
        for (int i = threadIdx.x; i < d; i += NT) {
            const int dst = (transpose && perm) ? perm[i] : i;
            const float sg = (transpose && signs && signs[dst] < 0) ? -1.f : 1.f;
            T *col = xt + dst;
#pragma unroll 4
            for (int r = 0; r < rows; ++r) col[(int64_t)r * d] = from_f32<T>(sg * v[r * d + row_pos<SWZ>(i)]);
        }
    }
}

template <typename T, int NT, bool BIG, bool SWZ>
harp_status_t launch_blockowner_swz(const harp_plan *plan, const StageTable &st, const float *blocks, void *x, int64_t n_rows,
                                    int transpose, cudaStream_t stream) {
    auto kern = harp_blockowner_kernel<T, NT, BIG, SWZ>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
        return HARP_ERR_CUDA;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t d = plan->d;
    const int per_sm = 1;                                               // CTAs per SM (see __launch_bounds__)
    int64_t r = ((227 * 1024) / per_sm - 1024) / (d * (int64_t)sizeof(float));   // what shared memory holds
    if (r < 1) r = (227 * 1024) / (d * (int64_t)sizeof(float));
    r = std::min<int64_t>(r, (n_rows + (int64_t)sms * per_sm - 1) / ((int64_t)sms * per_sm));   // one wave when the batch allows it
    r = std::max<int64_t>(1, std::min<int64_t>(r, 64));
    const int64_t grid = (n_rows + r - 1) / r;
    if (grid > 0x7fffffffLL) return HARP_ERR_BAD_DIM;
    kern<<<(unsigned)grid, NT, (size_t)r * d * sizeof(float), stream>>>((T *)x, n_rows, (int)d, (int)r, st,
                                                                              blocks, plan->d_perm, plan->d_signs, transpose);
    g_harp_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}

template <typename T, int NT, bool BIG>
harp_status_t launch_blockowner(const harp_plan *plan, const StageTable &st, const float *blocks, void *x, int64_t n_rows,
                                int transpose, cudaStream_t stream) {
    // the bank swizzle permutes inside aligned runs of 128 coordinates
    return plan->d % 128 == 0 ? launch_blockowner_swz<T, NT, BIG, true>(plan, st, blocks, x, n_rows, transpose, stream)
                              : launch_blockowner_swz<T, NT, BIG, false>(plan, st, blocks, x, n_rows, transpose, stream);
}

// ---------------------------------------------------------------------------------------
// Block-owner kernel on a transposed tile.  The tile is kept as [coordinate][row] with the row
// index fastest, so a thread that owns a block reads and writes four rows of one coordinate with
// one 16-byte access: a quarter of the shared-memory instructions of the row-major form, which is
// bound by their issue rate.  Coordinate x lives at tpos(x) * R4 (R4 = padded row count, a
// multiple of 4 with R4/4 odd): tpos XORs the low three index bits with bits 3 and 4 so that the
// eight lanes of a quarter-warp -- eight neighbouring blocks of any stage, eight neighbouring
// coordinates or coordinate quads in the copies -- fall into eight different bank groups
// (needs d to be a multiple of 32).  The copies transpose 4 x 4 in registers.
__device__ __forceinline__ int tpos(int x) { return x ^ (((x >> 4) & 1) * 5) ^ (((x >> 3) & 1) * 2); }

__device__ __forceinline__ float4 f4_scale(float4 a, float k) { return make_float4(a.x * k, a.y * k, a.z * k, a.w * k); }
__device__ __forceinline__ float4 f4_fma(float4 a, float k, float4 c) {
    return make_float4(fmaf(a.x, k, c.x), fmaf(a.y, k, c.y), fmaf(a.z, k, c.z), fmaf(a.w, k, c.w));
}

template <int B>
__device__ __forceinline__ void stage_blocks_t(float *v, int n_rg, int R4, int d, int s, const float *__restrict__ Kt, int transpose,
                                               int tid, int nthr) {
    const int nblk = d / B;
    for (int c = tid; c < nblk; c += nthr) {
        const int alpha = c / s, beta = c - alpha * s;
        const int base = alpha * B * s + beta;
        int pos[B];
#pragma unroll
        for (int i = 0; i < B; ++i) pos[i] = tpos(base + i * s) * R4;
        float K[B][B];
        const float *Kc = Kt + c;                // element-major: entry k of block c at Kt[k * nblk + c]
#pragma unroll
        for (int i = 0; i < B; ++i)
#pragma unroll
            for (int j = 0; j < B; ++j) K[i][j] = __ldg(Kc + (size_t)(transpose ? j * B + i : i * B + j) * nblk);
#pragma unroll 2
        for (int rg = 0; rg < n_rg; ++rg) {
            float4 in[B];
#pragma unroll
            for (int i = 0; i < B; ++i) in[i] = *reinterpret_cast<const float4 *>(v + pos[i] + 4 * rg);
#pragma unroll
            for (int j = 0; j < B; ++j) {
                float4 a = f4_scale(in[0], K[0][j]);
#pragma unroll
                for (int i = 1; i < B; ++i) a = f4_fma(in[i], K[i][j], a);
                *reinterpret_cast<float4 *>(v + pos[j] + 4 * rg) = a;
            }
        }
    }
}


// ---- the two ends of the stage list done on the way in / out of the transposed tile ----------------
// Stage 0 of the table (stride 1, radix 4): a thread that copies the quad of coordinates 4m .. 4m+3 of
// four rows between global memory and the tile owns block m of that stage, so the stage is applied in
// registers during the copy: forward on the way in (after the signs), transpose on the way out (before
// them).  One shared-memory pass and one barrier less, and the arithmetic runs under the HBM transfer.
template <typename T>
__device__ __forceinline__ void copy_in_with_stage0(const T *xt, float *v, int rows, int n_rg, int R4, int d,
                                                    const float *__restrict__ Kt, const int8_t *__restrict__ signs, int tid, int nthr) {
    const int nq = d >> 2;
    for (int m = tid; m < nq; m += nthr) {
        float K[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float sg = (signs && signs[4 * m + i] < 0) ? -1.f : 1.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) K[i][j] = sg * __ldg(Kt + (size_t)(i * 4 + j) * nq + m);     // sign folded into the row
        }
        int pos[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) pos[j] = tpos(4 * m + j) * R4;
        float e[4][4], nx[4][4];
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
            if (rr < rows) load4<T>(xt + (int64_t)rr * d + 4 * m, e[rr]);
            else e[rr][0] = e[rr][1] = e[rr][2] = e[rr][3] = 0.f;
        }
        for (int rg = 0; rg < n_rg; ++rg) {
            if (rg + 1 < n_rg) {                        // next row group in flight while this one is multiplied
#pragma unroll
                for (int rr = 0; rr < 4; ++rr) {
                    if (4 * (rg + 1) + rr < rows) load4<T>(xt + (int64_t)(4 * (rg + 1) + rr) * d + 4 * m, nx[rr]);
                    else nx[rr][0] = nx[rr][1] = nx[rr][2] = nx[rr][3] = 0.f;
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float4 a = f4_scale(make_float4(e[0][0], e[1][0], e[2][0], e[3][0]), K[0][j]);
#pragma unroll
                for (int i = 1; i < 4; ++i) a = f4_fma(make_float4(e[0][i], e[1][i], e[2][i], e[3][i]), K[i][j], a);
                *reinterpret_cast<float4 *>(v + pos[j] + 4 * rg) = a;
            }
#pragma unroll
            for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                for (int i = 0; i < 4; ++i) e[rr][i] = nx[rr][i];
        }
    }
}

template <typename T>
__device__ __forceinline__ void copy_out_with_stage0(T *xt, const float *v, int rows, int n_rg, int R4, int d,
                                                     const float *__restrict__ Kt, const int8_t *__restrict__ signs, int tid, int nthr) {
    const int nq = d >> 2;
    for (int m = tid; m < nq; m += nthr) {
        float K[4][4];                                  // K[i][j] of the transposed block, sign of output j folded in
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float sg = (signs && signs[4 * m + j] < 0) ? -1.f : 1.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) K[i][j] = sg * __ldg(Kt + (size_t)(j * 4 + i) * nq + m);
        }
        int pos[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) pos[j] = tpos(4 * m + j) * R4;
        for (int rg = 0; rg < n_rg; ++rg) {
            float4 in[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) in[i] = *reinterpret_cast<const float4 *>(v + pos[i] + 4 * rg);
            float4 o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float4 a = f4_scale(in[0], K[0][j]);
#pragma unroll
                for (int i = 1; i < 4; ++i) a = f4_fma(in[i], K[i][j], a);
                o[j] = a;
            }
            const float e[4][4] = {{o[0].x, o[1].x, o[2].x, o[3].x}, {o[0].y, o[1].y, o[2].y, o[3].y},
                                   {o[0].z, o[1].z, o[2].z, o[3].z}, {o[0].w, o[1].w, o[2].w, o[3].w}};
#pragma unroll
            for (int rr = 0; rr < 4; ++rr)
                if (4 * rg + rr < rows) store4<T>(xt + (int64_t)(4 * rg + rr) * d + 4 * m, e[rr]);
        }
    }
}

// The top stage of the table (stride >= 32, so neighbouring lanes own neighbouring coordinates): its
// results go from registers straight to global memory (forward), or its operands come straight from
// global memory (transpose); a warp moves 128 contiguous bytes of a row per access.
template <typename T, int B>
__device__ __forceinline__ void stage_to_global(T *xt, const float *v, int rows, int n_rg, int R4, int d, int s,
                                                const float *__restrict__ Kt, int tid, int nthr) {
    const int nblk = d / B;
    for (int c = tid; c < nblk; c += nthr) {
        const int alpha = c / s, beta = c - alpha * s;
        const int base = alpha * B * s + beta;
        int pos[B];
#pragma unroll
        for (int i = 0; i < B; ++i) pos[i] = tpos(base + i * s) * R4;
        float K[B][B];
#pragma unroll
        for (int i = 0; i < B; ++i)
#pragma unroll
            for (int j = 0; j < B; ++j) K[i][j] = __ldg(Kt + (size_t)(i * B + j) * nblk + c);
        for (int rg = 0; rg < n_rg; ++rg) {
            float4 in[B];
#pragma unroll
            for (int i = 0; i < B; ++i) in[i] = *reinterpret_cast<const float4 *>(v + pos[i] + 4 * rg);
#pragma unroll
            for (int j = 0; j < B; ++j) {
                float4 a = f4_scale(in[0], K[0][j]);
#pragma unroll
                for (int i = 1; i < B; ++i) a = f4_fma(in[i], K[i][j], a);
                T *dst = xt + (int64_t)(4 * rg) * d + base + j * s;
                const float o[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                for (int rr = 0; rr < 4; ++rr)
                    if (4 * rg + rr < rows) dst[(int64_t)rr * d] = from_f32<T>(o[rr]);
            }
        }
    }
}

template <typename T, int B>
__device__ __forceinline__ void stage_from_global(const T *xt, float *v, int rows, int n_rg, int R4, int d, int s,
                                                  const float *__restrict__ Kt, int tid, int nthr) {
    const int nblk = d / B;
    for (int c = tid; c < nblk; c += nthr) {
        const int alpha = c / s, beta = c - alpha * s;
        const int base = alpha * B * s + beta;
        int pos[B];
#pragma unroll
        for (int i = 0; i < B; ++i) pos[i] = tpos(base + i * s) * R4;
        float K[B][B];                                  // transposed block
#pragma unroll
        for (int i = 0; i < B; ++i)
#pragma unroll
            for (int j = 0; j < B; ++j) K[i][j] = __ldg(Kt + (size_t)(j * B + i) * nblk + c);
#pragma unroll 2
        for (int rg = 0; rg < n_rg; ++rg) {
            float4 in[B];
#pragma unroll
            for (int i = 0; i < B; ++i) {
                const T *src = xt + (int64_t)(4 * rg) * d + base + i * s;
                float e[4];
#pragma unroll
                for (int rr = 0; rr < 4; ++rr) e[rr] = 4 * rg + rr < rows ? to_f32<T>(src[(int64_t)rr * d]) : 0.f;
                in[i] = make_float4(e[0], e[1], e[2], e[3]);
            }
#pragma unroll
            for (int j = 0; j < B; ++j) {
                float4 a = f4_scale(in[0], K[0][j]);
#pragma unroll
                for (int i = 1; i < B; ++i) a = f4_fma(in[i], K[i][j], a);
                *reinterpret_cast<float4 *>(v + pos[j] + 4 * rg) = a;
            }
        }
    }
}

template <typename T, int NT, bool BIG, int MINB>
__global__ void __launch_bounds__(NT, MINB)
harp_rowvec_kernel(T *__restrict__ x, int64_t n_rows, int d, int rows_per_cta, int R4, StageTable st,
                   const float *__restrict__ blocks, const int32_t *__restrict__ perm,
                   const int8_t *__restrict__ signs, int transpose, int fuse_lo, int fuse_hi) {
    extern __shared__ __align__(16) float v[];       // [d][R4]
    const int64_t row0 = (int64_t)blockIdx.x * rows_per_cta;
    const int rows = (int)min((int64_t)rows_per_cta, n_rows - row0);
    const int n_rg = (rows + 3) >> 2;
    T *xt = x + row0 * d;
    const int tid = threadIdx.x, nthr = NT;
    const bool aligned = d % 4 == 0 && (reinterpret_cast<uintptr_t>(x) % (4 * sizeof(T))) == 0;
    // fuse_lo / fuse_hi (host: no permutation, aligned rows): stage 0 and the top stage run on the way
    // in and out of the tile
    const int top = st.m - 1;
    // a1-a3: load, sign, gather (forward) -- or plain load (transpose)
    if (!transpose && fuse_lo) {
        copy_in_with_stage0<T>(xt, v, rows, n_rg, R4, d, blocks + st.off[0], signs, tid, nthr);
    } else if (transpose && fuse_hi) {
        const float *Kt = blocks + st.off[top];
        const int b = st.b[top];
        if (b == 2) stage_from_global<T, 2>(xt, v, rows, n_rg, R4, d, st.s[top], Kt, tid, nthr);
        else if (b == 3) stage_from_global<T, 3>(xt, v, rows, n_rg, R4, d, st.s[top], Kt, tid, nthr);
        else stage_from_global<T, 4>(xt, v, rows, n_rg, R4, d, st.s[top], Kt, tid, nthr);
    } else if (aligned && (transpose || !perm)) {
        const int nq = d >> 2;
        for (int w = tid; w < nq * n_rg; w += nthr) {
            const int rg = w / nq, m = w - rg * nq;
            float e[4][4];
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
                if (4 * rg + rr < rows) load4<T>(xt + (int64_t)(4 * rg + rr) * d + 4 * m, e[rr]);
                else e[rr][0] = e[rr][1] = e[rr][2] = e[rr][3] = 0.f;
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float sg = (!transpose && signs && signs[4 * m + k] < 0) ? -1.f : 1.f;
                *reinterpret_cast<float4 *>(v + tpos(4 * m + k) * R4 + 4 * rg) =
                    make_float4(sg * e[0][k], sg * e[1][k], sg * e[2][k], sg * e[3][k]);
            }
        }
    } else {
        for (int w = tid; w < d * n_rg; w += nthr) {
            const int rg = w / d, i = w - rg * d;
            const int src = (!transpose && perm) ? perm[i] : i;
            const float sg = (!transpose && signs && signs[src] < 0) ? -1.f : 1.f;
            float e[4];
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) e[rr] = 4 * rg + rr < rows ? sg * to_f32<T>(xt[(int64_t)(4 * rg + rr) * d + src]) : 0.f;
            *reinterpret_cast<float4 *>(v + tpos(i) * R4 + 4 * rg) = make_float4(e[0], e[1], e[2], e[3]);
        }
    }
    __syncthreads();
    for (int k = 0; k < st.m; ++k) {
        const int t = transpose ? st.m - 1 - k : k;
        if ((t == 0 && fuse_lo) || (t == top && fuse_hi)) continue;      // done during a copy
        const float *Kt = blocks + st.off[t];
        const int b = st.b[t];
        if (b == 2) stage_blocks_t<2>(v, n_rg, R4, d, st.s[t], Kt, transpose, tid, nthr);
        else if (b == 3) stage_blocks_t<3>(v, n_rg, R4, d, st.s[t], Kt, transpose, tid, nthr);
        else if (b == 4) stage_blocks_t<4>(v, n_rg, R4, d, st.s[t], Kt, transpose, tid, nthr);
        else if (BIG) {
            if (b == 5) stage_blocks_t<5>(v, n_rg, R4, d, st.s[t], Kt, transpose, tid, nthr);
            else if (b == 6) stage_blocks_t<6>(v, n_rg, R4, d, st.s[t], Kt, transpose, tid, nthr);
            else if (b == 7) stage_blocks_t<7>(v, n_rg, R4, d, st.s[t], Kt, transpose, tid, nthr);
            else stage_blocks_t<8>(v, n_rg, R4, d, st.s[t], Kt, transpose, tid, nthr);
        }
        __syncthreads();
    }
    // a5: store -- or scatter and sign (transpose)
    if (transpose && fuse_lo) {
        copy_out_with_stage0<T>(xt, v, rows, n_rg, R4, d, blocks + st.off[0], signs, tid, nthr);
    } else if (!transpose && fuse_hi) {
        const float *Kt = blocks + st.off[top];
        const int b = st.b[top];
        if (b == 2) stage_to_global<T, 2>(xt, v, rows, n_rg, R4, d, st.s[top], Kt, tid, nthr);
        else if (b == 3) stage_to_global<T, 3>(xt, v, rows, n_rg, R4, d, st.s[top], Kt, tid, nthr);
        else stage_to_global<T, 4>(xt, v, rows, n_rg, R4, d, st.s[top], Kt, tid, nthr);
    } else if (aligned && (!transpose || !perm)) {
        const int nq = d >> 2;
        for (int w = tid; w < nq * n_rg; w += nthr) {
            const int rg = w / nq, m = w - rg * nq;
            float4 q[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float sg = (transpose && signs && signs[4 * m + k] < 0) ? -1.f : 1.f;
                q[k] = f4_scale(*reinterpret_cast<const float4 *>(v + tpos(4 * m + k) * R4 + 4 * rg), sg);
            }
            const float e[4][4] = {{q[0].x, q[1].x, q[2].x, q[3].x}, {q[0].y, q[1].y, q[2].y, q[3].y},
                                   {q[0].z, q[1].z, q[2].z, q[3].z}, {q[0].w, q[1].w, q[2].w, q[3].w}};
#pragma unroll
            for (int rr = 0; rr < 4; ++rr)
                if (4 * rg + rr < rows) store4<T>(xt + (int64_t)(4 * rg + rr) * d + 4 * m, e[rr]);
        }
    } else {
        for (int w = tid; w < d * n_rg; w += nthr) {
            const int rg = w / d, i = w - rg * d;
            const int dst = (transpose && perm) ? perm[i] : i;
            const float sg = (transpose && signs && signs[dst] < 0) ? -1.f : 1.f;
            const float4 q = *reinterpret_cast<const float4 *>(v + tpos(i) * R4 + 4 * rg);
            const float e[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int rr = 0; rr < 4; ++rr)
                if (4 * rg + rr < rows) xt[(int64_t)(4 * rg + rr) * d + dst] = from_f32<T>(sg * e[rr]);
        }
    }
}

template <typename T, int NT, bool BIG, int MINB = 1>
harp_status_t launch_rowvec(const harp_plan *plan, const StageTable &st, const float *blocks, void *x, int64_t n_rows,
                            int transpose, cudaStream_t stream) {
    auto kern = harp_rowvec_kernel<T, NT, BIG, MINB>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
        return HARP_ERR_CUDA;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t d = plan->d;
    // groups of four rows per CTA: an odd number (bank spread), as many as shared memory holds,
    // but no more than one wave of CTAs needs
    // MINB CTAs share an SM (and its shared memory): while one multiplies, another copies
    int64_t g_max = (226 * 1024 / MINB) / (d * 16);
    if (g_max % 2 == 0) --g_max;
    if (g_max < 1) return HARP_ERR_UNSUPPORTED;
    int64_t g = ((n_rows + (int64_t)sms * MINB - 1) / ((int64_t)sms * MINB) + 3) / 4;
    g = std::max<int64_t>(1, std::min<int64_t>(g, std::min<int64_t>(g_max, 15)));
    const int64_t g_pad = g | 1;                     // g_pad <= g_max because g_max is odd
    const int64_t r = 4 * g;
    const int64_t grid = (n_rows + r - 1) / r;
    if (grid > 0x7fffffffLL) return HARP_ERR_BAD_DIM;
    // the ends of the stage list on the way in and out: identity permutation, aligned rows, stage 0 of
    // radix 4 and stride 1, a top stage of radix <= 4 whose stride keeps a warp's accesses contiguous,
    // at least three stages (so that the two ends are different stages with a barrier between them)
    const bool ends_ok = !plan->d_perm && d % 4 == 0 && (reinterpret_cast<uintptr_t>(x) % (4 * sizeof(T))) == 0 && st.m >= 3;
    const int fuse_lo = ends_ok && st.b[0] == 4 && st.s[0] == 1;
    const int fuse_hi = ends_ok && st.b[st.m - 1] <= 4 && st.s[st.m - 1] >= 32;
    kern<<<(unsigned)grid, NT, (size_t)d * 16 * g_pad, stream>>>((T *)x, n_rows, (int)d, (int)r, (int)(4 * g_pad), st, blocks,
                                                              plan->d_perm, plan->d_signs, transpose, fuse_lo, fuse_hi);
    g_harp_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}

template <typename T, int ITEMS>
harp_status_t launch(const harp_plan *plan, void *x, int64_t n_rows, int rows_per_cta, int transpose,
                     cudaStream_t stream) {
    auto kern = harp_generic_kernel<T, ITEMS>;
    const size_t smem = (size_t)rows_per_cta * plan->d * sizeof(float);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
        return HARP_ERR_CUDA;
    const int64_t grid = (n_rows + rows_per_cta - 1) / rows_per_cta;
    if (grid > 0x7fffffffLL) return HARP_ERR_BAD_DIM;
    kern<<<(unsigned)grid, kThreads, smem, stream>>>((T *)x, n_rows, (int)plan->d, rows_per_cta, plan->st,
                                                      plan->d_blocks, plan->d_perm, plan->d_signs, transpose);
    g_harp_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}

}  // namespace

// Fuse runs of consecutive stages whose radices multiply to at most 4 into one dense stage (the
// product of their block kernels on the coordinates they touch, computed in fp64, rounded once to
// fp32): the same linear map with fewer stages, i.e. fewer barriers and shared-memory round trips.
harp_status_t harp_generic_build(harp_plan *plan) {
    const int m = plan->st.m;
    const int64_t d = plan->d;
    std::vector<harp_fuse::HostPhase> groups;
    for (int t = 0; t < m;) {
        int64_t prod = plan->st.b[t];
        int t1 = t + 1;
        while (t1 < m && prod * plan->st.b[t1] <= 4) prod *= plan->st.b[t1++];
        groups.push_back({t, t1, (int)prod, plan->st.s[t], 0, 1});
        t = t1;
    }
    // element-major copy of the block kernels of stage table tab (see harp_plan::d_bo_blocks)
    auto upload_element_major = [&](const StageTable &tab, const float *src) -> harp_status_t {
        size_t total = 0;
        for (int t = 0; t < tab.m; ++t) total = std::max(total, (size_t)tab.off[t] + (size_t)d * tab.b[t]);
        std::vector<float> em;
        try {
            em.resize(total);
        } catch (const std::bad_alloc &) {
            return HARP_ERR_ALLOC;
        }
        for (int t = 0; t < tab.m; ++t) {
            const int b = tab.b[t];
            const int64_t nblk = d / b;
            for (int64_t c = 0; c < nblk; ++c)
                for (int k = 0; k < b * b; ++k) em[(size_t)(tab.off[t] + k * nblk + c)] = src[tab.off[t] + c * b * b + k];
        }
        if (cudaMalloc(&plan->d_bo_blocks, sizeof(float) * std::max<size_t>(1, total)) != cudaSuccess) return HARP_ERR_ALLOC;
        if (cudaMemcpy(plan->d_bo_blocks, em.data(), sizeof(float) * total, cudaMemcpyHostToDevice) != cudaSuccess)
            return HARP_ERR_CUDA;
        return HARP_OK;
    };
    int max_b = 0;
    for (int t = 0; t < m; ++t) max_b = std::max(max_b, (int)plan->st.b[t]);
    if ((int)groups.size() == m)                                        // nothing to fuse
        return max_b <= 8 ? upload_element_major(plan->st, plan->h_blocks.data()) : HARP_OK;
    StageTable ft{};
    ft.m = (int32_t)groups.size();
    int64_t off = 0;
    for (size_t k = 0; k < groups.size(); ++k) {
        ft.b[k] = groups[k].B;
        ft.s[k] = (int32_t)groups[k].S;
        ft.off[k] = off;
        off += d * groups[k].B;
    }
    std::vector<float> fb;
    try {
        fb.resize((size_t)off);
    } catch (const std::bad_alloc &) {
        return HARP_ERR_ALLOC;
    }
    std::vector<double> F;
    for (size_t k = 0; k < groups.size(); ++k) {
        const int B = groups[k].B;
        const int64_t S = groups[k].S;
        for (int64_t c = 0; c < d / B; ++c) {
            const int64_t alpha = c / S, beta = c % S;
            harp_fuse::fused_block(plan, groups[k], alpha * B * S + beta, F);
            float *dst = fb.data() + ft.off[k] + c * B * B;
            for (int i = 0; i < B * B; ++i) dst[i] = (float)F[(size_t)i];
        }
    }
    if (cudaMalloc(&plan->d_fused_blocks, sizeof(float) * (size_t)off) != cudaSuccess) return HARP_ERR_ALLOC;
    if (cudaMemcpy(plan->d_fused_blocks, fb.data(), sizeof(float) * (size_t)off, cudaMemcpyHostToDevice) != cudaSuccess)
        return HARP_ERR_CUDA;
    plan->fused = ft;
    int max_fb = 0;
    for (int t = 0; t < ft.m; ++t) max_fb = std::max(max_fb, (int)ft.b[t]);
    return max_fb <= 8 ? upload_element_major(ft, fb.data()) : HARP_OK;
}

harp_status_t harp_generic_supported(const harp_plan *plan, harp_dtype_t dtype) {
    (void)dtype;
    if (plan->d > (int64_t)kThreads * kMaxItems) return HARP_ERR_UNSUPPORTED;
    if ((size_t)plan->d * sizeof(float) > 227u * 1024u) return HARP_ERR_UNSUPPORTED;
    return HARP_OK;
}

harp_status_t harp_generic_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                                 int transpose, cudaStream_t stream) {
    harp_status_t ok = harp_generic_supported(plan, dtype);
    if (ok != HARP_OK) return ok;
    const int64_t d = plan->d;
    const bool use_fused = plan->fused.m > 0 && plan->d_fused_blocks;
    const StageTable &bst = use_fused ? plan->fused : plan->st;
    const float *bblk = plan->d_bo_blocks;       // element-major, for the block-owner kernels (radices <= 8)
    int max_radix = 0;
    for (int t = 0; t < bst.m; ++t) max_radix = std::max(max_radix, (int)bst.b[t]);
    if (max_radix <= 8 && !bblk) return HARP_ERR_UNSUPPORTED;
    const bool rowvec = d % 32 == 0 && d * 16 <= 226 * 1024 && !plan->opt_no_rowvec;
    if (rowvec && max_radix <= 4) {
        return dtype == HARP_F32 ? launch_rowvec<float, 512, false>(plan, bst, bblk, x, n_rows, transpose, stream)
                                 : launch_rowvec<__nv_bfloat16, 512, false>(plan, bst, bblk, x, n_rows, transpose, stream);
    }
    if (rowvec && max_radix <= 8) {
        return dtype == HARP_F32 ? launch_rowvec<float, 256, true>(plan, bst, bblk, x, n_rows, transpose, stream)
                                 : launch_rowvec<__nv_bfloat16, 256, true>(plan, bst, bblk, x, n_rows, transpose, stream);
    }
    if (max_radix <= 4) {      // 1024 threads, 64 registers: the block kernel takes at most 16 of them
        return dtype == HARP_F32 ? launch_blockowner<float, 1024, false>(plan, bst, bblk, x, n_rows, transpose, stream)
                                 : launch_blockowner<__nv_bfloat16, 1024, false>(plan, bst, bblk, x, n_rows, transpose, stream);
    }
    if (max_radix <= 8) {      // 256 threads so that an 8 x 8 block kernel stays in registers
        return dtype == HARP_F32 ? launch_blockowner<float, 256, true>(plan, bst, bblk, x, n_rows, transpose, stream)
                                 : launch_blockowner<__nv_bfloat16, 256, true>(plan, bst, bblk, x, n_rows, transpose, stream);
    }
    // rows per CTA: as many as registers (kMaxItems) and shared memory allow, at most 8,
    // but keep at least ~2 CTAs per SM in flight when the batch is small.
    int r = (int)((int64_t)kThreads * kMaxItems / d);
    const int r_smem = (int)((227 * 1024) / (d * (int64_t)sizeof(float)));
    if (r > r_smem) r = r_smem;
    if (r > 8) r = 8;
    while (r > 1 && (n_rows + r - 1) / r < 296) --r;
    if (r < 1) r = 1;
    const int64_t items = ((int64_t)r * d + kThreads - 1) / kThreads;
#define HARP_GEN_DISPATCH(T)                                                                  \
    if (items <= 4) return launch<T, 4>(plan, x, n_rows, r, transpose, stream);               \
    if (items <= 8) return launch<T, 8>(plan, x, n_rows, r, transpose, stream);               \
    if (items <= 16) return launch<T, 16>(plan, x, n_rows, r, transpose, stream);             \
    return launch<T, 32>(plan, x, n_rows, r, transpose, stream);
    if (dtype == HARP_F32) {
        HARP_GEN_DISPATCH(float)
    } else {
        HARP_GEN_DISPATCH(__nv_bfloat16)
    }
#undef HARP_GEN_DISPATCH
}
