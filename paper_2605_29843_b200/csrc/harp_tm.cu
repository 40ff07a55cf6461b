// Tensor-memory path (tcgen05.mma + TMEM + bulk tensor copies): rows as the M dimension.
//
// A tile is 128 rows x 256 coordinates, seen as a 16 x 16 array [q][e] of the row's coordinates
// (e contiguous in memory, q at a stride).  One thread of an epilogue warpgroup owns one row of the
// tile and one lane of tensor memory, so every regrouping of a row's coordinates between stages
// (Algorithm 1's reshape/transpose) is register naming inside a thread: no shuffle, no shared-memory
// transposition.  A stage group ("phase", stages fused at plan time into dense 16 x 16 blocks as in
// the other tensor-core paths) is one tcgen05.mma per block: D[128 x 16] = A[128 x 16] * F_c, with A
// (bf16 pairs) and D (fp32) in tensor memory and F_c, shared by the 128 rows, in shared memory.  Block
// kernels are fetched once per 128 rows instead of once per 16.
//
// A pass streams tiles HBM/L2 -> shared memory (bulk tensor copy, mbarrier completion) -> registers ->
// tensor memory -> ... -> registers -> shared memory -> bulk tensor store, in place.  Dimensions with
// more than 256 coordinates take several passes (Eq. 7: a stage mixes one digit, so a pass that holds
// two digits of every row of a tile can run the stages of those digits).
#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "harp_fuse.h"
#include "harp_internal.h"
#include "harp_tm_ptx.cuh"

namespace {

using namespace harp_tm;

constexpr int kRows = 128;               // rows per tile = lanes of tensor memory
constexpr int kTileBytes = 65536;        // 128 rows x 256 bf16
constexpr int kNBuf = 3;                 // tile buffers in shared memory (ring; output staged in place)
constexpr int kFragBytes = 8192;         // 16 blocks x 16 x 16 bf16 per phase
constexpr int kThreads = 384;            // 12 warps: producer, MMA (chunk 0), store, MMA (chunk 1), 2 x 4 epilogue
constexpr uint32_t kSpin = 1u << 22;     // limit of every wait
constexpr int TM_I = 0, TM_O = 1;        // a phase contracts the inner (e) or the outer (q) index
constexpr int FMT_C = 0, FMT_S = 1;      // contiguous 256 coordinates / 16 segments of 16

// tensor-memory columns
constexpr uint32_t kColA1 = 0, kColA2 = 128, kColD = 256;

struct TmParams {
    const uint8_t *frags;       // [n_col_tiles][n_ph][16 blocks][512 bytes]
    int32_t n_row_tiles, n_col_tiles;
    int32_t lo_count;           // FMT_S: tile column index = hi * lo_count + lo
    int32_t tiles_per_cta;      // ceil(n_tiles / gridDim.x)
    int32_t *err;               // device word, set non-zero when a wait gave up
};

// byte offset of the 16-byte chunk (q, h) (coordinates e = 8h .. 8h+7 of segment q) of row r
template <int FMT>
__device__ __forceinline__ uint32_t chunk_off(int r, int q, int h) {
    if (FMT == FMT_C) {
        // four 128-row x 128-byte boxes, 128-byte swizzle: chunk index xor (row mod 8)
        const int c8 = ((q & 3) << 1) | h;
        return (uint32_t)((q >> 2) * 16384 + r * 128 + ((c8 ^ (r & 7)) << 4));
    }
    // one box [q][row][32 bytes], 32-byte swizzle: chunk bit xor address bit 7
    return (uint32_t)(q * 4096 + r * 32 + ((h ^ ((r >> 2) & 1)) << 4));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Per-section cycle counters (build with -DHARP_TM_TIMING): summed over CTAs by one thread per role.
//  0 tiles | producer: 1 wait for a free buffer, 2 issue | MMA: 3 wait for A, 4 issue
//  store: 5 wait for a finished tile, 6 wait for the store to have read it
//  epilogue (row 0 of warpgroup 0): 7 wait for the tile, 8 row -> A, 9 wait for D (phase 1), 10 D -> A (between
//  the phases), 11 wait for D (phase 2), 12 D -> tile buffer
__device__ long long g_tm_timing[16];
#ifdef HARP_TM_TIMING
#define TM_DECL long long acc[16] = {0}
#define TM_T(var) const long long var = clock64()
#define TM_ACC(slot, a, b) acc[slot] += (b) - (a)
#else
#define TM_DECL
#define TM_T(var)
#define TM_ACC(slot, a, b)
#endif

struct Waiter {
    volatile int *dead;
    int32_t *err;
    // false when the wait gave up (here or elsewhere in the CTA)
    __device__ __forceinline__ bool operator()(uint32_t bar, uint32_t parity, int code) const {
        for (uint32_t it = 0; it < kSpin; ++it) {
            if (mbar_try(bar, parity)) return true;
            if ((it & 63) == 63 && *dead) return false;
        }
        *dead = 1;
        atomicExch(err, code);
        return false;
    }
};

// cross-block packing of one D chunk (8 blocks x 16 columns): p[j*4 + m] = (D[2m][j], D[2m+1][j]) as bf16x2
__device__ __forceinline__ void pack_cross(uint32_t d_addr, uint32_t (&p)[64]) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        uint32_t d0[32], d1[32];
        tmem_ld32(d_addr + half * 64, d0);
        tmem_ld32(d_addr + half * 64 + 32, d1);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            p[j * 4 + half * 2 + 0] = pack_bf16x2(__uint_as_float(d0[j]), __uint_as_float(d0[16 + j]));
            p[j * 4 + half * 2 + 1] = pack_bf16x2(__uint_as_float(d1[j]), __uint_as_float(d1[16 + j]));
        }
    }
}

// One pass.  K0, K1: index contracted by the first / second phase (K1 < 0: one phase).  XPOSE: the
// result is stored with inner and outer index exchanged (element (q, e) of the result tile goes to
// segment e, offset q).
template <int FMT, int K0, int K1, int XPOSE>
__global__ void __launch_bounds__(kThreads, 1)
harp_tm_kernel(const __grid_constant__ CUtensorMap tmap, const TmParams P) {
    constexpr int NPH = K1 < 0 ? 1 : 2;
    constexpr int KLAST = K1 < 0 ? K0 : K1;
    // after the last phase block index and column are (q, e) or (e, q); the store wants 8 consecutive e
    constexpr bool CROSS_OUT = (KLAST == TM_O) != (XPOSE != 0);

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[3 * kNBuf + 5];
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t buf0 = smem0;                                   // kNBuf tile buffers
    const uint32_t frag0 = smem0 + kNBuf * kTileBytes;             // 2 fragment slots
    const uint32_t bar_full = smem_u32(&bars[0]);                  // + 8 b
    const uint32_t bar_empty = smem_u32(&bars[kNBuf]);
    const uint32_t bar_out = smem_u32(&bars[2 * kNBuf]);
    const uint32_t bar_a = smem_u32(&bars[3 * kNBuf]);             // two: A of the first phase, per warpgroup
    const uint32_t bar_a2 = smem_u32(&bars[3 * kNBuf + 2]);        // A of the second phase (both warpgroups)
    const uint32_t bar_d = smem_u32(&bars[3 * kNBuf + 3]);         // two: D chunk of a warpgroup

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int b = 0; b < kNBuf; ++b) {
            mbar_init(bar_full + 8 * b, 1);
            mbar_init(bar_empty + 8 * b, 1);
            mbar_init(bar_out + 8 * b, 256);
        }
        mbar_init(bar_a, 128);
        mbar_init(bar_a + 8, 128);
        mbar_init(bar_a2, 256);
        mbar_init(bar_d, 1);
        mbar_init(bar_d + 8, 1);
        dead_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    const Waiter wait{&dead_s, P.err};
    // Barriers and tensor memory are set up; nothing above touches the rows.  Launched with the programmatic
    // stream-serialisation attribute this point is reached while the kernel before this one in the stream is
    // still finishing on other SMs; the rows are read and written only after it has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int64_t n_tiles = (int64_t)P.n_row_tiles * P.n_col_tiles;
    const int64_t t_begin = (int64_t)blockIdx.x * P.tiles_per_cta;
    const int64_t t_end = t_begin + P.tiles_per_cta < n_tiles ? t_begin + P.tiles_per_cta : n_tiles;

    if (warp == 0) {
        // ---------------- producer: tiles and block fragments into shared memory ----------------
        if (lane == 0) {
            int cur_col = -1, slot = 1;
            int64_t issued = 0;
            TM_DECL;
            for (int64_t t = t_begin; t < t_end; ++t) {
                const int64_t i = t - t_begin;
                const int b = (int)(i % kNBuf);
                const uint32_t par = (uint32_t)((i / kNBuf) & 1);
                TM_T(c0);
                if (!wait(bar_empty + 8 * b, par ^ 1, 1)) break;
                TM_T(c1);
                TM_ACC(1, c0, c1);
                const int col = (int)(t / P.n_row_tiles), row0 = (int)(t % P.n_row_tiles) * kRows;
                uint32_t bytes = kTileBytes;
                const bool new_frag = col != cur_col;
                if (new_frag) {
                    // the slot about to be overwritten was last read by tiles <= i - 2: wait for their MMAs
                    if (i >= 2 && !wait(bar_out + 8 * (int)((i - 2) % kNBuf), (uint32_t)(((i - 2) / kNBuf) & 1), 2)) break;
                    cur_col = col;
                    slot ^= 1;
                    bytes += NPH * kFragBytes;
                }
                mbar_expect_tx(bar_full + 8 * b, bytes);
                if (new_frag)
                    bulk_load(frag0 + slot * (NPH * kFragBytes), P.frags + (size_t)col * (NPH * kFragBytes),
                              NPH * kFragBytes, bar_full + 8 * b);
                const uint32_t dst = buf0 + b * kTileBytes;
                if (FMT == FMT_C) {
#pragma unroll
                    for (int a = 0; a < 4; ++a) tma_load_2d(dst + a * 16384, &tmap, col * 256 + a * 64, row0, bar_full + 8 * b);
                } else {
                    const int hi = col / P.lo_count, lo = col % P.lo_count;
                    tma_load_3d(dst, &tmap, lo * 16, row0, hi * 16, bar_full + 8 * b);
                }
                issued = i + 1;
                TM_T(c2);
                TM_ACC(2, c1, c2);
            }
#ifdef HARP_TM_TIMING
            atomicAdd((unsigned long long *)&g_tm_timing[0], (unsigned long long)(t_end > t_begin ? t_end - t_begin : 0));
            atomicAdd((unsigned long long *)&g_tm_timing[1], (unsigned long long)acc[1]);
            atomicAdd((unsigned long long *)&g_tm_timing[2], (unsigned long long)acc[2]);
#endif
            if (dead_s) {
                // leave no copy in flight: bounded wait for the loads issued last
                for (int64_t k = issued > kNBuf ? issued - kNBuf : 0; k < issued; ++k)
                    for (uint32_t it = 0; it < kSpin; ++it)
                        if (mbar_try(bar_full + 8 * (int)(k % kNBuf), (uint32_t)((k / kNBuf) & 1))) break;
            }
        }
    } else if (warp == 1 || warp == 3) {
        // ---------------- MMA issue: warp 1 for chunk 0 (blocks 0-7), warp 3 for chunk 1 ----------------
        if (lane == 0) {
            const int g = warp == 1 ? 0 : 1;
            const uint32_t idesc = instr_desc(128, 16);
            int cur_col = -1, slot = 1;
            uint32_t ua = 0;
            TM_DECL;
            for (int64_t t = t_begin; t < t_end; ++t) {
                const int col = (int)(t / P.n_row_tiles);
                if (col != cur_col) { cur_col = col; slot ^= 1; }
                bool ok = true;
#pragma unroll
                for (int ph = 0; ph < NPH; ++ph) {
                    TM_T(c0);
                    // the first phase needs this chunk's own blocks of A (written by its warpgroup), the second
                    // the whole of A (pairs from both warpgroups)
                    if (!wait(ph == 0 ? bar_a + 8 * g : bar_a2, ua & 1, 3)) { ok = false; break; }
                    TM_T(c1);
                    TM_ACC(3, c0, c1);
                    tc_fence_after();
                    const uint32_t a_col = ph == 0 ? kColA1 : kColA2;
                    const uint32_t fbase = frag0 + slot * (NPH * kFragBytes) + ph * kFragBytes;
#pragma unroll
                    for (int blk = 0; blk < 8; ++blk) {
                        const int c = g * 8 + blk;
                        mma_ts(tmem + kColD + c * 16, tmem + a_col + c * 8, smem_desc(fbase + c * 512, 128, 256), idesc);
                    }
                    mma_commit(bar_d + 8 * g);
                    TM_T(c2);
                    TM_ACC(4, c1, c2);
                }
                ++ua;
                if (!ok) break;
            }
#ifdef HARP_TM_TIMING
            if (g == 0) {
                atomicAdd((unsigned long long *)&g_tm_timing[3], (unsigned long long)acc[3]);
                atomicAdd((unsigned long long *)&g_tm_timing[4], (unsigned long long)acc[4]);
            }
#endif
        }
    } else if (warp == 2) {
        // ---------------- store: finished tiles back to global memory ----------------
        if (lane == 0) {
            TM_DECL;
            for (int64_t t = t_begin; t < t_end; ++t) {
                const int64_t i = t - t_begin;
                const int b = (int)(i % kNBuf);
                TM_T(c0);
                if (!wait(bar_out + 8 * b, (uint32_t)((i / kNBuf) & 1), 4)) break;
                TM_T(c1);
                TM_ACC(5, c0, c1);
                const int col = (int)(t / P.n_row_tiles), row0 = (int)(t % P.n_row_tiles) * kRows;
                const uint32_t src = buf0 + b * kTileBytes;
                if (FMT == FMT_C) {
#pragma unroll
                    for (int a = 0; a < 4; ++a) tma_store_2d(&tmap, col * 256 + a * 64, row0, src + a * 16384);
                } else {
                    const int hi = col / P.lo_count, lo = col % P.lo_count;
                    tma_store_3d(&tmap, lo * 16, row0, hi * 16, src);
                }
                bulk_commit();
                bulk_wait_read0();
                mbar_arrive(bar_empty + 8 * b);
                TM_T(c2);
                TM_ACC(6, c1, c2);
            }
            bulk_wait0();
#ifdef HARP_TM_TIMING
            atomicAdd((unsigned long long *)&g_tm_timing[5], (unsigned long long)acc[5]);
            atomicAdd((unsigned long long *)&g_tm_timing[6], (unsigned long long)acc[6]);
#endif
        }
    } else if (warp >= 4) {
        // ---------------- epilogue warpgroups: thread = row = lane of tensor memory ----------------
        const int g = (warp - 4) >> 2;                      // chunk of 8 blocks this warpgroup owns
        const int r = ((warp & 3) << 5) | lane;             // row of the tile
        const uint32_t tlane = tmem + ((uint32_t)((warp & 3) << 5) << 16);
        uint32_t ud = 0;
        TM_DECL;
        // row r of the tile in buffer `src` -> this warpgroup's half of the first phase's A operand
        auto row_to_a1 = [&](uint32_t src) {
            uint32_t a[64];
            if (K0 == TM_I) {
                // blocks q = 8g .. 8g+7, K = e: the row's own order
#pragma unroll
                for (int beta = 0; beta < 8; ++beta)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint4 v = lds128(src + chunk_off<FMT>(r, 8 * g + beta, h));
                        a[beta * 8 + h * 4 + 0] = v.x; a[beta * 8 + h * 4 + 1] = v.y;
                        a[beta * 8 + h * 4 + 2] = v.z; a[beta * 8 + h * 4 + 3] = v.w;
                    }
            } else {
                // blocks e = 8g .. 8g+7, K = q: pair (q = 2m, 2m+1) at fixed e
                uint32_t c[16][4];
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const uint4 v = lds128(src + chunk_off<FMT>(r, q, g));
                    c[q][0] = v.x; c[q][1] = v.y; c[q][2] = v.z; c[q][3] = v.w;
                }
#pragma unroll
                for (int eps = 0; eps < 8; ++eps)
#pragma unroll
                    for (int m = 0; m < 8; ++m)
                        a[eps * 8 + m] = prmt(c[2 * m][eps >> 1], c[2 * m + 1][eps >> 1], (eps & 1) ? 0x7632u : 0x5410u);
            }
            tmem_st64(tlane + kColA1 + 64 * g, a);
        };
        for (int64_t t = t_begin; t < t_end; ++t) {
            const int64_t i = t - t_begin;
            const int b = (int)(i % kNBuf);
            const uint32_t buf = buf0 + b * kTileBytes;
            TM_T(e0);
            // two-phase passes fetch the next tile's row early (see below); then this tile's A is already there
            const bool a1_done = NPH == 2 && i > 0;
            if (!a1_done && !wait(bar_full + 8 * b, (uint32_t)((i / kNBuf) & 1), 5)) break;
            TM_T(e1);
            TM_ACC(7, e0, e1);
            if (!a1_done) {
                row_to_a1(buf);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar_a + 8 * g);
            }
            TM_T(e2);
            TM_ACC(8, e1, e2);
            if (!wait(bar_d + 8 * g, ud & 1, 6)) break;
            ++ud;
            tc_fence_after();
            TM_T(e3);
            TM_ACC(9, e2, e3);
            bool next_a1 = false;
            if (NPH == 2) {
                // --- between the phases: D (fp32) -> A of the other index (bf16 pairs over neighbouring blocks) ---
                uint32_t p[64];
                pack_cross(tlane + kColD + 128 * g, p);
                // A of the second phase is shared by both chunks: the other chunk's second-phase products of the
                // tile before must be complete, which that tile's out barrier implies (its warpgroup read them)
                if (i > 0 && !wait(bar_out + 8 * (int)((i - 1) % kNBuf), (uint32_t)(((i - 1) / kNBuf) & 1), 8)) break;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const uint32_t v4[4] = {p[j * 4 + 0], p[j * 4 + 1], p[j * 4 + 2], p[j * 4 + 3]};
                    tmem_st4(tlane + kColA2 + j * 8 + 4 * g, v4);
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar_a2);
                TM_T(e4);
                TM_ACC(10, e3, e4);
                // While the second phase's products run: the next tile's row into this warpgroup's half of the
                // first phase's A (its own first-phase products of this tile are complete, nobody else reads that
                // half).  The barrier that releases the next tile's first phase is arrived on further down, once
                // this tile's accumulators have been read.
                if (t + 1 < t_end) {
                    const int64_t i2 = i + 1;
                    if (!wait(bar_full + 8 * (int)(i2 % kNBuf), (uint32_t)((i2 / kNBuf) & 1), 5)) break;
                    row_to_a1(buf0 + (int)(i2 % kNBuf) * kTileBytes);
                    tmem_wait_st();
                    next_a1 = true;
                }
                if (!wait(bar_d + 8 * g, ud & 1, 7)) break;
                ++ud;
                tc_fence_after();
                TM_T(e5);
                TM_ACC(11, e4, e5);
            }
            TM_T(e6);
            // --- result back into the tile buffer (in place), rounded once to bf16 ---
            if (CROSS_OUT) {
                uint32_t p[64];
                pack_cross(tlane + kColD + 128 * g, p);
                if (next_a1) {                      // accumulators read: the next tile's first phase may overwrite them
                    tc_fence_before();
                    mbar_arrive(bar_a + 8 * g);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    sts128(buf + chunk_off<FMT>(r, j, g), p[j * 4 + 0], p[j * 4 + 1], p[j * 4 + 2], p[j * 4 + 3]);
            } else {
                uint32_t o4[16][4];
#pragma unroll
                for (int pair = 0; pair < 4; ++pair) {
                    uint32_t d[32];
                    tmem_ld32(tlane + kColD + 128 * g + 32 * pair, d);
                    tmem_wait_ld();
#pragma unroll
                    for (int bb = 0; bb < 2; ++bb)
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int o = bb * 16 + h * 8;
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                o4[pair * 4 + bb * 2 + h][u] = pack_bf16x2(__uint_as_float(d[o + 2 * u]), __uint_as_float(d[o + 2 * u + 1]));
                        }
                }
                if (next_a1) {
                    tc_fence_before();
                    mbar_arrive(bar_a + 8 * g);
                }
#pragma unroll
                for (int k = 0; k < 16; ++k)        // chunk (q = 8g + k/2, h = k & 1)
                    sts128(buf + chunk_off<FMT>(r, 8 * g + (k >> 1), k & 1), o4[k][0], o4[k][1], o4[k][2], o4[k][3]);
            }
            tc_fence_before();
            fence_async_smem();
            mbar_arrive(bar_out + 8 * b);
            TM_T(e7);
            TM_ACC(12, e6, e7);
        }
#ifdef HARP_TM_TIMING
        if (warp == 4 && lane == 0)
            for (int k = 7; k <= 12; ++k) atomicAdd((unsigned long long *)&g_tm_timing[k], (unsigned long long)acc[k]);
#endif
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------

struct TmPass {
    int fmt = FMT_C;
    int k0 = TM_I, k1 = -1, xpose = 0;
    int n_col_tiles = 0, lo_count = 1;
    uint8_t *d_frags = nullptr;
};

}  // namespace

struct TmPlan {
    std::vector<TmPass> pass[2];     // [0] forward, [1] transpose: the whole processor (empty if only the slab part exists)
    // the stages below stride 256 alone, on slabs of 256 contiguous coordinates (any d that is a multiple
    // of 256, identity permutation): the first pass of the two-pass paths for wide rows
    TmPass slab[2];
    bool has_slab = false;
    bool slab_shared = false;        // slab[] are copies of entries of pass[] (natural order, d = 256 or 4096)
    int slab_stages = 0;             // stages [0, slab_stages) are the slab's
    int32_t *d_err = nullptr;
    int n_sm = 0;
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    });
    return fn;
}

// A memory digit position holds one natural digit; tab maps the position's value to the digit's value.
struct Held {
    int digit;
    int tab[16];
};

struct Builder {
    const harp_plan *plan;
    int n_dig;                        // 2 (d = 256) or 3 (d = 4096)
    harp_fuse::HostPhase phase[3];    // natural digit -> stages
    Held held[3];                     // state of the memory positions
    int final_tab[3][16];             // transpose direction: table each digit must end with
    int dir;                          // 0 forward, 1 transpose
    int64_t wide_cols = 0;            // > 0: a slab pass of a wide row, tile column c = coordinates [256 c, 256 c + 256)
    std::vector<uint8_t> img;

    int64_t perm_of(int64_t i) const { return plan->h_perm.empty() ? i : plan->h_perm[(size_t)i]; }
    double sign_of(int64_t i) const { return plan->h_signs.empty() ? 1.0 : (double)plan->h_signs[(size_t)perm_of(i)]; }

    // fragments of one pass; positions: inner = 0, outer = po, tile column = the remaining position(s)
    bool add_pass(TmPlan *tp, int fmt, int k0, int k1, int xpose, TmPass *slab_out = nullptr) {
        const int po = fmt == FMT_C ? 1 : 2;                 // outer position
        const int pc = n_dig == 2 ? -1 : (fmt == FMT_C ? 2 : 1);   // position indexing the tile column
        const int n_col = wide_cols > 0 ? (int)wide_cols : (pc < 0 ? 1 : 16);
        const int nph = k1 < 0 ? 1 : 2;
        img.assign((size_t)n_col * nph * kFragBytes, 0);
        Held h[3] = {held[0], held[1], held[2]};
        for (int ph = 0; ph < nph; ++ph) {
            const int k = ph == 0 ? k0 : k1;
            const int pk = k == TM_I ? 0 : po;               // contracted position
            const int pb = k == TM_I ? po : 0;               // position indexing the block
            const int dg = h[pk].digit;
            const harp_fuse::HostPhase &hp = phase[dg];
            int nmap[16];
            for (int n = 0; n < 16; ++n) nmap[n] = dir == 0 ? n : final_tab[dg][n];
            std::vector<double> F;
            for (int col = 0; col < n_col; ++col)
                for (int blk = 0; blk < 16; ++blk) {
                    int64_t base = (int64_t)h[pb].tab[blk] * (phase[h[pb].digit].S);
                    if (wide_cols > 0) base += (int64_t)col * 256;
                    else if (pc >= 0) base += (int64_t)h[pc].tab[col] * (phase[h[pc].digit].S);
                    harp_fuse::fused_block(plan, hp, base, F);          // F[in][out] of the forward map
                    uint8_t *dst = img.data() + ((size_t)col * nph + ph) * kFragBytes + (size_t)blk * 512;
                    for (int n = 0; n < 16; ++n)
                        for (int kk = 0; kk < 16; ++kk) {
                            const int vin = h[pk].tab[kk], vout = nmap[n];   // digit values on the input / output side
                            double v;
                            if (dir == 0) {
                                v = F[(size_t)vin * 16 + vout];
                                if (hp.t0 == 0) v *= sign_of(base + (int64_t)vin * hp.S);
                            } else {
                                v = F[(size_t)vout * 16 + vin];
                                if (hp.t0 == 0) v *= sign_of(base + (int64_t)vout * hp.S);
                            }
                            const uint16_t bits = harp_fuse::f2bf(v);
                            std::memcpy(dst + (n / 8) * 256 + (kk / 8) * 128 + (n % 8) * 16 + (kk % 8) * 2, &bits, 2);
                        }
                }
            for (int n = 0; n < 16; ++n) h[pk].tab[n] = nmap[n];
        }
        if (xpose) std::swap(h[0], h[po]);
        for (int p = 0; p < 3; ++p) held[p] = h[p];
        TmPass ps;
        ps.fmt = fmt; ps.k0 = k0; ps.k1 = k1; ps.xpose = xpose;
        ps.n_col_tiles = n_col; ps.lo_count = 16;
        if (cudaMalloc(&ps.d_frags, img.size()) != cudaSuccess) { cudaGetLastError(); return false; }
        if (slab_out) *slab_out = ps;
        else tp->pass[dir].push_back(ps);
        if (cudaMemcpy(ps.d_frags, img.data(), img.size(), cudaMemcpyHostToDevice) != cudaSuccess) return false;
        return true;
    }
};

template <int FMT, int K0, int K1, int XP>
cudaError_t launch_one(const CUtensorMap &map, const TmParams &prm, int grid, size_t smem, cudaStream_t s) {
    static std::once_flag once;
    static cudaError_t attr = cudaSuccess;
    std::call_once(once, [&] {
        attr = cudaFuncSetAttribute(harp_tm_kernel<FMT, K0, K1, XP>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 1024);
    });
    if (attr != cudaSuccess) return attr;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute la[1];
    la[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    la[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = la;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, harp_tm_kernel<FMT, K0, K1, XP>, map, prm);
    return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace

void harp_tm_destroy(harp_plan *plan) {
    if (!plan->tm) return;
    for (int dir = 0; dir < 2; ++dir)
        for (TmPass &p : plan->tm->pass[dir])
            if (p.d_frags) cudaFree(p.d_frags);
    for (int dir = 0; dir < 2; ++dir)
        if (!plan->tm->slab_shared && plan->tm->slab[dir].d_frags) cudaFree(plan->tm->slab[dir].d_frags);
    if (plan->tm->d_err) cudaFree(plan->tm->d_err);
    delete plan->tm;
    plan->tm = nullptr;
}

harp_status_t harp_tm_build(harp_plan *plan) {
    const int64_t d = plan->d;
    if (d % 256 != 0) return HARP_ERR_UNSUPPORTED;
    if (!encode_fn()) return HARP_ERR_UNSUPPORTED;
    const bool whole = d == 256 || d == 4096;        // the whole processor as passes of this path
    const int n_dig = d == 256 ? 2 : 3;
    // group the stages into phases whose radices multiply to 16 (all of them, or the two below stride 256)
    Builder bld;
    bld.plan = plan;
    bld.n_dig = whole ? n_dig : 2;
    int t = 0;
    for (int dg = 0; dg < (whole ? n_dig : 2); ++dg) {
        int prod = 1, t0 = t;
        while (t < plan->st.m && prod < 16) prod *= plan->st.b[t++];
        if (prod != 16) return HARP_ERR_UNSUPPORTED;
        bld.phase[dg] = harp_fuse::HostPhase{t0, t, 16, plan->st.s[t0], 0, 1};
    }
    if (whole && t != plan->st.m) return HARP_ERR_UNSUPPORTED;
    if (!whole) {
        // wide row: only the slab part, on rows whose coordinates are already in the permuted order (the caller
        // moves them); the sign of a coordinate is read through the permutation (sign_of)
        TmPlan *tp = new (std::nothrow) TmPlan();
        if (!tp) return HARP_ERR_ALLOC;
        plan->tm = tp;
        Held ident[3];
        for (int p = 0; p < 3; ++p) { ident[p].digit = p; for (int v = 0; v < 16; ++v) ident[p].tab[v] = v; }
        for (int dg = 0; dg < 2; ++dg)
            for (int v = 0; v < 16; ++v) bld.final_tab[dg][v] = v;
        bld.wide_cols = d / 256;
        bool ok = true;
        for (int dir = 0; dir < 2 && ok; ++dir) {
            bld.dir = dir;
            for (int p = 0; p < 3; ++p) bld.held[p] = ident[p];
            ok = dir == 0 ? bld.add_pass(tp, FMT_C, TM_I, TM_O, 0, &tp->slab[0]) : bld.add_pass(tp, FMT_C, TM_O, TM_I, 0, &tp->slab[1]);
        }
        tp->has_slab = ok;
        tp->slab_stages = t;
        if (ok && cudaMalloc(&tp->d_err, sizeof(int32_t)) != cudaSuccess) ok = false;
        if (ok && cudaMemset(tp->d_err, 0, sizeof(int32_t)) != cudaSuccess) ok = false;
        if (ok && cudaDeviceGetAttribute(&tp->n_sm, cudaDevAttrMultiProcessorCount, plan->device) != cudaSuccess) ok = false;
        if (!ok) {
            cudaGetLastError();
            harp_tm_destroy(plan);
            return HARP_ERR_ALLOC;
        }
        return HARP_OK;
    }
    // the permutation must move whole 16-ary digits: position digit p of perm[i] depends on one digit of i
    Held init[3];
    int pos_of_digit[3] = {-1, -1, -1};
    for (int p = 0; p < n_dig; ++p) {
        int found = -1;
        for (int dg = 0; dg < n_dig && found < 0; ++dg) {
            int64_t w = 1;
            for (int k = 0; k < dg; ++k) w *= 16;
            int fwd[16];
            for (int v = 0; v < 16; ++v) fwd[v] = -1;
            bool ok = true;
            for (int64_t i = 0; i < d && ok; ++i) {
                int64_t x = plan->h_perm.empty() ? i : plan->h_perm[(size_t)i];
                for (int k = 0; k < p; ++k) x /= 16;
                const int xv = (int)(x % 16), iv = (int)((i / w) % 16);
                if (fwd[iv] < 0) fwd[iv] = xv;
                else if (fwd[iv] != xv) ok = false;
            }
            if (ok) {
                found = dg;
                init[p].digit = dg;
                for (int v = 0; v < 16; ++v) init[p].tab[fwd[v]] = v;     // position value -> digit value
            }
        }
        if (found < 0 || pos_of_digit[found] >= 0) return HARP_ERR_UNSUPPORTED;
        pos_of_digit[found] = p;
    }
    if (n_dig == 2) { init[2].digit = 2; for (int v = 0; v < 16; ++v) init[2].tab[v] = v; }
    const bool natural = pos_of_digit[0] == 0 && pos_of_digit[1] == 1 && (n_dig == 2 || pos_of_digit[2] == 2);
    const bool reversed = n_dig == 3 && pos_of_digit[0] == 2 && pos_of_digit[1] == 1 && pos_of_digit[2] == 0;
    if (!natural && !reversed) return HARP_ERR_UNSUPPORTED;

    TmPlan *tp = new (std::nothrow) TmPlan();
    if (!tp) return HARP_ERR_ALLOC;
    plan->tm = tp;
    bool ok = true;
    Held ident[3];
    for (int p = 0; p < 3; ++p) { ident[p].digit = p; for (int v = 0; v < 16; ++v) ident[p].tab[v] = v; }
    for (int dg = 0; dg < n_dig; ++dg)
        for (int v = 0; v < 16; ++v) bld.final_tab[dg][v] = init[pos_of_digit[dg]].tab[v];
    // forward: from the caller's order to the natural order, digits 0, 1, 2 in turn
    bld.dir = 0;
    for (int p = 0; p < 3; ++p) bld.held[p] = init[p];
    if (natural) {
        ok = ok && bld.add_pass(tp, FMT_C, TM_I, TM_O, 0);
        if (n_dig == 3) ok = ok && bld.add_pass(tp, FMT_S, TM_O, -1, 0);
    } else {
        ok = ok && bld.add_pass(tp, FMT_S, TM_O, -1, 1);      // digit 0 sits at position 2: contract, exchange with position 0
        ok = ok && bld.add_pass(tp, FMT_C, TM_O, -1, 0);
        ok = ok && bld.add_pass(tp, FMT_S, TM_O, -1, 0);
    }
    // transpose: from the natural order back to the caller's, digits 2, 1, 0
    bld.dir = 1;
    for (int p = 0; p < 3; ++p) bld.held[p] = ident[p];
    if (natural) {
        if (n_dig == 3) ok = ok && bld.add_pass(tp, FMT_S, TM_O, -1, 0);
        ok = ok && bld.add_pass(tp, FMT_C, TM_O, TM_I, 0);
    } else {
        ok = ok && bld.add_pass(tp, FMT_S, TM_O, -1, 0);
        ok = ok && bld.add_pass(tp, FMT_C, TM_O, -1, 0);
        ok = ok && bld.add_pass(tp, FMT_S, TM_I, -1, 1);
    }
    if (ok && natural && plan->h_perm.empty()) {
        // the pass over contiguous slabs is also the lower pass of the two-pass path
        tp->slab[0] = tp->pass[0].front();
        tp->slab[1] = tp->pass[1].back();
        tp->has_slab = tp->slab_shared = true;
        tp->slab_stages = bld.phase[1].t1;
    }
    if (ok && cudaMalloc(&tp->d_err, sizeof(int32_t)) != cudaSuccess) ok = false;
    if (ok && cudaMemset(tp->d_err, 0, sizeof(int32_t)) != cudaSuccess) ok = false;
    if (ok && cudaDeviceGetAttribute(&tp->n_sm, cudaDevAttrMultiProcessorCount, plan->device) != cudaSuccess) ok = false;
    if (!ok) {
        cudaGetLastError();
        harp_tm_destroy(plan);
        return HARP_ERR_ALLOC;
    }
    return HARP_OK;
}

namespace {

// tensor maps of one call: rows as 2-D boxes of 64 columns, and (d > 256) as 16 runs of 16 per row
harp_status_t encode_maps(void *x, int64_t n_rows, int64_t d, bool need_s, CUtensorMap *map_c, CUtensorMap *map_s) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return HARP_ERR_UNSUPPORTED;
    const cuuint32_t ones[3] = {1, 1, 1};
    {
        const cuuint64_t gdim[2] = {(cuuint64_t)d, (cuuint64_t)n_rows};
        const cuuint64_t gstr[1] = {(cuuint64_t)d * 2};
        const cuuint32_t box[2] = {64, 128};
        if (enc(map_c, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x, gdim, gstr, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return HARP_ERR_CUDA;
    }
    if (need_s) {
        // coordinates as (e within a run of 256, row, run): 16 elements of each of 16 runs per row
        const cuuint64_t gdim[3] = {256, (cuuint64_t)n_rows, (cuuint64_t)(d / 256)};
        const cuuint64_t gstr[2] = {(cuuint64_t)d * 2, 512};
        const cuuint32_t box[3] = {16, 128, 16};
        if (enc(map_s, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, x, gdim, gstr, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return HARP_ERR_CUDA;
    }
    return HARP_OK;
}

harp_status_t run_pass(const TmPlan *tp, const TmPass &ps, const CUtensorMap &map, int64_t n_rows, cudaStream_t stream) {
    const int n_row_tiles = (int)((n_rows + kRows - 1) / kRows);
    TmParams prm;
    prm.frags = ps.d_frags;
    prm.n_row_tiles = n_row_tiles;
    prm.n_col_tiles = ps.n_col_tiles;
    prm.lo_count = ps.lo_count;
    prm.err = tp->d_err;
    const int64_t n_tiles = (int64_t)n_row_tiles * ps.n_col_tiles;
    const int grid = (int)std::min<int64_t>(n_tiles, tp->n_sm);
    prm.tiles_per_cta = (int)((n_tiles + grid - 1) / grid);
    const int nph = ps.k1 < 0 ? 1 : 2;
    const size_t smem = 1024 + (size_t)kNBuf * kTileBytes + 2 * (size_t)nph * kFragBytes;
    cudaError_t e = cudaErrorInvalidValue;
    if (ps.fmt == FMT_C && ps.k0 == TM_I && ps.k1 == TM_O) e = launch_one<FMT_C, TM_I, TM_O, 0>(map, prm, grid, smem, stream);
    else if (ps.fmt == FMT_C && ps.k0 == TM_O && ps.k1 == TM_I) e = launch_one<FMT_C, TM_O, TM_I, 0>(map, prm, grid, smem, stream);
    else if (ps.fmt == FMT_C && ps.k0 == TM_O && ps.k1 < 0) e = launch_one<FMT_C, TM_O, -1, 0>(map, prm, grid, smem, stream);
    else if (ps.fmt == FMT_S && ps.k0 == TM_O && ps.k1 < 0 && !ps.xpose) e = launch_one<FMT_S, TM_O, -1, 0>(map, prm, grid, smem, stream);
    else if (ps.fmt == FMT_S && ps.k0 == TM_O && ps.k1 < 0 && ps.xpose) e = launch_one<FMT_S, TM_O, -1, 1>(map, prm, grid, smem, stream);
    else if (ps.fmt == FMT_S && ps.k0 == TM_I && ps.k1 < 0 && ps.xpose) e = launch_one<FMT_S, TM_I, -1, 1>(map, prm, grid, smem, stream);
    if (e != cudaSuccess) return HARP_ERR_CUDA;
    g_harp_launches.fetch_add(1, std::memory_order_relaxed);
    return HARP_OK;
}

bool tm_args_ok(const void *x, int64_t n_rows, harp_dtype_t dtype) {
    return dtype == HARP_BF16 && (reinterpret_cast<uintptr_t>(x) & 15u) == 0 && n_rows <= ((int64_t)1 << 30);
}

}  // namespace

harp_status_t harp_tm_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype, int transpose,
                            cudaStream_t stream) {
    const TmPlan *tp = plan->tm;
    if (!tp || tp->pass[0].empty() || !tm_args_ok(x, n_rows, dtype)) return HARP_ERR_UNSUPPORTED;
    CUtensorMap map_c, map_s;
    harp_status_t st = encode_maps(x, n_rows, plan->d, plan->d > 256, &map_c, &map_s);
    for (const TmPass &ps : tp->pass[transpose ? 1 : 0])
        if (st == HARP_OK) st = run_pass(tp, ps, ps.fmt == FMT_C ? map_c : map_s, n_rows, stream);
    return st;
}

// Stages [0, harp_tm_slab_stages) only -- those below stride 256, with the sign diagonal -- on slabs of 256
// contiguous coordinates (identity permutation): the lower pass of the two-pass paths for wide rows.
int harp_tm_slab_stages(const harp_plan *plan) {
    const TmPlan *tp = plan->tm;
    if (!tp) return 0;
    if (tp->has_slab) return tp->slab_stages;
    return 0;
}

harp_status_t harp_tm_slab_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype, int transpose,
                                 cudaStream_t stream) {
    const TmPlan *tp = plan->tm;
    if (!tp || !tp->has_slab || !tm_args_ok(x, n_rows, dtype)) return HARP_ERR_UNSUPPORTED;
    CUtensorMap map_c, map_s;
    const harp_status_t st = encode_maps(x, n_rows, plan->d, false, &map_c, &map_s);
    if (st != HARP_OK) return st;
    return run_pass(tp, tp->slab[transpose ? 1 : 0], map_c, n_rows, stream);
}

// Copies the per-section cycle counters to out[16] (zeros unless built with -DHARP_TM_TIMING) and
// clears them if asked.
extern "C" int32_t harp_debug_tm_timing(int64_t *out, int32_t reset) {
    if (!out) return -1;
    if (cudaMemcpyFromSymbol(out, g_tm_timing, sizeof(long long) * 16) != cudaSuccess) return -1;
    if (reset) {
        const long long zero[16] = {0};
        if (cudaMemcpyToSymbol(g_tm_timing, zero, sizeof(zero)) != cudaSuccess) return -1;
    }
    return 0;
}

// Non-zero if a kernel of this plan's tensor-memory path gave up on a wait since the plan was built
// (synchronises the device copy of the error word; for tests).
int32_t harp_tm_error_word(const harp_plan *plan) {
    if (!plan->tm || !plan->tm->d_err) return 0;
    int32_t v = 0;
    if (cudaMemcpy(&v, plan->tm->d_err, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
    return v;
}
