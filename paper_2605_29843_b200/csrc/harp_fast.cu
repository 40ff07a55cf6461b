// Tensor-core path for bf16 rows (sm_100a).
//
// Plan time: adjacent stages are fused into "phases" whose dense block has size
// B in {8, 16} (two radix-4 stages -> one 16x16 block, four radix-2 stages -> 16x16, one
// radix-8 stage -> 8x8, ...).  A fused block is the product of its stages' kernels on the B
// coordinates it touches, computed in fp64 and rounded once to bf16; the sign diagonal is
// folded into the first phase.  Per phase the blocks are stored in the register layout of
// mma.sync (one 16-byte load per lane and block).
//
// Run time: a CTA keeps a tile of 16 whole rows in shared memory as bf16 (one HBM read and
// one HBM write per row) and runs the phases on it.  A phase is a batch of tiny GEMMs
// out[16 rows x B] = in[16 rows x B] . F_c[B x B] (fp32 accumulate), one per block c, with
// the 16 rows as the M dimension of mma.sync.m16n8k16.  Coordinates of a block that are
// not adjacent in memory are fetched for eight neighbouring blocks at once with 16-byte
// loads and re-paired with byte permutes, so that shared memory is only touched with
// 16-byte, bank-conflict-free accesses; every thread writes exactly the locations it
// read, so a phase needs no barrier between its loads and stores.
//
// Permutations.  Identity: the tile is copied in and out with coalesced 16-byte accesses.
// Mixed-radix digit reversal of the plan's own schedule: the tile is copied in coalesced in
// source order, the phases run in place on the source-ordered layout (a digit reversal
// maps every phase onto a digit group again, only with other strides), and the one phase
// next to the output does the reordering inside shared memory: all of its operands are
// read into registers, the CTA synchronises, and the results are written in output order.
// Any other permutation that maps every aligned run of eight source coordinates onto the
// same slot of eight different first-phase blocks is gathered (forward) or scattered
// (transpose) in global memory with 16-byte accesses by the first/last phase.  All other
// permutations use the generic kernel.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>

#include "harp_internal.h"
#include "harp_mma.cuh"
#include "harp_fuse.h"

namespace {

constexpr int kMaxPhases = 8;
constexpr int kTileRows = 16;
constexpr int kThreads = 512;

enum PhaseMode : int32_t {
    MODE_CC = 0,   // contiguous block in shared memory, in place (ldmatrix / stmatrix)
    MODE_SS = 1,   // strided block in shared memory, eight blocks per item, in place
    MODE_GS = 2,   // operands gathered from global memory, result to contiguous smem blocks
    MODE_CG = 3,   // operands from contiguous smem blocks, result scattered to global memory
    MODE_PO = 4,   // contiguous smem blocks in, CTA barrier, strided smem out (reorders the tile)
    MODE_PI = 5    // strided smem in, CTA barrier, contiguous smem blocks out (reorders the tile)
};

struct PhaseDesc {
    const uint4 *bfrag;        // [item][block in item][lane] fragments
    int32_t items_off;         // index of the per-item table inside FastParams::tables
    int32_t n_items;
    int32_t mode;
    int32_t B;                 // 8 or 16
    int32_t lane_step;         // element offset between the slots of lanes q and q+1
    int32_t j_off[4];          // element offsets of a lane's slots
};

struct FastParams {
    int32_t n_phases;
    int32_t d;
    int32_t pitch;             // elements per shared-memory row
    int32_t copy_in;           // table offset of the chunk map used to load the tile, or -1
    int32_t copy_out;          // table offset of the chunk map used to store the tile, or -1
    // tables, copied to shared memory when the kernel starts: chunk maps (shared-memory element
    // offset of every 8-coordinate chunk of a row) and the per-phase item tables
    const int32_t *tables;
    int32_t tables_len;
    PhaseDesc ph[kMaxPhases];
};

// ----------------------------------------------------------------------------- device

struct TileCtx {
    uint32_t sbase;          // shared address of the tile
    const int32_t *tab;      // tables in shared memory
    int pitch, lane, warp, g, q;
    __nv_bfloat16 *xA, *xB;  // global rows g and g+8 of the tile (clamped to the batch)
    bool okA, okB;
};

// ---- MODE_SS, B = 16: load / store of one item's operands
__device__ __forceinline__ void ss16_load(const TileCtx &c, const PhaseDesc &ph, int it, uint4 (&raw)[4][2], uint4 (&bf)[8]) {
    const uint32_t a0 = c.sbase + 2u * (uint32_t)(c.g * c.pitch + c.q * ph.lane_step + c.tab[ph.items_off + it]);
    const uint32_t a1 = a0 + 2u * (uint32_t)(8 * c.pitch);
    const uint4 *bp = ph.bfrag + (size_t)it * 256 + c.lane;
#pragma unroll
    for (int e = 0; e < 8; ++e) bf[e] = __ldg(bp + e * 32);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        raw[j][0] = lds128(a0 + 2u * ph.j_off[j]);
        raw[j][1] = lds128(a1 + 2u * ph.j_off[j]);
    }
}
__device__ __forceinline__ void ss16_store(const TileCtx &c, const PhaseDesc &ph, int it, const uint4 (&raw)[4][2]) {
    const uint32_t a0 = c.sbase + 2u * (uint32_t)(c.g * c.pitch + c.q * ph.lane_step + c.tab[ph.items_off + it]);
    const uint32_t a1 = a0 + 2u * (uint32_t)(8 * c.pitch);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        sts128(a0 + 2u * ph.j_off[j], raw[j][0]);
        sts128(a1 + 2u * ph.j_off[j], raw[j][1]);
    }
}
// ---- MODE_GS: operands from global memory
__device__ __forceinline__ void gs_load(const TileCtx &c, const PhaseDesc &ph, int it, uint4 (&raw)[4][2], uint4 (&bf)[8]) {
    const int32_t *tab = c.tab + ph.items_off + it * 24;
    const uint4 *bp = ph.bfrag + (size_t)it * 256 + c.lane;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int off = tab[c.q * ph.lane_step + ph.j_off[j]];
        raw[j][0] = ldg128_stream(c.xA + off);
        raw[j][1] = ldg128_stream(c.xB + off);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) bf[e] = __ldg(bp + e * 32);
}
__device__ __forceinline__ void gs_store(const TileCtx &c, const PhaseDesc &ph, int it, const uint32_t (&mats)[8][4]) {
    const int32_t *tab = c.tab + ph.items_off + it * 24 + 16;
    const int mrow = (c.lane & 7) + ((c.lane >> 3) & 1) * 8, mcol = (c.lane >> 4) * 8;
#pragma unroll
    for (int e = 0; e < 8; ++e)
        stmatrix_x4(c.sbase + 2u * (uint32_t)(mrow * c.pitch + tab[e] + mcol), mats[e][0], mats[e][1], mats[e][2], mats[e][3]);
}

template <int NT>
__global__ void __launch_bounds__(NT, 1)
harp_fast_kernel(__nv_bfloat16 *__restrict__ x, int64_t n_rows, int64_t n_tiles, FastParams P) {
    constexpr int NW = NT / 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TileCtx c;
    c.sbase = smem_u32(smem_raw);
    c.pitch = P.pitch;
    c.lane = threadIdx.x & 31;
    c.warp = threadIdx.x >> 5;
    c.g = c.lane >> 2;
    c.q = c.lane & 3;
    const int d = P.d, pitch = P.pitch;
    int32_t *tab_s = reinterpret_cast<int32_t *>(smem_raw + (size_t)kTileRows * pitch * 2);
    for (int i = threadIdx.x; i < P.tables_len; i += NT) tab_s[i] = __ldg(P.tables + i);
    c.tab = tab_s;
    __syncthreads();
    const int warp = c.warp, lane = c.lane;

    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int64_t row0 = tile * kTileRows;
        // rows past the end of the batch are computed on a copy of the last row and never stored
        const int64_t last = n_rows - 1;
        c.okA = row0 + c.g < n_rows;
        c.okB = row0 + c.g + 8 < n_rows;
        c.xA = x + min(row0 + c.g, last) * d;
        c.xB = x + min(row0 + c.g + 8, last) * d;

        if (P.copy_in >= 0) {
            // a thread owns the same 16-byte chunks of every row; no index arithmetic per chunk
            const int32_t *cmap = tab_s + P.copy_in;
            const int chunks = d >> 3;
            for (int ch = threadIdx.x; ch < chunks; ch += NT) {
                const uint32_t dst = c.sbase + 2u * (uint32_t)cmap[ch];
                const __nv_bfloat16 *src = x + row0 * d + 8 * ch;
                const __nv_bfloat16 *last_src = x + last * d + 8 * ch;
#pragma unroll 4
                for (int r = 0; r < kTileRows; ++r)
                    cp_async16(dst + 2u * (uint32_t)(r * pitch), row0 + r <= last ? src + (int64_t)r * d : last_src);
            }
            cp_async_wait_all();
            __syncthreads();
        }

        for (int p = 0; p < P.n_phases; ++p) {
            const PhaseDesc &ph = P.ph[p];
            const int n = ph.n_items;
            if (ph.mode == MODE_CC) {
                // lane -> (matrix row, 8-column half) of the 16x16 (or 16x8) operand tile
                const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
                if (ph.B == 16) {
#pragma unroll 4
                    for (int it = warp; it < n; it += NW) {
                        const uint32_t addr = c.sbase + 2u * (uint32_t)(mrow * pitch + tab_s[ph.items_off + it] + mcol);
                        const uint4 bf = __ldg(ph.bfrag + (size_t)it * 32 + lane);
                        uint32_t a[4];
                        ldmatrix_x4(a, addr);
                        float c0[4], c1[4];
                        mma_k16(c0, a, bf.x, bf.y);
                        mma_k16(c1, a, bf.z, bf.w);
                        stmatrix_x4(addr, pack_bf16(c0[0], c0[1]), pack_bf16(c0[2], c0[3]), pack_bf16(c1[0], c1[1]),
                                    pack_bf16(c1[2], c1[3]));
                    }
                } else {
                    const uint32_t *bf8 = reinterpret_cast<const uint32_t *>(ph.bfrag);
                    const int mrow2 = (lane & 15);
#pragma unroll 4
                    for (int it = warp; it < n; it += NW) {
                        const uint32_t addr = c.sbase + 2u * (uint32_t)(mrow2 * pitch + tab_s[ph.items_off + it]);
                        const uint32_t bf = __ldg(bf8 + (size_t)it * 32 + lane);
                        uint32_t a[2];
                        ldmatrix_x2(a, addr);
                        float c0[4];
                        mma_k8(c0, a, bf);
                        stmatrix_x2(addr, pack_bf16(c0[0], c0[1]), pack_bf16(c0[2], c0[3]));
                    }
                }
            } else if (ph.mode == MODE_SS && ph.B == 16) {
                // software pipeline over this warp's items: operands of the next item are in
                // flight while the current one is multiplied
                uint4 rawA[4][2], rawB[4][2], bfA[8], bfB[8];
                uint32_t unused[8][4];
                int it = warp;
                {
                    for (; it < n; it += NW) {
                        ss16_load(c, ph, it, rawA, bfA);
                        octet_mma16<true>(rawA, bfA, unused);
                        ss16_store(c, ph, it, rawA);
                    }
                }
                if (false && it < n) ss16_load(c, ph, it, rawA, bfA);
                while (false && it < n) {
                    const int it2 = it + NW;
                    if (it2 < n) ss16_load(c, ph, it2, rawB, bfB);
                    octet_mma16<true>(rawA, bfA, unused);
                    ss16_store(c, ph, it, rawA);
                    if (it2 >= n) break;
                    const int it3 = it2 + NW;
                    if (it3 < n) ss16_load(c, ph, it3, rawA, bfA);
                    octet_mma16<true>(rawB, bfB, unused);
                    ss16_store(c, ph, it2, rawB);
                    it = it3;
                }
            } else if (ph.mode == MODE_SS) {
                const uint32_t *bf8 = reinterpret_cast<const uint32_t *>(ph.bfrag);
                for (int it = warp; it < n; it += NW) {
                    const uint32_t a0 = c.sbase + 2u * (uint32_t)(c.g * pitch + c.q * ph.lane_step + tab_s[ph.items_off + it]);
                    const uint32_t a1 = a0 + 2u * (uint32_t)(8 * pitch);
                    uint4 raw[2][2];
                    uint32_t bf[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) bf[e] = __ldg(bf8 + (size_t)it * 256 + e * 32 + lane);
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        raw[j][0] = lds128(a0 + 2u * ph.j_off[j]);
                        raw[j][1] = lds128(a1 + 2u * ph.j_off[j]);
                    }
                    octet_mma8(raw, bf);
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        sts128(a0 + 2u * ph.j_off[j], raw[j][0]);
                        sts128(a1 + 2u * ph.j_off[j], raw[j][1]);
                    }
                }
            } else if (ph.mode == MODE_GS) {
                uint4 rawA[4][2], rawB[4][2], bfA[8], bfB[8];
                uint32_t mats[8][4];
                int it = warp;
                {
                    for (; it < n; it += NW) {
                        gs_load(c, ph, it, rawA, bfA);
                        octet_mma16<false>(rawA, bfA, mats);
                        gs_store(c, ph, it, mats);
                    }
                }
                if (false && it < n) gs_load(c, ph, it, rawA, bfA);
                while (false && it < n) {
                    const int it2 = it + NW;
                    if (it2 < n) gs_load(c, ph, it2, rawB, bfB);
                    octet_mma16<false>(rawA, bfA, mats);
                    gs_store(c, ph, it, mats);
                    if (it2 >= n) break;
                    const int it3 = it2 + NW;
                    if (it3 < n) gs_load(c, ph, it3, rawA, bfA);
                    octet_mma16<false>(rawB, bfB, mats);
                    gs_store(c, ph, it2, mats);
                    it = it3;
                }
            } else if (ph.mode == MODE_PO) {
                // every operand of the phase is read before the barrier, every result is written
                // after it; a warp owns at most two items: the first is multiplied before the
                // barrier, the second only loaded
                const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
                const int it0 = warp, it1 = warp + NW;
                uint4 out[4][2];
                uint32_t a1[8][4];
                if (it0 < n) {
                    const int32_t *tab = tab_s + ph.items_off + it0 * 12;
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        float acc[2][2][4];
#pragma unroll
                        for (int ee = 0; ee < 2; ++ee) {
                            const int e = 2 * w + ee;
                            const uint4 bf = __ldg(ph.bfrag + (size_t)it0 * 256 + e * 32 + lane);
                            uint32_t a[4];
                            ldmatrix_x4(a, c.sbase + 2u * (uint32_t)(mrow * pitch + tab[e] + mcol));
                            mma_k16(acc[ee][0], a, bf.x, bf.y);
                            mma_k16(acc[ee][1], a, bf.z, bf.w);
                        }
#pragma unroll
                        for (int k = 0; k < 2; ++k)
#pragma unroll
                            for (int i = 0; i < 2; ++i)
#pragma unroll
                                for (int h = 0; h < 2; ++h)
                                    set_word(out[i + 2 * k][h], w, pack_bf16(acc[0][k][i + 2 * h], acc[1][k][i + 2 * h]));
                    }
                }
                if (it1 < n) {
                    const int32_t *tab = tab_s + ph.items_off + it1 * 12;
#pragma unroll
                    for (int e = 0; e < 8; ++e) ldmatrix_x4(a1[e], c.sbase + 2u * (uint32_t)(mrow * pitch + tab[e] + mcol));
                }
                __syncthreads();
                if (it0 < n) {
                    const uint32_t o0 = c.sbase + 2u * (uint32_t)(c.g * pitch + c.q * ph.lane_step + tab_s[ph.items_off + it0 * 12 + 8]);
                    const uint32_t o1 = o0 + 2u * (uint32_t)(8 * pitch);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        sts128(o0 + 2u * ph.j_off[j], out[j][0]);
                        sts128(o1 + 2u * ph.j_off[j], out[j][1]);
                    }
                }
                if (it1 < n) {
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        float acc[2][2][4];
#pragma unroll
                        for (int ee = 0; ee < 2; ++ee) {
                            const int e = 2 * w + ee;
                            const uint4 bf = __ldg(ph.bfrag + (size_t)it1 * 256 + e * 32 + lane);
                            mma_k16(acc[ee][0], a1[e], bf.x, bf.y);
                            mma_k16(acc[ee][1], a1[e], bf.z, bf.w);
                        }
#pragma unroll
                        for (int k = 0; k < 2; ++k)
#pragma unroll
                            for (int i = 0; i < 2; ++i)
#pragma unroll
                                for (int h = 0; h < 2; ++h)
                                    set_word(out[i + 2 * k][h], w, pack_bf16(acc[0][k][i + 2 * h], acc[1][k][i + 2 * h]));
                    }
                    const uint32_t o0 = c.sbase + 2u * (uint32_t)(c.g * pitch + c.q * ph.lane_step + tab_s[ph.items_off + it1 * 12 + 8]);
                    const uint32_t o1 = o0 + 2u * (uint32_t)(8 * pitch);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        sts128(o0 + 2u * ph.j_off[j], out[j][0]);
                        sts128(o1 + 2u * ph.j_off[j], out[j][1]);
                    }
                }
            } else if (ph.mode == MODE_PI) {
                const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
                const int it0 = warp, it1 = warp + NW;
                uint32_t mats[8][4];
                uint4 raw1[4][2];
                if (it0 < n) {
                    const uint32_t i0 = c.sbase + 2u * (uint32_t)(c.g * pitch + c.q * ph.lane_step + tab_s[ph.items_off + it0 * 12 + 8]);
                    const uint32_t i1 = i0 + 2u * (uint32_t)(8 * pitch);
                    uint4 raw[4][2], bf[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) bf[e] = __ldg(ph.bfrag + (size_t)it0 * 256 + e * 32 + lane);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        raw[j][0] = lds128(i0 + 2u * ph.j_off[j]);
                        raw[j][1] = lds128(i1 + 2u * ph.j_off[j]);
                    }
                    octet_mma16<false>(raw, bf, mats);
                }
                if (it1 < n) {
                    const uint32_t i0 = c.sbase + 2u * (uint32_t)(c.g * pitch + c.q * ph.lane_step + tab_s[ph.items_off + it1 * 12 + 8]);
                    const uint32_t i1 = i0 + 2u * (uint32_t)(8 * pitch);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        raw1[j][0] = lds128(i0 + 2u * ph.j_off[j]);
                        raw1[j][1] = lds128(i1 + 2u * ph.j_off[j]);
                    }
                }
                __syncthreads();
                if (it0 < n) {
                    const int32_t *tab = tab_s + ph.items_off + it0 * 12;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        stmatrix_x4(c.sbase + 2u * (uint32_t)(mrow * pitch + tab[e] + mcol), mats[e][0], mats[e][1], mats[e][2], mats[e][3]);
                }
                if (it1 < n) {
                    uint4 bf[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) bf[e] = __ldg(ph.bfrag + (size_t)it1 * 256 + e * 32 + lane);
                    octet_mma16<false>(raw1, bf, mats);
                    const int32_t *tab = tab_s + ph.items_off + it1 * 12;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        stmatrix_x4(c.sbase + 2u * (uint32_t)(mrow * pitch + tab[e] + mcol), mats[e][0], mats[e][1], mats[e][2], mats[e][3]);
                }
            } else {   // MODE_CG: operands from contiguous smem blocks, results scattered to global memory
                const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
                for (int it = warp; it < n; it += NW) {
                    const int32_t *tab = tab_s + ph.items_off + it * 24;
                    uint4 bf[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) bf[e] = __ldg(ph.bfrag + (size_t)it * 256 + e * 32 + lane);
                    uint4 out[4][2];
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        float acc[2][2][4];
#pragma unroll
                        for (int ee = 0; ee < 2; ++ee) {
                            const int e = 2 * w + ee;
                            uint32_t a[4];
                            ldmatrix_x4(a, c.sbase + 2u * (uint32_t)(mrow * pitch + tab[16 + e] + mcol));
                            mma_k16(acc[ee][0], a, bf[e].x, bf[e].y);
                            mma_k16(acc[ee][1], a, bf[e].z, bf[e].w);
                        }
#pragma unroll
                        for (int k = 0; k < 2; ++k)
#pragma unroll
                            for (int i = 0; i < 2; ++i)
#pragma unroll
                                for (int h = 0; h < 2; ++h)
                                    set_word(out[i + 2 * k][h], w, pack_bf16(acc[0][k][i + 2 * h], acc[1][k][i + 2 * h]));
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int off = tab[c.q * ph.lane_step + ph.j_off[j]];
                        if (c.okA) stg128(c.xA + off, out[j][0]);
                        if (c.okB) stg128(c.xB + off, out[j][1]);
                    }
                }
            }
            __syncthreads();
        }

        if (P.copy_out >= 0) {
            const int32_t *cmap = tab_s + P.copy_out;
            const int chunks = d >> 3;
            const int rows = (int)min((int64_t)kTileRows, n_rows - row0);
            for (int ch = threadIdx.x; ch < chunks; ch += NT) {
                const uint32_t src = c.sbase + 2u * (uint32_t)cmap[ch];
                __nv_bfloat16 *dst = x + row0 * d + 8 * ch;
#pragma unroll 4
                for (int r = 0; r < rows; ++r) stg128(dst + (int64_t)r * d, lds128(src + 2u * (uint32_t)(r * pitch)));
            }
            __syncthreads();
        }
    }
}

}  // namespace

// ----------------------------------------------------------------------------- host

struct FastPlan {
    FastParams fwd{}, bwd{};
    size_t smem_bytes = 0;
    std::vector<void *> dev_allocs;
    int max_ctas = 0;
};

namespace {

using namespace harp_fuse;

template <typename T>
T *upload(FastPlan *fp, const std::vector<T> &v, harp_status_t &st) {
    if (st != HARP_OK) return nullptr;
    void *p = nullptr;
    if (cudaMalloc(&p, std::max<size_t>(16, v.size() * sizeof(T))) != cudaSuccess) { st = HARP_ERR_ALLOC; return nullptr; }
    fp->dev_allocs.push_back(p);
    if (!v.empty() && cudaMemcpy(p, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) st = HARP_ERR_CUDA;
    return static_cast<T *>(p);
}

}  // namespace

harp_status_t harp_fast_build(harp_plan *plan) {
    const int64_t d = plan->d;
    const int m = plan->st.m;
    if (d % 8 != 0) return HARP_ERR_UNSUPPORTED;

    // ---- group stages into phases with fused size 8 or 16
    std::vector<HostPhase> phases;
    {
        int t = 0;
        while (t < m) {
            int64_t prod = 1;
            int t1 = t;
            while (t1 < m && prod * plan->st.b[t1] <= 16) prod *= plan->st.b[t1++];
            if (prod != 8 && prod != 16) return HARP_ERR_UNSUPPORTED;
            phases.push_back({t, t1, (int)prod, plan->st.s[t], 0, 1});
            t = t1;
        }
    }
    const int np = (int)phases.size();
    if (np > kMaxPhases) return HARP_ERR_UNSUPPORTED;

    // ---- permutation kind
    const bool identity = plan->h_perm.empty();
    bool digitrev = false;
    if (!identity && np >= 2 && phases[0].B == 16 && phases[np - 1].B == 16) {
        digitrev = true;
        for (int64_t i = 0; i < d && digitrev; ++i) {
            int64_t rem = i, src = 0, w = d;
            for (int t = 0; t < m; ++t) {
                w /= plan->st.b[t];
                src += (rem % plan->st.b[t]) * w;
                rem /= plan->st.b[t];
            }
            digitrev = plan->h_perm[(size_t)i] == src;
        }
        if (d / 16 / 8 > 2 * (kThreads / 32)) digitrev = false;      // a warp holds at most two items over the barrier
    }
    std::vector<int64_t> inv;                                        // source coordinate -> natural coordinate
    if (!identity) {
        inv.resize((size_t)d);
        for (int64_t i = 0; i < d; ++i) inv[(size_t)plan->h_perm[(size_t)i]] = i;
    }

    // ---- shared-memory layouts.  "nat": coordinates in the plan's own order; "src": in the
    // order of the rows in global memory before the gather (digit-reversal scheme only).
    // A layout gives every phase's local index an element stride W with W/8 mod 8 not in {0,4}.
    struct Layout {
        std::vector<int64_t> S, W;      // per phase: coordinate stride and shared-memory stride
        std::vector<int> lm;            // per phase: lane multiplier (1 or 2)
        int64_t extent = 0;
    };
    auto make_layout = [&](const std::vector<int> &order, const std::vector<int64_t> &strides) {
        Layout L;
        L.S = strides;
        L.W.assign((size_t)np, 0);
        L.lm.assign((size_t)np, 1);
        int64_t W = 1;
        bool first = true;
        for (int p : order) {
            if (!first) {
                W = (W + 7) / 8 * 8;
                while (((W / 8) % 8) == 0 || ((W / 8) % 8) == 4) W += 8;
                L.lm[(size_t)p] = ((W / 8) % 2 == 0) ? 1 : 2;
            }
            first = false;
            L.W[(size_t)p] = W;
            W *= phases[(size_t)p].B;
        }
        L.extent = W;
        return L;
    };
    std::vector<int> order_nat((size_t)np), order_src((size_t)np);
    std::vector<int64_t> S_nat((size_t)np), S_src((size_t)np);
    for (int p = 0; p < np; ++p) {
        order_nat[(size_t)p] = p;
        order_src[(size_t)p] = np - 1 - p;
        S_nat[(size_t)p] = phases[(size_t)p].S;
        S_src[(size_t)p] = d / (phases[(size_t)p].S * phases[(size_t)p].B);   // prod of radices above the phase
    }
    const Layout Lnat = make_layout(order_nat, S_nat);
    const Layout Lsrc = digitrev ? make_layout(order_src, S_src) : Lnat;
    int64_t pitch = (std::max(Lnat.extent, Lsrc.extent) + 7) / 8 * 8;
    if ((pitch / 8) % 2 == 0) pitch += 8;
    const size_t tile_bytes = (size_t)kTileRows * pitch * 2;
    if (tile_bytes > 227u * 1024u) return HARP_ERR_UNSUPPORTED;

    // local index of phase p: natural r <-> source r' (digits of the group in reverse order)
    auto nat_local_of_src_local = [&](int p, int rs) {
        const HostPhase &hp = phases[(size_t)p];
        int r = 0, wsrc = hp.B;
        int64_t wnat = 1;
        for (int t = hp.t0; t < hp.t1; ++t) {
            wsrc /= plan->st.b[t];
            r += (int)(((rs / wsrc) % plan->st.b[t]) * wnat);
            wnat *= plan->st.b[t];
        }
        return r;
    };
    auto phys_nat = [&](int64_t pos) {
        int64_t o = 0;
        for (int p = 0; p < np; ++p) o += ((pos / Lnat.S[(size_t)p]) % phases[(size_t)p].B) * Lnat.W[(size_t)p];
        return o;
    };
    // source coordinate j: its phase-p source-local index is (j / S_src[p]) % B_p, written with the
    // group's digits reversed; the layout only needs that index
    auto phys_src = [&](int64_t j) {
        int64_t o = 0;
        for (int p = 0; p < np; ++p) o += ((j / Lsrc.S[(size_t)p]) % phases[(size_t)p].B) * Lsrc.W[(size_t)p];
        return o;
    };

    // ---- first-phase octets for the global gather/scatter scheme
    const int B0 = phases[0].B;
    const int64_t nblk0 = d / B0;
    std::vector<std::vector<int64_t>> octets;
    if (!identity && !digitrev) {
        if (B0 != 16 || nblk0 % 8 != 0) return HARP_ERR_UNSUPPORTED;
        std::vector<int64_t> order((size_t)nblk0);
        for (int64_t c = 0; c < nblk0; ++c) order[(size_t)c] = c;
        const int32_t *pm = plan->h_perm.data();
        std::sort(order.begin(), order.end(), [&](int64_t a, int64_t b) { return pm[a * B0] < pm[b * B0]; });
        for (int64_t i = 0; i < nblk0; i += 8) {
            std::vector<int64_t> oc(order.begin() + i, order.begin() + i + 8);
            for (int r = 0; r < B0; ++r) {
                const int32_t s0 = pm[oc[0] * B0 + r];
                if (s0 % 8 != 0) return HARP_ERR_UNSUPPORTED;
                for (int e = 1; e < 8; ++e)
                    if (pm[oc[(size_t)e] * B0 + r] != s0 + e) return HARP_ERR_UNSUPPORTED;
            }
            octets.push_back(oc);
        }
    }

    FastPlan *fp = new (std::nothrow) FastPlan();
    if (!fp) return HARP_ERR_ALLOC;
    harp_status_t st = HARP_OK;

    std::vector<int32_t> chunk_nat((size_t)(d / 8)), chunk_src((size_t)(d / 8));
    for (int64_t c = 0; c < d / 8; ++c) {
        chunk_nat[(size_t)c] = (int32_t)phys_nat(8 * c);
        chunk_src[(size_t)c] = (int32_t)phys_src(8 * c);
    }

    auto sign_v = [&](int64_t i) -> double {             // sign seen by coordinate i after the gather
        if (plan->h_signs.empty()) return 1.0;
        const int64_t src = identity ? i : plan->h_perm[(size_t)i];
        return (double)plan->h_signs[(size_t)src];
    };
    static const int joff1_16[4] = {0, 4, 8, 12}, joff2_16[4] = {0, 1, 8, 9};
    static const int joff1_8[4] = {0, 4, 0, 0}, joff2_8[4] = {0, 1, 0, 0};

    for (int dir = 0; dir < 2 && st == HARP_OK; ++dir) {  // 0 = forward, 1 = transpose
        FastParams &P = dir == 0 ? fp->fwd : fp->bwd;
        P.n_phases = np;
        P.d = (int32_t)d;
        P.pitch = (int32_t)pitch;
        std::vector<int32_t> tables(chunk_nat);
        const int32_t off_nat = 0;
        const int32_t off_src = (int32_t)tables.size();
        tables.insert(tables.end(), chunk_src.begin(), chunk_src.end());
        if (identity) {
            P.copy_in = off_nat;
            P.copy_out = off_nat;
        } else if (digitrev) {
            P.copy_in = dir == 0 ? off_src : off_nat;
            P.copy_out = dir == 0 ? off_nat : off_src;
        } else {
            P.copy_in = dir == 0 ? -1 : off_nat;
            P.copy_out = dir == 0 ? off_nat : -1;
        }
        for (int k = 0; k < np && st == HARP_OK; ++k) {
            const int p = dir == 0 ? k : np - 1 - k;     // phase executed k-th
            const HostPhase &hp = phases[(size_t)p];
            PhaseDesc &D = P.ph[k];
            const int B = hp.B;
            int mode;
            if (identity) mode = p == 0 ? MODE_CC : MODE_SS;
            else if (digitrev) mode = p == np - 1 ? (dir == 0 ? MODE_PO : MODE_PI) : MODE_SS;
            else mode = p == 0 ? (dir == 0 ? MODE_GS : MODE_CG) : MODE_SS;
            D.mode = mode;
            D.B = B;
            // Which layout do the strided accesses of this phase use, and with which slot geometry?
            const bool src_side = digitrev && mode == MODE_SS;          // in place on the source-ordered layout
            const Layout &L = src_side ? Lsrc : Lnat;
            const int lm = (mode == MODE_GS || mode == MODE_CG || mode == MODE_CC) ? 1 : L.lm[(size_t)p];
            const int *jo = B == 16 ? (lm == 1 ? joff1_16 : joff2_16) : (lm == 1 ? joff1_8 : joff2_8);
            if (mode == MODE_GS || mode == MODE_CG) {    // these index the item table by slot
                D.lane_step = lm;
                for (int j = 0; j < 4; ++j) D.j_off[j] = jo[j];
            } else {
                D.lane_step = (int32_t)(lm * L.W[(size_t)p]);
                for (int j = 0; j < 4; ++j) D.j_off[j] = (int32_t)(jo[j] * L.W[(size_t)p]);
            }
            // local index seen by the strided / contiguous side of the operand, as a natural local index
            auto strided_nat = [&](int slot) {
                const int r = strided_slot(slot, B, lm);
                return src_side ? nat_local_of_src_local(p, r) : r;
            };
            auto contig_nat = [&](int slot) {            // contiguous blocks of PO/PI live in the source layout
                return (mode == MODE_PO || mode == MODE_PI) ? nat_local_of_src_local(p, slot) : slot;
            };
            // enumerate items and the natural base coordinate of every block
            std::vector<int32_t> items;
            std::vector<int64_t> block_base;             // natural coordinate of local index 0, per block in item order
            int ints_per_item = 1;
            if (mode == MODE_CC) {
                for (int64_t c = 0; c < nblk0; ++c) {
                    items.push_back((int32_t)phys_nat(c * B0));
                    block_base.push_back(c * B0);
                }
            } else if (mode == MODE_SS && !src_side) {
                const int64_t span = hp.S * B;
                for (int64_t hi = 0; hi < d; hi += span)
                    for (int64_t lo = 0; lo < hp.S; lo += 8) {
                        items.push_back((int32_t)phys_nat(hi + lo));
                        for (int e = 0; e < 8; ++e) block_base.push_back(hi + lo + e);
                    }
            } else if (mode == MODE_SS) {
                // source coordinates with source-local index 0 in this phase and a multiple of 8 below
                const int64_t Ss = Lsrc.S[(size_t)p], span = Ss * B;
                for (int64_t hi = 0; hi < d; hi += span)
                    for (int64_t lo = 0; lo < Ss; lo += 8) {
                        items.push_back((int32_t)phys_src(hi + lo));
                        for (int e = 0; e < 8; ++e) block_base.push_back(inv[(size_t)(hi + lo + e)]);
                    }
            } else if (mode == MODE_PO || mode == MODE_PI) {
                // octets of blocks that are neighbours in natural order; each block is 16 contiguous
                // source coordinates
                ints_per_item = 12;
                const int64_t span = hp.S * B;
                for (int64_t hi = 0; hi < d; hi += span)
                    for (int64_t lo = 0; lo < hp.S; lo += 8) {
                        for (int e = 0; e < 8; ++e) {
                            items.push_back((int32_t)phys_src(plan->h_perm[(size_t)(hi + lo + e)]));
                            block_base.push_back(hi + lo + e);
                        }
                        items.push_back((int32_t)phys_nat(hi + lo));
                        items.push_back(0); items.push_back(0); items.push_back(0);
                    }
            } else {
                ints_per_item = 24;
                for (const auto &oc : octets) {
                    for (int r = 0; r < 16; ++r) items.push_back(plan->h_perm[(size_t)(oc[0] * B0 + r)]);
                    for (int e = 0; e < 8; ++e) {
                        items.push_back((int32_t)phys_nat(oc[(size_t)e] * B0));
                        block_base.push_back(oc[(size_t)e] * B0);
                    }
                }
            }
            D.n_items = (int32_t)(items.size() / (size_t)ints_per_item);
            // every address the kernel will form from these tables must stay inside the tile / the row
            {
                bool ok = true;
                const int nj = B == 16 ? 4 : 2;
                auto strided_ok = [&](int64_t b) {
                    bool o = b >= 0;
                    for (int qq = 0; qq < 4; ++qq)
                        for (int j = 0; j < nj; ++j) {
                            const int64_t a = b + (int64_t)qq * D.lane_step + D.j_off[j];
                            o = o && a % 8 == 0 && a + 8 <= pitch;
                        }
                    return o;
                };
                auto contig_ok = [&](int64_t b) { return b >= 0 && b % 8 == 0 && b + B <= pitch; };
                if (mode == MODE_CC) {
                    for (int32_t b : items) ok = ok && contig_ok(b);
                } else if (mode == MODE_SS) {
                    for (int32_t b : items) ok = ok && strided_ok(b);
                } else if (mode == MODE_PO || mode == MODE_PI) {
                    ok = ok && B == 16 && D.n_items <= 2 * (kThreads / 32);
                    for (size_t i = 0; i < items.size(); i += 12) {
                        for (int e = 0; e < 8; ++e) ok = ok && contig_ok(items[i + e]);
                        ok = ok && strided_ok(items[i + 8]);
                    }
                } else {
                    for (size_t i = 0; i < items.size(); i += 24) {
                        for (int r = 0; r < 16; ++r) ok = ok && items[i + r] >= 0 && items[i + r] % 8 == 0 && items[i + r] + 8 <= d;
                        for (int e = 0; e < 8; ++e) ok = ok && contig_ok(items[i + 16 + e]);
                    }
                }
                if (!ok) { st = HARP_ERR_UNSUPPORTED; break; }
            }
            D.items_off = (int32_t)tables.size();
            tables.insert(tables.end(), items.begin(), items.end());
            // fragments: B[k-slot][n-slot] = G[local index of the k-slot][local index of the n-slot]
            const bool in_strided = (mode == MODE_SS || mode == MODE_GS || mode == MODE_PI);
            const bool out_strided = (mode == MODE_SS || mode == MODE_CG || mode == MODE_PO);
            const int words_per_lane = B == 16 ? 4 : 1;
            std::vector<uint32_t> frag(block_base.size() * 32 * words_per_lane);
            std::vector<double> F;
            for (size_t bi = 0; bi < block_base.size(); ++bi) {
                fused_block(plan, hp, block_base[bi], F);
                // G[r_in][r_out] (natural local indices): what this phase applies in this direction, signs folded in
                auto G = [&](int rin, int rout) -> double {
                    double v = dir == 0 ? F[(size_t)rin * B + rout] : F[(size_t)rout * B + rin];
                    if (p == 0 && dir == 0) v *= sign_v(block_base[bi] + (int64_t)rin * hp.S);
                    if (p == 0 && dir == 1) v *= sign_v(block_base[bi] + (int64_t)rout * hp.S);
                    return v;
                };
                auto kin = [&](int kappa) { return in_strided ? strided_nat(kappa) : contig_nat(kappa); };
                auto nout = [&](int nu) { return out_strided ? strided_nat(nu) : contig_nat(nu); };
                for (int lane = 0; lane < 32; ++lane) {
                    const int gg = lane >> 2, qq = lane & 3;
                    uint32_t *dst = frag.data() + (bi * 32 + lane) * words_per_lane;
                    if (B == 16) {
                        for (int nt = 0; nt < 2; ++nt) {
                            const int n = nout(8 * nt + gg);
                            const uint32_t b0 = f2bf(G(kin(2 * qq), n)) | ((uint32_t)f2bf(G(kin(2 * qq + 1), n)) << 16);
                            const uint32_t b1 = f2bf(G(kin(2 * qq + 8), n)) | ((uint32_t)f2bf(G(kin(2 * qq + 9), n)) << 16);
                            dst[2 * nt] = b0;
                            dst[2 * nt + 1] = b1;
                        }
                    } else {
                        const int n = nout(gg);
                        dst[0] = f2bf(G(kin(2 * qq), n)) | ((uint32_t)f2bf(G(kin(2 * qq + 1), n)) << 16);
                    }
                }
            }
            D.bfrag = reinterpret_cast<const uint4 *>(upload(fp, frag, st));
        }
        P.tables = upload(fp, tables, st);
        P.tables_len = (int32_t)tables.size();
        fp->smem_bytes = std::max(fp->smem_bytes, tile_bytes + tables.size() * sizeof(int32_t));
    }
    if (st == HARP_OK && fp->smem_bytes > 227u * 1024u) st = HARP_ERR_UNSUPPORTED;
    if (st == HARP_OK) {
        if (cudaFuncSetAttribute(harp_fast_kernel<kThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            st = HARP_ERR_CUDA;
        int dev = 0, sms = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        fp->max_ctas = sms > 0 ? sms : 148;
    }
    plan->fast = fp;
    if (st != HARP_OK) {
        cudaGetLastError();
        harp_fast_destroy(plan);
        return st;
    }
    return HARP_OK;
}

void harp_fast_destroy(harp_plan *plan) {
    if (!plan->fast) return;
    for (void *p : plan->fast->dev_allocs) cudaFree(p);
    delete plan->fast;
    plan->fast = nullptr;
}

harp_status_t harp_fast_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype, int transpose,
                              cudaStream_t stream) {
    const FastPlan *fp = plan->fast;
    if (!fp || dtype != HARP_BF16) return HARP_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(x) & 15u) != 0) return HARP_ERR_UNSUPPORTED;
    const int64_t n_tiles = (n_rows + kTileRows - 1) / kTileRows;
    const int grid = (int)std::min<int64_t>(n_tiles, fp->max_ctas);
    harp_fast_kernel<kThreads><<<grid, kThreads, fp->smem_bytes, stream>>>(static_cast<__nv_bfloat16 *>(x), n_rows, n_tiles,
                                                                 transpose ? fp->bwd : fp->fwd);
    g_harp_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}
