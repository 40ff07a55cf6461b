// Tensor-core path for wide rows (bf16, identity permutation): two passes over column groups.
//
// A row of d = S_mid * U coordinates is seen as a U x S_mid array.  The stages with stride
// below S_mid ("lower") only mix coordinates inside one slab of S_mid contiguous
// coordinates; the remaining ("upper") stages only mix coordinates that share the position
// l inside their slab.  So the transform is done in two passes, each of which gives a CTA
// a column group and many rows:
//   pass 1: column group = one slab (S_mid contiguous coordinates), lower stages;
//   pass 2: column group = Lw neighbouring positions l in every slab (U segments of Lw
//           coordinates), upper stages.
// Within a pass a CTA keeps the fused block kernels of its column group resident in shared
// memory for all the rows it processes (they are never re-read from L2), and works on
// tiles of 16*MT rows: coalesced cp.async in, phases as batches of small mma.sync products
// with the rows as the M dimension (see harp_fast.cu for the operand handling), coalesced
// stores out.  Tiles are small, so several CTAs share an SM and their copies overlap with
// each other's arithmetic.
//
// The host can walk over the batch in row chunks small enough to stay in L2 and launch
// pass 1 and pass 2 for a chunk back to back, so that the second pass finds the rows in L2
// (HBM then sees one read and one write per row; only L2 sees two).  See harp_split_build for
// the default chunk size.
//
// Radices that do not fill an 8- or 16-wide block (7, 2, ...) are zero-padded inside the
// fragments; padded slots read a valid coordinate and are never stored.
//
// A plan with a permutation takes the same two passes and one more kernel that moves the
// coordinates of every row (harp_gather_rows_kernel: whole rows through shared memory, in place):
// before the passes in the forward direction, after them in the transpose direction.  The sign
// diagonal stays folded into the first phase's fragments, read through the permutation.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "harp_internal.h"
#include "harp_mma.cuh"
#include "harp_fuse.h"

using namespace harp_fuse;

namespace {

constexpr int kSplitThreads = 256;
constexpr int kSplitWarps = kSplitThreads / 32;
constexpr int kMaxSplitPhases = 6;

struct SplitPhase {
    int32_t mode;              // 0 = contiguous blocks (ldmatrix), 1 = strided blocks, eight per item
    int32_t B, B_real;         // operand width (8 or 16) and number of real coordinates in a block
    int32_t lane_step;         // element offset between the slots of lanes q and q+1
    int32_t j_off[4];          // element offsets of a lane's slots
    int32_t lm, jr[4];         // local index of slot j of lane q is lm*q + jr[j]
    int32_t items_off, n_items;
    int32_t bfrag_off;         // word offset of the phase's fragments inside a column group's block
    int32_t paired;            // mode 0, B = 8: blocks 2k and 2k+1 are neighbours in the tile; a warp takes both at once
};

struct SplitPass {
    int32_t n_phases, n_cg, n_chunks, pitch, MT, mt_shift;
    int32_t n_buf;             // 2: the next tile is copied in while this one is multiplied; 1: single buffer
    int32_t cg_stride;         // global element offset between column groups
    int32_t row_stride;        // d
    int32_t chunk_off;         // tables[chunk_off + 2c] = global offset, [.. + 1] = smem offset of 16-byte chunk c
    const int32_t *tables;
    int32_t tables_len;
    const uint32_t *bfrag;     // [column group][bfrag_words]
    int32_t bfrag_words;
    SplitPhase ph[kMaxSplitPhases];
};

// Programmatic dependent launch: everything above this call reads only the plan's tables, so a
// kernel launched with the stream-serialisation attribute runs it while the kernel before it in
// the stream is still busy; the rows are touched only after that kernel has completed.  The next
// kernel in the stream may then start its own preamble.  Without the attribute both are no-ops.
__device__ __forceinline__ void rows_ready_barrier() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// B16: the pass has 16-wide phases (more registers, two CTAs per SM); otherwise only 8-wide ones.
template <bool B16>
__global__ void __launch_bounds__(kSplitThreads, B16 ? 2 : 3)
harp_split_kernel(__nv_bfloat16 *__restrict__ x, int64_t row_begin, int64_t row_end, SplitPass P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, q = lane & 3;
    const int pitch = P.pitch, MT = P.MT, mt_shift = P.mt_shift;
    const int tile_rows = 16 * MT;
    const size_t tile_bytes = (size_t)tile_rows * pitch * 2;          // a multiple of 16
    const uint32_t sbase0 = smem_u32(smem_raw);                        // tile buffer(s), then tables, then fragments
    const int n_buf = P.n_buf;
    int32_t *tab_s = reinterpret_cast<int32_t *>(smem_raw + n_buf * tile_bytes);
    const uint32_t bf_s = sbase0 + (uint32_t)((n_buf * tile_bytes + (size_t)P.tables_len * 4 + 15) / 16 * 16);

    const int cg = blockIdx.x % P.n_cg, part = blockIdx.x / P.n_cg, n_parts = gridDim.x / P.n_cg;
    __nv_bfloat16 *xg = x + (size_t)cg * P.cg_stride;
    const int64_t n_tiles = (row_end - row_begin + tile_rows - 1) / tile_rows;
    const int64_t rs = P.row_stride;

    // resident data of this column group: fragments (asynchronously; the first tile's wait covers
    // them) and tables
    {
        const uint32_t *src = P.bfrag + (size_t)cg * P.bfrag_words;
        for (int i = threadIdx.x * 4; i < P.bfrag_words; i += kSplitThreads * 4) cp_async16(bf_s + 4u * i, src + i);
    }
    for (int i = threadIdx.x; i < P.tables_len; i += kSplitThreads) tab_s[i] = __ldg(P.tables + i);

    // copy geometry: cp_cols threads share a row and cp_rows rows are copied per step; a thread
    // keeps the offsets of its (at most four) chunks of a row in registers
    const int cp_cols = min(P.n_chunks, kSplitThreads), cp_rows = kSplitThreads / cp_cols;
    const int cp_r = threadIdx.x / cp_cols, cp_c = threadIdx.x - cp_r * cp_cols;
    const bool copier = cp_r < cp_rows;
    const bool single_chunk = P.n_chunks <= kSplitThreads;
    int32_t goff[4], soff[4];
#pragma unroll
    for (int mth = 0; mth < 4; ++mth) {
        const int ch = cp_c + mth * cp_cols;
        const bool in = ch < P.n_chunks;
        goff[mth] = in ? __ldg(P.tables + P.chunk_off + 2 * ch) : -1;
        soff[mth] = in ? 2 * __ldg(P.tables + P.chunk_off + 2 * ch + 1) : 0;
    }

    // With two buffers the copy of the next tile is in flight while this one is multiplied; passes
    // whose occupancy is limited by shared memory rather than registers use one buffer instead.
    auto copy_in = [&](int64_t tile, uint32_t sb) {
        const int64_t row0 = row_begin + tile * tile_rows;
        // rows past the end are computed on a copy of the last row and never stored
        if (copier) {
            if (row0 + tile_rows <= row_end && single_chunk) {
                const __nv_bfloat16 *src = xg + (row0 + cp_r) * rs + goff[0];
                uint32_t dst = sb + 2u * (uint32_t)(cp_r * pitch) + soff[0];
                const int64_t src_step = (int64_t)cp_rows * rs;
                const uint32_t dst_step = 2u * (uint32_t)(cp_rows * pitch);
#pragma unroll 4
                for (int r = cp_r; r < tile_rows; r += cp_rows, src += src_step, dst += dst_step) cp_async16(dst, src);
            } else {
                const __nv_bfloat16 *last_row = xg + (row_end - 1) * rs;
                const __nv_bfloat16 *src = xg + (row0 + cp_r) * rs;
                uint32_t dst = sb + 2u * (uint32_t)(cp_r * pitch);
                const int64_t src_step = (int64_t)cp_rows * rs;
                const uint32_t dst_step = 2u * (uint32_t)(cp_rows * pitch);
                int64_t row = row0 + cp_r;
                for (int r = cp_r; r < tile_rows; r += cp_rows, src += src_step, dst += dst_step, row += cp_rows) {
                    const __nv_bfloat16 *s0 = row < row_end ? src : last_row;
#pragma unroll
                    for (int mth = 0; mth < 4; ++mth)
                        if (goff[mth] >= 0) cp_async16(dst + soff[mth], s0 + goff[mth]);
                }
            }
        }
        cp_async_commit();
    };

    rows_ready_barrier();
    int buf = 0;
    if (n_buf == 2 && part < n_tiles) copy_in(part, sbase0);
    for (int64_t tile = part; tile < n_tiles; tile += n_parts) {
        const int64_t row0 = row_begin + tile * tile_rows;
        const bool full_tile = row0 + tile_rows <= row_end;
        const uint32_t sbase = sbase0 + (uint32_t)(buf * tile_bytes);
        if (n_buf == 2) {
            if (tile + n_parts < n_tiles) {
                copy_in(tile + n_parts, sbase0 + (uint32_t)((buf ^ 1) * tile_bytes));
                cp_async_wait_group<1>();
            } else {
                cp_async_wait_group<0>();
            }
            buf ^= 1;
        } else {
            copy_in(tile, sbase0);
            cp_async_wait_group<0>();
        }
        __syncthreads();

        for (int p = 0; p < P.n_phases; ++p) {
            const SplitPhase &ph = P.ph[p];
            if (ph.mode == 0) {
                // contiguous blocks: one warp takes a block through all row groups of the tile
                if (B16 && ph.B == 16) {
                    const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
                    const uint32_t lane_addr = sbase + 2u * (uint32_t)(mrow * pitch + mcol);
                    for (int it = warp; it < ph.n_items; it += kSplitWarps) {
                        const uint4 bf = lds128(bf_s + 4u * (uint32_t)(ph.bfrag_off + (it * 32 + lane) * 4));
                        uint32_t addr = lane_addr + 2u * (uint32_t)tab_s[ph.items_off + it];
                        for (int mt = 0; mt < MT; ++mt, addr += 32u * (uint32_t)pitch) {
                            uint32_t a[4];
                            ldmatrix_x4(a, addr);
                            float c0[4], c1[4];
                            mma_k16(c0, a, bf.x, bf.y);
                            mma_k16(c1, a, bf.z, bf.w);
                            stmatrix_x4(addr, pack_bf16(c0[0], c0[1]), pack_bf16(c0[2], c0[3]), pack_bf16(c1[0], c1[1]),
                                        pack_bf16(c1[2], c1[3]));
                        }
                    }
                } else if (ph.paired) {
                    // two neighbouring 8-wide blocks per ldmatrix.x4 / stmatrix.x4: half the shared-memory instructions
                    const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
                    const uint32_t lane_addr = sbase + 2u * (uint32_t)(mrow * pitch + mcol);
                    for (int it = 2 * warp; it < ph.n_items; it += 2 * kSplitWarps) {
                        const uint32_t bfa = bf_s + 4u * (uint32_t)(ph.bfrag_off + it * 32 + lane);
                        const uint32_t bf0 = lds32(bfa), bf1 = lds32(bfa + 128);
                        uint32_t addr = lane_addr + 2u * (uint32_t)tab_s[ph.items_off + it];
                        for (int mt = 0; mt < MT; ++mt, addr += 32u * (uint32_t)pitch) {
                            uint32_t a[4];
                            ldmatrix_x4(a, addr);
                            const uint32_t a_lo[2] = {a[0], a[1]}, a_hi[2] = {a[2], a[3]};
                            float c0[4], c1[4];
                            mma_k8(c0, a_lo, bf0);
                            mma_k8(c1, a_hi, bf1);
                            stmatrix_x4(addr, pack_bf16(c0[0], c0[1]), pack_bf16(c0[2], c0[3]), pack_bf16(c1[0], c1[1]),
                                        pack_bf16(c1[2], c1[3]));
                        }
                    }
                } else {
                    const uint32_t lane_addr = sbase + 2u * (uint32_t)((lane & 15) * pitch);
                    for (int it = warp; it < ph.n_items; it += kSplitWarps) {
                        const uint32_t bf = lds32(bf_s + 4u * (uint32_t)(ph.bfrag_off + it * 32 + lane));
                        uint32_t addr = lane_addr + 2u * (uint32_t)tab_s[ph.items_off + it];
                        for (int mt = 0; mt < MT; ++mt, addr += 32u * (uint32_t)pitch) {
                            uint32_t a[2];
                            ldmatrix_x2(a, addr);
                            float c0[4];
                            mma_k8(c0, a, bf);
                            stmatrix_x2(addr, pack_bf16(c0[0], c0[1]), pack_bf16(c0[2], c0[3]));
                        }
                    }
                }
            } else if (B16 && ph.B == 16) {
                // strided blocks, eight per item; work unit = (item, row group).  Per-lane slot
                // offsets: padded slots read slot 0 and are not stored.
                uint32_t so[4];
                bool ok[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    ok[j] = ph.lm * q + ph.jr[j] < ph.B_real;
                    so[j] = ok[j] ? 2u * (uint32_t)(q * ph.lane_step + ph.j_off[j]) : 0u;
                }
                const int n_work = ph.n_items << mt_shift;
                for (int w = warp; w < n_work; w += kSplitWarps) {
                    const int it = w >> mt_shift, mt = w & (MT - 1);
                    const uint32_t a0 = sbase + 2u * (uint32_t)((mt * 16 + g) * pitch + tab_s[ph.items_off + it]);
                    const uint32_t a1 = a0 + 16u * (uint32_t)pitch;
                    const uint32_t bfa = bf_s + 4u * (uint32_t)(ph.bfrag_off + (it * 256 + lane) * 4);
                    uint4 raw[4][2], bf[8];
                    uint32_t unused[8][4];
#pragma unroll
                    for (int e = 0; e < 8; ++e) bf[e] = lds128(bfa + e * 512);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        raw[j][0] = lds128(a0 + so[j]);
                        raw[j][1] = lds128(a1 + so[j]);
                    }
                    octet_mma16<true>(raw, bf, unused);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (ok[j]) {
                            sts128(a0 + so[j], raw[j][0]);
                            sts128(a1 + so[j], raw[j][1]);
                        }
                    }
                }
            } else {
                uint32_t so[2];
                bool ok[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    ok[j] = ph.lm * q + ph.jr[j] < ph.B_real;
                    so[j] = ok[j] ? 2u * (uint32_t)(q * ph.lane_step + ph.j_off[j]) : 0u;
                }
                const int n_work = ph.n_items << mt_shift;
                for (int w = warp; w < n_work; w += kSplitWarps) {
                    const int it = w >> mt_shift, mt = w & (MT - 1);
                    const uint32_t a0 = sbase + 2u * (uint32_t)((mt * 16 + g) * pitch + tab_s[ph.items_off + it]);
                    const uint32_t a1 = a0 + 16u * (uint32_t)pitch;
                    // the eight blocks' fragment words of a lane: two 16-byte loads ([half][lane][4 words] per item)
                    const uint32_t bfa = bf_s + 4u * (uint32_t)(ph.bfrag_off + it * 256 + lane * 4);
                    uint4 raw[2][2];
                    uint32_t bf[8];
                    {
                        const uint4 f0 = lds128(bfa), f1 = lds128(bfa + 512);
                        bf[0] = f0.x; bf[1] = f0.y; bf[2] = f0.z; bf[3] = f0.w;
                        bf[4] = f1.x; bf[5] = f1.y; bf[6] = f1.z; bf[7] = f1.w;
                    }
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        raw[j][0] = lds128(a0 + so[j]);
                        raw[j][1] = lds128(a1 + so[j]);
                    }
                    octet_mma8(raw, bf);
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        if (ok[j]) {
                            sts128(a0 + so[j], raw[j][0]);
                            sts128(a1 + so[j], raw[j][1]);
                        }
                    }
                }
            }
            __syncthreads();
        }

        if (copier) {
            if (full_tile && single_chunk) {
                __nv_bfloat16 *dstg = xg + (row0 + cp_r) * rs + goff[0];
                uint32_t srcs = sbase + 2u * (uint32_t)(cp_r * pitch) + soff[0];
                const int64_t g_step = (int64_t)cp_rows * rs;
                const uint32_t s_step = 2u * (uint32_t)(cp_rows * pitch);
#pragma unroll 4
                for (int r = cp_r; r < tile_rows; r += cp_rows, dstg += g_step, srcs += s_step) stg128(dstg, lds128(srcs));
            } else {
                __nv_bfloat16 *dstg = xg + (row0 + cp_r) * rs;
                uint32_t srcs = sbase + 2u * (uint32_t)(cp_r * pitch);
                const int64_t g_step = (int64_t)cp_rows * rs;
                const uint32_t s_step = 2u * (uint32_t)(cp_rows * pitch);
                int64_t row = row0 + cp_r;
                for (int r = cp_r; r < tile_rows && row < row_end; r += cp_rows, dstg += g_step, srcs += s_step, row += cp_rows) {
#pragma unroll
                    for (int mth = 0; mth < 4; ++mth)
                        if (goff[mth] >= 0) stg128(dstg + goff[mth], lds128(srcs + soff[mth]));
                }
            }
        }
        __syncthreads();
    }
    cp_async_wait_all();      // a CTA without tiles must not exit with copies in flight
}

// ---------------------------------------------------------------------------------------
// Upper pass with one dense block per position l: all upper stages are fused into a single
// U x U matrix F_l (U = d / S_mid <= 64, zero-padded to KP = 16*KS).  The tile is stored
// transposed, [row][l][u], so that a block is KP contiguous values: operands come from
// ldmatrix, results go back with stmatrix, and the 2-byte transposition is done in registers
// by the copies (eight 16-byte loads -> 8x8 transpose -> eight 16-byte stores).
struct UpperPass {
    int32_t n_cg, Lw, U, KP, NT, pitch, MT;
    int32_t l_skew;            // elements added to the tile offset of a position per octet of positions
    int32_t S_mid, row_stride;
    const uint32_t *bfrag;     // [column group][l][n-tile][k-step][lane][2]
    int32_t bfrag_words;
};

__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

template <int KS>
__global__ void __launch_bounds__(kSplitThreads, 2)
harp_upper_kernel(__nv_bfloat16 *__restrict__ x, int64_t row_begin, int64_t row_end, UpperPass P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t sbase = smem_u32(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int pitch = P.pitch, MT = P.MT, KP = P.KP, NT = P.NT;
    const int tile_rows = 16 * MT;
    const uint32_t bf_s = sbase + (uint32_t)(((size_t)tile_rows * pitch * 2 + 15) / 16 * 16);
    const int cg = blockIdx.x % P.n_cg, part = blockIdx.x / P.n_cg, n_parts = gridDim.x / P.n_cg;
    __nv_bfloat16 *xg = x + (size_t)cg * P.Lw;
    const int64_t n_tiles = (row_end - row_begin + tile_rows - 1) / tile_rows;
    const int64_t rs = P.row_stride;
    {
        const uint32_t *src = P.bfrag + (size_t)cg * P.bfrag_words;
        for (int i = threadIdx.x * 4; i < P.bfrag_words; i += kSplitThreads * 4) cp_async16(bf_s + 4u * i, src + i);
    }
    // copy geometry: a thread owns one (octet of l, octet of u) unit and walks over rows
    const int lo_n = P.Lw >> 3, uo_n = KP >> 3;
    const int units_per_row = lo_n * uo_n;
    const int cp_rows = kSplitThreads / units_per_row;
    const int cp_r = threadIdx.x / units_per_row, un = threadIdx.x - cp_r * units_per_row;
    const int uo = un / lo_n, lo = un - uo * lo_n;
    const int mt_shift = MT == 4 ? 2 : (MT == 2 ? 1 : 0);

    rows_ready_barrier();
    for (int64_t tile = part; tile < n_tiles; tile += n_parts) {
        const int64_t row0 = row_begin + tile * tile_rows;
        // ---- copy in, transposing: unit = (row, octet of l, octet of u)
        for (int r = cp_r; r < tile_rows && cp_r < cp_rows; r += cp_rows) {
            const int64_t row = min(row0 + r, row_end - 1);
            const __nv_bfloat16 *src = xg + row * rs + 8 * lo;
            uint4 in[8], out[8];
#pragma unroll
            for (int uu = 0; uu < 8; ++uu) {
                const int u = 8 * uo + uu;
                in[uu] = u < P.U ? ldg128_stream(src + (int64_t)u * P.S_mid) : make_uint4(0u, 0u, 0u, 0u);
            }
            transpose8x8_b16(in, out);
            const uint32_t dst = sbase + 2u * (uint32_t)(r * pitch + (8 * lo) * KP + 8 * uo);
#pragma unroll
            for (int ll = 0; ll < 8; ++ll) sts128(dst + 2u * (uint32_t)(ll * KP), out[ll]);
        }
        cp_async_wait_all();
        __syncthreads();

        // ---- one dense block per (l, row group)
        {
            const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
            const int n_work = P.Lw * MT;
            for (int w = warp; w < n_work; w += kSplitWarps) {
                const int l = w >> mt_shift, mt = w & (MT - 1);
                const uint32_t addr = sbase + 2u * (uint32_t)((mt * 16 + mrow) * pitch + l * KP + mcol);
                uint32_t a[KS][4];
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) ldmatrix_x4(a[ks], addr + 32u * ks);
                const uint32_t bfa = bf_s + 8u * (uint32_t)((l * NT * KS) * 32 + lane);
                float acc[2 * KS][4];
#pragma unroll
                for (int nt = 0; nt < 2 * KS; ++nt) {
                    acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
                    if (nt < NT) {
#pragma unroll
                        for (int ks = 0; ks < KS; ++ks) {
                            const uint2 b = lds64(bfa + 256u * (uint32_t)(nt * KS + ks));
                            mma_k16_acc(acc[nt], a[ks], b.x, b.y);
                        }
                    }
                }
#pragma unroll
                for (int c = 0; c < KS; ++c)
                    stmatrix_x4(addr + 32u * c, pack_bf16(acc[2 * c][0], acc[2 * c][1]), pack_bf16(acc[2 * c][2], acc[2 * c][3]),
                                pack_bf16(acc[2 * c + 1][0], acc[2 * c + 1][1]), pack_bf16(acc[2 * c + 1][2], acc[2 * c + 1][3]));
            }
        }
        __syncthreads();

        // ---- copy out, transposing back
        for (int r = cp_r; r < tile_rows && cp_r < cp_rows && row0 + r < row_end; r += cp_rows) {
            const uint32_t srcs = sbase + 2u * (uint32_t)(r * pitch + (8 * lo) * KP + 8 * uo);
            uint4 in[8], out[8];
#pragma unroll
            for (int ll = 0; ll < 8; ++ll) in[ll] = lds128(srcs + 2u * (uint32_t)(ll * KP));
            transpose8x8_b16(in, out);
            __nv_bfloat16 *dstg = xg + (row0 + r) * rs + 8 * lo;
#pragma unroll
            for (int uu = 0; uu < 8; ++uu) {
                const int u = 8 * uo + uu;
                if (u < P.U) stg128(dstg + (int64_t)u * P.S_mid, out[uu]);
            }
        }
        __syncthreads();
    }
    cp_async_wait_all();
}

// The same pass with the fragments of F_l in registers (KS <= 3, i.e. U <= 48): warp w owns positions
// w and w + 8 of a column group of sixteen, loads their fragments once from global memory and keeps
// them for every row the CTA sees.  Shared memory holds the tile twice: a staging buffer that cp.async
// fills with the rows as they are in global memory ([row][octet of l][u][8 values of l], the 16-byte
// chunks of a u-octet XOR-swizzled by the octet's index), and the operand buffer [row][l][u] that the
// transposing copy (eight 16-byte loads -> 8x8 transpose in registers -> eight 16-byte stores) writes
// and ldmatrix / stmatrix work on.  The staging buffer of the next tile fills while this tile is
// multiplied and written back, so the copy's latency is hidden without holding registers for it.
// The positions of the second octet are shifted by l_skew elements in the operand buffer so that the
// two position octets of a transposing copy fall into different bank groups.
// Per-section cycle counts of harp_upper_reg_kernel (build with -DHARP_UPPER_TIMING): thread 0 of CTA 0 prints
// the cycles it spent in  0 wait for the staged rows | 1 transposing copy | 2 issue of the next stage |
// 3 products | 4 copy out.
#ifdef HARP_UPPER_TIMING
#define UP_DECL long long up_acc[5] = {0, 0, 0, 0, 0}, up_last = clock64()
#define UP_MARK(k) do { if (threadIdx.x == 0) { const long long now_ = clock64(); up_acc[k] += now_ - up_last; up_last = now_; } } while (0)
#define UP_DUMP do { if (threadIdx.x == 0 && blockIdx.x == 0) printf("upper sections: wait %lld  transpose %lld  stage %lld  products %lld  out %lld  tiles %lld\n", up_acc[0], up_acc[1], up_acc[2], up_acc[3], up_acc[4], (long long)((n_tiles - part + n_parts - 1) / n_parts)); } while (0)
#else
#define UP_DECL do { } while (0)
#define UP_MARK(k) do { } while (0)
#define UP_DUMP do { } while (0)
#endif

template <int KS>
__global__ void __launch_bounds__(kSplitThreads, 2)
harp_upper_reg_kernel(__nv_bfloat16 *__restrict__ x, int64_t row_begin, int64_t row_end, UpperPass P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int pitch = P.pitch, MT = P.MT, KP = P.KP, NT = P.NT, U = P.U;
    const int tile_rows = 16 * MT;
    const uint32_t sbase = smem_u32(smem_raw);                                  // operand buffer
    const uint32_t stage = sbase + (uint32_t)(((size_t)tile_rows * pitch * 2 + 15) / 16 * 16);
    const uint32_t stage_row = 32u * (uint32_t)KP + 64u;                        // bytes per row: 2 octets of l x KP chunks, the second shifted by 4 chunks
    const int cg = blockIdx.x % P.n_cg, part = blockIdx.x / P.n_cg, n_parts = gridDim.x / P.n_cg;
    __nv_bfloat16 *xg = x + (size_t)cg * P.Lw;
    const int64_t n_tiles = (row_end - row_begin + tile_rows - 1) / tile_rows;
    const int64_t rs = P.row_stride;
    // fragments of this warp's two positions
    uint2 bfr[2][2 * KS][KS];
#pragma unroll
    for (int li = 0; li < 2; ++li) {
        const uint2 *src = reinterpret_cast<const uint2 *>(P.bfrag + (size_t)cg * P.bfrag_words) +
                           (size_t)(warp + 8 * li) * NT * KS * 32 + lane;
#pragma unroll
        for (int nt = 0; nt < 2 * KS; ++nt)
#pragma unroll
            for (int ks = 0; ks < KS; ++ks)
                bfr[li][nt][ks] = nt < NT ? __ldg(src + (nt * KS + ks) * 32) : make_uint2(0u, 0u);
    }
    // transposing copies: a thread owns one (octet of l, octet of u) unit and walks over rows
    const int uo_n = KP >> 3;
    const int units_per_row = 2 * uo_n;
    const int cp_rows = kSplitThreads / units_per_row;
    const int cp_r = threadIdx.x / units_per_row, un = threadIdx.x - cp_r * units_per_row;
    const int lo = un / uo_n, uo = un - lo * uo_n;
    const int unit_off = (8 * lo) * KP + lo * P.l_skew + 8 * uo;
    const uint32_t unit_stage = (uint32_t)(lo * (KP + 4) + 8 * uo) * 16u;
    // copy out: the two position octets of a (row, u) in neighbouring lanes, so that a pair of lanes writes a whole sector
    const int lo_w = un & 1, uo_w = un >> 1;
    const int unit_off_w = (8 * lo_w) * KP + lo_w * P.l_skew + 8 * uo_w;

    // rows of a tile as they are, into the staging buffer: chunk = (row, u, octet of l); a thread's chunks are
    // kSplitThreads apart in (row, u, l8) order, stepped without a division
    const int per_row = 2 * U;
    const int c_r0 = threadIdx.x / per_row, c_rem0 = threadIdx.x - c_r0 * per_row;
    const int step_r = kSplitThreads / per_row, step_rem = kSplitThreads - step_r * per_row;
    auto stage_in = [&](int64_t tile) {
        const int64_t row0 = row_begin + tile * tile_rows;
        int r = c_r0, rem = c_rem0;
        while (r < tile_rows) {
            const int u = rem >> 1, l8 = rem & 1;
            const int64_t row = min(row0 + r, row_end - 1);
            const uint32_t dst = stage + (uint32_t)r * stage_row + (uint32_t)(l8 * (KP + 4) + (u & ~7) + ((u & 7) ^ ((u >> 3) & 7))) * 16u;
            cp_async16(dst, xg + row * rs + (int64_t)u * P.S_mid + 8 * l8);
            r += step_r;
            rem += step_rem;
            if (rem >= per_row) { rem -= per_row; ++r; }
        }
        cp_async_commit();
    };

    rows_ready_barrier();
    UP_DECL;
    if (part < n_tiles) stage_in(part);
    for (int64_t tile = part; tile < n_tiles; tile += n_parts) {
        const int64_t row0 = row_begin + tile * tile_rows;
        cp_async_wait_group<0>();
        __syncthreads();
        UP_MARK(0);
        // ---- staging buffer -> operand buffer, transposing: unit = (row, octet of l, octet of u)
        for (int r = cp_r; r < tile_rows && cp_r < cp_rows; r += cp_rows) {
            const uint32_t src = stage + (uint32_t)r * stage_row + unit_stage;
            uint4 in[8], out[8];
#pragma unroll
            for (int uu = 0; uu < 8; ++uu)
                in[uu] = 8 * uo + uu < U ? lds128(src + 16u * (uint32_t)(uu ^ (uo & 7))) : make_uint4(0u, 0u, 0u, 0u);
            transpose8x8_b16(in, out);
            const uint32_t dst = sbase + 2u * (uint32_t)(r * pitch + unit_off);
#pragma unroll
            for (int ll = 0; ll < 8; ++ll) sts128(dst + 2u * (uint32_t)(ll * KP), out[ll]);
        }
        __syncthreads();
        UP_MARK(1);
        if (tile + n_parts < n_tiles) stage_in(tile + n_parts);       // lands under the products and the copy out
        UP_MARK(2);

        // ---- one dense block per (l, row group); the fragments stay where they are
        {
            const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
#pragma unroll
            for (int li = 0; li < 2; ++li) {
                const uint32_t addr0 = sbase + 2u * (uint32_t)(mrow * pitch + (warp + 8 * li) * KP + li * P.l_skew + mcol);
                for (int mt = 0; mt < MT; ++mt) {
                    const uint32_t addr = addr0 + 32u * (uint32_t)(mt * pitch);
                    uint32_t a[KS][4];
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) ldmatrix_x4(a[ks], addr + 32u * ks);
#pragma unroll
                    for (int c = 0; c < KS; ++c) {
                        float acc[2][4];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            acc[h][0] = acc[h][1] = acc[h][2] = acc[h][3] = 0.f;
#pragma unroll
                            for (int ks = 0; ks < KS; ++ks) mma_k16_acc(acc[h], a[ks], bfr[li][2 * c + h][ks].x, bfr[li][2 * c + h][ks].y);
                        }
                        stmatrix_x4(addr + 32u * c, pack_bf16(acc[0][0], acc[0][1]), pack_bf16(acc[0][2], acc[0][3]),
                                    pack_bf16(acc[1][0], acc[1][1]), pack_bf16(acc[1][2], acc[1][3]));
                    }
                }
            }
        }
        __syncthreads();
        UP_MARK(3);

        // ---- copy out, transposing back
        for (int r = cp_r; r < tile_rows && cp_r < cp_rows && row0 + r < row_end; r += cp_rows) {
            const uint32_t srcs = sbase + 2u * (uint32_t)(r * pitch + unit_off_w);
            uint4 in[8], out[8];
#pragma unroll
            for (int ll = 0; ll < 8; ++ll) in[ll] = lds128(srcs + 2u * (uint32_t)(ll * KP));
            transpose8x8_b16(in, out);
            __nv_bfloat16 *dstg = xg + (row0 + r) * rs + 8 * lo_w;
#pragma unroll
            for (int uu = 0; uu < 8; ++uu) {
                const int u = 8 * uo_w + uu;
                if (u < U) stg128(dstg + (int64_t)u * P.S_mid, out[uu]);
            }
        }
        // (the next iteration's barrier separates these reads from the next transposing copy)
        UP_MARK(4);
    }
    UP_DUMP;
    cp_async_wait_all();
}

// ---------------------------------------------------------------------------------------
// Fixed permutation of wide rows, in place: out[i] = in[table[i]] for every row (Theorem 1's
// permutation convention: table = the plan's permutation in the forward direction, its inverse
// in the transpose direction).  A CTA keeps the table in shared memory as 16-bit indices and
// takes groups of R whole rows through two buffers: the next group is copied in (cp.async) while
// this one is gathered with 2-byte shared-memory reads and written back with 16-byte stores.  The
// move is exact: no arithmetic touches the values.
constexpr int kGatherThreads = 512;

__global__ void __launch_bounds__(kGatherThreads, 1)
harp_gather_rows_kernel(__nv_bfloat16 *__restrict__ x, int64_t n_rows, int32_t d, int32_t R, const uint16_t *__restrict__ table) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t sbase = smem_u32(smem_raw);
    const uint32_t tab_s = sbase;                                   // d 16-bit indices
    const uint32_t row_bytes = 2u * (uint32_t)d;
    const uint32_t buf_s = sbase + row_bytes;                       // two buffers of R rows
    const uint32_t buf_bytes = (uint32_t)R * row_bytes;
    const int chunks = d >> 3;                                      // 16-byte chunks per row
    for (int c = threadIdx.x; c < chunks; c += kGatherThreads) cp_async16(tab_s + 16u * c, table + 8 * c);
    const int64_t n_groups = (n_rows + R - 1) / R;
    auto copy_in = [&](int64_t grp, uint32_t dst) {
        const int64_t row0 = grp * R;
        const int rows = (int)min((int64_t)R, n_rows - row0);
        const __nv_bfloat16 *src = x + row0 * d;
        for (int c = threadIdx.x; c < rows * chunks; c += kGatherThreads) cp_async16(dst + 16u * c, src + 8 * (int64_t)c);
        cp_async_commit();
    };
    int buf = 0;
    if ((int64_t)blockIdx.x < n_groups) copy_in(blockIdx.x, buf_s);
    for (int64_t grp = blockIdx.x; grp < n_groups; grp += gridDim.x) {
        cp_async_wait_group<0>();
        __syncthreads();                                            // this group is here; the other buffer is free
        if (grp + gridDim.x < n_groups) copy_in(grp + gridDim.x, buf_s + (uint32_t)(buf ^ 1) * buf_bytes);
        const int64_t row0 = grp * R;
        const int rows = (int)min((int64_t)R, n_rows - row0);
        const uint32_t src_s = buf_s + (uint32_t)buf * buf_bytes;
        for (int c = threadIdx.x; c < rows * chunks; c += kGatherThreads) {
            const int r = c / chunks, cc = c - r * chunks;
            const uint4 idx = lds128(tab_s + 16u * cc);
            const uint32_t rb = src_s + (uint32_t)r * row_bytes;
            auto pick = [&](uint32_t pair) {
                uint32_t lo, hi;
                asm volatile("ld.shared.u16 %0, [%1];" : "=r"(lo) : "r"(rb + 2u * (pair & 0xffffu)));
                asm volatile("ld.shared.u16 %0, [%1];" : "=r"(hi) : "r"(rb + 2u * (pair >> 16)));
                return lo | (hi << 16);
            };
            uint4 out;
            out.x = pick(idx.x);
            out.y = pick(idx.y);
            out.z = pick(idx.z);
            out.w = pick(idx.w);
            stg128(x + (row0 + r) * d + 8 * cc, out);
        }
        buf ^= 1;
    }
    cp_async_wait_all();
}

// ------------------------------------------------------------------------------- host

struct PassHost {
    SplitPass fwd{}, bwd{};
    size_t smem_bytes = 0;
    bool present = false;
    bool has16 = false;
};

}  // namespace

struct SplitPlan {
    PassHost pass[2];          // [0] lower stages on slabs, [1] upper stages on position groups
    std::vector<void *> dev_allocs;
    int64_t chunk_rows = 0;    // rows per L2-resident chunk
    int sms = 148;
    int lower_stages = 0;      // pass[0] covers stages [0, lower_stages)
    // plans with a permutation: 16-bit gather tables ([0] forward = the permutation, [1] transpose = its inverse)
    const uint16_t *gather[2] = {nullptr, nullptr};
    int gather_rows = 1;       // rows per buffer of the gather kernel
    size_t gather_smem = 0;
    // dense upper pass (replaces pass[1] when set)
    bool dense_upper = false;
    bool up_in_regs = false;   // fragments in registers (harp_upper_reg_kernel)
    UpperPass up_fwd{}, up_bwd{};
    size_t up_smem = 0;
    int up_ks = 0;
};

namespace {

struct GPhase {                // a fused group of stages
    int t0, t1;
    int B, B_real;
    int64_t S;                 // natural stride
};

template <typename T>
T *upload_s(SplitPlan *sp, const std::vector<T> &v, harp_status_t &st) {
    if (st != HARP_OK) return nullptr;
    void *p = nullptr;
    if (cudaMalloc(&p, std::max<size_t>(16, v.size() * sizeof(T))) != cudaSuccess) { st = HARP_ERR_ALLOC; return nullptr; }
    sp->dev_allocs.push_back(p);
    if (!v.empty() && cudaMemcpy(p, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) st = HARP_ERR_CUDA;
    return static_cast<T *>(p);
}

// One pass.  `phs`: the pass's phases.  Tile coordinates: an innermost index of `inner` positions
// (stride 1 in memory, not mixed by this pass unless it is phase 0 of pass 1) followed by the
// phases' local indices.  For pass 1, inner = 1 and phase 0 is contiguous; for pass 2, inner = Lw.
harp_status_t build_pass(const harp_plan *plan, SplitPlan *sp, PassHost &ph_out, const std::vector<GPhase> &phs, bool lower,
                         int64_t S_mid, int64_t U, int inner) {
    const int64_t d = plan->d;
    const int np = (int)phs.size();
    if (np == 0 || np > kMaxSplitPhases) return HARP_ERR_UNSUPPORTED;
    // ---- layout of a tile row
    std::vector<int64_t> W((size_t)np);
    std::vector<int> lm((size_t)np, 1);
    int64_t ext = inner;
    for (int p = 0; p < np; ++p) {
        if (!(lower && p == 0)) {
            ext = (ext + 7) / 8 * 8;
            while (((ext / 8) % 8) == 0 || ((ext / 8) % 8) == 4) ext += 8;
            lm[(size_t)p] = ((ext / 8) % 2 == 0) ? 1 : 2;
        }
        W[(size_t)p] = ext;
        ext *= phs[(size_t)p].B_real;
    }
    int64_t pitch = (ext + 7) / 8 * 8;
    if ((pitch / 8) % 2 == 0) pitch += 8;
    // local strides of the phases inside the tile's own coordinate system
    // pass 1: tile coordinate t in [0, S_mid): local index of phase p = (t / S_p) % B_real
    // pass 2: tile coordinate (l', u): local index of phase p = (u / (S_p / S_mid)) % B_real
    auto phys = [&](int64_t lpos, int64_t u) {       // lpos: position inside the inner run / slab
        int64_t o = 0;
        if (lower) {
            for (int p = 0; p < np; ++p) o += ((lpos / phs[(size_t)p].S) % phs[(size_t)p].B_real) * W[(size_t)p];
        } else {
            o = lpos;
            for (int p = 0; p < np; ++p) o += ((u / (phs[(size_t)p].S / S_mid)) % phs[(size_t)p].B_real) * W[(size_t)p];
        }
        return o;
    };
    const int n_cg = lower ? (int)U : (int)(S_mid / inner);
    const int n_chunks = lower ? (int)(S_mid / 8) : (int)(U * inner / 8);
    // rows per tile: as many 16-row groups as fit ~40 KB
    // (measured on 65536 rows of d = 28672: slabs of 512 coordinates with 64-row tiles and two CTAs per SM are 4 %
    // faster than with 32-row tiles and three; for the position groups of the upper pass larger tiles gain nothing.
    // The launch shrinks the tile for batches that do not fill it.)
    int MT = (int)std::max<int64_t>(1, std::min<int64_t>(4, ((lower ? 80 : 40) * 1024) / (pitch * 2 * 16)));
    if (MT == 3) MT = 2;
    if (n_chunks > 4 * kSplitThreads) return HARP_ERR_UNSUPPORTED;

    // ---- tables: chunk map, then items per phase (identical for all column groups and both directions)
    std::vector<int32_t> tables;
    for (int c = 0; c < n_chunks; ++c) {
        if (lower) {
            tables.push_back(8 * c);
            tables.push_back((int32_t)phys(8 * c, 0));
        } else {
            const int per = inner / 8;
            const int64_t u = c / per, lc = (c % per) * 8;
            tables.push_back((int32_t)(u * S_mid + lc));
            tables.push_back((int32_t)phys(lc, u));
        }
    }
    struct ItemSet { std::vector<int32_t> bases; std::vector<int64_t> block_rel; int mode; };   // block_rel: (lpos, u) packed
    std::vector<ItemSet> sets((size_t)np);
    for (int p = 0; p < np; ++p) {
        const GPhase &gp = phs[(size_t)p];
        ItemSet &is = sets[(size_t)p];
        if (lower && p == 0) {
            is.mode = 0;
            if (gp.B != gp.B_real) return HARP_ERR_UNSUPPORTED;
            for (int64_t c = 0; c < S_mid / gp.B; ++c) {
                is.bases.push_back((int32_t)phys(c * gp.B, 0));
                is.block_rel.push_back(c * gp.B);
            }
        } else if (lower) {
            is.mode = 1;
            const int64_t span = gp.S * gp.B_real;
            for (int64_t hi = 0; hi < S_mid; hi += span)
                for (int64_t lo = 0; lo < gp.S; lo += 8) {
                    is.bases.push_back((int32_t)phys(hi + lo, 0));
                    for (int e = 0; e < 8; ++e) is.block_rel.push_back(hi + lo + e);
                }
        } else {
            is.mode = 1;
            const int64_t su = gp.S / S_mid, span = su * gp.B_real;      // in units of u
            for (int64_t hi = 0; hi < U; hi += span)
                for (int64_t lo = 0; lo < su; ++lo)
                    for (int64_t lc = 0; lc < inner; lc += 8) {
                        is.bases.push_back((int32_t)phys(lc, hi + lo));
                        for (int e = 0; e < 8; ++e) is.block_rel.push_back((hi + lo) * S_mid + lc + e);   // relative natural coordinate
                    }
        }
    }

    static const int joff1_16[4] = {0, 4, 8, 12}, joff2_16[4] = {0, 1, 8, 9};
    static const int joff1_8[4] = {0, 4, 0, 0}, joff2_8[4] = {0, 1, 0, 0};
    harp_status_t st = HARP_OK;
    for (int dir = 0; dir < 2 && st == HARP_OK; ++dir) {
        SplitPass &P = dir == 0 ? ph_out.fwd : ph_out.bwd;
        P.n_phases = np;
        P.n_cg = n_cg;
        P.n_chunks = n_chunks;
        P.pitch = (int32_t)pitch;
        P.MT = MT;
        P.mt_shift = MT == 4 ? 2 : (MT == 2 ? 1 : 0);
        P.cg_stride = lower ? (int32_t)S_mid : inner;
        P.row_stride = (int32_t)d;
        P.chunk_off = 0;
        std::vector<int32_t> tab(tables);
        int32_t words = 0;
        std::vector<int32_t> frag_off((size_t)np);
        for (int k = 0; k < np; ++k) {
            const int p = dir == 0 ? k : np - 1 - k;
            const GPhase &gp = phs[(size_t)p];
            const ItemSet &is = sets[(size_t)p];
            SplitPhase &D = P.ph[k];
            D.mode = is.mode;
            D.B = gp.B;
            D.B_real = gp.B_real;
            const int l = is.mode == 0 ? 1 : lm[(size_t)p];
            const int *jo = gp.B == 16 ? (l == 1 ? joff1_16 : joff2_16) : (l == 1 ? joff1_8 : joff2_8);
            D.lm = l;
            D.lane_step = (int32_t)(l * W[(size_t)p]);
            for (int j = 0; j < 4; ++j) { D.jr[j] = jo[j]; D.j_off[j] = (int32_t)(jo[j] * W[(size_t)p]); }
            D.items_off = (int32_t)tab.size();
            D.n_items = (int32_t)is.bases.size();
            D.paired = 0;
            if (is.mode == 0 && gp.B == 8 && is.bases.size() % 2 == 0) {
                D.paired = 1;
                for (size_t i = 0; i + 1 < is.bases.size(); i += 2) D.paired = D.paired && is.bases[i + 1] == is.bases[i] + 8;
            }
            tab.insert(tab.end(), is.bases.begin(), is.bases.end());
            D.bfrag_off = words;
            frag_off[(size_t)p] = words;
            words += (int32_t)(is.block_rel.size() * 32 * (gp.B == 16 ? 4 : 1));
            // bounds of every address formed from the tables
            bool ok = true;
            const int nj = gp.B == 16 ? 4 : 2;
            for (int32_t b : is.bases) {
                if (is.mode == 0) ok = ok && b >= 0 && b % 8 == 0 && b + gp.B <= pitch;
                else
                    for (int qq = 0; qq < 4; ++qq)
                        for (int j = 0; j < nj; ++j) {
                            if (l * qq + jo[j] >= gp.B_real) continue;
                            const int64_t a = (int64_t)b + (int64_t)qq * D.lane_step + D.j_off[j];
                            ok = ok && b >= 0 && a % 8 == 0 && a + 8 <= pitch;
                        }
            }
            if (!ok) return HARP_ERR_UNSUPPORTED;
        }
        words = (words + 3) / 4 * 4;
        P.bfrag_words = words;
        P.tables_len = (int32_t)tab.size();
        P.tables = upload_s(sp, tab, st);
        // ---- fragments for every column group
        std::vector<uint32_t> frag((size_t)n_cg * words, 0u);
        std::vector<double> F;
        for (int cgi = 0; cgi < n_cg; ++cgi) {
            const int64_t cg_base = lower ? (int64_t)cgi * S_mid : (int64_t)cgi * inner;
            for (int p = 0; p < np; ++p) {
                const GPhase &gp = phs[(size_t)p];
                const ItemSet &is = sets[(size_t)p];
                const int B = gp.B, Br = gp.B_real;
                const int l = is.mode == 0 ? 1 : lm[(size_t)p];
                HostPhase hp{gp.t0, gp.t1, Br, gp.S, 0, 1};
                const int wpl = B == 16 ? 4 : 1;
                for (size_t bi = 0; bi < is.block_rel.size(); ++bi) {
                    const int64_t base = cg_base + is.block_rel[bi];
                    fused_block(plan, hp, base, F);
                    auto G = [&](int rin, int rout) -> double {
                        if (rin >= Br || rout >= Br) return 0.0;
                        double v = dir == 0 ? F[(size_t)rin * Br + rout] : F[(size_t)rout * Br + rin];
                        if (gp.t0 == 0 && !plan->h_signs.empty()) {
                            const int64_t pos = base + (int64_t)(dir == 0 ? rin : rout) * gp.S;
                            v *= (double)plan->h_signs[(size_t)(plan->h_perm.empty() ? pos : plan->h_perm[(size_t)pos])];
                        }
                        return v;
                    };
                    auto slot = [&](int s) { return is.mode == 0 ? s : strided_slot(s, B, l); };
                    uint32_t *dst0 = frag.data() + (size_t)cgi * words + frag_off[(size_t)p] + bi * 32 * wpl;
                    // 8-wide strided phases: the words of an item's eight blocks sit together per lane,
                    // [item][blocks 0-3 | 4-7][lane][4 words], so that a lane fetches them with two 16-byte loads
                    const bool grouped = is.mode == 1 && B == 8;
                    uint32_t *grp0 = frag.data() + (size_t)cgi * words + frag_off[(size_t)p] + (bi / 8) * 256 + ((bi % 8) / 4) * 128 + (bi % 4);
                    for (int lane = 0; lane < 32; ++lane) {
                        const int gg = lane >> 2, qq = lane & 3;
                        uint32_t *dst = grouped ? grp0 + lane * 4 : dst0 + lane * wpl;
                        if (B == 16) {
                            for (int nt = 0; nt < 2; ++nt) {
                                const int n = slot(8 * nt + gg);
                                dst[2 * nt] = f2bf(G(slot(2 * qq), n)) | ((uint32_t)f2bf(G(slot(2 * qq + 1), n)) << 16);
                                dst[2 * nt + 1] = f2bf(G(slot(2 * qq + 8), n)) | ((uint32_t)f2bf(G(slot(2 * qq + 9), n)) << 16);
                            }
                        } else {
                            const int n = slot(gg);
                            dst[0] = f2bf(G(slot(2 * qq), n)) | ((uint32_t)f2bf(G(slot(2 * qq + 1), n)) << 16);
                        }
                    }
                }
            }
        }
        P.bfrag = upload_s(sp, frag, st);
        const size_t tile_bytes = (size_t)16 * MT * pitch * 2;
        bool any16 = false;
        for (const GPhase &gp : phs) any16 = any16 || gp.B == 16;
        const size_t one = (tile_bytes + tab.size() * 4 + 15) / 16 * 16 + (size_t)words * 4;
        P.n_buf = (any16 && one + tile_bytes <= 100u * 1024u) ? 2 : 1;
        const size_t need = (P.n_buf * tile_bytes + tab.size() * 4 + 15) / 16 * 16 + (size_t)words * 4;
        ph_out.smem_bytes = std::max(ph_out.smem_bytes, need);
    }
    if (st == HARP_OK && ph_out.smem_bytes > 110u * 1024u) return HARP_ERR_UNSUPPORTED;
    ph_out.present = true;
    for (const GPhase &gp : phs) ph_out.has16 = ph_out.has16 || gp.B == 16;
    return st;
}


// All upper stages fused into one U x U block per position l (U <= 64).
harp_status_t build_dense_upper(const harp_plan *plan, SplitPlan *sp, int t0, int64_t S_mid, int64_t U) {
    if (U > 64 || U < 2) return HARP_ERR_UNSUPPORTED;
    const int KP = (int)((U + 15) / 16 * 16), KS = KP / 16, NT = (int)((U + 7) / 8);
    const int64_t per_l_words = (int64_t)NT * KS * 64;
    // U <= 48 and sixteen positions per column group: the fragments of two positions fit a warp's registers
    const bool in_regs = KS <= 3 && S_mid % 16 == 0;
    int Lw = 16;
    if (!in_regs && (S_mid % 16 != 0 || 16 * per_l_words * 4 > 80 * 1024)) Lw = 8;
    if (S_mid % Lw != 0) return HARP_ERR_UNSUPPORTED;
    const int l_skew = in_regs ? 32 : 0;
    int64_t pitch = (int64_t)Lw * KP + l_skew;
    if ((pitch / 8) % 2 == 0) pitch += 8;
    const int64_t frag_bytes = in_regs ? 0 : Lw * per_l_words * 4;
    int MT = 1;
    // in_regs: the tile twice (operand buffer and the staging buffer of 32 KP + 64 bytes per row)
    auto tile_bytes = [&](int mt) { return (int64_t)16 * mt * (pitch * 2 + (in_regs ? 32 * KP + 64 : 0)); };
    while (MT < 4 && tile_bytes(2 * MT) + frag_bytes <= (in_regs ? 110 : 100) * 1024) MT *= 2;
    const size_t smem = in_regs ? ((size_t)16 * MT * pitch * 2 + 15) / 16 * 16 + (size_t)16 * MT * (32 * KP + 64)
                                : ((size_t)16 * MT * pitch * 2 + 15) / 16 * 16 + (size_t)frag_bytes;
    if (smem > 110u * 1024u) return HARP_ERR_UNSUPPORTED;
    if ((Lw / 8) * (KP / 8) > kSplitThreads) return HARP_ERR_UNSUPPORTED;
    const int n_cg = (int)(S_mid / Lw);
    harp_status_t st = HARP_OK;
    HostPhase hp{t0, plan->st.m, (int)U, S_mid, 0, 1};
    std::vector<double> F;
    for (int dir = 0; dir < 2 && st == HARP_OK; ++dir) {
        UpperPass &P = dir == 0 ? sp->up_fwd : sp->up_bwd;
        P.n_cg = n_cg; P.Lw = Lw; P.U = (int32_t)U; P.KP = KP; P.NT = NT; P.pitch = (int32_t)pitch; P.MT = MT;
        P.l_skew = l_skew;
        P.S_mid = (int32_t)S_mid; P.row_stride = (int32_t)plan->d;
        P.bfrag_words = (int32_t)(Lw * per_l_words);
        std::vector<uint32_t> frag((size_t)n_cg * P.bfrag_words, 0u);
        for (int cgi = 0; cgi < n_cg; ++cgi)
            for (int l = 0; l < Lw; ++l) {
                const int64_t base = (int64_t)cgi * Lw + l;
                fused_block(plan, hp, base, F);
                auto G = [&](int rin, int rout) -> double {
                    if (rin >= U || rout >= U) return 0.0;
                    return dir == 0 ? F[(size_t)rin * U + rout] : F[(size_t)rout * U + rin];
                };
                uint32_t *dst0 = frag.data() + (size_t)cgi * P.bfrag_words + (size_t)l * per_l_words;
                for (int nt = 0; nt < NT; ++nt)
                    for (int ks = 0; ks < KS; ++ks)
                        for (int lane = 0; lane < 32; ++lane) {
                            const int gg = lane >> 2, qq = lane & 3;
                            const int n = 8 * nt + gg, k0 = 16 * ks + 2 * qq;
                            uint32_t *dst = dst0 + ((size_t)(nt * KS + ks) * 32 + lane) * 2;
                            dst[0] = f2bf(G(k0, n)) | ((uint32_t)f2bf(G(k0 + 1, n)) << 16);
                            dst[1] = f2bf(G(k0 + 8, n)) | ((uint32_t)f2bf(G(k0 + 9, n)) << 16);
                        }
            }
        P.bfrag = upload_s(sp, frag, st);
    }
    sp->dense_upper = true;
    sp->up_in_regs = in_regs;
    sp->up_smem = smem;
    sp->up_ks = KS;
    return st;
}

}  // namespace

harp_status_t harp_split_build(harp_plan *plan) {
    const int64_t d = plan->d;
    const int m = plan->st.m;
    if (d % 8 != 0) return HARP_ERR_UNSUPPORTED;
    const bool permuted = !plan->h_perm.empty();
    if (permuted && d > 65536) return HARP_ERR_UNSUPPORTED;                         // 16-bit gather tables
    // ---- group stages: as many as fit a 16-wide block; smaller products are zero-padded to 8 or 16.
    // A radix above 16 ends the grouping: it and everything after it form the dense upper block.
    std::vector<GPhase> phs;
    int t_big = m;
    for (int t = 0; t < m;) {
        if (plan->st.b[t] > 16) { t_big = t; break; }
        int64_t prod = 1;
        int t1 = t;
        while (t1 < m && prod * plan->st.b[t1] <= 16) prod *= plan->st.b[t1++];
        phs.push_back({t, t1, prod <= 8 ? 8 : 16, (int)prod, plan->st.s[t]});
        t = t1;
    }
    if (phs.empty() || phs[0].B != phs[0].B_real) return HARP_ERR_UNSUPPORTED;   // octets run along the first phase
    // ---- split point: the longest prefix whose slab has at most 512 coordinates
    int k = 0;
    int64_t S_mid = 1;
    while (k < (int)phs.size() && S_mid * phs[(size_t)k].B_real <= 512) S_mid *= phs[(size_t)k++].B_real;
    if (k == 0 || S_mid % 8 != 0) return HARP_ERR_UNSUPPORTED;
    const int64_t U = d / S_mid;
    std::vector<GPhase> lower(phs.begin(), phs.begin() + k), upper(phs.begin() + k, phs.end());
    const int Lw = 16;
    const bool want_dense = t_big < m || (getenv("HARP_UPPER_DENSE") && atoi(getenv("HARP_UPPER_DENSE")) && U > 1);
    if (t_big < m && k != (int)phs.size()) return HARP_ERR_UNSUPPORTED;            // big radix must follow the slab directly
    if (!want_dense && !upper.empty() && S_mid % Lw != 0) return HARP_ERR_UNSUPPORTED;

    SplitPlan *sp = new (std::nothrow) SplitPlan();
    if (!sp) return HARP_ERR_ALLOC;
    sp->lower_stages = lower.back().t1;
    harp_status_t st = build_pass(plan, sp, sp->pass[0], lower, true, S_mid, U, 1);
    if (st == HARP_OK && want_dense) st = build_dense_upper(plan, sp, lower.back().t1, S_mid, U);
    else if (st == HARP_OK && !upper.empty()) st = build_pass(plan, sp, sp->pass[1], upper, false, S_mid, U, Lw);
    if (st == HARP_OK &&
        (cudaFuncSetAttribute(harp_split_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_split_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_split_kernel<true>, cudaFuncAttributePreferredSharedMemoryCarveout, 100) != cudaSuccess ||
         cudaFuncSetAttribute(harp_split_kernel<false>, cudaFuncAttributePreferredSharedMemoryCarveout, 100) != cudaSuccess ||
         cudaFuncSetAttribute(harp_upper_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_upper_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_upper_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_upper_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_upper_reg_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_upper_reg_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_upper_reg_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess))
        st = HARP_ERR_CUDA;
    if (st == HARP_OK && permuted) {
        std::vector<uint16_t> fwd((size_t)d), bwd((size_t)d);
        for (int64_t i = 0; i < d; ++i) {
            fwd[(size_t)i] = (uint16_t)plan->h_perm[(size_t)i];
            bwd[(size_t)plan->h_perm[(size_t)i]] = (uint16_t)i;
        }
        sp->gather[0] = upload_s(sp, fwd, st);
        sp->gather[1] = upload_s(sp, bwd, st);
        // table + two buffers of R rows in about 200 KB
        const size_t row_bytes = (size_t)d * 2;
        sp->gather_rows = (int)std::max<size_t>(1, std::min<size_t>(16, (200u * 1024u - row_bytes) / (2 * row_bytes)));
        sp->gather_smem = row_bytes * (1 + 2 * (size_t)sp->gather_rows);
        if (sp->gather_smem > 227u * 1024u) st = HARP_ERR_UNSUPPORTED;
        else if (st == HARP_OK && cudaFuncSetAttribute(harp_gather_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                       (int)sp->gather_smem) != cudaSuccess)
            st = HARP_ERR_CUDA;
    }
    if (st == HARP_OK) {
        int dev = 0, sms = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms > 0) sp->sms = sms;
        // Rows per chunk.  A chunk that fits L2 lets the second pass read what the first wrote
        // without going to HBM, but every chunk costs two launches and two partial waves; with
        // the present kernels (bound by instruction issue, not by HBM) large chunks are faster,
        // so the default is one chunk of up to 8 GiB.  HARP_SPLIT_CHUNK_MB overrides it.
        const char *e = getenv("HARP_SPLIT_CHUNK_MB");
        const int64_t chunk_bytes = (int64_t)(e ? atoi(e) : 8192) << 20;
        sp->chunk_rows = std::max<int64_t>(64, chunk_bytes / (d * 2) / 64 * 64);
    }
    plan->split = sp;
    if (st != HARP_OK) {
        cudaGetLastError();
        harp_split_destroy(plan);
        return st;
    }
    return HARP_OK;
}

void harp_split_destroy(harp_plan *plan) {
    if (!plan->split) return;
    for (void *p : plan->split->dev_allocs) cudaFree(p);
    delete plan->split;
    plan->split = nullptr;
}

// Launch of one pass.  overlap: let the kernel's preamble run under the tail of the kernel before it
// in the stream (see rows_ready_barrier); used for small row counts, where a pass lasts a few
// microseconds and the preamble is a large part of it.
template <typename PassT>
cudaError_t launch_pass(void (*kern)(__nv_bfloat16 *, int64_t, int64_t, PassT), unsigned grid, size_t smem, cudaStream_t stream,
                        bool overlap, __nv_bfloat16 *x, int64_t r0, int64_t r1, const PassT &P) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kSplitThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, x, r0, r1, P);
}

constexpr int64_t kOverlapMaxRows = 64;
constexpr int64_t kTmSlabMinRows = 1024;

harp_status_t harp_split_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype, int transpose,
                               cudaStream_t stream) {
    const SplitPlan *sp = plan->split;
    if (!sp || dtype != HARP_BF16) return HARP_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(x) & 15u) != 0) return HARP_ERR_UNSUPPORTED;
    __nv_bfloat16 *xb = static_cast<__nv_bfloat16 *>(x);
    const bool two = sp->pass[1].present || sp->dense_upper;
    // (with the attribute on for every batch size an apply of 32768 rows at d = 14336 took 940 us instead of 907,
    // 65536 rows at d = 28672 5.2 ms instead of 4.8: large batches are launched plainly)
    const bool overlap = n_rows <= kOverlapMaxRows;
    auto gather = [&](int dir) -> harp_status_t {
        const int64_t n_groups = (n_rows + sp->gather_rows - 1) / sp->gather_rows;
        const unsigned grid = (unsigned)std::min<int64_t>(n_groups, sp->sms);
        harp_gather_rows_kernel<<<grid, kGatherThreads, sp->gather_smem, stream>>>(xb, n_rows, (int32_t)plan->d, sp->gather_rows,
                                                                                   sp->gather[dir]);
        g_harp_launches.fetch_add(1, std::memory_order_relaxed);
        return cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
    };
    if (sp->gather[0] && !transpose) {
        const harp_status_t gs = gather(0);
        if (gs != HARP_OK) return gs;
    }
    for (int64_t r0 = 0; r0 < n_rows; r0 += sp->chunk_rows) {
        const int64_t r1 = std::min(n_rows, r0 + (two ? sp->chunk_rows : n_rows));
        for (int s = 0; s < (two ? 2 : 1); ++s) {
            const int pi = transpose ? (two ? 1 - s : 0) : s;
            if (pi == 1 && sp->dense_upper) {
                const UpperPass &P = transpose ? sp->up_bwd : sp->up_fwd;
                const int64_t tile_rows = 16 * P.MT;
                const int64_t n_tiles = (r1 - r0 + tile_rows - 1) / tile_rows;
                const int per_sm = std::max<int>(1, std::min<int>(2, (int)((220 * 1024) / (sp->up_smem + 1024))));
                int64_t parts = std::max<int64_t>(1, ((int64_t)sp->sms * per_sm) / P.n_cg);
                parts = std::min(parts, n_tiles);
                const unsigned grid = (unsigned)(parts * P.n_cg);
                cudaError_t err;
                if (sp->up_in_regs) {
                    switch (sp->up_ks) {
                        case 1: err = launch_pass(harp_upper_reg_kernel<1>, grid, sp->up_smem, stream, overlap, xb, r0, r1, P); break;
                        case 2: err = launch_pass(harp_upper_reg_kernel<2>, grid, sp->up_smem, stream, overlap, xb, r0, r1, P); break;
                        default: err = launch_pass(harp_upper_reg_kernel<3>, grid, sp->up_smem, stream, overlap, xb, r0, r1, P); break;
                    }
                } else
                switch (sp->up_ks) {
                    case 1: err = launch_pass(harp_upper_kernel<1>, grid, sp->up_smem, stream, overlap, xb, r0, r1, P); break;
                    case 2: err = launch_pass(harp_upper_kernel<2>, grid, sp->up_smem, stream, overlap, xb, r0, r1, P); break;
                    case 3: err = launch_pass(harp_upper_kernel<3>, grid, sp->up_smem, stream, overlap, xb, r0, r1, P); break;
                    default: err = launch_pass(harp_upper_kernel<4>, grid, sp->up_smem, stream, overlap, xb, r0, r1, P); break;
                }
                g_harp_launches.fetch_add(1, std::memory_order_relaxed);
                if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return HARP_ERR_CUDA;
                continue;
            }
            // lower pass on slabs of 256 coordinates: the tensor-memory kernel (128-row tiles, bulk tensor
            // copies) when the plan has it and the batch fills its tiles
            if (pi == 0 && r1 - r0 >= kTmSlabMinRows && harp_tm_slab_stages(plan) == sp->lower_stages) {
                const harp_status_t ts = harp_tm_slab_apply(plan, xb + r0 * plan->d, r1 - r0, dtype, transpose, stream);
                if (ts == HARP_OK) continue;
                if (ts != HARP_ERR_UNSUPPORTED) return ts;
            }
            const PassHost &ph = sp->pass[pi];
            SplitPass P = transpose ? ph.bwd : ph.fwd;
            while (P.MT > 1 && 16 * (int64_t)(P.MT / 2) >= r1 - r0) {     // a small batch takes the smallest tile that holds it
                P.MT /= 2;
                --P.mt_shift;
            }
            const int64_t tile_rows = 16 * P.MT;
            const int64_t n_tiles = (r1 - r0 + tile_rows - 1) / tile_rows;
            // one wave of CTAs, each keeping its column group for as many tiles as possible
            const int per_sm = std::max<int>(1, std::min<int>(ph.has16 ? 2 : 3, (int)((220 * 1024) / (ph.smem_bytes + 1024))));
            int64_t parts = std::max<int64_t>(1, ((int64_t)sp->sms * per_sm) / P.n_cg);
            parts = std::min(parts, n_tiles);
            const int64_t grid = parts * P.n_cg;
            const cudaError_t err =
                ph.has16 ? launch_pass(harp_split_kernel<true>, (unsigned)grid, ph.smem_bytes, stream, overlap, xb, r0, r1, P)
                         : launch_pass(harp_split_kernel<false>, (unsigned)grid, ph.smem_bytes, stream, overlap, xb, r0, r1, P);
            g_harp_launches.fetch_add(1, std::memory_order_relaxed);
            if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return HARP_ERR_CUDA;
        }
        if (!two) break;
    }
    if (sp->gather[0] && transpose) return gather(1);
    return HARP_OK;
}
