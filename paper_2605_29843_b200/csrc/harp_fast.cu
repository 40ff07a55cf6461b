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
// the order of the direction's input (source order forward, output order for the transpose),
// the phases run in place on a layout ordered the same way (a digit reversal maps every phase
// onto a digit group again, only with other strides), and the last phase of the direction
// reorders inside shared memory, in place: an item of that phase reads eight blocks that are
// neighbours in the order of the direction's output (16 contiguous values of the layout each,
// ldmatrix) and writes its sixteen eight-block runs into the same sixteen 16-byte slots; the
// copy to global memory follows a chunk map.
// Any other permutation that maps every aligned run of eight source coordinates onto the
// same slot of eight different first-phase blocks is gathered (forward) or scattered
// (transpose) in global memory with 16-byte accesses by the first/last phase.  All other
// permutations use the generic kernel.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>

#include "harp_internal.h"
#include "harp_mma.cuh"
#include "harp_fuse.h"
#include "harp_tm_ptx.cuh"

namespace {

constexpr int kMaxPhases = 8;
constexpr int kTileRows = 16;
constexpr int kThreads = 512;

enum PhaseMode : int32_t {
    MODE_CC = 0,   // contiguous block in shared memory, in place (ldmatrix / stmatrix)
    MODE_SS = 1,   // strided block in shared memory, eight blocks per item, in place
    MODE_GS = 2,   // operands gathered from global memory, result to contiguous smem blocks
    MODE_CG = 3,   // operands from contiguous smem blocks, result scattered to global memory
    MODE_PO = 4    // contiguous smem blocks in, eight-block runs out to the same slots (reorders the tile in place)
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
    // phases whose block fragments a CTA keeps in tensor memory for all its tiles (bit p = phase p):
    // warp w reads the fragments of its own items w and w + 16 from its 32 lanes, 32 columns per item
    uint32_t tm_mask;
    PhaseDesc ph[kMaxPhases];
};

// Per-section cycle counters of the whole-row kernel (build with -DHARP_FAST_TIMING): thread 0 of every CTA
// reads the clock after the barrier that ends a section; sums over CTAs and tiles.
//  0 tiles | 1 copy in | 2 .. 2+kMaxPhases-1 phase k | 10 copy out
__device__ long long g_fast_timing[16];
#ifdef HARP_FAST_TIMING
#define FAST_MARK(slot) do { if (threadIdx.x == 0) { const long long now_ = clock64(); tacc[slot] += now_ - tlast; tlast = now_; } } while (0)
#else
#define FAST_MARK(slot) do { } while (0)
#endif

// fragments of one item (eight blocks, one uint4 per lane and block): from tensor memory when the
// phase is kept there, else from global memory
__device__ __forceinline__ void load_frag8(uint4 (&bf)[8], const uint4 *bp, bool in_tm, uint32_t tm_addr) {
    if (in_tm) {
        uint32_t v[32];
        harp_tm::tmem_ld32(tm_addr, v);
        harp_tm::tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 8; ++e) bf[e] = make_uint4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) bf[e] = __ldg(bp + e * 32);
    }
}

// ----------------------------------------------------------------------------- device

struct TileCtx {
    uint32_t sbase;          // shared address of the tile
    const int32_t *tab;      // tables in shared memory
    int pitch, lane, warp, g, q;
    __nv_bfloat16 *xA, *xB;  // global rows g and g+8 of the tile (clamped to the batch)
    bool okA, okB;
    uint32_t tm_warp;        // tensor-memory address of this warp's fragment columns
};
// tensor-memory address of item `it` of the phase kept in slot `slot` (0 or 1), for the calling warp
__device__ __forceinline__ uint32_t tm_item(const TileCtx &c, int slot, int it) {
    return c.tm_warp + (uint32_t)((slot * 2 + (it >> 4)) * 32);
}

// ---- MODE_SS, B = 16: load / store of one item's operands
__device__ __forceinline__ void ss16_load(const TileCtx &c, const PhaseDesc &ph, int it, uint4 (&raw)[4][2], uint4 (&bf)[8],
                                          int tm_slot) {
    const uint32_t a0 = c.sbase + 2u * (uint32_t)(c.g * c.pitch + c.q * ph.lane_step + c.tab[ph.items_off + it]);
    const uint32_t a1 = a0 + 2u * (uint32_t)(8 * c.pitch);
    const uint4 *bp = ph.bfrag + (size_t)it * 256 + c.lane;
    load_frag8(bf, bp, tm_slot >= 0, tm_item(c, tm_slot, it));
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
__device__ __forceinline__ void gs_load(const TileCtx &c, const PhaseDesc &ph, int it, uint4 (&raw)[4][2], uint4 (&bf)[8],
                                        int tm_slot) {
    const int32_t *tab = c.tab + ph.items_off + it * 24;
    const uint4 *bp = ph.bfrag + (size_t)it * 256 + c.lane;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int off = tab[c.q * ph.lane_step + ph.j_off[j]];
        raw[j][0] = ldg128_stream(c.xA + off);
        raw[j][1] = ldg128_stream(c.xB + off);
    }
    load_frag8(bf, bp, tm_slot >= 0, tm_item(c, tm_slot, it));
}
__device__ __forceinline__ void gs_store(const TileCtx &c, const PhaseDesc &ph, int it, const uint32_t (&mats)[8][4]) {
    const int32_t *tab = c.tab + ph.items_off + it * 24 + 16;
    const int mrow = (c.lane & 7) + ((c.lane >> 3) & 1) * 8, mcol = (c.lane >> 4) * 8;
#pragma unroll
    for (int e = 0; e < 8; ++e)
        stmatrix_x4(c.sbase + 2u * (uint32_t)(mrow * c.pitch + tab[e] + mcol), mats[e][0], mats[e][1], mats[e][2], mats[e][3]);
}

// MODES: bit m set = the code of phase mode m is compiled in.  The host launches the variant
// that holds exactly the modes of the plan's direction, so that the register allocation of one
// scheme does not pay for the others.
__host__ __device__ constexpr uint32_t bit(int mode) { return 1u << mode; }
constexpr uint32_t kModesGeneral = bit(MODE_CC) | bit(MODE_SS) | bit(MODE_GS) | bit(MODE_CG);
constexpr uint32_t kModesReorderOut = bit(MODE_SS) | bit(MODE_PO);   // the digit-reversal scheme, both directions

template <int NT, uint32_t MODES>
__global__ void __launch_bounds__(NT, 1)
harp_fast_kernel(__nv_bfloat16 *__restrict__ x, int64_t n_rows, int64_t n_tiles, int stagger, FastParams P) {
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
    // ---- block fragments of up to two phases into tensor memory, once per CTA ----
    uint32_t &tm_base_s = *reinterpret_cast<uint32_t *>(tab_s + P.tables_len);   // one word after the tables
    if (P.tm_mask) {
        if (c.warp == 0) harp_tm::tmem_alloc(smem_u32(&tm_base_s), 512);
        harp_tm::tc_fence_before();
    }
    __syncthreads();
    c.tm_warp = 0;
    if (P.tm_mask) {
        harp_tm::tc_fence_after();
        c.tm_warp = tm_base_s + ((uint32_t)((c.warp & 3) * 32) << 16) + (uint32_t)((c.warp >> 2) * 128);
        int slot = 0;
        for (int p = 0; p < P.n_phases; ++p) {
            if (!((P.tm_mask >> p) & 1u)) continue;
            for (int it = c.warp; it < P.ph[p].n_items; it += NW) {
                uint32_t v[32];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint4 f = __ldg(P.ph[p].bfrag + (size_t)it * 256 + e * 32 + c.lane);
                    v[4 * e] = f.x; v[4 * e + 1] = f.y; v[4 * e + 2] = f.z; v[4 * e + 3] = f.w;
                }
                harp_tm::tmem_st32(tm_item(c, slot, it), v);
            }
            ++slot;
        }
        harp_tm::tmem_wait_st();
    }
    const int warp = c.warp, lane = c.lane;

    // All CTAs have the same work, so without this they copy their tiles in step and share the
    // HBM bandwidth at those moments while it idles during the phases.  Three classes of CTAs
    // start a quarter of a tile period apart (a bounded wait on the clock; only used when every
    // CTA has several tiles, so the delay is small against the run).
    if (stagger > 0) {
        const long long wait = (long long)(blockIdx.x % 3) * stagger, t0 = clock64();
        while (clock64() - t0 < wait) { }
    }
    // Everything above reads the plan's data only.  Launched with the programmatic stream-serialisation
    // attribute, a CTA gets here while the kernel before it in the stream is still running on other SMs
    // (tables, tensor-memory fill and the start delay then cost nothing); the rows are touched only after
    // that kernel has completed.  The kernel after this one may start its own preamble as SMs become free.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#ifdef HARP_FAST_TIMING
    long long tacc[16] = {0}, tlast = clock64();
#endif
    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int64_t row0 = tile * kTileRows;
#ifdef HARP_FAST_TIMING
        if (threadIdx.x == 0) { tacc[0] += 1; tlast = clock64(); }
#endif
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
        FAST_MARK(1);

        for (int p = 0; p < P.n_phases; ++p) {
            const PhaseDesc &ph = P.ph[p];
            const int n = ph.n_items;
            const int tm_slot = ((P.tm_mask >> p) & 1u) ? __popc(P.tm_mask & ((1u << p) - 1u)) : -1;
            if ((MODES & bit(MODE_CC)) && ph.mode == MODE_CC) {
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
            } else if ((MODES & bit(MODE_SS)) && ph.mode == MODE_SS && ph.B == 16) {
                // (prefetching the next item's operands or fragments in registers was measured: the
                // kernel sits at the register limit and every variant that holds more spills)
                uint4 raw[4][2], bf[8];
                uint32_t unused[8][4];
                for (int it = warp; it < n; it += NW) {
                    ss16_load(c, ph, it, raw, bf, tm_slot);
                    octet_mma16<true>(raw, bf, unused);
                    ss16_store(c, ph, it, raw);
                }
            } else if ((MODES & bit(MODE_SS)) && ph.mode == MODE_SS) {
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
            } else if ((MODES & bit(MODE_GS)) && ph.mode == MODE_GS) {
                uint4 raw[4][2], bf[8];
                uint32_t mats[8][4];
                for (int it = warp; it < n; it += NW) {
                    gs_load(c, ph, it, raw, bf, tm_slot);
                    octet_mma16<false>(raw, bf, mats);
                    gs_store(c, ph, it, mats);
                }
            } else if ((MODES & bit(MODE_PO)) && ph.mode == MODE_PO) {
                // contiguous blocks in (ldmatrix), eight-block runs out to the same sixteen 16-byte
                // slots the item read (a per-item table names them): in place, no barrier
                const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
                for (int it = warp; it < n; it += NW) {
                    const int32_t *tab = tab_s + ph.items_off + it * 24;
                    uint4 bf[8], out[4][2];
                    load_frag8(bf, ph.bfrag + (size_t)it * 256 + lane, tm_slot >= 0, tm_item(c, tm_slot, it));
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        float acc[2][2][4];
#pragma unroll
                        for (int ee = 0; ee < 2; ++ee) {
                            const int e = 2 * w + ee;
                            uint32_t a[4];
                            ldmatrix_x4(a, c.sbase + 2u * (uint32_t)(mrow * pitch + tab[e] + mcol));
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
                    // every lane's ldmatrix of this item precedes these stores in program order
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t o0 = c.sbase + 2u * (uint32_t)(c.g * pitch + tab[8 + c.q + 4 * j]);
                        sts128(o0, out[j][0]);
                        sts128(o0 + 2u * (uint32_t)(8 * pitch), out[j][1]);
                    }
                }
            } else if ((MODES & bit(MODE_CG)) && ph.mode == MODE_CG) {   // operands from contiguous smem blocks, results scattered to global memory
                const int mrow = (lane & 7) + ((lane >> 3) & 1) * 8, mcol = (lane >> 4) * 8;
                for (int it = warp; it < n; it += NW) {
                    const int32_t *tab = tab_s + ph.items_off + it * 24;
                    uint4 bf[8];
                    load_frag8(bf, ph.bfrag + (size_t)it * 256 + lane, tm_slot >= 0, tm_item(c, tm_slot, it));
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
            FAST_MARK(2 + p);
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
        FAST_MARK(10);
    }
#ifdef HARP_FAST_TIMING
    if (threadIdx.x == 0)
        for (int k = 0; k < 16; ++k)
            if (tacc[k]) atomicAdd((unsigned long long *)&g_fast_timing[k], (unsigned long long)tacc[k]);
#endif
    if (P.tm_mask) {
        harp_tm::tc_fence_before();
        __syncthreads();
        if (c.warp == 0) harp_tm::tmem_dealloc(tm_base_s, 512);
    }
}

}  // namespace

// ----------------------------------------------------------------------------- host

struct FastPlan {
    FastParams fwd{}, bwd{};
    size_t smem_bytes = 0;
    int variant_fwd = 0, variant_bwd = 0;     // which compiled set of phase modes each direction needs
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
    }
    std::vector<int64_t> inv;                                        // source coordinate -> natural coordinate
    if (!identity) {
        inv.resize((size_t)d);
        for (int64_t i = 0; i < d; ++i) inv[(size_t)plan->h_perm[(size_t)i]] = i;
    }

    // ---- shared-memory layouts.  "nat": coordinates in the plan's own order; "src": in the
    // order of the rows in global memory before the gather (digit-reversal scheme only).
    // Local index r of a phase sits at element offset r*W + (r/4)*gp.  The four lanes q of a
    // quarter-warp hold local indices lm*q + const, lm*W (+ gp when lm = 4) elements apart; that
    // distance should be 2 or 6 (mod 8) 16-byte slots, which together with the odd row pitch puts
    // the eight accesses of a quarter-warp into eight bank groups.  The strides also decide how
    // the chunk copies of the tile hit the banks.  W (padding), gp (gap after every fourth step)
    // and lm are chosen per phase by coordinate descent on the number of shared-memory wavefronts
    // of the strided phases and of the two tile copies.
    struct Layout {
        std::vector<int64_t> S, W, gp;  // per phase: coordinate stride, shared-memory stride, gap
        std::vector<int> lm;            // per phase: lane multiplier (1, 2 or 4)
        int64_t extent = 0;
        int64_t off(int p, int64_t r) const { return r * W[(size_t)p] + (r / 4) * gp[(size_t)p]; }
    };
    struct Choice { int pad, gap, lm; };                 // pad and gap in 16-byte slots
    auto make_layout = [&](const std::vector<int> &order, const std::vector<int64_t> &strides,
                           const std::vector<Choice> &ch, Layout &L) {
        L.S = strides;
        L.W.assign((size_t)np, 0);
        L.gp.assign((size_t)np, 0);
        L.lm.assign((size_t)np, 1);
        int64_t W = 1;
        bool first = true;
        for (int p : order) {
            const int B = phases[(size_t)p].B;
            const Choice &c = ch[(size_t)p];
            int64_t gp = 0;
            if (!first) {
                W = (W + 7) / 8 * 8 + 8 * c.pad;
                gp = 8 * c.gap;
                if (c.lm == 4 && B != 16) return false;
                if (c.lm == 2 && gp != 0) return false;  // the lanes' slots would straddle a gap
                L.lm[(size_t)p] = c.lm;
            } else if (c.pad || c.gap || c.lm != 1) {
                return false;
            }
            first = false;
            L.W[(size_t)p] = W;
            L.gp[(size_t)p] = gp;
            W = W * B + (B / 4 - 1) * gp;
        }
        L.extent = W;
        return true;
    };
    auto pitch_of = [&](const Layout &L) {
        int64_t pt = (L.extent + 7) / 8 * 8;
        if ((pt / 8) % 2 == 0) pt += 8;
        return pt;
    };
    auto worst_bank = [](const std::vector<int64_t> &slots) {   // wavefronts of one quarter-warp access
        int cnt[8] = {0, 0, 0, 0, 0, 0, 0, 0}, worst = 0;
        for (int64_t s : slots) worst = std::max(worst, ++cnt[((s % 8) + 8) % 8]);
        return worst;
    };
    std::vector<int> order_nat((size_t)np), order_src((size_t)np);
    std::vector<int64_t> S_nat((size_t)np), S_src((size_t)np);
    for (int p = 0; p < np; ++p) {
        order_nat[(size_t)p] = p;
        order_src[(size_t)p] = np - 1 - p;
        S_nat[(size_t)p] = phases[(size_t)p].S;
        S_src[(size_t)p] = d / (phases[(size_t)p].S * phases[(size_t)p].B);   // prod of radices above the phase
    }
    // offset of a coordinate in a layout (coordinate in the layout's own order)
    auto phys_in = [&](const Layout &L, int64_t pos) {
        int64_t o = 0;
        for (int p = 0; p < np; ++p) o += L.off(p, (pos / L.S[(size_t)p]) % phases[(size_t)p].B);
        return o;
    };
    // In the digit-reversal scheme the phases run on the layout ordered like the input of the
    // direction (source order forward, output order for the transpose) and the last phase reorders
    // in place: an item is eight blocks that are neighbours in the direction's output order
    // (coordinates hi + lo + e there), each 16 contiguous coordinates of the layout, and slot
    // (e, h) = (sl & 7, sl >> 3) of these sixteen 16-byte slots receives one run of eight
    // neighbouring output coordinates (see reorder_slots below).
    auto reorder_off = [&](const Layout &L, int dir, int64_t hi, int64_t lo, int sl) {
        const int64_t co = hi + lo + (sl & 7);
        return phys_in(L, dir == 0 ? (int64_t)plan->h_perm[(size_t)co] : inv[(size_t)co]) + 8 * (sl >> 3);
    };
    // Stores of the reordering phase.  The four lanes q of a quarter-warp write the slots of the output runs
    // r = q + 4j in two neighbouring rows.  Starting from the identity, pairs of runs are swapped while that
    // lowers the number of shared-memory wavefronts (judged on the first item; the other items differ by a
    // constant offset).  Returns the wavefronts of one item's four store steps (4 = conflict-free) and, if
    // asked, the assignment.
    auto reorder_store_wavefronts = [&](const Layout &L, int dir, int64_t pitch_el, int *slot_of_out) {
        int slot_of[16];
        for (int r = 0; r < 16; ++r) slot_of[r] = r;
        int64_t off16[16];
        for (int sl = 0; sl < 16; ++sl) off16[sl] = reorder_off(L, dir, 0, 0, sl) / 8;
        auto slot_cost = [&]() {
            int total = 0;
            for (int j = 0; j < 4; ++j) {
                int cnt[8] = {0, 0, 0, 0, 0, 0, 0, 0}, worst = 0;
                for (int q = 0; q < 4; ++q)
                    for (int row = 0; row < 2; ++row) {
                        const int64_t sidx = off16[slot_of[q + 4 * j]] + row * (pitch_el / 8);
                        worst = std::max(worst, ++cnt[((sidx % 8) + 8) % 8]);
                    }
                total += worst;
            }
            return total;
        };
        int cur = slot_cost();
        for (bool improved = true; improved && cur > 4;) {
            improved = false;
            for (int a = 0; a < 16; ++a)
                for (int b = a + 1; b < 16; ++b) {
                    std::swap(slot_of[a], slot_of[b]);
                    const int c2 = slot_cost();
                    if (c2 < cur) { cur = c2; improved = true; }
                    else std::swap(slot_of[a], slot_of[b]);
                }
        }
        if (slot_of_out) for (int r = 0; r < 16; ++r) slot_of_out[r] = slot_of[r];
        return cur;
    };
    // scheme 0: plain (both tile copies follow the layout); 1: L is the source-ordered layout of
    // the forward reordering scheme; 2: L is the output-ordered layout of the transpose one
    auto layout_cost = [&](const Layout &L, int scheme) {
        const int64_t pc = pitch_of(L) / 8;
        double cost = 1e-7 * (double)L.extent;
        // strided phases: lanes q = 0..3 of two neighbouring rows
        const std::vector<int> &order = scheme == 1 ? order_src : order_nat;
        for (size_t k = 1; k < order.size(); ++k) {
            const int p = order[k];
            const int64_t step = L.lm[(size_t)p] * L.W[(size_t)p] + (L.lm[(size_t)p] == 4 ? L.gp[(size_t)p] : 0);
            std::vector<int64_t> slots;
            for (int q = 0; q < 4; ++q)
                for (int row = 0; row < 2; ++row) slots.push_back(q * step / 8 + row * pc);
            cost += 2.0 * worst_bank(slots);
        }
        // tile copies: eight neighbouring chunks of one row per quarter-warp
        auto map_cost = [&](auto loc) {
            double sum = 0;
            for (int64_t c0 = 0; c0 < d / 8; c0 += 8) {
                std::vector<int64_t> slots;
                for (int64_t c = c0; c < std::min(d / 8, c0 + 8); ++c) slots.push_back(loc(c) / 8);
                sum += worst_bank(slots);
            }
            return sum / (double)((d / 8 + 7) / 8);
        };
        cost += map_cost([&](int64_t c) { return phys_in(L, 8 * c); });
        if (scheme != 0) {
            // stride of the reordering phase in the order of the direction's output
            const int pr = scheme == 1 ? np - 1 : 0;
            const int64_t So = scheme == 1 ? phases[(size_t)pr].S : S_src[(size_t)pr], Bo = phases[(size_t)pr].B;
            cost += map_cost([&](int64_t c) {
                const int64_t o = 8 * c, span = So * Bo;                              // o = hi + lo + r*So
                return reorder_off(L, scheme - 1, o / span * span, o % So, (int)((o / So) % Bo));
            });
            // the reordering phase's own stores: 1.0 when conflict-free
            if (Bo == 16 && So % 8 == 0) cost += 0.25 * reorder_store_wavefronts(L, scheme - 1, pitch_of(L), nullptr);
        } else {
            cost += map_cost([&](int64_t c) { return phys_in(L, 8 * c); });
        }
        return cost;
    };
    auto search_layout = [&](const std::vector<int> &order, const std::vector<int64_t> &strides, int src_scheme, Layout &best) {
        // start: the smallest padding that makes every strided phase conflict-free on its own
        std::vector<Choice> ch((size_t)np, Choice{0, 0, 1});
        {
            int64_t W = 1;
            bool first = true;
            for (int p : order) {
                if (!first) {
                    W = (W + 7) / 8 * 8;
                    int pad = 0;
                    while (((W / 8 + pad) % 8) == 0 || ((W / 8 + pad) % 8) == 4) ++pad;
                    ch[(size_t)p] = Choice{pad, 0, ((W / 8 + pad) % 2 == 0) ? 1 : 2};
                    W += 8 * pad;
                }
                first = false;
                W *= phases[(size_t)p].B;
            }
        }
        if (!make_layout(order, strides, ch, best)) return false;
        double best_cost = layout_cost(best, src_scheme);
        if (order.size() == 3) {
            // two free phases: try every pair of choices
            const int p1 = order[1], p2 = order[2];
            for (int c1 = 0; c1 < 96; ++c1)
                for (int c2 = 0; c2 < 96; ++c2) {
                    std::vector<Choice> trial = ch;
                    trial[(size_t)p1] = Choice{c1 % 8, (c1 / 8) % 4, 1 << (c1 / 32)};
                    trial[(size_t)p2] = Choice{c2 % 8, (c2 / 8) % 4, 1 << (c2 / 32)};
                    Layout L;
                    if (!make_layout(order, strides, trial, L)) continue;
                    if ((size_t)kTileRows * pitch_of(L) * 2 > 200u * 1024u) continue;
                    // skip layouts whose strided phases are not conflict-free on their own
                    bool clean = true;
                    const int64_t pc = pitch_of(L) / 8;
                    for (int p : {p1, p2}) {
                        const int64_t step = L.lm[(size_t)p] * L.W[(size_t)p] + (L.lm[(size_t)p] == 4 ? L.gp[(size_t)p] : 0);
                        std::vector<int64_t> slots;
                        for (int q = 0; q < 4; ++q)
                            for (int row = 0; row < 2; ++row) slots.push_back(q * step / 8 + row * pc);
                        clean = clean && worst_bank(slots) == 1;
                    }
                    if (!clean) continue;
                    const double c = layout_cost(L, src_scheme);
                    if (c < best_cost - 1e-12) { best_cost = c; best = L; ch = trial; }
                }
            return true;
        }
        for (int sweep = 0; sweep < 3; ++sweep) {
            bool improved = false;
            for (size_t k = 1; k < order.size(); ++k) {
                const int p = order[k];
                for (int pad = 0; pad < 8; ++pad)
                    for (int gap = 0; gap < 4; ++gap)
                        for (int lm = 1; lm <= 4; lm *= 2) {
                            std::vector<Choice> trial = ch;
                            trial[(size_t)p] = Choice{pad, gap, lm};
                            Layout L;
                            if (!make_layout(order, strides, trial, L)) continue;
                            if ((size_t)kTileRows * pitch_of(L) * 2 > 200u * 1024u) continue;
                            const double c = layout_cost(L, src_scheme);
                            if (c < best_cost - 1e-12) { best_cost = c; best = L; ch = trial; improved = true; }
                        }
            }
            if (!improved) break;
        }
        return true;
    };
    Layout Lnat, Lsrc;
    if (!search_layout(order_nat, S_nat, digitrev ? 2 : 0, Lnat)) return HARP_ERR_UNSUPPORTED;
    if (digitrev) {
        if (!search_layout(order_src, S_src, 1, Lsrc)) return HARP_ERR_UNSUPPORTED;
    } else {
        Lsrc = Lnat;
    }
    // (the transpose direction of the digit-reversal scheme also uses the output-ordered layout)
    int64_t pitch = std::max(pitch_of(Lsrc), pitch_of(Lnat));
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
    auto phys_nat = [&](int64_t pos) { return phys_in(Lnat, pos); };
    // source coordinate j: its phase-p source-local index is (j / S_src[p]) % B_p, written with the
    // group's digits reversed; the layout only needs that index
    auto phys_src = [&](int64_t j) { return phys_in(Lsrc, j); };

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
    // Digit reversal: the last phase of either direction reorders the tile in place (see
    // reorder_off).  After it slot slot_of[r] of an item holds, for local index r in output order,
    // the eight blocks' values: a run of eight neighbouring output coordinates.
    // reorder_slots[dir][item][r] is that slot's offset and chunk_out[dir] the chunk map of the
    // copy to global memory that follows from it.
    std::vector<int32_t> reorder_slots[2], chunk_out[2];
    for (int dir = 0; dir < 2 && digitrev; ++dir) {
        const Layout &L = dir == 0 ? Lsrc : Lnat;
        const int pr = dir == 0 ? np - 1 : 0;
        const int64_t So = dir == 0 ? phases[(size_t)pr].S : S_src[(size_t)pr], span = So * phases[(size_t)pr].B;
        int slot_of[16];
        const int store_wavefronts = reorder_store_wavefronts(L, dir, pitch, slot_of);
        if (getenv("HARP_DEBUG_LAYOUT")) {
            fprintf(stderr, "dir %d: reorder-phase store wavefronts per item %d (ideal 4); W =", dir, store_wavefronts);
            for (int p = 0; p < np; ++p) fprintf(stderr, " (%lld,%lld,%d)", (long long)L.W[(size_t)p], (long long)L.gp[(size_t)p], L.lm[(size_t)p]);
            fprintf(stderr, " pitch %lld\n", (long long)pitch);
        }
        chunk_out[dir].assign((size_t)(d / 8), 0);
        for (int64_t hi = 0; hi < d; hi += span)
            for (int64_t lo = 0; lo < So; lo += 8)
                for (int r = 0; r < 16; ++r) {
                    const int32_t off = (int32_t)reorder_off(L, dir, hi, lo, slot_of[r]);
                    reorder_slots[dir].push_back(off);
                    chunk_out[dir][(size_t)((hi + lo + (int64_t)r * So) / 8)] = off;
                }
    }

    auto sign_v = [&](int64_t i) -> double {             // sign seen by coordinate i after the gather
        if (plan->h_signs.empty()) return 1.0;
        const int64_t src = identity ? i : plan->h_perm[(size_t)i];
        return (double)plan->h_signs[(size_t)src];
    };
    static const int joff1_16[4] = {0, 4, 8, 12}, joff2_16[4] = {0, 1, 8, 9}, joff4_16[4] = {0, 1, 2, 3};
    static const int joff1_8[4] = {0, 4, 0, 0}, joff2_8[4] = {0, 1, 0, 0};

    for (int dir = 0; dir < 2 && st == HARP_OK; ++dir) {  // 0 = forward, 1 = transpose
        FastParams &P = dir == 0 ? fp->fwd : fp->bwd;
        P.n_phases = np;
        P.d = (int32_t)d;
        P.pitch = (int32_t)pitch;
        // chunk maps: output order and source order in their layouts, and (digit reversal) where the
        // in-place reordering phase of this direction leaves the chunks of its output
        std::vector<int32_t> tables(chunk_nat);
        const int32_t off_nat = 0;
        const int32_t off_src = (int32_t)tables.size();
        tables.insert(tables.end(), chunk_src.begin(), chunk_src.end());
        const int32_t off_out = (int32_t)tables.size();
        if (digitrev) tables.insert(tables.end(), chunk_out[dir].begin(), chunk_out[dir].end());
        if (identity) {
            P.copy_in = off_nat;
            P.copy_out = off_nat;
        } else if (digitrev) {
            P.copy_in = dir == 0 ? off_src : off_nat;
            P.copy_out = off_out;
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
            else if (digitrev) mode = p == (dir == 0 ? np - 1 : 0) ? MODE_PO : MODE_SS;
            else mode = p == 0 ? (dir == 0 ? MODE_GS : MODE_CG) : MODE_SS;
            D.mode = mode;
            D.B = B;
            // Which layout do the strided accesses of this phase use, and with which slot geometry?
            // digit reversal: the forward direction works on the source-ordered layout, the transpose
            // on the output-ordered one
            const bool src_side = digitrev && dir == 0 && mode == MODE_SS;
            const Layout &L = src_side ? Lsrc : Lnat;
            const int lm = (mode == MODE_GS || mode == MODE_CG || mode == MODE_CC || mode == MODE_PO)
                               ? 1 : L.lm[(size_t)p];   // table-indexed slots use the plain map
            const int *jo = B == 16 ? (lm == 1 ? joff1_16 : lm == 2 ? joff2_16 : joff4_16) : (lm == 1 ? joff1_8 : joff2_8);
            if (mode == MODE_GS || mode == MODE_CG) {    // these index the item table by slot
                D.lane_step = lm;
                for (int j = 0; j < 4; ++j) D.j_off[j] = jo[j];
            } else {
                // the slots of one lane group never straddle a gap: q*lm steps with lm = 4, j steps otherwise
                D.lane_step = (int32_t)(lm * L.W[(size_t)p] + (lm == 4 ? L.gp[(size_t)p] : 0));
                for (int j = 0; j < 4; ++j) D.j_off[j] = (int32_t)L.off(p, jo[j]);
            }
            // local index seen by the strided / contiguous side of the operand, as a natural local index
            auto strided_nat = [&](int slot) {
                const int r = strided_slot(slot, B, lm);
                // the strided side counts in source order in the forward in-place phases and in the
                // reordering phase of the transpose, whose output is source-ordered
                const bool in_src_order = src_side || (mode == MODE_PO && dir == 1);
                return in_src_order ? nat_local_of_src_local(p, r) : r;
            };
            auto contig_nat = [&](int slot) {            // the forward reordering phase reads contiguous source blocks
                return (mode == MODE_PO && dir == 0) ? nat_local_of_src_local(p, slot) : slot;
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
            } else if (mode == MODE_PO) {
                // octets of blocks that are neighbours in the order of this direction's output; each
                // block is 16 contiguous coordinates of the layout the direction works on
                ints_per_item = 24;
                const int64_t So = dir == 0 ? hp.S : S_src[(size_t)p], span = So * B;
                size_t item_no = 0;
                for (int64_t hi = 0; hi < d; hi += span)
                    for (int64_t lo = 0; lo < So; lo += 8, ++item_no) {
                        for (int e = 0; e < 8; ++e) {
                            // natural coordinate of the block's local index 0
                            const int64_t nb = dir == 0 ? hi + lo + e : inv[(size_t)(hi + lo + e)];
                            items.push_back((int32_t)(dir == 0 ? phys_src(plan->h_perm[(size_t)nb]) : phys_nat(nb)));
                            block_base.push_back(nb);
                        }
                        for (int r = 0; r < 16; ++r) items.push_back(reorder_slots[dir][item_no * 16 + (size_t)r]);
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
                } else if (mode == MODE_PO) {
                    ok = ok && B == 16 && (dir == 0 ? hp.S : S_src[(size_t)p]) % 8 == 0;
                    for (size_t i = 0; i < items.size(); i += 24) {
                        for (int e = 0; e < 8; ++e) ok = ok && contig_ok(items[i + e]);
                        for (int r = 0; r < 16; ++r) ok = ok && items[i + 8 + r] >= 0 && items[i + 8 + r] % 8 == 0 && items[i + 8 + r] + 8 <= pitch;
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
            const bool in_strided = (mode == MODE_SS || mode == MODE_GS);
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
        // up to two phases whose items come eight blocks at a time keep their fragments in tensor memory
        // (2 x 32 items x 4 KB fill its 256 KB)
        P.tm_mask = 0;
        {
            int kept = 0;
            for (int k = 0; k < np && kept < 2; ++k) {
                const PhaseDesc &D = P.ph[k];
                const bool eight = D.B == 16 && (D.mode == MODE_SS || D.mode == MODE_GS || D.mode == MODE_PO || D.mode == MODE_CG);
                if (eight && D.n_items <= 2 * (kThreads / 32)) { P.tm_mask |= 1u << k; ++kept; }
            }
        }
        P.tables = upload(fp, tables, st);
        P.tables_len = (int32_t)tables.size();
        fp->smem_bytes = std::max(fp->smem_bytes, tile_bytes + tables.size() * sizeof(int32_t) + 16);
    }
    if (st == HARP_OK && fp->smem_bytes > 227u * 1024u) st = HARP_ERR_UNSUPPORTED;
    if (st == HARP_OK) {
        if (cudaFuncSetAttribute(harp_fast_kernel<kThreads, kModesGeneral>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(harp_fast_kernel<kThreads, kModesReorderOut>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            st = HARP_ERR_CUDA;
        fp->variant_fwd = digitrev ? 1 : 0;
        fp->variant_bwd = digitrev ? 1 : 0;
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

// Copies the per-section cycle counters to out[16] (zeros unless built with -DHARP_FAST_TIMING) and clears
// them if asked.
extern "C" int32_t harp_debug_fast_timing(int64_t *out, int32_t reset) {
    if (!out) return -1;
    if (cudaMemcpyFromSymbol(out, g_fast_timing, sizeof(long long) * 16) != cudaSuccess) return -1;
    if (reset) {
        const long long zero[16] = {0};
        if (cudaMemcpyToSymbol(g_fast_timing, zero, sizeof(zero)) != cudaSuccess) return -1;
    }
    return 0;
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
    __nv_bfloat16 *xb = static_cast<__nv_bfloat16 *>(x);
    FastParams P = transpose ? fp->bwd : fp->fwd;
    // fragments in tensor memory pay from the second tile of a CTA on; a CTA with one tile streams them
    if (n_tiles < 2 * (int64_t)grid) P.tm_mask = 0;
    // a quarter of a tile period, estimated from the measured 28 k cycles per tile of d = 4096 with
    // three phases (the gain is flat between half and the full value)
    const int stagger = n_tiles >= 4 * (int64_t)grid ? (int)(0.57 * (double)P.d * P.n_phases) : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = fp->smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t err;
    switch (transpose ? fp->variant_bwd : fp->variant_fwd) {
        case 1: err = cudaLaunchKernelEx(&cfg, harp_fast_kernel<kThreads, kModesReorderOut>, xb, n_rows, n_tiles, stagger, P); break;
        default: err = cudaLaunchKernelEx(&cfg, harp_fast_kernel<kThreads, kModesGeneral>, xb, n_rows, n_tiles, stagger, P); break;
    }
    g_harp_launches.fetch_add(1, std::memory_order_relaxed);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? HARP_OK : HARP_ERR_CUDA;
}
