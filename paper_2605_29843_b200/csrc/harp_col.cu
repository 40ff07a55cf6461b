// Column-side tensor-core kernels for two-sided processing (bf16, identity permutation).
//
// W~ = Q_out^T W Q_in needs the processor Q_out applied down every column of the row-major
// matrix W.  Here the "batch" (the vectors that share block kernels) is the set of columns,
// which is the contiguous direction of memory, and a coordinate of the transform is a row
// index.  A CTA takes a tile of [positions x NC columns], keeps it in shared memory as
// [position][NC] and treats 16 neighbouring columns as the M dimension of mma.sync: the
// operand of a block (B positions x 16 columns) is read with ldmatrix.trans from B rows of
// 16 bytes and written back with stmatrix.trans -- no transposition of W, no gather, no
// byte permutes.  Rows of the tile are padded (odd row pitch and odd position strides, in
// 16-byte units) so that the eight row addresses of an ldmatrix hit eight bank groups.
//
// As in harp_split.cu the coordinate range d_out = S_mid * U is covered in two passes (lower
// stages inside slabs of S_mid positions, upper stages across slabs), each CTA keeping the
// fragments of its position group resident while it walks over column tiles.
#include <algorithm>
#include <cstdlib>
#include <new>

#include "harp_internal.h"
#include "harp_mma.cuh"
#include "harp_fuse.h"

using namespace harp_fuse;

namespace {

constexpr int kColThreads = 256;
constexpr int kColWarps = kColThreads / 32;
constexpr int kMaxColPhases = 6;

struct ColPhase {
    int32_t B, B_real;         // operand width (8 or 16), real block size
    int32_t wr;                // distance, in tile rows, between consecutive slots of a block
    int32_t items_off, n_items;
    int32_t bfrag_off;         // word offset inside the position group's fragment block
};

struct ColPass {
    int32_t n_phases, n_cg, n_pos, n_rows_phys, rowbytes, NC;
    int32_t cg_stride;         // positions between consecutive position groups
    int32_t map_off;           // tables[map_off + 2i] = position offset inside the group, [+1] = tile row
    const int32_t *tables;
    int32_t tables_len;
    const uint32_t *bfrag;
    int32_t bfrag_words;
    ColPhase ph[kMaxColPhases];
};

__device__ __forceinline__ void ldmatrix_x4_t(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2_t(uint32_t (&r)[2], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void stmatrix_x4_t(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
__device__ __forceinline__ void stmatrix_x2_t(uint32_t addr, uint32_t r0, uint32_t r1) {
    asm volatile("stmatrix.sync.aligned.m8n8.x2.trans.shared.b16 [%0], {%1,%2};" ::"r"(addr), "r"(r0), "r"(r1) : "memory");
}
__device__ __forceinline__ uint32_t lds32c(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// W: n_pos_total x ld (row-major); columns [0, n_cols) are processed, n_cols a multiple of 8.
__global__ void __launch_bounds__(kColThreads, 2)
harp_col_kernel(__nv_bfloat16 *__restrict__ W, int64_t ld, int64_t n_cols, ColPass P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t sbase = smem_u32(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rowbytes = P.rowbytes, NC = P.NC, MT = NC >> 4;
    const size_t tile_bytes = (size_t)P.n_rows_phys * rowbytes;          // includes one scratch row for padded slots
    int32_t *tab_s = reinterpret_cast<int32_t *>(smem_raw + tile_bytes);
    const uint32_t bf_s = sbase + (uint32_t)((tile_bytes + (size_t)P.tables_len * 4 + 15) / 16 * 16);
    const int scratch_row = P.n_rows_phys - 1;

    const int cg = blockIdx.x % P.n_cg, part = blockIdx.x / P.n_cg, n_parts = gridDim.x / P.n_cg;
    __nv_bfloat16 *Wg = W + (int64_t)cg * P.cg_stride * ld;
    {
        const uint32_t *src = P.bfrag + (size_t)cg * P.bfrag_words;
        for (int i = threadIdx.x * 4; i < P.bfrag_words; i += kColThreads * 4) cp_async16(bf_s + 4u * i, src + i);
    }
    for (int i = threadIdx.x; i < P.tables_len; i += kColThreads) tab_s[i] = __ldg(P.tables + i);
    __syncthreads();
    const int32_t *rmap = tab_s + P.map_off;

    // copy geometry: cpr threads share a tile row (NC/8 chunks of 16 bytes)
    const int cpr = NC >> 3, rows_per_step = kColThreads / cpr;
    const int cp_r = threadIdx.x / cpr, cp_c = threadIdx.x - cp_r * cpr;

    const int64_t n_tiles = (n_cols + NC - 1) / NC;
    for (int64_t tile = part; tile < n_tiles; tile += n_parts) {
        const int64_t c0 = tile * NC;
        const bool col_ok = c0 + 8 * cp_c < n_cols;                       // chunks past the last column are skipped
        // columns past the end are filled from the last valid chunk (finite values), never stored
        const int64_t csrc = col_ok ? c0 + 8 * cp_c : (n_cols - 8);
        for (int i = cp_r; i < P.n_pos; i += rows_per_step)
            cp_async16(sbase + (uint32_t)(rmap[2 * i + 1] * rowbytes + 16 * cp_c), Wg + (int64_t)rmap[2 * i] * ld + csrc);
        cp_async_wait_all();
        __syncthreads();

        for (int p = 0; p < P.n_phases; ++p) {
            const ColPhase &ph = P.ph[p];
            // a warp takes a block through all 16-column groups of the tile: the block's fragment and
            // addresses are set up once
            if (ph.B == 16) {
                const int k = (lane & 7) + 8 * (lane >> 4), mch = (lane >> 3) & 1;
                const bool real = k < ph.B_real;
                const uint32_t lane_ld = sbase + (uint32_t)((real ? k * ph.wr : 0) * rowbytes + 16 * mch);
                const uint32_t lane_scr = sbase + (uint32_t)(scratch_row * rowbytes + 16 * mch);
                for (int it = warp; it < ph.n_items; it += kColWarps) {
                    const uint32_t row_off = (uint32_t)(tab_s[ph.items_off + it] * rowbytes);
                    const uint4 bf = lds128(bf_s + 4u * (uint32_t)(ph.bfrag_off + (it * 32 + lane) * 4));
                    uint32_t ld_addr = lane_ld + row_off, st_addr = real ? ld_addr : lane_scr;
#pragma unroll 2
                    for (int mt = 0; mt < MT; ++mt, ld_addr += 32, st_addr += 32) {
                        uint32_t a[4];
                        ldmatrix_x4_t(a, ld_addr);
                        float c0f[4], c1f[4];
                        mma_k16(c0f, a, bf.x, bf.y);
                        mma_k16(c1f, a, bf.z, bf.w);
                        stmatrix_x4_t(st_addr, pack_bf16(c0f[0], c0f[1]), pack_bf16(c0f[2], c0f[3]), pack_bf16(c1f[0], c1f[1]),
                                      pack_bf16(c1f[2], c1f[3]));
                    }
                }
            } else if ((MT & 1) == 0) {
                // 8-wide blocks: two 16-column groups per ldmatrix.x4 / stmatrix.x4 (lanes 16-31 address the second
                // group), the block's fragment used twice: half the shared-memory instructions
                const int k = lane & 7, mch = lane >> 3;
                const bool real = k < ph.B_real;
                const uint32_t lane_ld = sbase + (uint32_t)((real ? k * ph.wr : 0) * rowbytes + 16 * mch);
                const uint32_t lane_scr = sbase + (uint32_t)(scratch_row * rowbytes + 16 * mch);
                for (int it = warp; it < ph.n_items; it += kColWarps) {
                    const uint32_t row_off = (uint32_t)(tab_s[ph.items_off + it] * rowbytes);
                    const uint32_t bf = lds32c(bf_s + 4u * (uint32_t)(ph.bfrag_off + it * 32 + lane));
                    uint32_t ld_addr = lane_ld + row_off, st_addr = real ? ld_addr : lane_scr;
#pragma unroll 2
                    for (int mt = 0; mt < MT; mt += 2, ld_addr += 64, st_addr += 64) {
                        uint32_t a[4];
                        ldmatrix_x4_t(a, ld_addr);
                        const uint32_t a_lo[2] = {a[0], a[1]}, a_hi[2] = {a[2], a[3]};
                        float c0f[4], c1f[4];
                        mma_k8(c0f, a_lo, bf);
                        mma_k8(c1f, a_hi, bf);
                        stmatrix_x4_t(st_addr, pack_bf16(c0f[0], c0f[1]), pack_bf16(c0f[2], c0f[3]), pack_bf16(c1f[0], c1f[1]),
                                      pack_bf16(c1f[2], c1f[3]));
                    }
                }
            } else {
                const int k = lane & 7, mch = (lane >> 3) & 1;
                const bool real = k < ph.B_real;
                const uint32_t lane_ld = sbase + (uint32_t)((real ? k * ph.wr : 0) * rowbytes + 16 * mch);
                const uint32_t lane_scr = sbase + (uint32_t)(scratch_row * rowbytes + 16 * mch);
                for (int it = warp; it < ph.n_items; it += kColWarps) {
                    const uint32_t row_off = (uint32_t)(tab_s[ph.items_off + it] * rowbytes);
                    const uint32_t bf = lds32c(bf_s + 4u * (uint32_t)(ph.bfrag_off + it * 32 + lane));
                    uint32_t ld_addr = lane_ld + row_off, st_addr = real ? ld_addr : lane_scr;
#pragma unroll 2
                    for (int mt = 0; mt < MT; ++mt, ld_addr += 32, st_addr += 32) {
                        uint32_t a[2];
                        ldmatrix_x2_t(a, ld_addr);
                        float c0f[4];
                        mma_k8(c0f, a, bf);
                        stmatrix_x2_t(st_addr, pack_bf16(c0f[0], c0f[1]), pack_bf16(c0f[2], c0f[3]));
                    }
                }
            }
            __syncthreads();
        }

        if (col_ok)
            for (int i = cp_r; i < P.n_pos; i += rows_per_step)
                stg128(Wg + (int64_t)rmap[2 * i] * ld + csrc, lds128(sbase + (uint32_t)(rmap[2 * i + 1] * rowbytes + 16 * cp_c)));
        __syncthreads();
    }
    cp_async_wait_all();
}

}  // namespace

struct ColPlan {
    ColPass pass[2];
    size_t smem[2] = {0, 0};
    int n_pass = 0;
    std::vector<void *> dev_allocs;
    int sms = 148;
};

namespace {

struct CPhase { int t0, t1, B, B_real; int64_t S; };

template <typename T>
T *upload_c(ColPlan *cp, const std::vector<T> &v, harp_status_t &st) {
    if (st != HARP_OK) return nullptr;
    void *p = nullptr;
    if (cudaMalloc(&p, std::max<size_t>(16, v.size() * sizeof(T))) != cudaSuccess) { st = HARP_ERR_ALLOC; return nullptr; }
    cp->dev_allocs.push_back(p);
    if (!v.empty() && cudaMemcpy(p, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) st = HARP_ERR_CUDA;
    return static_cast<T *>(p);
}

// lower = true : position group = slab u (positions u*S_mid + t, t < S_mid), phases = lower ones
// lower = false: position group = Lr neighbouring t in every slab (positions t0 + t' + S_mid*u), phases = upper ones
harp_status_t build_col_pass(const harp_plan *plan, ColPlan *cp, int which, const std::vector<CPhase> &phs, bool lower,
                             int64_t S_mid, int64_t U, int Lr) {
    const int np = (int)phs.size();
    if (np == 0 || np > kMaxColPhases) return HARP_ERR_UNSUPPORTED;
    // tile-row stride of every phase's local index: odd, so eight consecutive slots fall into eight bank groups
    std::vector<int64_t> wr((size_t)np);
    int64_t ext = 1;
    for (int p = 0; p < np; ++p) {
        if (ext % 2 == 0) ++ext;
        wr[(size_t)p] = ext;
        ext *= phs[(size_t)p].B_real;
    }
    const int64_t group_rows = ext;                           // rows of one l (pass 2) or of the slab (pass 1)
    const int64_t n_rows_phys = (lower ? group_rows : group_rows * Lr) + 1;      // + scratch row
    const int n_pos = lower ? (int)S_mid : (int)(U * Lr);
    auto tile_row = [&](int64_t tl, int64_t u) {              // tl: position inside the slab (pass 1) or l' (pass 2)
        int64_t o = 0;
        if (lower) {
            for (int p = 0; p < np; ++p) o += ((tl / phs[(size_t)p].S) % phs[(size_t)p].B_real) * wr[(size_t)p];
        } else {
            o = tl * group_rows;
            for (int p = 0; p < np; ++p) o += ((u / (phs[(size_t)p].S / S_mid)) % phs[(size_t)p].B_real) * wr[(size_t)p];
        }
        return o;
    };
    // fragments and tables
    std::vector<int32_t> tab;
    ColPass &P = cp->pass[which];
    P.n_phases = np;
    P.n_cg = lower ? (int32_t)U : (int32_t)(S_mid / Lr);
    P.n_pos = n_pos;
    P.n_rows_phys = (int32_t)n_rows_phys;
    P.cg_stride = lower ? (int32_t)S_mid : Lr;
    P.map_off = 0;
    for (int i = 0; i < n_pos; ++i) {
        if (lower) { tab.push_back(i); tab.push_back((int32_t)tile_row(i, 0)); }
        else {
            const int64_t u = i / Lr, tl = i % Lr;
            tab.push_back((int32_t)(u * S_mid + tl));
            tab.push_back((int32_t)tile_row(tl, u));
        }
    }
    std::vector<std::vector<int64_t>> block_rel((size_t)np);
    int32_t words = 0;
    std::vector<int32_t> frag_off((size_t)np);
    for (int p = 0; p < np; ++p) {
        const CPhase &gp = phs[(size_t)p];
        ColPhase &D = P.ph[p];
        D.B = gp.B; D.B_real = gp.B_real; D.wr = (int32_t)wr[(size_t)p];
        D.items_off = (int32_t)tab.size();
        if (lower) {
            const int64_t span = gp.S * gp.B_real;
            for (int64_t hi = 0; hi < S_mid; hi += span)
                for (int64_t lo = 0; lo < gp.S; ++lo) {
                    tab.push_back((int32_t)tile_row(hi + lo, 0));
                    block_rel[(size_t)p].push_back(hi + lo);
                }
        } else {
            const int64_t su = gp.S / S_mid, span = su * gp.B_real;
            for (int64_t tl = 0; tl < Lr; ++tl)
                for (int64_t hi = 0; hi < U; hi += span)
                    for (int64_t lo = 0; lo < su; ++lo) {
                        tab.push_back((int32_t)tile_row(tl, hi + lo));
                        block_rel[(size_t)p].push_back((hi + lo) * S_mid + tl);
                    }
        }
        D.n_items = (int32_t)block_rel[(size_t)p].size();
        D.bfrag_off = words;
        frag_off[(size_t)p] = words;
        words += D.n_items * 32 * (gp.B == 16 ? 4 : 1);
        // every slot row must lie inside the tile
        for (size_t i = 0; i < block_rel[(size_t)p].size(); ++i) {
            const int64_t b = tab[(size_t)D.items_off + i];
            if (b < 0 || b + (int64_t)(gp.B_real - 1) * D.wr >= n_rows_phys - 1) return HARP_ERR_UNSUPPORTED;
        }
    }
    words = (words + 3) / 4 * 4;
    P.bfrag_words = words;
    // column tile: 64 columns if the tile, tables and fragments fit about 100 KB, else 32
    int NC = 64;
    auto need = [&](int nc) { return ((size_t)n_rows_phys * (size_t)(nc * 2 + 16) + tab.size() * 4 + 15) / 16 * 16 + (size_t)words * 4; };
    if (need(NC) > 100u * 1024u) NC = 32;
    if (need(NC) > 110u * 1024u) return HARP_ERR_UNSUPPORTED;
    P.NC = NC;
    P.rowbytes = NC * 2 + 16;
    cp->smem[which] = need(NC);
    harp_status_t st = HARP_OK;
    P.tables_len = (int32_t)tab.size();
    P.tables = upload_c(cp, tab, st);
    std::vector<uint32_t> frag((size_t)P.n_cg * words, 0u);
    std::vector<double> F;
    for (int cgi = 0; cgi < P.n_cg; ++cgi) {
        const int64_t cg_base = (int64_t)cgi * P.cg_stride;
        for (int p = 0; p < np; ++p) {
            const CPhase &gp = phs[(size_t)p];
            const int B = gp.B, Br = gp.B_real;
            HostPhase hp{gp.t0, gp.t1, Br, gp.S, 0, 1};
            const int wpl = B == 16 ? 4 : 1;
            for (size_t bi = 0; bi < block_rel[(size_t)p].size(); ++bi) {
                const int64_t base = cg_base + block_rel[(size_t)p][bi];
                fused_block(plan, hp, base, F);
                auto G = [&](int rin, int rout) -> double {
                    if (rin >= Br || rout >= Br) return 0.0;
                    double v = F[(size_t)rin * Br + rout];
                    if (gp.t0 == 0 && !plan->h_signs.empty()) v *= (double)plan->h_signs[(size_t)(base + (int64_t)rin * gp.S)];
                    return v;
                };
                uint32_t *dst0 = frag.data() + (size_t)cgi * words + frag_off[(size_t)p] + bi * 32 * wpl;
                for (int lane = 0; lane < 32; ++lane) {
                    const int gg = lane >> 2, qq = lane & 3;
                    uint32_t *dst = dst0 + lane * wpl;
                    if (B == 16) {
                        for (int nt = 0; nt < 2; ++nt) {
                            const int n = 8 * nt + gg;
                            dst[2 * nt] = f2bf(G(2 * qq, n)) | ((uint32_t)f2bf(G(2 * qq + 1, n)) << 16);
                            dst[2 * nt + 1] = f2bf(G(2 * qq + 8, n)) | ((uint32_t)f2bf(G(2 * qq + 9, n)) << 16);
                        }
                    } else {
                        dst[0] = f2bf(G(2 * qq, gg)) | ((uint32_t)f2bf(G(2 * qq + 1, gg)) << 16);
                    }
                }
            }
        }
    }
    P.bfrag = upload_c(cp, frag, st);
    return st;
}

}  // namespace

harp_status_t harp_col_build(harp_plan *plan) {
    const int64_t d = plan->d;
    const int m = plan->st.m;
    if (!plan->h_perm.empty()) return HARP_ERR_UNSUPPORTED;
    std::vector<CPhase> phs;
    for (int t = 0; t < m;) {
        int64_t prod = 1;
        int t1 = t;
        while (t1 < m && prod * plan->st.b[t1] <= 16) prod *= plan->st.b[t1++];
        if (t1 == t) return HARP_ERR_UNSUPPORTED;
        phs.push_back({t, t1, prod <= 8 ? 8 : 16, (int)prod, plan->st.s[t]});
        t = t1;
    }
    int k = 0;
    int64_t S_mid = 1;
    while (k < (int)phs.size() && S_mid * phs[(size_t)k].B_real <= 512) S_mid *= phs[(size_t)k++].B_real;
    if (k == 0) return HARP_ERR_UNSUPPORTED;
    const int64_t U = d / S_mid;
    std::vector<CPhase> lower(phs.begin(), phs.begin() + k), upper(phs.begin() + k, phs.end());
    int Lr = 16;
    while (Lr > 1 && S_mid % Lr != 0) Lr /= 2;
    ColPlan *cp = new (std::nothrow) ColPlan();
    if (!cp) return HARP_ERR_ALLOC;
    harp_status_t st = build_col_pass(plan, cp, 0, lower, true, S_mid, U, 1);
    cp->n_pass = 1;
    if (st == HARP_OK && !upper.empty()) {
        // as many neighbouring positions per group as shared memory allows
        st = HARP_ERR_UNSUPPORTED;
        for (; Lr >= 2 && st == HARP_ERR_UNSUPPORTED; Lr /= 2) st = build_col_pass(plan, cp, 1, upper, false, S_mid, U, Lr);
        cp->n_pass = 2;
    }
    if (st == HARP_OK &&
        (cudaFuncSetAttribute(harp_col_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024) != cudaSuccess ||
         cudaFuncSetAttribute(harp_col_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100) != cudaSuccess))
        st = HARP_ERR_CUDA;
    if (st == HARP_OK) {
        int dev = 0, sms = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms > 0) cp->sms = sms;
    }
    plan->col = cp;
    if (st != HARP_OK) {
        cudaGetLastError();
        harp_col_destroy(plan);
        return st;
    }
    return HARP_OK;
}

void harp_col_destroy(harp_plan *plan) {
    if (!plan->col) return;
    for (void *p : plan->col->dev_allocs) cudaFree(p);
    delete plan->col;
    plan->col = nullptr;
}

// Apply plan (forward) down the columns of W (dim(plan) x n_cols, row-major, leading dimension ld).
harp_status_t harp_col_apply(const harp_plan *plan, void *W, int64_t n_cols, int64_t ld, harp_dtype_t dtype, cudaStream_t stream) {
    const ColPlan *cp = plan->col;
    if (!cp || dtype != HARP_BF16) return HARP_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(W) & 15u) != 0 || n_cols % 8 != 0 || ld % 8 != 0 || n_cols < 8) return HARP_ERR_UNSUPPORTED;
    for (int s = 0; s < cp->n_pass; ++s) {
        const ColPass &P = cp->pass[s];
        const int64_t n_tiles = (n_cols + P.NC - 1) / P.NC;
        // up to three CTAs per SM (70 registers per thread): the pass with the small tile gains from the third
        // (two-sided product of the 8192 x 28672 matrix 1.14 -> 1.10 ms); 32-column tiles were measured slower
        const int per_sm = std::max<int>(1, std::min<int>(3, (int)((220 * 1024) / (cp->smem[s] + 1024))));
        int64_t parts = std::max<int64_t>(1, ((int64_t)cp->sms * per_sm) / P.n_cg);
        parts = std::min(parts, n_tiles);
        harp_col_kernel<<<(unsigned)(parts * P.n_cg), kColThreads, cp->smem[s], stream>>>(static_cast<__nv_bfloat16 *>(W), ld, n_cols, P);
        g_harp_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return HARP_ERR_CUDA;
    }
    return HARP_OK;
}
