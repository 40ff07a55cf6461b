// Internal declarations shared by the translation units of libharp.so.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "harp.h"

#define HARP_MAX_STAGES 24

// Stage geometry handed to kernels by value.
struct StageTable {
    int32_t m;
    int32_t b[HARP_MAX_STAGES];       // radix b_t
    int32_t s[HARP_MAX_STAGES];       // stride s_t = prod_{j<t} b_j
    int64_t off[HARP_MAX_STAGES];     // offset (in floats) of stage t in the block array
};

struct FastPlan;   // tensor-core path data, whole rows per CTA (harp_fast.cu)
struct SplitPlan;  // tensor-core path data, two passes over column groups (harp_split.cu)
struct TmPlan;    // tensor-memory path data: tcgen05.mma, rows as the M dimension (harp_tm.cu)
struct ColPlan;    // tensor-core path data for applying the plan down the columns of a matrix (harp_col.cu)

struct harp_plan {
    int64_t d = 0;
    int device = 0;
    StageTable st{};
    int64_t n_params = 0;
    float *d_blocks = nullptr;        // [sum_t d*b_t] fp32, stage after stage
    float *d_blocks_em = nullptr;     // the same stages element-major: entry k of block c of stage t at off[t] + k*D_t + c
    // the same map with runs of small-radix stages fused into dense blocks of size <= 4 (fewer
    // stages for the CUDA-core kernel); fused.m == 0 if nothing could be fused
    StageTable fused{};
    float *d_fused_blocks = nullptr;
    // block kernels of the stage table the block-owner kernels use (fused if present, else st),
    // element-major: entry k = i*b + j of block c of stage t at off[t] + k * (d / b_t) + c, so that
    // neighbouring threads (neighbouring blocks) read neighbouring words
    float *d_bo_blocks = nullptr;
    int32_t *d_perm = nullptr;        // nullptr = identity
    int8_t *d_signs = nullptr;        // nullptr = all +1
    // host copies (used to derive kernel-specific layouts)
    std::vector<int32_t> h_perm;
    std::vector<int8_t> h_signs;
    std::vector<float> h_blocks;
    FastPlan *fast = nullptr;
    SplitPlan *split = nullptr;
    ColPlan *col = nullptr;
    TmPlan *tm = nullptr;
    // test-only switch, read from the environment once, when the plan is built (HARP_NO_ROWVEC=1: the
    // CUDA-core kernels keep their tile row-major)
    bool opt_no_rowvec = false;
    // staging owned by harp_apply_host
    static constexpr int kStages = 4;
    void *stage_buf[kStages] = {nullptr, nullptr, nullptr, nullptr};
    int64_t stage_bytes = 0;
    cudaStream_t stage_stream[kStages] = {nullptr, nullptr, nullptr, nullptr};
};

extern std::atomic<int64_t> g_harp_launches;

// generic CUDA-core path (harp_generic.cu)
harp_status_t harp_generic_build(harp_plan *plan);   // fused stage table for the block-owner kernel
harp_status_t harp_generic_supported(const harp_plan *plan, harp_dtype_t dtype);
harp_status_t harp_generic_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                                 int transpose, cudaStream_t stream);

// tensor-core path (harp_fast.cu)
harp_status_t harp_fast_build(harp_plan *plan);     // HARP_OK or HARP_ERR_UNSUPPORTED (plan->fast stays null)
void harp_fast_destroy(harp_plan *plan);
harp_status_t harp_fast_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                              int transpose, cudaStream_t stream);

// tensor-core path for wide rows (harp_split.cu)
harp_status_t harp_split_build(harp_plan *plan);
void harp_split_destroy(harp_plan *plan);
harp_status_t harp_split_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                               int transpose, cudaStream_t stream);

// tensor-memory path (harp_tm.cu)
harp_status_t harp_tm_build(harp_plan *plan);
void harp_tm_destroy(harp_plan *plan);
harp_status_t harp_tm_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                            int transpose, cudaStream_t stream);
int32_t harp_tm_error_word(const harp_plan *plan);
// the stages below stride 256 alone (lower pass of the two-pass paths); 0 stages = not available
int harp_tm_slab_stages(const harp_plan *plan);
harp_status_t harp_tm_slab_apply(const harp_plan *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                                 int transpose, cudaStream_t stream);

// column-side apply for two-sided processing (harp_col.cu): plan applied down the columns of a
// dim(plan) x n_cols row-major matrix with leading dimension ld
harp_status_t harp_col_build(harp_plan *plan);
void harp_col_destroy(harp_plan *plan);
harp_status_t harp_col_apply(const harp_plan *plan, void *W, int64_t n_cols, int64_t ld, harp_dtype_t dtype,
                             cudaStream_t stream);

// out-of-place matrix transpose, rows x cols -> cols x rows (harp_two_sided.cu)
harp_status_t harp_transpose_matrix(const void *src, void *dst, int64_t rows, int64_t cols,
                                    harp_dtype_t dtype, cudaStream_t stream);

static inline size_t harp_dtype_size(harp_dtype_t t) { return t == HARP_F32 ? 4 : 2; }
