// C ABI of libharp.so: plan construction and validation, dispatch, two-sided
// processing, the host-buffer pipeline.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>

#include "harp_internal.h"

std::atomic<int64_t> g_harp_launches{0};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" const char *harp_status_string(harp_status_t s) {
    switch (s) {
        case HARP_OK: return "ok";
        case HARP_ERR_NULL: return "null pointer";
        case HARP_ERR_BAD_DIM: return "bad dimension";
        case HARP_ERR_BAD_SCHEDULE: return "bad radix schedule";
        case HARP_ERR_BAD_PERM: return "perm is not a bijection";
        case HARP_ERR_BAD_SIGNS: return "signs must be +1 or -1";
        case HARP_ERR_BAD_DTYPE: return "bad dtype";
        case HARP_ERR_DIM_MISMATCH: return "dimension mismatch";
        case HARP_ERR_UNSUPPORTED: return "unsupported by this build";
        case HARP_ERR_ALLOC: return "allocation failed";
        case HARP_ERR_CUDA: return "CUDA error";
        case HARP_ERR_TOO_LARGE: return "exceeds a fixed capacity";
    }
    return "unknown status";
}

extern "C" int32_t harp_plan_error_word(const harp_plan_t *plan) { return plan ? harp_tm_error_word(plan) : -1; }

extern "C" int64_t harp_launch_count(void) { return g_harp_launches.load(std::memory_order_relaxed); }

extern "C" harp_status_t harp_plan_create(harp_plan_t **out, int64_t d, int32_t n_stages,
                                          const int32_t *radices, const int32_t *perm,
                                          const int8_t *signs, const float *const *blocks) {
    // ---- validation: before any CUDA call ----
    if (!out || !radices || !blocks) return HARP_ERR_NULL;
    if (d < 2 || d > (1 << 20)) return HARP_ERR_BAD_DIM;
    if (n_stages < 1 || n_stages > HARP_MAX_STAGES) return HARP_ERR_BAD_SCHEDULE;
    int64_t prod = 1;
    for (int t = 0; t < n_stages; ++t) {
        if (radices[t] < 2 || radices[t] > d) return HARP_ERR_BAD_SCHEDULE;
        prod *= radices[t];
        if (prod > d) return HARP_ERR_BAD_SCHEDULE;
    }
    if (prod != d) return HARP_ERR_BAD_SCHEDULE;
    for (int t = 0; t < n_stages; ++t)
        if (!blocks[t]) return HARP_ERR_NULL;
    if (perm) {
        std::vector<uint8_t> seen((size_t)d, 0);
        for (int64_t i = 0; i < d; ++i) {
            const int32_t p = perm[i];
            if (p < 0 || p >= d || seen[(size_t)p]) return HARP_ERR_BAD_PERM;
            seen[(size_t)p] = 1;
        }
    }
    if (signs)
        for (int64_t i = 0; i < d; ++i)
            if (signs[i] != 1 && signs[i] != -1) return HARP_ERR_BAD_SIGNS;

    harp_plan *p = new (std::nothrow) harp_plan();
    if (!p) return HARP_ERR_ALLOC;
    p->d = d;
    p->opt_no_rowvec = getenv("HARP_NO_ROWVEC") != nullptr;
    p->st.m = n_stages;
    int64_t s = 1, off = 0;
    for (int t = 0; t < n_stages; ++t) {
        p->st.b[t] = radices[t];
        p->st.s[t] = (int32_t)s;
        p->st.off[t] = off;
        s *= radices[t];
        off += d * radices[t];
    }
    p->n_params = off;
    try {
        p->h_blocks.resize((size_t)off);
        for (int t = 0; t < n_stages; ++t)
            std::memcpy(p->h_blocks.data() + p->st.off[t], blocks[t], sizeof(float) * (size_t)d * radices[t]);
        bool identity = true;
        if (perm)
            for (int64_t i = 0; i < d && identity; ++i) identity = perm[i] == (int32_t)i;
        if (perm && !identity) p->h_perm.assign(perm, perm + d);
        bool all_plus = true;
        if (signs)
            for (int64_t i = 0; i < d && all_plus; ++i) all_plus = signs[i] == 1;
        if (signs && !all_plus) p->h_signs.assign(signs, signs + d);
    } catch (const std::bad_alloc &) {
        delete p;
        return HARP_ERR_ALLOC;
    }

    // ---- device copies ----
    if (cudaGetDevice(&p->device) != cudaSuccess) { delete p; return HARP_ERR_CUDA; }
    harp_status_t st = HARP_OK;
    if (cudaMalloc(&p->d_blocks, sizeof(float) * (size_t)off) != cudaSuccess) st = HARP_ERR_ALLOC;
    if (st == HARP_OK && !p->h_perm.empty() && cudaMalloc(&p->d_perm, sizeof(int32_t) * (size_t)d) != cudaSuccess)
        st = HARP_ERR_ALLOC;
    if (st == HARP_OK && !p->h_signs.empty() && cudaMalloc(&p->d_signs, (size_t)d) != cudaSuccess)
        st = HARP_ERR_ALLOC;
    if (st == HARP_OK &&
        cudaMemcpy(p->d_blocks, p->h_blocks.data(), sizeof(float) * (size_t)off, cudaMemcpyHostToDevice) != cudaSuccess)
        st = HARP_ERR_CUDA;
    if (st == HARP_OK) {         // element-major copy (neighbouring blocks' entries side by side), for the gradient kernels
        std::vector<float> em;
        try {
            em.resize((size_t)off);
        } catch (const std::bad_alloc &) {
            st = HARP_ERR_ALLOC;
        }
        for (int t = 0; st == HARP_OK && t < p->st.m; ++t) {
            const int64_t bb = (int64_t)p->st.b[t] * p->st.b[t], nblk = d / p->st.b[t];
            const float *src = p->h_blocks.data() + p->st.off[t];
            float *dst = em.data() + p->st.off[t];
            for (int64_t c = 0; c < nblk; ++c)
                for (int64_t k = 0; k < bb; ++k) dst[k * nblk + c] = src[c * bb + k];
        }
        if (st == HARP_OK && cudaMalloc(&p->d_blocks_em, sizeof(float) * (size_t)off) != cudaSuccess) st = HARP_ERR_ALLOC;
        if (st == HARP_OK &&
            cudaMemcpy(p->d_blocks_em, em.data(), sizeof(float) * (size_t)off, cudaMemcpyHostToDevice) != cudaSuccess)
            st = HARP_ERR_CUDA;
    }
    if (st == HARP_OK && p->d_perm &&
        cudaMemcpy(p->d_perm, p->h_perm.data(), sizeof(int32_t) * (size_t)d, cudaMemcpyHostToDevice) != cudaSuccess)
        st = HARP_ERR_CUDA;
    if (st == HARP_OK && p->d_signs &&
        cudaMemcpy(p->d_signs, p->h_signs.data(), (size_t)d, cudaMemcpyHostToDevice) != cudaSuccess)
        st = HARP_ERR_CUDA;
    if (st == HARP_OK) st = harp_generic_build(p);
    if (st == HARP_OK) {
        harp_status_t fs = harp_fast_build(p);
        if (fs != HARP_OK && fs != HARP_ERR_UNSUPPORTED) st = fs;
    }
    if (st == HARP_OK) {
        harp_status_t fs = harp_split_build(p);
        if (fs != HARP_OK && fs != HARP_ERR_UNSUPPORTED) st = fs;
    }
    if (st == HARP_OK) {
        harp_status_t fs = harp_tm_build(p);
        if (fs != HARP_OK && fs != HARP_ERR_UNSUPPORTED) st = fs;
    }
    if (st == HARP_OK) {
        harp_status_t fs = harp_col_build(p);
        if (fs != HARP_OK && fs != HARP_ERR_UNSUPPORTED) st = fs;
    }
    if (st != HARP_OK) {
        cudaGetLastError();
        harp_plan_destroy(p);
        return st;
    }
    *out = p;
    return HARP_OK;
}

extern "C" void harp_plan_destroy(harp_plan_t *p) {
    if (!p) return;
    {
        DeviceGuard g(p->device);
        harp_fast_destroy(p);
        harp_split_destroy(p);
        harp_col_destroy(p);
        harp_tm_destroy(p);
        for (int i = 0; i < harp_plan::kStages; ++i) {
            if (p->stage_stream[i]) { cudaStreamSynchronize(p->stage_stream[i]); cudaStreamDestroy(p->stage_stream[i]); }
            if (p->stage_buf[i]) cudaFree(p->stage_buf[i]);
        }
        if (p->d_blocks) cudaFree(p->d_blocks);
        if (p->d_blocks_em) cudaFree(p->d_blocks_em);
        if (p->d_fused_blocks) cudaFree(p->d_fused_blocks);
        if (p->d_bo_blocks) cudaFree(p->d_bo_blocks);
        if (p->d_perm) cudaFree(p->d_perm);
        if (p->d_signs) cudaFree(p->d_signs);
    }
    delete p;
}

extern "C" int64_t harp_plan_dim(const harp_plan_t *p) { return p ? p->d : -1; }

extern "C" harp_status_t harp_apply_ex(const harp_plan_t *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                                       int transpose, harp_kernel_t kernel, void *stream) {
    if (!plan) return HARP_ERR_NULL;
    if (dtype != HARP_F32 && dtype != HARP_BF16) return HARP_ERR_BAD_DTYPE;
    if (n_rows < 0) return HARP_ERR_BAD_DIM;
    if (kernel != HARP_KERNEL_AUTO && kernel != HARP_KERNEL_GENERIC && kernel != HARP_KERNEL_FAST &&
        kernel != HARP_KERNEL_SPLIT && kernel != HARP_KERNEL_TMEM)
        return HARP_ERR_UNSUPPORTED;
    if (n_rows == 0) return HARP_OK;
    if (!x) return HARP_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(x) & (harp_dtype_size(dtype) - 1)) != 0) return HARP_ERR_BAD_DIM;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    transpose = transpose ? 1 : 0;
    if (kernel == HARP_KERNEL_GENERIC) return harp_generic_apply(plan, x, n_rows, dtype, transpose, s);
    if (kernel == HARP_KERNEL_FAST) return harp_fast_apply(plan, x, n_rows, dtype, transpose, s);
    if (kernel == HARP_KERNEL_SPLIT) return harp_split_apply(plan, x, n_rows, dtype, transpose, s);
    if (kernel == HARP_KERNEL_TMEM) return harp_tm_apply(plan, x, n_rows, dtype, transpose, s);
    harp_status_t st;
    if (plan->d == 256 && n_rows >= 1024) {
        // one pass of the tensor-memory kernel covers the whole processor: several times the rate of the
        // 16-row tile kernels, whose per-tile block-kernel traffic dominates at this width
        st = harp_tm_apply(plan, x, n_rows, dtype, transpose, s);
        if (st != HARP_ERR_UNSUPPORTED) return st;
    }
    st = harp_fast_apply(plan, x, n_rows, dtype, transpose, s);
    if (st != HARP_ERR_UNSUPPORTED) return st;
    st = harp_split_apply(plan, x, n_rows, dtype, transpose, s);
    if (st != HARP_ERR_UNSUPPORTED) return st;
    return harp_generic_apply(plan, x, n_rows, dtype, transpose, s);
}

extern "C" harp_status_t harp_apply(const harp_plan_t *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                                    int transpose, void *stream) {
    return harp_apply_ex(plan, x, n_rows, dtype, transpose, HARP_KERNEL_AUTO, stream);
}

// Several passes: forward applies plans[0], plans[1], ... in turn; the transpose undoes them in
// the opposite order.
extern "C" harp_status_t harp_apply_passes(const harp_plan_t *const *plans, int32_t n_passes, void *x, int64_t n_rows,
                                           harp_dtype_t dtype, int transpose, void *stream) {
    if (!plans) return HARP_ERR_NULL;
    if (n_passes < 1) return HARP_ERR_BAD_SCHEDULE;
    for (int32_t k = 0; k < n_passes; ++k) {
        if (!plans[k]) return HARP_ERR_NULL;
        if (plans[k]->d != plans[0]->d) return HARP_ERR_DIM_MISMATCH;
    }
    for (int32_t k = 0; k < n_passes; ++k) {
        const harp_plan_t *p = plans[transpose ? n_passes - 1 - k : k];
        const harp_status_t st = harp_apply(p, x, n_rows, dtype, transpose, stream);
        if (st != HARP_OK) return st;
    }
    return HARP_OK;
}

extern "C" int64_t harp_two_sided_scratch_bytes(const harp_plan_t *plan_out, const harp_plan_t *plan_in,
                                                harp_dtype_t dtype) {
    if (!plan_out || !plan_in || (dtype != HARP_F32 && dtype != HARP_BF16)) return 0;
    const int64_t bytes = plan_out->d * plan_in->d * (int64_t)harp_dtype_size(dtype);
    return (bytes + 255) / 256 * 256;
}

extern "C" harp_status_t harp_apply_two_sided(void *W, harp_dtype_t dtype, const harp_plan_t *plan_out,
                                              const harp_plan_t *plan_in, void *scratch, void *stream) {
    if (!W || !plan_out || !plan_in) return HARP_ERR_NULL;
    if (dtype != HARP_F32 && dtype != HARP_BF16) return HARP_ERR_BAD_DTYPE;
    if ((reinterpret_cast<uintptr_t>(W) & (harp_dtype_size(dtype) - 1)) != 0) return HARP_ERR_BAD_DIM;
    if (scratch && (reinterpret_cast<uintptr_t>(scratch) & 255u) != 0) return HARP_ERR_BAD_DIM;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t d_out = plan_out->d, d_in = plan_in->d;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return HARP_ERR_CUDA;
    if (dev != plan_out->device || dev != plan_in->device) return HARP_ERR_DIM_MISMATCH;
    // row side: every row of W through Q_in
    harp_status_t st = harp_apply(plan_in, W, d_out, dtype, 0, s);
    if (st != HARP_OK) return st;
    // column side: every column of W through Q_out -- in place with the column kernels when the
    // plan has them (no scratch needed), otherwise as rows of W^T (transpose, apply, transpose back)
    st = harp_col_apply(plan_out, W, d_in, d_in, dtype, s);
    if (st != HARP_ERR_UNSUPPORTED) return st;
    bool own = false;
    if (!scratch) {
        if (cudaMallocAsync(&scratch, (size_t)harp_two_sided_scratch_bytes(plan_out, plan_in, dtype), s) != cudaSuccess) {
            cudaGetLastError();
            return HARP_ERR_ALLOC;
        }
        own = true;
    }
    st = harp_transpose_matrix(W, scratch, d_out, d_in, dtype, s);
    if (st == HARP_OK) st = harp_apply(plan_out, scratch, d_in, dtype, 0, s);
    if (st == HARP_OK) st = harp_transpose_matrix(scratch, W, d_in, d_out, dtype, s);
    if (own && cudaFreeAsync(scratch, s) != cudaSuccess && st == HARP_OK) st = HARP_ERR_CUDA;
    return st;
}

extern "C" harp_status_t harp_apply_host(harp_plan_t *plan, void *x_host, int64_t n_rows, harp_dtype_t dtype,
                                         int transpose) {
    if (!plan) return HARP_ERR_NULL;
    if (dtype != HARP_F32 && dtype != HARP_BF16) return HARP_ERR_BAD_DTYPE;
    if (n_rows < 0) return HARP_ERR_BAD_DIM;
    if (n_rows == 0) return HARP_OK;
    if (!x_host) return HARP_ERR_NULL;
    DeviceGuard g(plan->device);
    if (!g.ok) return HARP_ERR_CUDA;
    const int64_t row_bytes = plan->d * (int64_t)harp_dtype_size(dtype);
    // staging bytes per buffer: small enough that the first copy in and the last copy out, which
    // nothing overlaps, are a small part of the transfer
    const int64_t want = (int64_t)16 << 20;
    int64_t chunk_rows = std::max<int64_t>(1, want / row_bytes);
    const int64_t need = chunk_rows * row_bytes;
    if (plan->stage_bytes < need) {
        for (int i = 0; i < harp_plan::kStages; ++i) {
            if (plan->stage_buf[i]) { cudaFree(plan->stage_buf[i]); plan->stage_buf[i] = nullptr; }
            if (cudaMalloc(&plan->stage_buf[i], (size_t)need) != cudaSuccess) { cudaGetLastError(); plan->stage_bytes = 0; return HARP_ERR_ALLOC; }
        }
        plan->stage_bytes = need;
    }
    for (int i = 0; i < harp_plan::kStages; ++i)
        if (!plan->stage_stream[i] && cudaStreamCreateWithFlags(&plan->stage_stream[i], cudaStreamNonBlocking) != cudaSuccess)
            return HARP_ERR_CUDA;
    harp_status_t st = HARP_OK;
    int k = 0;
    for (int64_t r = 0; r < n_rows && st == HARP_OK; r += chunk_rows, ++k) {
        const int64_t rows = std::min(chunk_rows, n_rows - r);
        const int b = k % harp_plan::kStages;
        char *h = static_cast<char *>(x_host) + r * row_bytes;
        cudaStream_t s = plan->stage_stream[b];
        if (cudaMemcpyAsync(plan->stage_buf[b], h, (size_t)(rows * row_bytes), cudaMemcpyHostToDevice, s) != cudaSuccess) st = HARP_ERR_CUDA;
        if (st == HARP_OK) st = harp_apply(plan, plan->stage_buf[b], rows, dtype, transpose, s);
        if (st == HARP_OK && cudaMemcpyAsync(h, plan->stage_buf[b], (size_t)(rows * row_bytes), cudaMemcpyDeviceToHost, s) != cudaSuccess) st = HARP_ERR_CUDA;
    }
    for (int i = 0; i < harp_plan::kStages; ++i)
        if (cudaStreamSynchronize(plan->stage_stream[i]) != cudaSuccess && st == HARP_OK) st = HARP_ERR_CUDA;
    return st;
}
