// Plan-side helpers of the C ABI (host code): the greedy Mixed-Radix schedule, block kernels
// rebuilt from stored parameters (Givens angle / Cayley upper triangle, optionally int8 with a
// per-block scale), and the Kronecker fallback written as an ordinary stage list.
#include <algorithm>
#include <cmath>
#include <new>
#include <vector>

#include "harp_internal.h"

extern "C" int32_t harp_greedy_schedule(int64_t d, int32_t b_base, int32_t b_max, int32_t *radices, int32_t max_stages) {
    if (d < 2 || b_base < 2 || b_max < 2 || !radices || max_stages < 1) return -1;
    int32_t n = 0;
    int64_t r = d;
    auto push = [&](int64_t f) {
        if (n >= max_stages) return false;
        radices[n++] = (int32_t)f;
        return true;
    };
    while (r % b_base == 0) {
        if (!push(b_base)) return -1;
        r /= b_base;
    }
    for (int64_t f = std::min<int64_t>(b_max, r); f >= 2; --f)
        while (r % f == 0) {
            if (!push(f)) return -1;
            r /= f;
        }
    if (r != 1) {
        if (r > 0x7fffffffLL || !push(r)) return -1;
    }
    return n;
}

namespace {

bool is_pow2(int b) { return b > 0 && (b & (b - 1)) == 0; }

// H_b[i][j] = (-1)^popcount(i & j) / sqrt(b)
void sylvester(int b, std::vector<double> &g) {
    g.resize((size_t)b * b);
    const double s = 1.0 / std::sqrt((double)b);
    for (int i = 0; i < b; ++i)
        for (int j = 0; j < b; ++j) g[(size_t)i * b + j] = (__builtin_popcount((unsigned)(i & j)) & 1) ? -s : s;
}

// Q = (I + A)^{-1} (I - A) for skew-symmetric A given by its strict upper triangle (row-major, i < j):
// Gaussian elimination with partial pivoting on [I + A | I - A].  Returns false if singular.
bool cayley(int b, const double *upper, std::vector<double> &q) {
    std::vector<double> m((size_t)b * 2 * b, 0.0);
    const int w = 2 * b;
    int k = 0;
    for (int i = 0; i < b; ++i) {
        m[(size_t)i * w + i] += 1.0;
        m[(size_t)i * w + b + i] += 1.0;
        for (int j = i + 1; j < b; ++j, ++k) {
            const double a = upper[k];
            m[(size_t)i * w + j] += a;          // (I + A)_ij
            m[(size_t)j * w + i] -= a;          // (I + A)_ji = -a
            m[(size_t)i * w + b + j] -= a;      // (I - A)_ij
            m[(size_t)j * w + b + i] += a;
        }
    }
    for (int c = 0; c < b; ++c) {
        int piv = c;
        for (int r = c + 1; r < b; ++r)
            if (std::fabs(m[(size_t)r * w + c]) > std::fabs(m[(size_t)piv * w + c])) piv = r;
        if (std::fabs(m[(size_t)piv * w + c]) < 1e-300) return false;
        if (piv != c)
            for (int j = 0; j < w; ++j) std::swap(m[(size_t)piv * w + j], m[(size_t)c * w + j]);
        const double inv = 1.0 / m[(size_t)c * w + c];
        for (int j = c; j < w; ++j) m[(size_t)c * w + j] *= inv;
        for (int r = 0; r < b; ++r) {
            if (r == c) continue;
            const double f = m[(size_t)r * w + c];
            if (f == 0.0) continue;
            for (int j = c; j < w; ++j) m[(size_t)r * w + j] -= f * m[(size_t)c * w + j];
        }
    }
    q.resize((size_t)b * b);
    for (int i = 0; i < b; ++i)
        for (int j = 0; j < b; ++j) q[(size_t)i * b + j] = m[(size_t)i * w + b + j];
    return true;
}

}  // namespace

extern "C" int32_t harp_theta_params_per_block(int32_t b) { return b < 2 ? -1 : (b == 2 ? 1 : b * (b - 1) / 2); }

extern "C" harp_status_t harp_blocks_from_theta(int32_t b, int64_t n_blocks, const float *theta, const int8_t *theta_q,
                                                const float *scales, const float *mixer, float *out_blocks) {
    if (!out_blocks || (!theta && !theta_q) || (theta_q && !theta && !scales)) return HARP_ERR_NULL;
    if (b < 2 || b > 256 || n_blocks < 0) return HARP_ERR_BAD_SCHEDULE;
    if (!mixer && !is_pow2(b)) return HARP_ERR_NULL;         // no default mixer for a radix that is not a power of two
    const int np = harp_theta_params_per_block(b);
    std::vector<double> g, q, th((size_t)np);
    try {
        if (mixer) {
            g.resize((size_t)b * b);
            for (int i = 0; i < b * b; ++i) g[(size_t)i] = mixer[i];
        } else {
            sylvester(b, g);
        }
        q.resize((size_t)b * b);
    } catch (const std::bad_alloc &) {
        return HARP_ERR_ALLOC;
    }
    for (int64_t c = 0; c < n_blocks; ++c) {
        for (int k = 0; k < np; ++k)
            th[(size_t)k] = theta ? (double)theta[c * np + k] : (double)scales[c] * (double)theta_q[c * np + k];
        if (b == 2) {
            const double cs = std::cos(th[0]), sn = std::sin(th[0]);
            q[0] = cs; q[1] = -sn; q[2] = sn; q[3] = cs;
        } else if (!cayley(b, th.data(), q)) {
            return HARP_ERR_BAD_SCHEDULE;
        }
        float *dst = out_blocks + c * b * b;
        for (int i = 0; i < b; ++i)
            for (int j = 0; j < b; ++j) {
                double acc = 0.0;
                for (int k = 0; k < b; ++k) acc += q[(size_t)i * b + k] * g[(size_t)k * b + j];
                dst[i * b + j] = (float)acc;
            }
    }
    return HARP_OK;
}

// Chain rule from the block kernels back to the stored parameters.  K = Q G, so D = dL/dQ = (dL/dK) G^T.
// Givens: dL/dtheta = <D, dQ/dtheta>.  Cayley: with M = (I + A)^{-1} = (Q + I)/2, a change dA moves Q
// by -M dA (Q + I), hence dL/dA = -(1/2) (Q + I)^T D (Q + I)^T, and the parameter of the pair i < j
// (A_ij = a, A_ji = -a) collects (dL/dA)_ij - (dL/dA)_ji.
extern "C" harp_status_t harp_grad_theta(int32_t b, int64_t n_blocks, const float *theta, const float *mixer,
                                         const float *grad_blocks, float *grad_theta) {
    if (!theta || !grad_blocks || !grad_theta) return HARP_ERR_NULL;
    if (b < 2 || b > 256 || n_blocks < 0) return HARP_ERR_BAD_SCHEDULE;
    if (!mixer && !is_pow2(b)) return HARP_ERR_NULL;
    const int np = harp_theta_params_per_block(b);
    const size_t bb = (size_t)b * b;
    std::vector<double> g, q, th((size_t)np), dq, p, tmp;
    try {
        if (mixer) {
            g.resize(bb);
            for (size_t i = 0; i < bb; ++i) g[i] = mixer[i];
        } else {
            sylvester(b, g);
        }
        q.resize(bb); dq.resize(bb); p.resize(bb); tmp.resize(bb);
    } catch (const std::bad_alloc &) {
        return HARP_ERR_ALLOC;
    }
    for (int64_t c = 0; c < n_blocks; ++c) {
        const float *gk = grad_blocks + c * (int64_t)bb;
        for (int i = 0; i < b; ++i)                       // D = (dL/dK) G^T
            for (int k = 0; k < b; ++k) {
                double acc = 0.0;
                for (int j = 0; j < b; ++j) acc += (double)gk[i * b + j] * g[(size_t)k * b + j];
                dq[(size_t)i * b + k] = acc;
            }
        for (int k = 0; k < np; ++k) th[(size_t)k] = theta[c * np + k];
        float *out = grad_theta + c * np;
        if (b == 2) {
            const double cs = std::cos(th[0]), sn = std::sin(th[0]);
            out[0] = (float)(-sn * dq[0] - cs * dq[1] + cs * dq[2] - sn * dq[3]);
            continue;
        }
        if (!cayley(b, th.data(), q)) return HARP_ERR_BAD_SCHEDULE;
        for (int i = 0; i < b; ++i)                       // P = Q + I
            for (int j = 0; j < b; ++j) p[(size_t)i * b + j] = q[(size_t)i * b + j] + (i == j ? 1.0 : 0.0);
        for (int i = 0; i < b; ++i)                       // tmp = P^T D
            for (int j = 0; j < b; ++j) {
                double acc = 0.0;
                for (int k = 0; k < b; ++k) acc += p[(size_t)k * b + i] * dq[(size_t)k * b + j];
                tmp[(size_t)i * b + j] = acc;
            }
        auto ga = [&](int i, int j) {                     // (dL/dA)_ij = -(1/2) (tmp P^T)_ij
            double acc = 0.0;
            for (int k = 0; k < b; ++k) acc += tmp[(size_t)i * b + k] * p[(size_t)j * b + k];
            return -0.5 * acc;
        };
        int k = 0;
        for (int i = 0; i < b; ++i)
            for (int j = i + 1; j < b; ++j, ++k) out[k] = (float)(ga(i, j) - ga(j, i));
    }
    return HARP_OK;
}

namespace {

// One stage's block kernels through the device kernels: parameters up, blocks rebuilt on the GPU,
// blocks back (the plan builder fuses stages on the host).  HARP_ERR_UNSUPPORTED for radices the
// device kernels do not take.
harp_status_t stage_blocks_on_device(int b, int64_t n_blocks, const float *theta, const int8_t *theta_q, const float *scales,
                                     const float *mixer, float *out_host) {
    if (b > harp_theta_device_max_radix()) return HARP_ERR_UNSUPPORTED;
    if ((!theta && !theta_q) || (theta_q && !theta && !scales)) return HARP_ERR_NULL;
    if (!mixer && !is_pow2(b)) return HARP_ERR_NULL;
    const int np = harp_theta_params_per_block(b);
    void *d_theta = nullptr, *d_scales = nullptr, *d_mixer = nullptr, *d_out = nullptr;
    const size_t theta_bytes = (size_t)n_blocks * np * (theta ? sizeof(float) : 1);
    harp_status_t st = HARP_OK;
    auto up = [&](void **dst, const void *src, size_t bytes) {
        if (st != HARP_OK || !src) return;
        if (cudaMalloc(dst, std::max<size_t>(bytes, 16)) != cudaSuccess) { st = HARP_ERR_ALLOC; return; }
        if (cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice) != cudaSuccess) st = HARP_ERR_CUDA;
    };
    up(&d_theta, theta ? (const void *)theta : (const void *)theta_q, theta_bytes);
    if (!theta) up(&d_scales, scales, (size_t)n_blocks * sizeof(float));
    up(&d_mixer, mixer, (size_t)b * b * sizeof(float));
    const size_t out_bytes = (size_t)n_blocks * b * b * sizeof(float);
    if (st == HARP_OK && cudaMalloc(&d_out, std::max<size_t>(out_bytes, 16)) != cudaSuccess) st = HARP_ERR_ALLOC;
    if (st == HARP_OK)
        st = harp_blocks_from_theta_device(b, n_blocks, theta ? (const float *)d_theta : nullptr,
                                           theta ? nullptr : (const int8_t *)d_theta, (const float *)d_scales,
                                           (const float *)d_mixer, (float *)d_out, nullptr);
    if (st == HARP_OK && cudaMemcpy(out_host, d_out, out_bytes, cudaMemcpyDeviceToHost) != cudaSuccess) st = HARP_ERR_CUDA;
    if (st != HARP_OK) cudaGetLastError();
    cudaFree(d_theta); cudaFree(d_scales); cudaFree(d_mixer); cudaFree(d_out);
    return st;
}

}  // namespace

extern "C" harp_status_t harp_plan_create_from_theta(harp_plan_t **out, int64_t d, int32_t n_stages, const int32_t *radices,
                                                     const int32_t *perm, const int8_t *signs, const float *const *theta,
                                                     const int8_t *const *theta_q, const float *const *scales,
                                                     const float *const *mixers) {
    if (!out || !radices || (!theta && !theta_q)) return HARP_ERR_NULL;
    if (d < 2 || d > (1 << 20)) return HARP_ERR_BAD_DIM;
    if (n_stages < 1 || n_stages > HARP_MAX_STAGES) return HARP_ERR_BAD_SCHEDULE;
    int64_t prod = 1;
    for (int t = 0; t < n_stages; ++t) {
        if (radices[t] < 2 || radices[t] > d) return HARP_ERR_BAD_SCHEDULE;
        prod *= radices[t];
        if (prod > d) return HARP_ERR_BAD_SCHEDULE;
    }
    if (prod != d) return HARP_ERR_BAD_SCHEDULE;
    std::vector<std::vector<float>> blocks((size_t)n_stages);
    std::vector<const float *> ptrs((size_t)n_stages);
    for (int t = 0; t < n_stages; ++t) {
        const int b = radices[t];
        try {
            blocks[(size_t)t].resize((size_t)d * b);
        } catch (const std::bad_alloc &) {
            return HARP_ERR_ALLOC;
        }
        // rebuilt by the device kernels; radices beyond their limit by the host routine
        harp_status_t st = stage_blocks_on_device(b, d / b, theta ? theta[t] : nullptr, theta_q ? theta_q[t] : nullptr,
                                                  scales ? scales[t] : nullptr, mixers ? mixers[t] : nullptr,
                                                  blocks[(size_t)t].data());
        if (st == HARP_ERR_UNSUPPORTED)
            st = harp_blocks_from_theta(b, d / b, theta ? theta[t] : nullptr, theta_q ? theta_q[t] : nullptr,
                                        scales ? scales[t] : nullptr, mixers ? mixers[t] : nullptr, blocks[(size_t)t].data());
        if (st != HARP_OK) return st;
        ptrs[(size_t)t] = blocks[(size_t)t].data();
    }
    return harp_plan_create(out, d, n_stages, radices, perm, signs, ptrs.data());
}

extern "C" harp_status_t harp_plan_create_kronecker(harp_plan_t **out, int64_t n2, int32_t n_stages, const int32_t *radices,
                                                    const float *const *blocks_n2, int32_t K, const float *hk,
                                                    const int32_t *perm, const int8_t *signs) {
    if (!out || !radices || !blocks_n2 || !hk) return HARP_ERR_NULL;
    if (K < 2 || n2 < 2 || n_stages < 1 || n_stages + 1 > HARP_MAX_STAGES) return HARP_ERR_BAD_SCHEDULE;
    const int64_t d = (int64_t)K * n2;
    if (d > (1 << 20)) return HARP_ERR_BAD_DIM;
    int64_t prod = 1;
    for (int t = 0; t < n_stages; ++t) {
        if (radices[t] < 2 || !blocks_n2[t]) return HARP_ERR_BAD_SCHEDULE;
        prod *= radices[t];
        if (prod > n2) return HARP_ERR_BAD_SCHEDULE;
    }
    if (prod != n2) return HARP_ERR_BAD_SCHEDULE;
    // the table must be +-1 with H H^T = K I
    for (int i = 0; i < K; ++i)
        for (int j = 0; j < K; ++j) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                const float v = hk[i * K + k];
                if (v != 1.0f && v != -1.0f) return HARP_ERR_BAD_SIGNS;
                acc += (double)v * hk[j * K + k];
            }
            if (std::fabs(acc - (i == j ? K : 0)) > 1e-6) return HARP_ERR_BAD_SCHEDULE;
        }
    std::vector<int32_t> rad((size_t)n_stages + 1);
    std::vector<std::vector<float>> blocks((size_t)n_stages + 1);
    std::vector<const float *> ptrs((size_t)n_stages + 1);
    try {
        int64_t s = 1;
        for (int t = 0; t < n_stages; ++t) {
            const int b = radices[t];
            rad[(size_t)t] = b;
            const int64_t g_small = n2 / (b * s), bb = (int64_t)b * b;
            blocks[(size_t)t].resize((size_t)d * b);
            // block index of the wide plan: alpha = k*g_small + alpha', the K rows being the slowest index
            for (int64_t k = 0; k < K; ++k)
                for (int64_t a = 0; a < g_small; ++a)
                    for (int64_t be = 0; be < s; ++be) {
                        const float *src = blocks_n2[t] + (a * s + be) * bb;
                        float *dst = blocks[(size_t)t].data() + ((k * g_small + a) * s + be) * bb;
                        for (int64_t i = 0; i < bb; ++i) dst[i] = src[i];
                    }
            ptrs[(size_t)t] = blocks[(size_t)t].data();
            s *= b;
        }
        rad[(size_t)n_stages] = K;
        blocks[(size_t)n_stages].resize((size_t)n2 * K * K);
        const float inv = (float)(1.0 / std::sqrt((double)K));
        for (int64_t c = 0; c < n2; ++c)
            for (int i = 0; i < K * K; ++i) blocks[(size_t)n_stages][(size_t)(c * K * K + i)] = hk[i] * inv;
        ptrs[(size_t)n_stages] = blocks[(size_t)n_stages].data();
    } catch (const std::bad_alloc &) {
        return HARP_ERR_ALLOC;
    }
    return harp_plan_create(out, d, n_stages + 1, rad.data(), perm, signs, ptrs.data());
}
