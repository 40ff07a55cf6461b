// Host-side helpers shared by the tensor-core plan builders: stage grouping, fused block
// matrices (fp64), bf16 rounding, and the slot maps of the mma.sync operand layouts.
#pragma once

#include <cstring>
#include <vector>

#include "harp_internal.h"

namespace harp_fuse {

struct HostPhase {
    int t0, t1;          // stages [t0, t1)
    int B;               // fused block size
    int64_t S;           // natural stride of the phase (= s_{t0})
    int64_t W;           // shared-memory element stride of the phase's local index
    int lane_mult;       // 1, 2 or (B = 16 only) 4
};

inline uint16_t f2bf(double v) {
    const float f = (float)v;
    uint32_t u;
    std::memcpy(&u, &f, 4);
    const uint32_t r = u + 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(r >> 16);
}

// Fused block of phase hp for the block whose coordinates are base + r*S (r < B):
// F[r_in][r_out] in fp64, the product of the phase's stages restricted to those coordinates.
inline void fused_block(const harp_plan *plan, const HostPhase &hp, int64_t base, std::vector<double> &F) {
    const int B = hp.B;
    F.assign((size_t)B * B, 0.0);
    for (int r = 0; r < B; ++r) F[(size_t)r * B + r] = 1.0;
    std::vector<double> tmp((size_t)B * B);
    for (int t = hp.t0; t < hp.t1; ++t) {
        const int b = plan->st.b[t];
        const int64_t s = plan->st.s[t];
        const int64_t ls = s / hp.S;                     // local stride of this stage's digit
        const float *Kt = plan->h_blocks.data() + plan->st.off[t];
        std::fill(tmp.begin(), tmp.end(), 0.0);
        for (int r = 0; r < B; ++r) {                    // r = output local index
            const int digit = (int)((r / ls) % b);
            const int r_base = r - digit * (int)ls;
            const int64_t pos = base + (int64_t)r_base * hp.S;      // coordinate with the digit zeroed
            const int64_t alpha = pos / ((int64_t)b * s), beta = pos % s;
            const float *Kc = Kt + (alpha * s + beta) * b * b;
            for (int i = 0; i < b; ++i) {                // input digit
                const int r_in = r_base + i * (int)ls;
                const double k = (double)Kc[i * b + digit];
                for (int row = 0; row < B; ++row) tmp[(size_t)row * B + r] += F[(size_t)row * B + r_in] * k;
            }
        }
        F.swap(tmp);
    }
}

// slot maps: k-slot (or n-slot) index 0..B-1 of the MMA operand -> block-local index r
inline int strided_slot(int kappa, int B, int lane_mult) {
    const int qq = (kappa & 7) >> 1, i = kappa & 1, k = kappa >> 3;
    const int j = i + 2 * k;
    if (B == 16) {
        static const int joff1[4] = {0, 4, 8, 12}, joff2[4] = {0, 1, 8, 9}, joff4[4] = {0, 1, 2, 3};
        return lane_mult * qq + (lane_mult == 1 ? joff1[j] : lane_mult == 2 ? joff2[j] : joff4[j]);
    }
    static const int joff1[2] = {0, 4}, joff2[2] = {0, 1};
    return lane_mult * qq + (lane_mult == 1 ? joff1[j] : joff2[j]);
}


}  // namespace harp_fuse
