// Device helpers shared by the tensor-core kernels: shared-memory and global 16-byte
// accesses, ldmatrix/stmatrix, mma.sync (bf16 operands, fp32 accumulate), bf16 packing,
// and the "octet" block products used when a block's coordinates are strided in memory.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4 &v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ldg128_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void stg128(void *p, const uint4 &v) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void stmatrix_x4(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t (&r)[2], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void stmatrix_x2(uint32_t addr, uint32_t r0, uint32_t r1) {
    asm volatile("stmatrix.sync.aligned.m8n8.x2.shared.b16 [%0], {%1,%2};" ::"r"(addr), "r"(r0), "r"(r1) : "memory");
}
// D(16x8, fp32) = A(16x16, bf16) . B(16x8, bf16)
__device__ __forceinline__ void mma_k16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}
// D(16x8, fp32) += A(16x16, bf16) . B(16x8, bf16)
__device__ __forceinline__ void mma_k16_acc(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// D(16x8, fp32) = A(16x8, bf16) . B(8x8, bf16)
__device__ __forceinline__ void mma_k8(float (&c)[4], const uint32_t (&a)[2], uint32_t b0) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%7,%7,%7,%7};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(b0), "f"(0.f));
}
// {lo, hi} -> packed bf16x2, round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t pair_lo(uint32_t x, uint32_t y) { return __byte_perm(x, y, 0x5410); }
__device__ __forceinline__ uint32_t pair_hi(uint32_t x, uint32_t y) { return __byte_perm(x, y, 0x7632); }
__device__ __forceinline__ uint32_t word_of(const uint4 &v, int w) {
    return w == 0 ? v.x : (w == 1 ? v.y : (w == 2 ? v.z : v.w));
}
__device__ __forceinline__ void set_word(uint4 &v, int w, uint32_t x) {
    if (w == 0) v.x = x; else if (w == 1) v.y = x; else if (w == 2) v.z = x; else v.w = x;
}
// 8x8 transpose of 16-bit values held as eight uint4 (row i = in[i], eight values each)
__device__ __forceinline__ void transpose8x8_b16(const uint4 (&in)[8], uint4 (&out)[8]) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const uint32_t x = word_of(in[2 * m], k), y = word_of(in[2 * m + 1], k);
            set_word(out[2 * k], m, pair_lo(x, y));
            set_word(out[2 * k + 1], m, pair_hi(x, y));
        }
    }
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Eight neighbouring blocks at once (B = 16).  raw[j][h] holds, for slot j of this lane
// and row half h, the values of the eight blocks; bf[e] is block e's fragment.  STRIDED_OUT:
// results go back into raw (same slots, same rows); otherwise they are packed for stmatrix.
template <bool STRIDED_OUT>
__device__ __forceinline__ void octet_mma16(uint4 (&raw)[4][2], const uint4 (&bf)[8], uint32_t (&mats)[8][4]) {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        float acc[2][2][4];
#pragma unroll
        for (int ee = 0; ee < 2; ++ee) {
            uint32_t a[4];
            if (ee == 0) {
                a[0] = pair_lo(word_of(raw[0][0], w), word_of(raw[1][0], w));
                a[1] = pair_lo(word_of(raw[0][1], w), word_of(raw[1][1], w));
                a[2] = pair_lo(word_of(raw[2][0], w), word_of(raw[3][0], w));
                a[3] = pair_lo(word_of(raw[2][1], w), word_of(raw[3][1], w));
            } else {
                a[0] = pair_hi(word_of(raw[0][0], w), word_of(raw[1][0], w));
                a[1] = pair_hi(word_of(raw[0][1], w), word_of(raw[1][1], w));
                a[2] = pair_hi(word_of(raw[2][0], w), word_of(raw[3][0], w));
                a[3] = pair_hi(word_of(raw[2][1], w), word_of(raw[3][1], w));
            }
            mma_k16(acc[ee][0], a, bf[2 * w + ee].x, bf[2 * w + ee].y);
            mma_k16(acc[ee][1], a, bf[2 * w + ee].z, bf[2 * w + ee].w);
        }
        if (!STRIDED_OUT) {
#pragma unroll
            for (int ee = 0; ee < 2; ++ee) {
                mats[2 * w + ee][0] = pack_bf16(acc[ee][0][0], acc[ee][0][1]);
                mats[2 * w + ee][1] = pack_bf16(acc[ee][0][2], acc[ee][0][3]);
                mats[2 * w + ee][2] = pack_bf16(acc[ee][1][0], acc[ee][1][1]);
                mats[2 * w + ee][3] = pack_bf16(acc[ee][1][2], acc[ee][1][3]);
            }
        } else {
#pragma unroll
            for (int k = 0; k < 2; ++k)
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        set_word(raw[i + 2 * k][h], w, pack_bf16(acc[0][k][i + 2 * h], acc[1][k][i + 2 * h]));
        }
    }
}

// B = 8: slots j = 0, 1 only; one 32-bit fragment per block.
__device__ __forceinline__ void octet_mma8(uint4 (&raw)[2][2], const uint32_t (&bf)[8]) {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        float acc[2][4];
#pragma unroll
        for (int ee = 0; ee < 2; ++ee) {
            uint32_t a[2];
            if (ee == 0) {
                a[0] = pair_lo(word_of(raw[0][0], w), word_of(raw[1][0], w));
                a[1] = pair_lo(word_of(raw[0][1], w), word_of(raw[1][1], w));
            } else {
                a[0] = pair_hi(word_of(raw[0][0], w), word_of(raw[1][0], w));
                a[1] = pair_hi(word_of(raw[0][1], w), word_of(raw[1][1], w));
            }
            mma_k8(acc[ee], a, bf[2 * w + ee]);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int h = 0; h < 2; ++h) set_word(raw[i][h], w, pack_bf16(acc[0][i + 2 * h], acc[1][i + 2 * h]));
    }
}

