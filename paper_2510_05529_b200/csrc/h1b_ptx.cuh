// Thin inline-PTX wrappers used by the H1B-KV kernels (sm_100a): mbarrier with
// bounded waits, non-multicast bulk async copies into this CTA's shared memory,
// warp-level fp16 tensor-core MMA, and a few scalar helpers.
#pragma once
#include <cstdint>
#include <cuda_fp16.h>

namespace h1b {

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait for a phase of an mbarrier, for at most `limit_ns`. Returns false when
// the limit ran out (the caller records an error and leaves; nothing spins
// forever).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
}

// Bulk async copy global -> this CTA's shared memory (no multicast); completion
// is signalled on `bar` as transferred bytes. Both addresses 16-byte aligned,
// `bytes` a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// 16-byte async copy global -> shared; `src_bytes` = 16, or 0 to fill the 16 bytes with zeros.
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
// Four 8x8 b16 matrices from shared memory (lane l gives the row address of matrix l/8, row l%8).
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two floats -> packed f16x2, round to nearest even; `lo` lands in bits 0-15.
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// D(16x8, f32) += A(16x16, f16, row) * B(16x8, f16, col). Subnormal f16 inputs keep their value, but
// lose alignment precision when summed with larger terms (see decode_chunk).
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Eight 4-bit codes of one packed word -> the four f16x2 registers of an MMA A fragment, as fp16
// SUBNORMALS taken in place: a code c at bits 4-7 of a half, everything else masked off, is the
// subnormal 16 * c * 2^-24 = c * 2^-20. The word holds codes at bits 0, 4, 8 and 12 of each half, so
// three of the four registers need a shift first. Bits 4-7 are used for all of them (and not bits
// 0-3, which would save two shifts) because the tensor core aligns the 16 products of one MMA by
// their exponent FIELDS: a subnormal with six leading zero bits loses about ten bits whenever
// weights of different magnitude meet in one block of tokens; with two leading zeros the loss is
// about 1e-6 relative, measured.
//   H1B_DEQUANT_TWO_SHIFTS (build option): codes at bits 2-5 and 6-9 instead, one shift fewer,
//   about 4e-6 relative.
#ifdef H1B_DEQUANT_TWO_SHIFTS
constexpr float kCodeScaleLo = 4194304.f;     // rows r:     code * 2^-22
constexpr float kCodeScaleHi = 262144.f;      // rows r + 8: code * 2^-18
__device__ __forceinline__ void codes_to_f16x2(uint32_t w, uint32_t (&a)[4]) {
    const uint32_t u = w << 2, t = w >> 6;
    a[0] = u & 0x003C003Cu; a[1] = u & 0x03C003C0u; a[2] = t & 0x003C003Cu; a[3] = t & 0x03C003C0u;
}
#else
constexpr float kCodeScaleLo = 1048576.f;     // every row: code * 2^-20
constexpr float kCodeScaleHi = 1048576.f;
__device__ __forceinline__ void codes_to_f16x2(uint32_t w, uint32_t (&a)[4]) {
    a[0] = (w << 4) & 0x00F000F0u; a[1] = w & 0x00F000F0u;
    a[2] = (w >> 4) & 0x00F000F0u; a[3] = (w >> 8) & 0x00F000F0u;
}
#endif

// D = A * B + Z, where Z is a quad of registers that the caller keeps at zero (see zero_quad): the
// accumulator starts at zero without four register moves per MMA.
__device__ __forceinline__ void mma_f16_16816_from(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                   uint32_t b0, uint32_t b1, const float (&z)[4]) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(z[0]), "f"(z[1]), "f"(z[2]), "f"(z[3]));
}

// Four zeros the compiler cannot see through, so that it keeps them in one register quad for the
// whole kernel instead of re-creating them wherever they are used.
__device__ __forceinline__ void zero_quad(float (&z)[4]) {
    asm volatile("mov.f32 %0, 0f00000000;\n\tmov.f32 %1, 0f00000000;\n\tmov.f32 %2, 0f00000000;\n\tmov.f32 %3, 0f00000000;"
                 : "=f"(z[0]), "=f"(z[1]), "=f"(z[2]), "=f"(z[3]));
}

__device__ __forceinline__ float2 half2_bits_to_float2(uint32_t h2) {
    __half2 h = *reinterpret_cast<__half2 *>(&h2);
    return __half22float2(h);
}

}  // namespace h1b
