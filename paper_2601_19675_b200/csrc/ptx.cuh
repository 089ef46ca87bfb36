// Device helpers shared by the small-batch kernels: mbarrier and bulk-copy wrappers with bounded
// waits, warp-level tensor-core instructions, and the expansion of packed codes into bf16 operands.
#pragma once

#include <stdint.h>

namespace lopro {

constexpr uint32_t kSpinLimit = 1u << 22;  // polls of one mbarrier wait before it gives up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// one poll that never suspends the thread
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// try_wait with a suspend-time hint (ns): the thread may stay parked that long before the instruction returns false
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Bounded wait for warps that expect to wait long: a failed poll backs off before the next one, so that the polls
// of many waiting warps do not crowd the shared-memory pipeline of the warps that work.
__device__ __forceinline__ bool mbar_wait_backoff(uint32_t bar, uint32_t parity, uint32_t limit = kSpinLimit) {
    for (uint32_t i = 0; i < limit; ++i) {
#if defined(RB_WAIT_HINT)
        if (mbar_try_wait_hint(bar, parity, RB_WAIT_HINT)) return true;
#else
        if (mbar_try_wait(bar, parity)) return true;
#endif
#if defined(RB_WAIT_SLEEP)
        __nanosleep(RB_WAIT_SLEEP);
#endif
    }
    return false;
}
// Bounded wait: false if the limit ran out (the caller records the time-out and carries on).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit = kSpinLimit) {
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// First product of a chain: D = A B with a zero C operand (no registers to clear).
__device__ __forceinline__ void mma_bf16_first(float (&d)[4], const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.0f));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

// two fp8 e4m3 values (low byte first) -> two fp16 values (exact)
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint16_t v) {
    uint32_t d;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(d) : "h"(v));
    return d;
}

// A-operand registers (m16n8k16, fp16) of the 16 x 16 piece at columns jj of a 16-row tile of the up-projection
// factor held in shared memory, rows r_pad entries apart: fp16 entries (A = U Sigma), or fp8 e4m3 entries (U of the
// FP8 low-rank record) converted exactly to fp16.
__device__ __forceinline__ void load_up_fragment(uint32_t (&a)[4], const unsigned char* tile, int r_pad, int gq, int tg, int jj,
                                                 bool lr8) {
    if (!lr8) {
        const __half* as = reinterpret_cast<const __half*>(tile);
        a[0] = *reinterpret_cast<const uint32_t*>(as + gq * r_pad + jj + 2 * tg);
        a[1] = *reinterpret_cast<const uint32_t*>(as + (gq + 8) * r_pad + jj + 2 * tg);
        a[2] = *reinterpret_cast<const uint32_t*>(as + gq * r_pad + jj + 8 + 2 * tg);
        a[3] = *reinterpret_cast<const uint32_t*>(as + (gq + 8) * r_pad + jj + 8 + 2 * tg);
    } else {
        a[0] = e4m3x2_to_f16x2(*reinterpret_cast<const uint16_t*>(tile + gq * r_pad + jj + 2 * tg));
        a[1] = e4m3x2_to_f16x2(*reinterpret_cast<const uint16_t*>(tile + (gq + 8) * r_pad + jj + 2 * tg));
        a[2] = e4m3x2_to_f16x2(*reinterpret_cast<const uint16_t*>(tile + gq * r_pad + jj + 8 + 2 * tg));
        a[3] = e4m3x2_to_f16x2(*reinterpret_cast<const uint16_t*>(tile + (gq + 8) * r_pad + jj + 8 + 2 * tg));
    }
}

constexpr uint32_t kMagic128 = 0x43004300u;  // two bf16 128.0 (ulp 1): 128.0 | c == 128 + c

// (a & mask) | magic in ONE logic instruction (truth table 0xEA), both constants held in registers --
// left to the compiler this becomes two instructions, since only one operand may be an immediate.
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t mask, uint32_t magic) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(mask), "r"(magic));
    return d;
}

template <int BITS>
__device__ __forceinline__ void expand_codes(uint32_t (&a)[16], const uint32_t (&w)[BITS]) {
    const uint32_t magic = kMagic128;
    if constexpr (BITS == 4) {
        const uint32_t mask = 0x000F000Fu;
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int rho = 0; rho < 4; ++rho) a[4 * j + rho] = and_or(w[j] >> (4 * rho), mask, magic);
    } else if constexpr (BITS == 2) {
        const uint32_t mask = 0x00030003u;
#pragma unroll
        for (int pi = 0; pi < 16; ++pi) a[pi] = and_or(w[pi >> 3] >> (2 * (pi & 7)), mask, magic);
    } else {
        const uint32_t mask = 0x00070007u;
#pragma unroll
        for (int pi = 0; pi < 15; ++pi) a[pi] = and_or(w[pi / 5] >> (3 * (pi % 5)), mask, magic);
        a[15] = ((w[0] >> 15) & 0x00010001u) | ((w[1] >> 14) & 0x00020002u) | ((w[2] >> 13) & 0x00040004u) | kMagic128;
    }
}

}  // namespace lopro
