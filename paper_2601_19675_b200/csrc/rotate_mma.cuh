// Permutation gather and partial block Walsh-Hadamard rotation (Eq. 5, Eq. 6) of many token rows, with the first
// four levels of the Hadamard recursion (Eq. 2) as a tensor-core product and the rest as register butterflies.
//
// H_b = H_{b/16} (x) H_16 in the natural (Kronecker) order: a block of b gathered entries is cut into tiles of 16;
// every tile is multiplied by H_16 (entries +-1, exact in bf16; fp32 accumulation) with mma.m16n8k16 -- tokens are
// the M dimension, so a warp rotates the same block of up to 8 token rows at once --, then the tiles are combined by
// log2(b/16) levels of add / subtract, which pair registers of the SAME lane (no shuffles), one scaling by 1/sqrt(b)
// and one rounding to bf16.  Against register-and-shuffle butterflies this is about a third of the instructions
// per entry, which is what bounds the rotation of a prefill batch (the data is read and written exactly once).
//
// A CTA stages TOK token rows of x in shared memory (the permutation scatters over the whole row) and its warps
// take the row's blocks in turn.  Lane l = 4 g + t: token g; of every 16-tile the gathered columns 2t, 2t+1, 2t+8,
// 2t+9 (the A fragment) and, after the product, the outputs 2t, 2t+1, 8+2t, 8+2t+1 (the D fragments of the two
// 8-column halves).  The identity prefix (b_I columns, Eq. 6) is gathered and stored by the same lanes.
// Requires 16 <= b_H <= 256, b_I a multiple of 16.  Writes no column sums.
#pragma once

#include "common.cuh"

namespace lopro {

// +-1 fragments of H_16 for the B operand (k x n, "col" layout): b0 = rows 2t, 2t+1, b1 = rows 2t+8, 2t+9 of
// column n = col; H_16[k][i] = (-1)^popcount(k & i).
__device__ __forceinline__ void h16_fragment(int t, int col, uint32_t (&b)[2]) {
    auto entry = [&](int k) { return (__popc(k & col) & 1) ? 0xBF80u : 0x3F80u; };
    b[0] = entry(2 * t) | (entry(2 * t + 1) << 16);
    b[1] = entry(2 * t + 8) | (entry(2 * t + 9) << 16);
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a2, const uint32_t (&b)[2]) {
    // rows g + 8 of A are empty (a1 = a3 = 0): at most 8 token rows per warp
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b[0]), "r"(b[1]), "f"(0.0f));
}

// The lane's four gathered entries of the 16-tile that starts at column k0, as two bf16 pairs.  xrow_s: shared-space
// address of the lane's staged row; off_s: shared-space address of the CTA's table of 16-bit column indices perm[k]
// (d_in <= 32768; clamped to the row when it was built, so that a perm that is no permutation cannot reach foreign
// memory).
__device__ __forceinline__ void gather_tile(uint32_t xrow_s, uint32_t off_s, int k0, int t, uint32_t& a0, uint32_t& a2) {
    uint32_t w0, w1;  // two 16-bit column indices each
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w0) : "r"(off_s + 2u * (uint32_t)(k0 + 2 * t)));
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w1) : "r"(off_s + 2u * (uint32_t)(k0 + 8 + 2 * t)));
    unsigned short v0, v1, v2, v3;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v0) : "r"(xrow_s + 2u * (w0 & 0xFFFFu)));
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v1) : "r"(xrow_s + 2u * (w0 >> 16)));
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v2) : "r"(xrow_s + 2u * (w1 & 0xFFFFu)));
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v3) : "r"(xrow_s + 2u * (w1 >> 16)));
    asm("mov.b32 %0, {%1,%2};" : "=r"(a0) : "h"(v0), "h"(v1));
    asm("mov.b32 %0, {%1,%2};" : "=r"(a2) : "h"(v2), "h"(v3));
}

template <int KT>
__device__ __forceinline__ void rotate_block_mma(uint32_t xrow, uint32_t perm,
                                                 int kb, int t, bool live, const uint32_t (&h0)[2], const uint32_t (&h1)[2],
                                                 float inv_sqrt_bh, __nv_bfloat16* __restrict__ orow) {
    float z[KT][4];
#pragma unroll
    for (int kt = 0; kt < KT; ++kt) {
        uint32_t a0, a2;  // lanes without a live row gather row 0 and store nothing
        gather_tile(xrow, perm, kb + 16 * kt, t, a0, a2);
        float d0[4], d1[4];
        mma_bf16_16816(d0, a0, a2, h0);
        mma_bf16_16816(d1, a0, a2, h1);
        z[kt][0] = d0[0];
        z[kt][1] = d0[1];
        z[kt][2] = d1[0];
        z[kt][3] = d1[1];
    }
#pragma unroll
    for (int h = 1; h < KT; h <<= 1)
#pragma unroll
        for (int kt = 0; kt < KT; ++kt)
            if ((kt & h) == 0) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float a = z[kt][e], b = z[kt + h][e];
                    z[kt][e] = a + b;
                    z[kt + h][e] = a - b;
                }
            }
    if (live) {
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) {
            __nv_bfloat16* o = orow + kb + 16 * kt + 2 * t;
            *reinterpret_cast<__nv_bfloat162*>(o) = __floats2bfloat162_rn(z[kt][0] * inv_sqrt_bh, z[kt][1] * inv_sqrt_bh);
            *reinterpret_cast<__nv_bfloat162*>(o + 8) = __floats2bfloat162_rn(z[kt][2] * inv_sqrt_bh, z[kt][3] * inv_sqrt_bh);
        }
    }
}

// Shared memory: rotate_mma_smem_bytes(TOK, n) -- the staged rows and a copy of perm (a lookup from global memory in
// front of every gather would put an L2 round trip into each tile's chain).  The rows are kept 16 bytes apart from a multiple of 128 bytes, so
// that the eight lanes that read the same gathered column of eight different rows hit eight different banks.
// `block` = index of the CTA's group of TOK token rows; blockDim.x = 256.
constexpr int kRotMmaPad = 8;  // bf16 entries between the staged rows
constexpr int kRotMmaMaxSmem = 200 * 1024;
__host__ __device__ inline size_t rotate_mma_smem_bytes(int tok, int n) {
    return (size_t)tok * (size_t)(n + kRotMmaPad) * 2 + (size_t)n * 2;  // the rows, then perm as 16-bit indices
}

template <int TOK>
__device__ __forceinline__ void rotate_mma_body(unsigned char* smem_raw, int block, const __nv_bfloat16* __restrict__ x,
                                                int64_t ldx, const int32_t* __restrict__ perm,
                                                __nv_bfloat16* __restrict__ xrot, int64_t ldo, int* __restrict__ status, int n,
                                                int b_i, int b_h, float inv_sqrt_bh, int T) {
    static_assert(TOK == 4 || TOK == 8, "token rows per CTA");
    unsigned short* xs = reinterpret_cast<unsigned short*>(smem_raw);  // [TOK][n + kRotMmaPad]
    const int stride = n + kRotMmaPad;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int t0 = block * TOK, nt = min(TOK, T - t0);
    if (status != nullptr && block == 0 && tid == 0) *status = LOPRO_OK;
    // stage the rows with asynchronous 16-byte copies: all of them in flight at once, one wait
    const int pieces = n >> 3;
    for (int r = 0; r < nt; ++r) {
        const __nv_bfloat16* src = x + (size_t)(t0 + r) * ldx;
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(xs + (size_t)r * stride);
        for (int c = tid; c < pieces; c += 256)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16u * (uint32_t)c), "l"(src + 8 * c) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    // the gather's column indices min(perm[k], n - 1) as 16-bit numbers, one table per CTA
    unsigned short* off_tab = xs + (size_t)TOK * stride;
    for (int c = tid; c < (n >> 2); c += 256) {
        const int4 p4 = __ldg(reinterpret_cast<const int4*>(perm) + c);
        const uint32_t last = (uint32_t)n - 1u;
        uint2 o2;
        o2.x = min((uint32_t)p4.x, last) | (min((uint32_t)p4.y, last) << 16);
        o2.y = min((uint32_t)p4.z, last) | (min((uint32_t)p4.w, last) << 16);
        reinterpret_cast<uint2*>(off_tab)[c] = o2;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    const int g = lane >> 2, t = lane & 3;
    const bool live = g < nt;
    const uint32_t xrow = (uint32_t)__cvta_generic_to_shared(xs + (size_t)(live ? g : 0) * stride);
    const uint32_t perm_s32 = (uint32_t)__cvta_generic_to_shared(off_tab);
    __nv_bfloat16* orow = xrot + (size_t)(t0 + (live ? g : 0)) * ldo;
    // identity prefix: gathered entries go out as they are
    for (int j = warp; j < (b_i >> 4); j += nwarps) {
        uint32_t a0, a2;
        gather_tile(xrow, perm_s32, 16 * j, t, a0, a2);
        if (live) {
            *reinterpret_cast<uint32_t*>(orow + 16 * j + 2 * t) = a0;
            *reinterpret_cast<uint32_t*>(orow + 16 * j + 8 + 2 * t) = a2;
        }
    }
    uint32_t h0[2], h1[2];
    h16_fragment(t, g, h0);
    h16_fragment(t, g + 8, h1);
    const int n_blk = (n - b_i) / b_h;
    for (int blk = warp; blk < n_blk; blk += nwarps) {
        const int kb = b_i + blk * b_h;
        switch (b_h) {
            case 16: rotate_block_mma<1>(xrow, perm_s32, kb, t, live, h0, h1, inv_sqrt_bh, orow); break;
            case 32: rotate_block_mma<2>(xrow, perm_s32, kb, t, live, h0, h1, inv_sqrt_bh, orow); break;
            case 64: rotate_block_mma<4>(xrow, perm_s32, kb, t, live, h0, h1, inv_sqrt_bh, orow); break;
            case 128: rotate_block_mma<8>(xrow, perm_s32, kb, t, live, h0, h1, inv_sqrt_bh, orow); break;
            default: rotate_block_mma<16>(xrow, perm_s32, kb, t, live, h0, h1, inv_sqrt_bh, orow); break;
        }
    }
}

inline bool rotate_mma_shape_ok(const lopro_desc& d) {
    return d.block_size >= 16 && d.block_size <= 256 && d.identity_cols % 16 == 0;
}

}  // namespace lopro
