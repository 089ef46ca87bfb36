// Small-batch forward (decode): y = W^ x~ + A t for up to 32 tokens per CTA, streaming the
// packed codes once from HBM (steps "Dequant(W_q) X" and "U (Sigma Y)" of Appendix A.3, summed
// as in Eq. 8).
//
// Arithmetic.  With w = s (c - z) per group,
//     sum_k w_k x~_k = s * ( sum_k (128 + c_k) x~_k  -  (128 + z) * sum_k x~_k ) ,
// so the tensor cores multiply the bf16 activations with the bf16 numbers 128 + c (exact: the
// code is OR-ed into the mantissa of 128.0, no conversion instruction), accumulate in fp32 over
// 64 columns, and the scale and zero-point enter once per 64 columns in fp32 together with the
// pre-computed column sums of x~.  The quantized weights are never rounded.
#include <stdlib.h>

#include "common.cuh"
#include "ptx.cuh"

namespace lopro {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsPerCta = kWarps * 16;
constexpr int kPrefetch = 8;  // 64-column steps of codes in flight per warp

struct DecodeParams {
    const uint32_t* codes;  // fragment layout
    const uint32_t* sz;     // (scale, zero) pairs, fragment layout
    const __half* A;        // [m][r_pad]
    const __nv_bfloat16* xrot;  // [T][n]
    const float* s64;           // [T][n/64]
    const __half* t;            // [T][r_pad]
    int s64_stride;
    void* y;
    int64_t ldy;
    int out_f32;
    int m, n, T;
    int gshift;      // log2(group_size / 64)
    int ng;          // groups per row
    int r_pad;
    int slice_steps; // 64-column steps (the whole K range)
    int panel_steps; // steps staged in shared memory at a time (multiple of kPrefetch)
};

// Streaming load of one lane's `BITS` code words (read once: keep them out of L1).
template <int BITS>
__device__ __forceinline__ void load_codes(uint32_t (&w)[BITS], const uint32_t* p) {
    if constexpr (BITS == 4) {
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3])
                     : "l"(p));
    } else if constexpr (BITS == 2) {
        asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];\n" : "=r"(w[0]), "=r"(w[1]) : "l"(p));
    } else {
        w[0] = __ldg(p);
        w[1] = __ldg(p + 1);
        w[2] = __ldg(p + 2);
    }
}

// General path: grid (row tiles of 128, 1, token chunks of 32); every warp streams the codes of its
// 16 rows over the whole K range with a register ring and writes its outputs directly.
template <int BITS, int NT>
__global__ void __launch_bounds__(kThreads)
decode_kernel(const DecodeParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int kTok = NT * 8;
    const int panel_cols = p.panel_steps * 64;
    const int xs_stride = panel_cols + 8;  // bf16 elements; +16 bytes makes the fragment loads conflict-free
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    float* ss = reinterpret_cast<float*>(smem_raw + (size_t)kTok * xs_stride * 2);  // [kTok][panel_steps]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, tg = lane & 3;
    const int mtile = blockIdx.x;
    const int tok0 = blockIdx.z * kDecodeMaxT;
    const int tc = min(kTok, p.T - tok0);  // live tokens of this CTA
    const int row0 = mtile * kRowsPerCta + warp * 16;
    const bool active = row0 < p.m;
    const int nsteps = p.n >> 6;
    const int s_begin = 0, s_end = p.slice_steps;

    float yacc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) yacc[nt][i] = 0.0f;

    // Register ring of code words and (scale, zero) pairs, kPrefetch steps deep.  The layer's own
    // data does not depend on the previous kernel, so the first loads are issued before the wait.
    uint32_t wbuf[kPrefetch][BITS];
    uint32_t szbuf[kPrefetch][2];
    const uint32_t* wbase = p.codes + ((size_t)(row0 >> 4) * nsteps * 32 + lane) * BITS;
    const uint32_t* szbase = p.sz + (size_t)(row0 >> 4) * p.ng * 16 + gq;
    auto issue = [&](int slot, int s) {
        load_codes<BITS>(wbuf[slot], wbase + (size_t)s * 32 * BITS);
        const uint32_t* q = szbase + (size_t)(s >> p.gshift) * 16;
        szbuf[slot][0] = __ldg(q);
        szbuf[slot][1] = __ldg(q + 8);
    };
    if (active) {
#pragma unroll
        for (int i = 0; i < kPrefetch; ++i)
            if (s_begin + i < s_end) issue(i, s_begin + i);
    }

    const uint32_t xs_u32 = (uint32_t)__cvta_generic_to_shared(xs);
    // ldmatrix row address of this lane: matrix i = lane / 8 covers columns [8 i, 8 i + 8) of a
    // 32-column span, row = token lane % 8.
    const uint32_t ldm_off = (uint32_t)((lane & 7) * xs_stride + (lane >> 3) * 8) * 2u;

    for (int ps = s_begin; ps < s_end; ps += p.panel_steps) {
        const int pe = min(ps + p.panel_steps, s_end);
        const int pcols = (pe - ps) * 64;
        __syncthreads();
        // stage the rotated activations and their 64-column sums of this panel
        for (int i = tid; i < kTok * (pcols / 8); i += kThreads) {
            const int tk = i / (pcols / 8), c = i % (pcols / 8);
            uint4 v = make_uint4(0, 0, 0, 0);
            if (tk < tc) v = __ldcg(reinterpret_cast<const uint4*>(p.xrot + (size_t)(tok0 + tk) * p.n + ps * 64) + c);
            *reinterpret_cast<uint4*>(xs + (size_t)tk * xs_stride + c * 8) = v;
        }
        for (int i = tid; i < kTok * (pe - ps); i += kThreads) {
            const int tk = i / (pe - ps), st = i % (pe - ps);
            ss[tk * p.panel_steps + st] = tk < tc ? __ldcg(p.s64 + (size_t)(tok0 + tk) * p.s64_stride + ps + st) : 0.0f;
        }
        __syncthreads();
        if (!active) continue;

        for (int s0 = ps; s0 < pe; s0 += kPrefetch) {
#pragma unroll
            for (int i = 0; i < kPrefetch; ++i) {
                const int s = s0 + i;
                if (s < pe) {
                    uint32_t w[BITS];
#pragma unroll
                    for (int b = 0; b < BITS; ++b) w[b] = wbuf[i][b];
                    const uint32_t sz_lo = szbuf[i][0], sz_hi = szbuf[i][1];
                    if (s + kPrefetch < s_end) issue(i, s + kPrefetch);

                    uint32_t a[16];
                    expand_codes<BITS>(a, w);
                    const float2 f_lo = __half22float2(*reinterpret_cast<const __half2*>(&sz_lo));
                    const float2 f_hi = __half22float2(*reinterpret_cast<const __half2*>(&sz_hi));
                    const float nsz_lo = -f_lo.x * (128.0f + f_lo.y), nsz_hi = -f_hi.x * (128.0f + f_hi.y);
                    const int sl = s - ps;  // step inside the panel
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                        uint32_t b[4];
                        const uint32_t base = xs_u32 + (uint32_t)(nt * 8 * xs_stride + sl * 64) * 2u + ldm_off;
                        ldmatrix_x4(b, base);
                        mma_bf16(acc, *reinterpret_cast<const uint32_t(*)[4]>(&a[0]), b[0], b[1]);
                        mma_bf16(acc, *reinterpret_cast<const uint32_t(*)[4]>(&a[4]), b[2], b[3]);
                        ldmatrix_x4(b, base + 64u);
                        mma_bf16(acc, *reinterpret_cast<const uint32_t(*)[4]>(&a[8]), b[0], b[1]);
                        mma_bf16(acc, *reinterpret_cast<const uint32_t(*)[4]>(&a[12]), b[2], b[3]);
                        const float sx0 = ss[(nt * 8 + 2 * tg) * p.panel_steps + sl];
                        const float sx1 = ss[(nt * 8 + 2 * tg + 1) * p.panel_steps + sl];
                        yacc[nt][0] = fmaf(f_lo.x, acc[0], fmaf(nsz_lo, sx0, yacc[nt][0]));
                        yacc[nt][1] = fmaf(f_lo.x, acc[1], fmaf(nsz_lo, sx1, yacc[nt][1]));
                        yacc[nt][2] = fmaf(f_hi.x, acc[2], fmaf(nsz_hi, sx0, yacc[nt][2]));
                        yacc[nt][3] = fmaf(f_hi.x, acc[3], fmaf(nsz_hi, sx1, yacc[nt][3]));
                    }
                }
            }
        }
    }

    // low-rank up-projection A t (fp16 tensor-core product, fp32 sum)
    if (active && p.r_pad > 0) {
        const __half* arow_lo = p.A + (size_t)(row0 + gq) * p.r_pad + 2 * tg;
        const __half* arow_hi = arow_lo + (size_t)8 * p.r_pad;
        for (int jj = 0; jj < p.r_pad; jj += 16) {
            uint32_t a[4];
            a[0] = __ldg(reinterpret_cast<const uint32_t*>(arow_lo + jj));
            a[1] = __ldg(reinterpret_cast<const uint32_t*>(arow_hi + jj));
            a[2] = __ldg(reinterpret_cast<const uint32_t*>(arow_lo + jj + 8));
            a[3] = __ldg(reinterpret_cast<const uint32_t*>(arow_hi + jj + 8));
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                uint32_t b0 = 0, b1 = 0;
                if (nt * 8 + gq < tc) {
                    const __half* trow = p.t + (size_t)(tok0 + nt * 8 + gq) * p.r_pad + jj + 2 * tg;
                    b0 = __ldcg(reinterpret_cast<const uint32_t*>(trow));
                    b1 = __ldcg(reinterpret_cast<const uint32_t*>(trow + 8));
                }
                mma_f16(yacc[nt], a, b0, b1);
            }
        }
    }

    // ---- write-out ---------------------------------------------------------------------------
    // accumulator element (nt, i): token nt*8 + 2 tg + (i & 1), row row0 + gq + 8 (i >> 1)
    if (active) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int tk = nt * 8 + 2 * tg + (i & 1), row = row0 + gq + 8 * (i >> 1);
                if (tk < tc) {
                    const size_t o = (size_t)(tok0 + tk) * p.ldy + row;
                    if (p.out_f32) reinterpret_cast<float*>(p.y)[o] = yacc[nt][i];
                    else reinterpret_cast<__nv_bfloat16*>(p.y)[o] = __float2bfloat16_rn(yacc[nt][i]);
                }
            }
    }
}

template <int BITS, int NT>
cudaError_t launch_nt(const DecodeParams& p, dim3 grid, cudaStream_t s) {
    const size_t smem = (size_t)NT * 8 * (p.panel_steps * 64 + 8) * 2 + (size_t)NT * 8 * p.panel_steps * 4;
    static unsigned long long attr_done = 0;
    constexpr int kMaxPanel = NT == 4 ? 16 : 32;
    constexpr int kMaxSmem = NT * 8 * (kMaxPanel * 64 + 8) * 2 + NT * 8 * kMaxPanel * 4;
    cudaError_t e = ensure_dynamic_smem(decode_kernel<BITS, NT>, kMaxSmem, &attr_done);
    if (e != cudaSuccess) return e;
    decode_kernel<BITS, NT><<<grid, kThreads, smem, s>>>(p);
    return cudaGetLastError();
}

template <int BITS>
cudaError_t launch_bits(const DecodeParams& p, int nt, dim3 grid, cudaStream_t s) {
    if (nt == 1) return launch_nt<BITS, 1>(p, grid, s);
    if (nt == 2) return launch_nt<BITS, 2>(p, grid, s);
    return launch_nt<BITS, 4>(p, grid, s);
}

}  // namespace

cudaError_t launch_decode(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, const uint8_t* ws,
                          const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int T, cudaStream_t s) {
    DecodeParams p;
    p.codes = reinterpret_cast<const uint32_t*>(blob + L.off[LOPRO_SEC_CODES]);
    p.sz = reinterpret_cast<const uint32_t*>(blob + L.off[LOPRO_SEC_SCALEZERO]);
    p.A = reinterpret_cast<const __half*>(blob + L.off[LOPRO_SEC_A]);
    p.xrot = reinterpret_cast<const __nv_bfloat16*>(ws + W.off_xrot);
    p.s64 = reinterpret_cast<const float*>(ws + W.off_s64);
    p.s64_stride = s64_stride(d.d_in);
    p.t = reinterpret_cast<const __half*>(ws + W.off_t);
    p.y = y;
    p.ldy = ldy;
    p.out_f32 = out_dtype == LOPRO_OUT_F32;
    p.m = d.d_out;
    p.n = d.d_in;
    p.T = T;
    int gs = d.group_size / 64, gshift = 0;
    while ((1 << gshift) < gs) ++gshift;
    p.gshift = gshift;
    p.ng = d.d_in / d.group_size;
    p.r_pad = d.rank > 0 ? L.r_pad : 0;
    p.slice_steps = d.d_in / 64;
    const int zc = (T + kDecodeMaxT - 1) / kDecodeMaxT;
    const int tl = T < kDecodeMaxT ? T : kDecodeMaxT;
    const int nt = tl <= 8 ? 1 : (tl <= 16 ? 2 : 4);
    const int max_panel = nt == 4 ? 16 : 32;  // 1024 or 2048 columns of x~ per panel
    p.panel_steps = p.slice_steps < max_panel ? round_up_int(p.slice_steps, kPrefetch) : max_panel;
    const int mt = (d.d_out + kRowsPerCta - 1) / kRowsPerCta;
    if (zc > 65535) return cudaErrorInvalidValue;
    dim3 grid(mt, 1, zc);
    switch (d.bits) {
        case 2: return launch_bits<2>(p, nt, grid, s);
        case 3: return launch_bits<3>(p, nt, grid, s);
        default: return launch_bits<4>(p, nt, grid, s);
    }
}

}  // namespace lopro
