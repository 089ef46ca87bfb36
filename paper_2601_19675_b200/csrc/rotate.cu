// Activation-side transform x~ = Q^T P^T x (Eq. 8; Eq. 5 permutation, Eq. 6 partial block
// Walsh-Hadamard rotation with the Sylvester recursion of Eq. 2), and the low-rank
// down-projection t = B x (Appendix A.3, "Y = V X").
#include <math.h>

#include "common.cuh"
#include "ptx.cuh"
#include "rotate_body.cuh"
#include "rotate_mma.cuh"

namespace lopro {

namespace {

template <int E, int TOK, bool DIRECT>
__global__ void __launch_bounds__(kRotThreads)
rotate_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, const int32_t* __restrict__ perm,
              __nv_bfloat16* __restrict__ xrot, int64_t ldo, float* __restrict__ s64, int s64_ld,
              int* __restrict__ status, int n, int b_i, int b_h, float inv_sqrt_bh, int T) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    rotate_body<E, TOK, DIRECT>(smem_raw, (int)blockIdx.x, x, ldx, perm, xrot, ldo, s64, s64_ld, status, n, b_i, b_h,
                                inv_sqrt_bh, T);
}

// t[tok][j] = sum_k B[j][k] x[tok][k]: one warp per row j of B and eight tokens, fp32 accumulation,
// one rounding to fp16.  Rows j >= rank of the padded B are zero and give t = 0.
__global__ void __launch_bounds__(256)
lowrank_down_kernel(const __half* __restrict__ B, const __nv_bfloat16* __restrict__ x, int64_t ldx,
                    __half* __restrict__ t, int n, int r_pad, int T) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int j = blockIdx.x * 8 + warp;
    const int tok0 = blockIdx.y * 8;
    if (j >= r_pad) return;
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
    const uint4* brow = reinterpret_cast<const uint4*>(B + (size_t)j * n);
    for (int c = lane; c < n / 8; c += 32) {
        const uint4 bw = __ldg(brow + c);
        const __half2* bh = reinterpret_cast<const __half2*>(&bw);
        float bf[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(bh[i]);
            bf[2 * i] = f.x;
            bf[2 * i + 1] = f.y;
        }
#pragma unroll
        for (int tk = 0; tk < 8; ++tk) {
            if (tok0 + tk < T) {
                const uint4 xw = __ldg(reinterpret_cast<const uint4*>(x + (size_t)(tok0 + tk) * ldx) + c);
                const __nv_bfloat162* xh = reinterpret_cast<const __nv_bfloat162*>(&xw);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 f = __bfloat1622float2(xh[i]);
                    acc[tk] = fmaf(bf[2 * i], f.x, acc[tk]);
                    acc[tk] = fmaf(bf[2 * i + 1], f.y, acc[tk]);
                }
            }
        }
    }
#pragma unroll
    for (int tk = 0; tk < 8; ++tk) {
        float s = acc[tk];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
        if (lane == 0 && tok0 + tk < T) t[(size_t)(tok0 + tk) * r_pad + j] = __float2half_rn(s);
    }
}

// Pulls the 128-byte line at p into L2.  Layer data (perm, B) is requested this way before griddepcontrol.wait and
// loaded after it: loads issued before the wait were measured to delay the CTA's passage through the wait by
// 0.5-0.9 us, which cost more than the L2 hit afterwards.
__device__ __forceinline__ void prefetch_l2(const void* p) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// One row j of B against TPR tokens: t[token][j] = sum_k B[j][k] x[token][k], fp32 accumulation over all of K, one
// rounding to fp16.  The row of B is pulled into L2 before griddepcontrol.wait, every load of the first 4096 columns
// is in flight before the first use.  Fewer tokens per CTA mean more CTAs and less to load per SM: this chain decides
// when the prologue ends.
template <int TPR>
__device__ __forceinline__ void lowrank_row(const __nv_bfloat16* __restrict__ x, int64_t ldx, const __half* __restrict__ B,
                                            __half* __restrict__ t, int n, int r_pad, int T, int rb, int tok0,
                                            const ImageOut& img) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ float part[8][TPR];
    const int j = rb % r_pad, tq = tok0 + TPR * (rb / r_pad);
    const __half* brow = B + (size_t)j * n;
    const int npass = (n + 2047) >> 11;
    if ((tid & 7) == 0) {  // one request per 128-byte line of the first 4096 columns of the row
#pragma unroll
        for (int ps = 0; ps < 2; ++ps) {
            const int k = ps * 2048 + tid * 8;
            if (k < n) prefetch_l2(brow + k);
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    uint4 pre[2];
#pragma unroll
    for (int ps = 0; ps < 2; ++ps) {
        const int k = ps * 2048 + tid * 8;
        pre[ps] = k < n ? __ldg(reinterpret_cast<const uint4*>(brow + k)) : make_uint4(0, 0, 0, 0);
    }
    float acc[TPR];
#pragma unroll
    for (int tk = 0; tk < TPR; ++tk) acc[tk] = 0.0f;
    auto load_x = [&](uint4 (&xw)[TPR], int k) {
#pragma unroll
        for (int tk = 0; tk < TPR; ++tk)
            xw[tk] = (k < n && tq + tk < T) ? __ldg(reinterpret_cast<const uint4*>(x + (size_t)(tq + tk) * ldx + k))
                                            : make_uint4(0, 0, 0, 0);
    };
    auto accumulate = [&](const uint4& bw, const uint4 (&xw)[TPR]) {
        float bf[8];
        const __half2* h = reinterpret_cast<const __half2*>(&bw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(h[i]);
            bf[2 * i] = f.x;
            bf[2 * i + 1] = f.y;
        }
#pragma unroll
        for (int tk = 0; tk < TPR; ++tk) {
            const __nv_bfloat162* xh = reinterpret_cast<const __nv_bfloat162*>(&xw[tk]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __bfloat1622float2(xh[i]);
                acc[tk] = fmaf(bf[2 * i], f.x, acc[tk]);
                acc[tk] = fmaf(bf[2 * i + 1], f.y, acc[tk]);
            }
        }
    };
    {   // the first two passes (all of K up to 4096 columns): every load is in flight before the first use,
        // so the dependent chain after the wait is one memory round trip
        uint4 x0[TPR], x1[TPR];
        load_x(x0, tid * 8);
        load_x(x1, 2048 + tid * 8);
        accumulate(pre[0], x0);
        accumulate(pre[1], x1);
    }
    for (int ps = 2; ps < npass; ++ps) {
        const int k = ps * 2048 + tid * 8;
        if (k >= n) break;
        uint4 xw[TPR];
        load_x(xw, k);
        accumulate(__ldg(reinterpret_cast<const uint4*>(brow + k)), xw);
    }
#pragma unroll
    for (int tk = 0; tk < TPR; ++tk) {
        float v = acc[tk];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
        if (lane == 0) part[warp][tk] = v;
    }
    __syncthreads();
    if (tid < TPR) {
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += part[w][tid];
        if (tq + tid < T) {
            const int tok = tq + tid;
            if (img.ximg == nullptr) {
                t[(size_t)tok * r_pad + j] = __float2half_rn(v);
            } else {
                // operand image: tile (token group, 64-column step of the rank), token row tl, swizzled 16-byte piece
                const int tgp = tok >> img.np_shift, tl = tok & (img.np - 1);
                unsigned char* tile = img.timg + ((size_t)tgp * img.lr_steps + (j >> 6)) * img.np * 128;
                *reinterpret_cast<__half*>(tile + tl * 128 + ((((j & 63) >> 3) ^ (tl & 7)) << 4) + (j & 7) * 2) =
                    __float2half_rn(v);
            }
        }
    }
}

// The same row job for the FP8 low-rank record (U, V, Sigma, s) that Algorithm 1 saves:
// t[token][j] = sigma[j] * sum_k V[j][k] * (x[token][k] / s[k]), V in fp8 e4m3 (exact in fp32), the quotient taken on
// the layer's side as V[j][k] * (1 / s[k]) in fp32 (once for all tokens), fp32 accumulation, one rounding to fp16.
template <int TPR>
__device__ __forceinline__ void lowrank_row_lr8(const __nv_bfloat16* __restrict__ x, int64_t ldx, const Lr8Args lr8,
                                                __half* __restrict__ t, int n, int r_pad, int T, int rb, int tok0) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ float part[8][TPR];
    const int j = rb % r_pad, tq = tok0 + TPR * (rb / r_pad);
    const uint8_t* vrow = lr8.V + (size_t)j * n;
    if ((tid & 15) == 0) {  // one request per 128-byte line of the first 4096 columns of the row of V; s likewise
#pragma unroll
        for (int ps = 0; ps < 2; ++ps) {
            const int k = ps * 2048 + tid * 8;
            if (k < n) prefetch_l2(vrow + k);
        }
    }
    if ((tid & 7) == 0) {
#pragma unroll
        for (int ps = 0; ps < 2; ++ps) {
            const int k = ps * 2048 + tid * 8;
            if (k < n) prefetch_l2(lr8.svec + k);
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float acc[TPR];
#pragma unroll
    for (int tk = 0; tk < TPR; ++tk) acc[tk] = 0.0f;
    auto load_x = [&](uint4 (&xw)[TPR], int k) {
#pragma unroll
        for (int tk = 0; tk < TPR; ++tk)
            xw[tk] = (k < n && tq + tk < T) ? __ldg(reinterpret_cast<const uint4*>(x + (size_t)(tq + tk) * ldx + k))
                                            : make_uint4(0, 0, 0, 0);
    };
    auto accumulate = [&](const uint2& vw, const uint4& sw, const uint4 (&xw)[TPR]) {
        float vs[8];  // V[j][k] / s[k]
        const uint32_t vv[2] = {vw.x, vw.y};
        const __half2* sh = reinterpret_cast<const __half2*>(&sw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t h2 = e4m3x2_to_f16x2((uint16_t)(vv[i >> 1] >> (16 * (i & 1))));
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h2));
            const float2 sf = __half22float2(sh[i]);
            vs[2 * i] = f.x * __frcp_rn(sf.x);
            vs[2 * i + 1] = f.y * __frcp_rn(sf.y);
        }
#pragma unroll
        for (int tk = 0; tk < TPR; ++tk) {
            const __nv_bfloat162* xh = reinterpret_cast<const __nv_bfloat162*>(&xw[tk]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __bfloat1622float2(xh[i]);
                acc[tk] = fmaf(vs[2 * i], f.x, acc[tk]);
                acc[tk] = fmaf(vs[2 * i + 1], f.y, acc[tk]);
            }
        }
    };
    const uint4 one = make_uint4(0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u);  // s = 1 where there is no column
    {   // the first two passes (all of K up to 4096 columns): every load in flight before the first use
        uint2 v0 = make_uint2(0, 0), v1 = make_uint2(0, 0);
        uint4 s0 = one, s1 = one, x0[TPR], x1[TPR];
        const int k0 = tid * 8, k1 = 2048 + tid * 8;
        if (k0 < n) {
            v0 = __ldg(reinterpret_cast<const uint2*>(vrow + k0));
            s0 = __ldg(reinterpret_cast<const uint4*>(lr8.svec + k0));
        }
        if (k1 < n) {
            v1 = __ldg(reinterpret_cast<const uint2*>(vrow + k1));
            s1 = __ldg(reinterpret_cast<const uint4*>(lr8.svec + k1));
        }
        load_x(x0, k0);
        load_x(x1, k1);
        accumulate(v0, s0, x0);
        accumulate(v1, s1, x1);
    }
    for (int k = 4096 + tid * 8; k < n; k += 2048) {
        uint4 xw[TPR];
        load_x(xw, k);
        accumulate(__ldg(reinterpret_cast<const uint2*>(vrow + k)), __ldg(reinterpret_cast<const uint4*>(lr8.svec + k)), xw);
    }
#pragma unroll
    for (int tk = 0; tk < TPR; ++tk) {
        float v = acc[tk];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
        if (lane == 0) part[warp][tk] = v;
    }
    __syncthreads();
    if (tid < TPR) {
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += part[w][tid];
        if (tq + tid < T) t[(size_t)(tq + tid) * r_pad + j] = __float2half_rn(v * __half2float(lr8.sigma[j]));
    }
}

// Tail of the prologue's rotation for one (token, chunk of 256 output columns) pair of a warp: v holds the 8
// gathered entries of the lane.  Register and shuffle butterflies, rounding to bf16, and the store of the entries
// and of their 64-column sums into the record of (stage, token) in the activation image.
__device__ __forceinline__ void rotate_tail(const float (&v)[8], unsigned char* __restrict__ act_image, int n, int b_i,
                                            int b_h, float inv_sqrt_bh, int t_pad, int tok, int col0, int lane,
                                            const ImageOut& img) {
    const bool rot = col0 >= b_i;  // whole Hadamard blocks lie on one side of b_I
    float r[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) r[e] = v[e];
#pragma unroll
    for (int h = 1; h < 8; h <<= 1) {
        if (h < b_h) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if ((e & h) == 0) {
                    const float a = r[e], b = r[e + h];
                    r[e] = a + b;
                    r[e + h] = a - b;
                }
            }
        }
    }
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        if (d * 8 < b_h) {
            const bool upper = (lane & d) != 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float other = __shfl_xor_sync(0xffffffffu, r[e], d);
                r[e] = upper ? other - r[e] : r[e] + other;
            }
        }
    }
    __nv_bfloat16 o[8];
    float sum = 0.0f;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        o[e] = rot ? __float2bfloat16_rn(r[e] * inv_sqrt_bh) : __float2bfloat16_rn(v[e]);
        sum += __bfloat162float(o[e]);
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    sum += __shfl_xor_sync(0xffffffffu, sum, 4);
    if (img.ximg != nullptr) {
        // operand image of the tcgen05 kernel: swizzled 16-byte piece of the (token group, step) tile, and the sum
        // over the run of 64, 128 or 256 columns (a warp's chunk of 256 columns holds whole runs)
        if (img.gs_shift >= 1) sum += __shfl_xor_sync(0xffffffffu, sum, 8);
        if (img.gs_shift >= 2) sum += __shfl_xor_sync(0xffffffffu, sum, 16);
        if (col0 < n) {
            const int tgp = tok >> img.np_shift, tl = tok & (img.np - 1);
            unsigned char* tile = img.ximg + ((size_t)tgp * img.nsteps + (col0 >> 6)) * img.np * 128;
            *reinterpret_cast<uint4*>(tile + tl * 128 + ((((col0 & 63) >> 3) ^ (tl & 7)) << 4)) =
                *reinterpret_cast<const uint4*>(o);
            if ((lane & ((8 << img.gs_shift) - 1)) == 0)
                img.sums[((size_t)tgp * img.n_sums + (col0 >> (6 + img.gs_shift))) * img.np + tl] = sum;
        }
        return;
    }
    if (col0 < n) {
        // record of (stage, token) in the activation image: 1024 entries, then the 16 sums
        unsigned char* rec = act_image + ((size_t)(col0 >> 10) * t_pad + tok) * kActRecord;
        *reinterpret_cast<uint4*>(rec + (col0 & 1023) * 2) = *reinterpret_cast<const uint4*>(o);
        if ((lane & 7) == 0) reinterpret_cast<float*>(rec + 2048)[(col0 & 1023) >> 6] = sum;
    }
}

constexpr int kPrologueMaxSmem = 200 * 1024;  // one row of x: d_in <= 102400

// Prologue of the small-batch forward (T <= 32, b_H <= 256, b_I a multiple of b_H).  Grid:
// x = the rows of B (8 / tpr CTAs each), then the rotation CTAs; y = groups of 8 tokens.
//  * a rotation CTA takes one token and 8 chunks of 256 output columns, warp w for chunk w (STAGED: the
//    token's row of x is copied to dynamic shared memory, 2 * d_in bytes, and the 8 entries of a lane are
//    gathered from there through perm), or one chunk and 8 tokens, warp w for token w (gather straight from
//    global memory); the entries are transformed with register and shuffle butterflies, rounded to bf16 and
//    stored together with their 64-column sums in the activation image that the streaming kernel copies to
//    shared memory;
//  * a row CTA computes t[token][j] = sum_k B[j][k] x[token][k] for one row j of B and `tpr` of the 8 tokens
//    (8 / tpr CTAs per row): the low-rank intermediate "Y = V X".
// Launched with programmatic stream serialization: perm and B (layer data) are pulled into L2 before the
// wait, everything is loaded after it.
// A launch for a single layer carries no sibling table (several hundred bytes of kernel parameters less).
struct NoPrologueSiblings {};
__device__ __forceinline__ void select_prologue_sibling(const NoPrologueSiblings&, const int32_t*&, const __half*&,
                                                        unsigned char*&, __half*&, const __nv_bfloat16*&, int&) {}
__device__ __forceinline__ void select_prologue_sibling(const PrologueSiblings& sibs, const int32_t*& perm, const __half*& B,
                                                        unsigned char*& act_image, __half*& t, const __nv_bfloat16*& x,
                                                        int& T) {
    // (a __grid_constant__ parameter: one constant-bank load per field at a computed index)
    const int z = (int)blockIdx.z;
    if (z > 0) {
        perm = sibs.perm[z - 1];
        B = sibs.B[z - 1];
        act_image = sibs.act[z - 1];
        t = sibs.t[z - 1];
    }
    if (sibs.own_rows) {
        x = sibs.x_of[z];
        T = sibs.T_of[z];
    }
}

template <bool STAGED, typename SIBS>
__global__ void __launch_bounds__(256)
prologue_kernel(const __nv_bfloat16* __restrict__ x0, int64_t ldx, const int32_t* __restrict__ perm0,
                const __half* __restrict__ B0, unsigned char* __restrict__ act_image0, __half* __restrict__ t0,
                int* __restrict__ status, int n, int b_i, int b_h, float inv_sqrt_bh, int r_pad, int t_pad, int T_grid,
                int tpr, const ImageOut img, const __grid_constant__ SIBS sibs, const Lr8Args lr8) {
    // sibling layers (grid z): the same x (or each its own rows), each layer its own permutation, B and outputs
    const int32_t* perm = perm0;
    const __half* B = B0;
    unsigned char* act_image = act_image0;
    __half* t = t0;
    const __nv_bfloat16* x = x0;
    int T = T_grid;  // T_grid shapes the grid; T is the number of token rows of this CTA's layer
    select_prologue_sibling(sibs, perm, B, act_image, t, x, T);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nchunks = (n + 255) >> 8;
    const int tok0 = blockIdx.y * 8;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int live = T_grid < 8 ? T_grid : 8;
    // the row CTAs come first in the grid, the rotation CTAs last
    const int nrow = (int)gridDim.x - (STAGED ? live * ((nchunks + 7) >> 3) : nchunks);
    if ((int)blockIdx.x < nrow) {
        const int rb = (int)blockIdx.x;
        if (lr8.V != nullptr) {
            if (tpr == 8) lowrank_row_lr8<8>(x, ldx, lr8, t, n, r_pad, T, rb, tok0);
            else if (tpr == 4) lowrank_row_lr8<4>(x, ldx, lr8, t, n, r_pad, T, rb, tok0);
            else if (tpr == 2) lowrank_row_lr8<2>(x, ldx, lr8, t, n, r_pad, T, rb, tok0);
            else lowrank_row_lr8<1>(x, ldx, lr8, t, n, r_pad, T, rb, tok0);
            return;
        }
        if (tpr == 8) lowrank_row<8>(x, ldx, B, t, n, r_pad, T, rb, tok0, img);
        else if (tpr == 4) lowrank_row<4>(x, ldx, B, t, n, r_pad, T, rb, tok0, img);
        else if (tpr == 2) lowrank_row<2>(x, ldx, B, t, n, r_pad, T, rb, tok0, img);
        else lowrank_row<1>(x, ldx, B, t, n, r_pad, T, rb, tok0, img);
        return;
    }

    // ---- rotation ----
    const int c = (int)blockIdx.x - nrow;
    if constexpr (!STAGED) {
        // one chunk of 256 output columns, warp w for token w; gather straight from global memory
        const int col0 = c * 256 + lane * 8;
        if (warp == 0 && (lane & 3) == 0 && col0 < n) prefetch_l2(perm + col0);  // the chunk's 1 KB of perm
        asm volatile("griddepcontrol.wait;" ::: "memory");
        int pidx[8];
        if (col0 < n) {
            const int4 p0 = __ldg(reinterpret_cast<const int4*>(perm + col0));
            const int4 p1 = __ldg(reinterpret_cast<const int4*>(perm + col0 + 4));
            pidx[0] = p0.x; pidx[1] = p0.y; pidx[2] = p0.z; pidx[3] = p0.w;
            pidx[4] = p1.x; pidx[5] = p1.y; pidx[6] = p1.z; pidx[7] = p1.w;
        }
        if (c == 0 && tok0 == 0 && blockIdx.z == 0) {
            if (status != nullptr && tid == 0) *status = LOPRO_OK;
            if (img.ximg != nullptr)
                for (int i = tid; i < img.n_counters; i += 256) img.counters[i] = 0;
        }
        const int tok = tok0 + warp;
        if (tok < T) {
            float v[8];
            const __nv_bfloat16* xrow = x + (size_t)tok * ldx;
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = col0 < n ? __bfloat162float(xrow[pidx[e]]) : 0.0f;
            rotate_tail(v, act_image, n, b_i, b_h, inv_sqrt_bh, t_pad, tok, col0, lane, img);
        }
    } else {
        // one token, 8 chunks: warp w takes chunk 8 * (c / live) + w.  perm and the token's row of x are independent
        // loads: one memory round trip, then the gather runs in shared memory
        extern __shared__ __align__(16) unsigned char prologue_smem[];
        __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(prologue_smem);
        const int tok = tok0 + c % live;
        const int col0 = ((c / live) * 8 + warp) * 256 + lane * 8;
        if ((lane & 3) == 0 && col0 < n) prefetch_l2(perm + col0);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (tok >= T) return;  // the whole CTA
        int pidx[8];
        if (col0 < n) {
            const int4 p0 = __ldg(reinterpret_cast<const int4*>(perm + col0));
            const int4 p1 = __ldg(reinterpret_cast<const int4*>(perm + col0 + 4));
            pidx[0] = p0.x; pidx[1] = p0.y; pidx[2] = p0.z; pidx[3] = p0.w;
            pidx[4] = p1.x; pidx[5] = p1.y; pidx[6] = p1.z; pidx[7] = p1.w;
        }
        const __nv_bfloat16* xrow = x + (size_t)tok * ldx;
        for (int base = 0; base < n; base += 4 * 2048) {
            uint4 w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k = base + i * 2048 + tid * 8;
                if (k < n) w[i] = __ldg(reinterpret_cast<const uint4*>(xrow + k));
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k = base + i * 2048 + tid * 8;
                if (k < n) *reinterpret_cast<uint4*>(xs + k) = w[i];
            }
        }
        __syncthreads();
        if (c == 0 && tok0 == 0 && blockIdx.z == 0) {  // (token 0 exists: T >= 1)
            if (status != nullptr && tid == 0) *status = LOPRO_OK;
            if (img.ximg != nullptr)
                for (int i = tid; i < img.n_counters; i += 256) img.counters[i] = 0;
        }
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = col0 < n ? __bfloat162float(xs[pidx[e]]) : 0.0f;
        rotate_tail(v, act_image, n, b_i, b_h, inv_sqrt_bh, t_pad, tok, col0, lane, img);
    }
}

template <int E, int TOK, bool DIRECT>
cudaError_t launch_rotate_etd(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                              __nv_bfloat16* xrot, int64_t ldo, float* s64, int* status, int T, cudaStream_t s) {
    const size_t smem = (size_t)d.d_in * (DIRECT ? 2 : 4) * TOK;
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(rotate_kernel<E, TOK, DIRECT>, TOK == 1 ? 32768 * 4 : 160 * 1024, &attr_done);
    if (e != cudaSuccess) return e;
    const float inv = (float)(1.0 / sqrt((double)d.block_size));
    rotate_kernel<E, TOK, DIRECT><<<(T + TOK - 1) / TOK, kRotThreads, smem, s>>>(
        x, ldx, perm, xrot, ldo, s64, s64_stride(d.d_in), status, d.d_in, d.identity_cols, d.block_size, inv, T);
    return cudaGetLastError();
}

// Results go straight from registers to global memory when the identity prefix ends on a 64-column step
// (16-byte stores and whole steps per lane group); otherwise they are collected in shared memory first.
// Four rows per CTA when there are many tokens and the rows fit shared memory, else one.
template <int E>
cudaError_t launch_rotate_e(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                            __nv_bfloat16* xrot, int64_t ldo, float* s64, int* status, int T, cudaStream_t s) {
    const bool direct = d.identity_cols % 64 == 0;
    const bool four = T >= 256 && (size_t)d.d_in * (direct ? 8 : 16) <= 160 * 1024;
    if (direct)
        return four ? launch_rotate_etd<E, 4, true>(d, perm, x, ldx, xrot, ldo, s64, status, T, s)
                    : launch_rotate_etd<E, 1, true>(d, perm, x, ldx, xrot, ldo, s64, status, T, s);
    return four ? launch_rotate_etd<E, 4, false>(d, perm, x, ldx, xrot, ldo, s64, status, T, s)
                : launch_rotate_etd<E, 1, false>(d, perm, x, ldx, xrot, ldo, s64, status, T, s);
}

}  // namespace

namespace {

template <int TOK>
__global__ void __launch_bounds__(256, 2)
rotate_mma_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, const int32_t* __restrict__ perm,
                  __nv_bfloat16* __restrict__ xrot, int64_t ldo, int* __restrict__ status, int n, int b_i, int b_h,
                  float inv_sqrt_bh, int T) {
    extern __shared__ __align__(16) unsigned char rot_smem[];
    rotate_mma_body<TOK>(rot_smem, (int)blockIdx.x, x, ldx, perm, xrot, ldo, status, n, b_i, b_h, inv_sqrt_bh, T);
}

template <int TOK>
cudaError_t launch_rotate_mma(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                              __nv_bfloat16* xrot, int64_t ldo, int* status, int T, cudaStream_t s) {
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(rotate_mma_kernel<TOK>, kRotMmaMaxSmem, &attr_done);
    if (e != cudaSuccess) return e;
    const float inv = (float)(1.0 / sqrt((double)d.block_size));
    rotate_mma_kernel<TOK><<<(T + TOK - 1) / TOK, 256, rotate_mma_smem_bytes(TOK, d.d_in), s>>>(
        x, ldx, perm, xrot, ldo, status, d.d_in, d.identity_cols, d.block_size, inv, T);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_rotate(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                          __nv_bfloat16* xrot, int64_t ldo, float* s64, int* status, int T, cudaStream_t s) {
    // many rows and no column sums wanted: the tensor-core form of the recursion, eight (or four) rows per CTA
    if (s64 == nullptr && T >= 16 && rotate_mma_shape_ok(d) && (reinterpret_cast<uintptr_t>(perm) % 16) == 0) {
        if (rotate_mma_smem_bytes(8, d.d_in) <= (size_t)kRotMmaMaxSmem / 2)
            return launch_rotate_mma<8>(d, perm, x, ldx, xrot, ldo, status, T, s);
        if (rotate_mma_smem_bytes(4, d.d_in) <= (size_t)kRotMmaMaxSmem)
            return launch_rotate_mma<4>(d, perm, x, ldx, xrot, ldo, status, T, s);
    }
    if (d.block_size <= 256) return launch_rotate_e<8>(d, perm, x, ldx, xrot, ldo, s64, status, T, s);
    if (d.block_size == 512) return launch_rotate_e<16>(d, perm, x, ldx, xrot, ldo, s64, status, T, s);
    return launch_rotate_e<32>(d, perm, x, ldx, xrot, ldo, s64, status, T, s);
}

bool prologue_supported(const lopro_desc& d, int T) {
    return T <= kDecodeMaxT && d.block_size <= 256 && d.identity_cols % d.block_size == 0 &&
           (size_t)d.d_in * 2 <= (size_t)kPrologueMaxSmem;
}

cudaError_t launch_prologue(const lopro_desc& d, const int32_t* perm, const __half* B, int r_pad,
                            const __nv_bfloat16* x, int64_t ldx, unsigned char* act_image, __half* t, int t_pad,
                            int* status, int T, cudaStream_t s, const ImageOut* img_out, const PrologueSiblings* siblings,
                            const Lr8Args* lr8_args) {
    const float inv = (float)(1.0 / sqrt((double)d.block_size));
    ImageOut img = {};
    if (img_out != nullptr) img = *img_out;
    PrologueSiblings sibs = {};
    if (siblings != nullptr) sibs = *siblings;
    Lr8Args lr8 = {};
    if (lr8_args != nullptr) lr8 = *lr8_args;
    cudaLaunchConfig_t cfg = {};
    // tokens per row CTA: as few as it takes to fill the SMs
    const int live = T < 8 ? T : 8;
    int tpr = 8;
    // (measured: with one group of tokens a CTA per (row, token) is best -- 256 CTAs for cfg2 --, with several
    // groups about one CTA per SM)
    const int want = T <= 8 ? 256 : 120;
    while (tpr > 1 && r_pad * ((live + tpr - 1) / tpr) * ((T + 7) / 8) < want) tpr >>= 1;
    const int row_ctas = d.rank > 0 ? r_pad * ((live + tpr - 1) / tpr) : 0;
    // rotation: a token's row of x is staged in shared memory and gathered from there; with very few (token,
    // chunk) pairs the gather straight from global memory, warp = token, is as fast (measured: 6.1 against 6.3 us
    // per layer forward for one token and 4096 columns, 15.4 against 16.9 us for 8 tokens and 11008 columns)
    const int nchunks = (d.d_in + 255) / 256, groups = (T + 7) / 8;
    const bool staged = nchunks * live * groups > 64;
    const int rot_ctas = staged ? live * ((nchunks + 7) / 8) : nchunks;
    if (staged && (size_t)d.d_in * 2 > 48 * 1024) {  // a row of x beyond the default limit
        static unsigned long long attr_done = 0;
        cudaError_t e = ensure_dynamic_smem(prologue_kernel<true, PrologueSiblings>, kPrologueMaxSmem, &attr_done);
        if (e == cudaSuccess) {
            static unsigned long long attr_done2 = 0;
            e = ensure_dynamic_smem(prologue_kernel<true, NoPrologueSiblings>, kPrologueMaxSmem, &attr_done2);
        }
        if (e != cudaSuccess) return e;
    }
    cfg.gridDim = dim3(row_ctas + rot_ctas, (T + 7) / 8, 1 + sibs.n);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = staged ? (size_t)d.d_in * 2 : 0;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    const int rp = d.rank > 0 ? r_pad : 0;
    if (sibs.n == 0 && !sibs.own_rows && option(LOPRO_OPT_ONE_KERNEL_SET) != 1) {
        const NoPrologueSiblings none;
        return staged ? cudaLaunchKernelEx(&cfg, prologue_kernel<true, NoPrologueSiblings>, x, ldx, perm, B, act_image, t, status,
                                           d.d_in, d.identity_cols, d.block_size, inv, rp, t_pad, T, tpr, img, none, lr8)
                      : cudaLaunchKernelEx(&cfg, prologue_kernel<false, NoPrologueSiblings>, x, ldx, perm, B, act_image, t, status,
                                           d.d_in, d.identity_cols, d.block_size, inv, rp, t_pad, T, tpr, img, none, lr8);
    }
    return staged ? cudaLaunchKernelEx(&cfg, prologue_kernel<true, PrologueSiblings>, x, ldx, perm, B, act_image, t, status, d.d_in,
                                       d.identity_cols, d.block_size, inv, rp, t_pad, T, tpr, img, sibs, lr8)
                  : cudaLaunchKernelEx(&cfg, prologue_kernel<false, PrologueSiblings>, x, ldx, perm, B, act_image, t, status, d.d_in,
                                       d.identity_cols, d.block_size, inv, rp, t_pad, T, tpr, img, sibs, lr8);
}

cudaError_t launch_lowrank_down(const lopro_desc& d, const __half* B, int r_pad, const __nv_bfloat16* x,
                                int64_t ldx, __half* t, int T, cudaStream_t s) {
    dim3 grid((r_pad + 7) / 8, (T + 7) / 8);
    lowrank_down_kernel<<<grid, 256, 0, s>>>(B, x, ldx, t, d.d_in, r_pad, T);
    return cudaGetLastError();
}

}  // namespace lopro
