// Low-rank down-projection t = B x for many tokens (Appendix A.3, "Y = V X"), on the tensor cores.
//
// x is bf16 and B is fp16; to keep the products exact each fp16 entry of B is split into two bf16
// numbers, B = B_hi + B_lo (the 11-bit significand of fp16 fits 8 + 8 bits), and both parts are
// multiplied with x by mma.sync with fp32 accumulation.  Grid: (128-token tiles, K slices); every
// CTA writes the fp32 partial sums of its K slice, a second small kernel adds the slices in order
// and rounds once to fp16.
#include <math.h>

#include "common.cuh"
#include "ptx.cuh"
#include "rotate_body.cuh"
#include "rotate_mma.cuh"

namespace lopro {

namespace {

constexpr int kLrThreads = 256;
constexpr int kLrTokens = 128;       // tokens per CTA (8 warps x 16)
constexpr int kLrChunk = 64;         // K columns staged per iteration
constexpr int kLrStride = kLrChunk + 8;  // bf16 elements per shared-memory row (+16 bytes: conflict-free ldmatrix)
constexpr int kLrMaxRank = 128;      // rows of B per CTA

// NJ = 8-wide column tiles of the output handled per CTA (rows of B / 8)
template <int NJ>
__device__ __forceinline__ void lowrank_body(unsigned char* smem_raw, int bx, int by, const __half* __restrict__ B,
                                             const __nv_bfloat16* __restrict__ x, int64_t ldx,
                                             float* __restrict__ partial, int n, int r_pad, int T, int j0,
                                             int slice_cols) {
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);   // [128][kLrStride]
    __nv_bfloat16* bh = xs + kLrTokens * kLrStride;                    // [NJ*8][kLrStride]
    __nv_bfloat16* bl = bh + NJ * 8 * kLrStride;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tok0 = bx * kLrTokens;
    const int kb = by * slice_cols, ke = min(n, kb + slice_cols);
    const int rows_b = min(NJ * 8, r_pad - j0);

    float acc[NJ][4];
#pragma unroll
    for (int j = 0; j < NJ; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[j][i] = 0.0f;

    const uint32_t xs_u = (uint32_t)__cvta_generic_to_shared(xs);
    const uint32_t bh_u = (uint32_t)__cvta_generic_to_shared(bh), bl_u = (uint32_t)__cvta_generic_to_shared(bl);
    // ldmatrix lane addresses: A operand (16 tokens x 16 columns), B operand (16 rows of B x 16 columns)
    const uint32_t a_off = (uint32_t)((warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1)) * kLrStride + 8 * (lane >> 4)) * 2u;
    const uint32_t b_off = (uint32_t)(((lane & 7) + 8 * (lane >> 4)) * kLrStride + 8 * ((lane >> 3) & 1)) * 2u;

    // global loads of one 64-column chunk, kept in registers while the previous chunk is multiplied
    constexpr int kXPer = kLrTokens * 8 / kLrThreads;                     // 16-byte pieces of x per thread
    constexpr int kBPer = (NJ * 8 * 8 + kLrThreads - 1) / kLrThreads;     // 16-byte pieces of B per thread
    uint4 xr[kXPer], br[kBPer];
    auto load_chunk = [&](int k0) {
#pragma unroll
        for (int u = 0; u < kXPer; ++u) {
            const int i = tid + u * kLrThreads, r = i >> 3, c = i & 7;
            xr[u] = tok0 + r < T ? __ldg(reinterpret_cast<const uint4*>(x + (size_t)(tok0 + r) * ldx + k0) + c)
                                 : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kBPer; ++u) {
            const int i = tid + u * kLrThreads, r = i >> 3, c = i & 7;
            br[u] = (i < NJ * 64 && r < rows_b) ? __ldg(reinterpret_cast<const uint4*>(B + (size_t)(j0 + r) * n + k0) + c)
                                                : make_uint4(0, 0, 0, 0);
        }
    };
    if (kb < ke) load_chunk(kb);
    for (int k0 = kb; k0 < ke; k0 += kLrChunk) {
        __syncthreads();  // the previous chunk has been multiplied
#pragma unroll
        for (int u = 0; u < kXPer; ++u) {
            const int i = tid + u * kLrThreads, r = i >> 3, c = i & 7;
            *reinterpret_cast<uint4*>(xs + r * kLrStride + c * 8) = xr[u];
        }
        // rows of B: fp16 -> (hi, lo) bf16
#pragma unroll
        for (int u = 0; u < kBPer; ++u) {
            const int i = tid + u * kLrThreads, r = i >> 3, c = i & 7;
            if (i < NJ * 64) {
                const __half2* h = reinterpret_cast<const __half2*>(&br[u]);
                uint4 hi, lo;
                uint32_t* hp = reinterpret_cast<uint32_t*>(&hi);
                uint32_t* lp = reinterpret_cast<uint32_t*>(&lo);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __half22float2(h[e]);
                    const __nv_bfloat162 bhi = __floats2bfloat162_rn(f.x, f.y);
                    const float2 fh = __bfloat1622float2(bhi);
                    const __nv_bfloat162 blo = __floats2bfloat162_rn(f.x - fh.x, f.y - fh.y);  // exact remainder
                    hp[e] = *reinterpret_cast<const uint32_t*>(&bhi);
                    lp[e] = *reinterpret_cast<const uint32_t*>(&blo);
                }
                *reinterpret_cast<uint4*>(bh + r * kLrStride + c * 8) = hi;
                *reinterpret_cast<uint4*>(bl + r * kLrStride + c * 8) = lo;
            }
        }
        if (k0 + kLrChunk < ke) load_chunk(k0 + kLrChunk);  // in flight during the products below
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kLrChunk; kk += 16) {
            uint32_t a[4];
            ldmatrix_x4(a, xs_u + a_off + kk * 2);
#pragma unroll
            for (int jp = 0; jp < NJ / 2; ++jp) {
                uint32_t b[4];
                ldmatrix_x4(b, bh_u + b_off + (uint32_t)(jp * 16 * kLrStride + kk) * 2u);
                mma_bf16(acc[2 * jp], a, b[0], b[1]);
                mma_bf16(acc[2 * jp + 1], a, b[2], b[3]);
                ldmatrix_x4(b, bl_u + b_off + (uint32_t)(jp * 16 * kLrStride + kk) * 2u);
                mma_bf16(acc[2 * jp], a, b[0], b[1]);
                mma_bf16(acc[2 * jp + 1], a, b[2], b[3]);
            }
        }
    }
    // partial[slice][token][j]
    const int gq = lane >> 2, tg = lane & 3;
#pragma unroll
    for (int j = 0; j < NJ; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int tok = tok0 + warp * 16 + gq + 8 * (i >> 1), col = j0 + j * 8 + 2 * tg + (i & 1);
            if (tok < T && col < r_pad) partial[((size_t)by * T + tok) * r_pad + col] = acc[j][i];
        }
}

template <int NJ>
__global__ void __launch_bounds__(kLrThreads)
lowrank_down_mma_kernel(const __half* __restrict__ B, const __nv_bfloat16* __restrict__ x, int64_t ldx,
                        float* __restrict__ partial, int n, int r_pad, int T, int j0, int slice_cols) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    lowrank_body<NJ>(smem_raw, (int)blockIdx.x, (int)blockIdx.y, B, x, ldx, partial, n, r_pad, T, j0, slice_cols);
}

// Rotation and low-rank down-projection of a many-token forward in ONE grid: the two read the same activations
// and do not depend on each other, so their CTAs run side by side (blocks [0, n_rot) rotate four token rows each,
// the rest are the (token tile, K slice) CTAs of the down-projection).  Launched with programmatic stream
// serialization: the dependents may be scheduled at once, the activations are read after the wait.
template <int NJ>
__global__ void __launch_bounds__(kLrThreads, NJ <= 8 ? 3 : 2)
rotate_lowrank_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, const int32_t* __restrict__ perm,
                      __nv_bfloat16* __restrict__ xrot, int64_t ldo, float* __restrict__ s64, int s64_ld,
                      int* __restrict__ status, int n, int b_i, int b_h, float inv_sqrt_bh, int T, int n_rot,
                      const __half* __restrict__ B, float* __restrict__ partial, int r_pad, int lr_gx, int slice_cols,
                      int mma_form, int rows_per_cta) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // The two kinds of CTA are dealt out evenly over the grid (rot_before(i) = rotation CTAs among the first i), so
    // that every wave of resident CTAs holds both: their memory and arithmetic phases then overlap instead of all
    // rotation CTAs loading at once and all of them computing at once.
    const unsigned total = gridDim.x, i = blockIdx.x;
    const int rot_before = (int)(((unsigned long long)i * (unsigned)n_rot) / total);
    const int rot_through = (int)(((unsigned long long)(i + 1) * (unsigned)n_rot) / total);
    if (rot_through > rot_before) {
        const int rb = rot_before;
        // (no 64-column sums: the tensor-core product that follows dequantizes the weights and needs none)
        if (rows_per_cta == 8)
            rotate_mma_body<8>(smem_raw, rb, x, ldx, perm, xrot, ldo, status, n, b_i, b_h, inv_sqrt_bh, T);
        else if (mma_form)
            rotate_mma_body<4>(smem_raw, rb, x, ldx, perm, xrot, ldo, status, n, b_i, b_h, inv_sqrt_bh, T);
        else
            rotate_body<8, 4, true>(smem_raw, rb, x, ldx, perm, xrot, ldo, s64, s64_ld, status, n, b_i, b_h,
                                    inv_sqrt_bh, T);
    } else {
        const int b = (int)i - rot_before;
        lowrank_body<NJ>(smem_raw, b % lr_gx, b / lr_gx, B, x, ldx, partial, n, r_pad, T, 0, slice_cols);
    }
}

// Adds the K slices in order and rounds once to fp16.  Safe under a programmatic launch: waits for the producer.
__global__ void lowrank_finish_kernel(const float* __restrict__ partial, __half* __restrict__ t, size_t count, int slices) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    float s = 0.0f;
    for (int k = 0; k < slices; ++k) s += partial[(size_t)k * count + i];
    t[i] = __float2half_rn(s);
}

}  // namespace

int lowrank_mma_slices(const lopro_desc& d, int T) {
    const int tiles = (T + kLrTokens - 1) / kLrTokens;
    int slices = 1;
    while (slices < 32 && tiles * slices < 512 && d.d_in / (slices * 2) >= 256 && (d.d_in / 64) % (slices * 2) == 0) slices *= 2;
    return slices;
}

// Bytes reserved for the K-slice sums of up to T tokens.  The slice count falls as the token tiles grow, so the
// need of a launch, slices(T) * T rows, is not monotone in T; the reservation is the largest need of any token
// count up to T (the slice count is constant within a tile count, so the last T of each tile count decides).
size_t lowrank_mma_scratch_bytes(const lopro_desc& d, int T) {
    const int r_pad = round_up_int(d.rank, 16);
    const int tiles = (T + kLrTokens - 1) / kLrTokens;
    size_t rows = 0;
    for (int tl = 1; tl <= tiles; ++tl) {
        const int t_last = tl * kLrTokens < T ? tl * kLrTokens : T;
        const size_t need = (size_t)lowrank_mma_slices(d, t_last) * (size_t)t_last;
        if (need > rows) rows = need;
    }
    return rows * (size_t)r_pad * 4;
}

cudaError_t launch_lowrank_down_mma(const lopro_desc& d, const __half* B, int r_pad, const __nv_bfloat16* x, int64_t ldx,
                                    float* partial, __half* t, int T, cudaStream_t s) {
    const int slices = lowrank_mma_slices(d, T);
    const int slice_cols = d.d_in / slices;
    dim3 grid((T + kLrTokens - 1) / kLrTokens, slices);
    for (int j0 = 0; j0 < r_pad; j0 += kLrMaxRank) {
        const int rows = r_pad - j0 < kLrMaxRank ? r_pad - j0 : kLrMaxRank;
        cudaError_t e;
        static unsigned long long done16 = 0, done8 = 0, done4 = 0, done2 = 0;
        if (rows > 64) {
            const int smem = (kLrTokens + 2 * 128) * kLrStride * 2;
            if ((e = ensure_dynamic_smem(lowrank_down_mma_kernel<16>, smem, &done16)) != cudaSuccess) return e;
            lowrank_down_mma_kernel<16><<<grid, kLrThreads, smem, s>>>(B, x, ldx, partial, d.d_in, r_pad, T, j0, slice_cols);
        } else if (rows > 32) {
            const int smem = (kLrTokens + 2 * 64) * kLrStride * 2;
            if ((e = ensure_dynamic_smem(lowrank_down_mma_kernel<8>, smem, &done8)) != cudaSuccess) return e;
            lowrank_down_mma_kernel<8><<<grid, kLrThreads, smem, s>>>(B, x, ldx, partial, d.d_in, r_pad, T, j0, slice_cols);
        } else if (rows > 16) {
            const int smem = (kLrTokens + 2 * 32) * kLrStride * 2;
            if ((e = ensure_dynamic_smem(lowrank_down_mma_kernel<4>, smem, &done4)) != cudaSuccess) return e;
            lowrank_down_mma_kernel<4><<<grid, kLrThreads, smem, s>>>(B, x, ldx, partial, d.d_in, r_pad, T, j0, slice_cols);
        } else {
            const int smem = (kLrTokens + 2 * 16) * kLrStride * 2;
            if ((e = ensure_dynamic_smem(lowrank_down_mma_kernel<2>, smem, &done2)) != cudaSuccess) return e;
            lowrank_down_mma_kernel<2><<<grid, kLrThreads, smem, s>>>(B, x, ldx, partial, d.d_in, r_pad, T, j0, slice_cols);
        }
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    const size_t count = (size_t)T * r_pad;
    lowrank_finish_kernel<<<(unsigned)((count + 255) / 256), 256, 0, s>>>(partial, t, count, slices);
    return cudaGetLastError();
}

namespace {

template <int NJ>
cudaError_t launch_rotate_lowrank_nj(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                                     __nv_bfloat16* xrot, int64_t ldo, float* s64, int* status, const __half* B, int r_pad,
                                     float* partial, int T, cudaStream_t s) {
    const int slices = lowrank_mma_slices(d, T);
    const int slice_cols = d.d_in / slices;
    // rotation CTAs: the tensor-core form of the recursion with 8 rows per CTA where that leaves room for three CTAs
    // per SM, with 4 rows otherwise; the register-and-shuffle form where the block size or prefix rules it out
    const bool mma_form = rotate_mma_shape_ok(d) && (reinterpret_cast<uintptr_t>(perm) % 16) == 0 &&
                          rotate_mma_smem_bytes(4, d.d_in) <= 160 * 1024;
    const int rows_per_cta = mma_form && rotate_mma_smem_bytes(8, d.d_in) <= 74 * 1024 ? 8 : 4;
    const int n_rot = (T + rows_per_cta - 1) / rows_per_cta, lr_gx = (T + kLrTokens - 1) / kLrTokens;
    const size_t smem_rot = mma_form ? rotate_mma_smem_bytes(rows_per_cta, d.d_in) : (size_t)d.d_in * 8;
    const size_t smem_lr = (size_t)(kLrTokens + 2 * NJ * 8) * kLrStride * 2;
    const size_t smem = smem_rot > smem_lr ? smem_rot : smem_lr;
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(rotate_lowrank_kernel<NJ>, 160 * 1024, &attr_done);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_rot + lr_gx * slices));
    cfg.blockDim = dim3(kLrThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    const float inv = (float)(1.0 / sqrt((double)d.block_size));
    return cudaLaunchKernelEx(&cfg, rotate_lowrank_kernel<NJ>, x, ldx, perm, xrot, ldo, s64, s64_stride(d.d_in), status,
                              d.d_in, d.identity_cols, d.block_size, inv, T, n_rot, B, partial, r_pad, lr_gx, slice_cols,
                              mma_form ? 1 : 0, rows_per_cta);
}

}  // namespace

namespace {

// The FP8 low-rank record folded for the tensor-core path: A[i][j] = fp16(U[i][j] sigma[j]) (the product of a 4-bit and an
// 11-bit significand is exact in fp32: one rounding), B[j][k] = fp16(V[j][k] / s[k]) (IEEE single division, then one
// rounding).  Two entries per thread; r_pad and n are even.
__global__ void __launch_bounds__(256)
lr8_fold_kernel(const uint8_t* __restrict__ U, const uint8_t* __restrict__ V, const __half* __restrict__ sigma,
                const __half* __restrict__ svec, __half* __restrict__ A, __half* __restrict__ B, size_t pairs_a, int r_pad,
                size_t pairs_b, int n) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < pairs_a) {
        const uint32_t h2 = e4m3x2_to_f16x2(reinterpret_cast<const uint16_t*>(U)[i]);
        const float2 u = __half22float2(*reinterpret_cast<const __half2*>(&h2));
        const int j = (int)((2 * i) % (size_t)r_pad);
        reinterpret_cast<__half2*>(A)[i] = __floats2half2_rn(u.x * __half2float(sigma[j]), u.y * __half2float(sigma[j + 1]));
    } else if (i - pairs_a < pairs_b) {
        const size_t b = i - pairs_a;
        const uint32_t h2 = e4m3x2_to_f16x2(reinterpret_cast<const uint16_t*>(V)[b]);
        const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&h2));
        const int k = (int)((2 * b) % (size_t)n);
        reinterpret_cast<__half2*>(B)[b] =
            __floats2half2_rn(__fdiv_rn(v.x, __half2float(svec[k])), __fdiv_rn(v.y, __half2float(svec[k + 1])));
    }
}

}  // namespace

// A plain launch (not a programmatic one): the buffers it writes may still be read by the tensor-core kernel of the
// previous forward on this stream.
cudaError_t launch_lr8_fold(const lopro_desc& d, int r_pad, const uint8_t* U, const uint8_t* V, const __half* sigma,
                            const __half* svec, __half* A, __half* B, cudaStream_t s) {
    const size_t pairs_a = (size_t)d.d_out * r_pad / 2, pairs_b = (size_t)r_pad * d.d_in / 2;
    const size_t blocks = (pairs_a + pairs_b + 255) / 256;
    if (blocks > 0x7fffffffull) return cudaErrorInvalidValue;
    lr8_fold_kernel<<<(unsigned)blocks, 256, 0, s>>>(U, V, sigma, svec, A, B, pairs_a, r_pad, pairs_b, d.d_in);
    return cudaGetLastError();
}

bool rotate_lowrank_supported(const lopro_desc& d, int T) {
    const int r_pad = round_up_int(d.rank, 16);
    // from 64 tokens on the one grid beats rotation and B x as two launches (11008 columns, 128 tokens: 84.6 -> 75.5 us
    // for the whole forward; 8192 columns: 145 -> 141)
    return d.rank > 0 && r_pad <= kLrMaxRank && T >= 64 && d.block_size <= 256 && d.identity_cols % 64 == 0 &&
           (size_t)d.d_in * 8 <= 160 * 1024;
}

cudaError_t launch_rotate_lowrank(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                                  __nv_bfloat16* xrot, int64_t ldo, float* s64, int* status, const __half* B, int r_pad,
                                  float* partial, __half* t, int T, cudaStream_t s) {
    cudaError_t e;
    if (r_pad > 64) e = launch_rotate_lowrank_nj<16>(d, perm, x, ldx, xrot, ldo, s64, status, B, r_pad, partial, T, s);
    else if (r_pad > 32) e = launch_rotate_lowrank_nj<8>(d, perm, x, ldx, xrot, ldo, s64, status, B, r_pad, partial, T, s);
    else if (r_pad > 16) e = launch_rotate_lowrank_nj<4>(d, perm, x, ldx, xrot, ldo, s64, status, B, r_pad, partial, T, s);
    else e = launch_rotate_lowrank_nj<2>(d, perm, x, ldx, xrot, ldo, s64, status, B, r_pad, partial, T, s);
    if (e != cudaSuccess) return e;
    // the K slices are added by a dependent launch that waits for the grid above
    const size_t count = (size_t)T * r_pad;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((count + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, lowrank_finish_kernel, (const float*)partial, t, count, lowrank_mma_slices(d, T));
}

}  // namespace lopro
