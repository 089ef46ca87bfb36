// Vector-quantized residual (the vector variant of the method: a codebook of 256 four-dimensional centroids per group
// of cb_rows x cb_cols rotated weights, one 8-bit index per four consecutive columns; or 64 two-dimensional centroids,
// one 6-bit index per two columns, the 3-bit form): packed record and forward.
// The forward is Eq. 8 with W^ looked up instead of dequantized: rotation and t = B x by the library's kernels, then
// one product kernel per group of up to 32 tokens.
#include "lopro_vq.h"

#include "common.cuh"
#include "ptx.cuh"

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstring>

namespace lopro {

namespace {

constexpr uint32_t kVqMagic = 0x5156504Cu;  // "LPVQ"
constexpr int kVqHeader = 256;
constexpr int kVqRowsPerCta = 64;           // four warps, sixteen rows each
constexpr int kVqBookBytes = 256 * 4 * 2;   // one codebook of 256 four-dimensional centroids
constexpr int kVqBook2Bytes = 64 * 2 * 2;   // one codebook of 64 two-dimensional centroids
inline int vq_dim(const lopro_vq_desc& d) { return d.dim == 0 ? 4 : d.dim; }
inline int vq_book_bytes(int dim) { return dim == 4 ? kVqBookBytes : kVqBook2Bytes; }
// bytes of a row's indices: one byte per four columns, or 6 bits per two columns
inline size_t vq_idx_row_bytes(size_t n, int dim) { return dim == 4 ? n / 4 : n / 8 * 3; }
// codebooks per shared-memory buffer (two buffers): 6 with one token tile (24 KB, seven CTAs per SM, so that two waves
// hold the grid of a 28672-row layer), 8 otherwise (the registers of the wider variants allow five CTAs per SM anyway)
constexpr int kVqSectionMax = 8;

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

struct VqLayout {
    size_t off_idx, off_books, off_perm, off_a, off_b, off_bitmap, total;
    int r_pad, n_rg, n_cg;
};

lopro_status vq_check(const lopro_vq_desc* d) {
    if (!d) return LOPRO_ERR_INVALID_ARG;
    if (d->d_in <= 0 || d->d_out <= 0 || d->cb_rows <= 0 || d->cb_cols <= 0) return LOPRO_ERR_INVALID_ARG;
    if (d->block_size < 2 || d->block_size > 1024 || (d->block_size & (d->block_size - 1))) return LOPRO_ERR_INVALID_ARG;
    if (d->identity_cols < 0 || d->identity_cols > d->d_in || (d->d_in - d->identity_cols) % d->block_size)
        return LOPRO_ERR_INVALID_ARG;
    if (d->rank < 0 || d->rank > 512 || d->d_in % d->cb_cols) return LOPRO_ERR_INVALID_ARG;
    if (d->dim != 0 && d->dim != 2 && d->dim != 4) return LOPRO_ERR_INVALID_ARG;
    if (d->d_in % 64 || d->d_out % kVqRowsPerCta || d->cb_rows % kVqRowsPerCta || d->cb_cols % 64) return LOPRO_ERR_UNSUPPORTED;
    if (d->d_in > 32768 || d->d_out > (1 << 20)) return LOPRO_ERR_UNSUPPORTED;
    return LOPRO_OK;
}

VqLayout vq_layout(const lopro_vq_desc& d) {
    VqLayout L;
    const size_t m = d.d_out, n = d.d_in;
    L.r_pad = round_up_int(d.rank, 16);
    L.n_rg = (d.d_out + d.cb_rows - 1) / d.cb_rows;
    L.n_cg = d.d_in / d.cb_cols;
    size_t off = kVqHeader;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off += round_up_size(bytes, 256);
        return at;
    };
    L.off_idx = take(m * vq_idx_row_bytes(n, vq_dim(d)));
    L.off_books = take((size_t)L.n_rg * L.n_cg * vq_book_bytes(vq_dim(d)));
    L.off_perm = take(n * 4);
    L.off_a = take(m * (size_t)L.r_pad * 2);
    L.off_b = take((size_t)L.r_pad * n * 2);
    L.off_bitmap = take((n + 31) / 32 * 4);  // scratch of the permutation check
    L.total = off;
    return L;
}

// The rotation and the low-rank down-projection are those of the scalar forward: they see this descriptor.
lopro_desc as_scalar_desc(const lopro_vq_desc& d) {
    lopro_desc s = {};
    s.d_in = d.d_in;
    s.d_out = d.d_out;
    s.bits = 4;
    s.group_size = 64;
    s.block_size = d.block_size;
    s.identity_cols = d.identity_cols;
    s.rank = d.rank;
    s.layout = LOPRO_LAYOUT_FRAGMENT;
    s.lowrank_format = LOPRO_LOWRANK_FOLDED_F16;
    return s;
}

struct VqWorkspace {
    size_t off_status, off_xrot, off_t, off_part, total;
    int r_pad;
};

VqWorkspace vq_workspace(const lopro_vq_desc& d, int T) {
    VqWorkspace W;
    W.r_pad = round_up_int(d.rank, 16);
    size_t off = 0;
    W.off_status = off;
    off += 256;
    W.off_xrot = off;
    off += round_up_size((size_t)T * d.d_in * 2, 256);
    W.off_t = off;
    off += round_up_size((size_t)T * (W.r_pad > 0 ? W.r_pad : 16) * 2, 256);
    W.off_part = off;
    off += d.rank > 0 && T > kDecodeMaxT ? round_up_size(lowrank_mma_scratch_bytes(as_scalar_desc(d), T), 256) : 0;
    W.total = off;
    return W;
}

__global__ void vq_perm_check_kernel(const int32_t* __restrict__ perm, int n, uint32_t* __restrict__ bitmap, int* flag) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int p = perm[i];
    if ((unsigned)p >= (unsigned)n) {
        *flag = 1;
        return;
    }
    const uint32_t bit = 1u << (p & 31);
    if (atomicOr(bitmap + (p >> 5), bit) & bit) *flag = 1;
}

// 6-bit indices, one per byte -> the packed bit stream: four indices (24 bits) per thread; an index of 64 or more
// raises the flag and is reduced modulo 64
__global__ void vq_pack6_kernel(const uint8_t* __restrict__ idx, size_t quads, uint8_t* __restrict__ out, int* flag) {
    const size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= quads) return;
    const uchar4 v = reinterpret_cast<const uchar4*>(idx)[q];
    if ((v.x | v.y | v.z | v.w) & 0xC0) *flag = 1;
    const uint32_t w = (v.x & 63u) | ((v.y & 63u) << 6) | ((v.z & 63u) << 12) | ((v.w & 63u) << 18);
    out[3 * q] = (uint8_t)w;
    out[3 * q + 1] = (uint8_t)(w >> 8);
    out[3 * q + 2] = (uint8_t)(w >> 16);
}

__global__ void vq_identity_perm_kernel(int32_t* __restrict__ perm, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) perm[i] = i;
}

// rows of a factor matrix into rows padded to r_pad (zeros beyond r)
__global__ void vq_copy_padded_kernel(const __half* __restrict__ src, int rows, int cols, int cols_pad, __half* __restrict__ dst) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)rows * cols_pad) return;
    const int r = (int)(i / cols_pad), c = (int)(i % cols_pad);
    dst[i] = c < cols ? src[(size_t)r * cols + c] : __float2half(0.0f);
}

// t[tok][j] = sum_k B[j][k] x[tok][k] for one row j of B and up to 8 tokens per CTA (grid: r_pad x token groups):
// 16-byte loads strided over the row, fp32 sums, one rounding to fp16.
__global__ void __launch_bounds__(256) vq_lowrank_down_kernel(const __half* __restrict__ B, const __nv_bfloat16* __restrict__ x,
                                                              int64_t ldx, __half* __restrict__ t, int n, int r_pad, int T) {
    __shared__ float part[8][8];
    const int j = blockIdx.x, tok0 = blockIdx.y * 8, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nt = min(8, T - tok0);
    float acc[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) acc[q] = 0.0f;
    for (int c = tid; c < (n >> 3); c += 256) {
        const uint4 bv = __ldg(reinterpret_cast<const uint4*>(B + (size_t)j * n) + c);
        const __half2* bh = reinterpret_cast<const __half2*>(&bv);
        float bf[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __half22float2(bh[e]);
            bf[2 * e] = f.x;
            bf[2 * e + 1] = f.y;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q)
            if (q < nt) {
                const uint4 xv = __ldg(reinterpret_cast<const uint4*>(x + (size_t)(tok0 + q) * ldx) + c);
                const __nv_bfloat162* xh = reinterpret_cast<const __nv_bfloat162*>(&xv);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __bfloat1622float2(xh[e]);
                    acc[q] = fmaf(bf[2 * e], f.x, acc[q]);
                    acc[q] = fmaf(bf[2 * e + 1], f.y, acc[q]);
                }
            }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], o);
        if (lane == 0) part[warp][q] = acc[q];
    }
    __syncthreads();
    if (tid < nt) {
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += part[w][tid];
        t[(size_t)(tok0 + tid) * r_pad + j] = __float2half_rn(v);
    }
}

struct VqParams {
    const uint8_t* idx;          // [m][n / 4] bytes, or [m] rows of n / 2 six-bit indices
    const unsigned char* books;  // [n_rg][n_cg][256][4] or [n_rg][n_cg][64][2] bf16
    const __half* A;             // [m][r_pad]
    const __nv_bfloat16* xrot;   // [T][n] rotated activations of this launch's tokens
    const __half* t;             // [T][r_pad]
    void* y;
    int64_t ldy;
    int out_f32, m, n, T, r_pad, cb_rows, cb_cols, n_cg, section;
};


// grid = m / 64, 128 threads: warp w owns rows 64 b + 16 w .. + 15 over all of K.  The codebooks of the CTA's row group
// sit in shared memory.  K is walked in super-tiles of 64 columns = 16 vectors per row: lane 4 g + t takes the
// vectors 4 t .. 4 t + 3 of rows g and g + 8 (one 32-bit word of indices per row), and product s of the four
// m16n8k16 products of a super-tile uses vector 4 t + s, i.e. the lane's k-slots {2t, 2t+1, 2t+8, 2t+9} stand for
// the columns 16 t + 4 s .. + 3.  The activation fragments follow the same assignment (32 contiguous bytes of a
// token's rotated row per lane and super-tile), so both operands agree on which column a k-slot means.
// KS = 4: the four warps share ONE 16-row tile and take every fourth super-tile each (grid = m / 16; four times the
// warps per SM for the same registers per warp, which is what hides the lookup latency); their sums meet in shared
// memory at the end.  KS = 1: a warp per tile over all of K (grid = m / 64).
// DIM = 2 (64 two-dimensional centroids, 6-bit indices): the lane's 16 columns of a super-tile are eight vectors, 48 bits
// of the row's index stream starting at bit 48 t -- two 32-bit words from the 4-byte boundary below, shifted by 16 bits
// for odd t --, and product s uses the vectors 2 s (k-slots 2t, 2t+1) and 2 s + 1 (k-slots 2t+8, 2t+9).
template <int NT, int KS, int DIM>
__global__ void __launch_bounds__(128) vq_decode_kernel(const VqParams p) {
    constexpr int kBook = DIM == 4 ? kVqBookBytes : kVqBook2Bytes;
    extern __shared__ __align__(16) unsigned char vq_smem[];  // two sections of p.section codebooks
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int row0 = KS == 1 ? blockIdx.x * kVqRowsPerCta + warp * 16 : blockIdx.x * 16;
    const int kq = KS == 1 ? 0 : warp;  // this warp's share of K: super-tiles S = kq (mod KS)
    const int rg = row0 / p.cb_rows;
    // The row group's codebooks pass through shared memory in sections of p.section books, the next section copied
    // asynchronously while the warps work on the present one (a CTA then holds 32 KB instead of all its books, and
    // every CTA of a large layer is resident at once).
    const unsigned char* books_g = p.books + (size_t)rg * p.n_cg * kBook;
    const int n_sections = (p.n_cg + p.section - 1) / p.section;
    auto copy_section = [&](int sec) {
        const int first = sec * p.section, cnt = min(p.section, p.n_cg - first);
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(vq_smem) + (uint32_t)((sec & 1) * p.section * kBook);
        const unsigned char* src = books_g + (size_t)first * kBook;
        for (int i = tid; i < cnt * (kBook / 16); i += 128)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16u * (uint32_t)i), "l"(src + 16 * (size_t)i) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    copy_section(0);
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nt][e] = 0.0f;
    // DIM 4: word t of the super-tile's four index words; DIM 2: the word that holds bit 48 t of its six
    const size_t row_bytes = DIM == 4 ? (size_t)(p.n / 4) : (size_t)(p.n / 8 * 3);
    const int word0 = DIM == 4 ? t : (6 * t) >> 2;
    constexpr int kWordsPerSuper = DIM == 4 ? 4 : 6;
    const uint32_t* idx_lo = reinterpret_cast<const uint32_t*>(p.idx + (size_t)(row0 + g) * row_bytes) + word0;
    const uint32_t* idx_hi = reinterpret_cast<const uint32_t*>(p.idx + (size_t)(row0 + g + 8) * row_bytes) + word0;
    const int n_super = p.n >> 6, per_book = p.cb_cols >> 6;
    // Everything a super-tile needs from global memory -- one word of indices per row and 32 bytes of every token's
    // rotated row -- is requested one super-tile ahead and kept in registers meanwhile (two register stages).
    struct Stage {
        uint32_t w_lo, w_hi;
        uint32_t w_lo2, w_hi2;  // DIM 2: the second word of the lane's 48 bits
        uint4 xa[NT], xb[NT];
    };
    const uint4* xptr[NT];
    bool live[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int tok = nt * 8 + g;
        live[nt] = tok < p.T;
        xptr[nt] = reinterpret_cast<const uint4*>(p.xrot + (size_t)(live[nt] ? tok : 0) * p.n + 16 * t);
    }
    auto fetch = [&](Stage& st, int S) {
        st.w_lo = __ldg(idx_lo + kWordsPerSuper * S);
        st.w_hi = __ldg(idx_hi + kWordsPerSuper * S);
        if (DIM == 2) {
            st.w_lo2 = __ldg(idx_lo + kWordsPerSuper * S + 1);
            st.w_hi2 = __ldg(idx_hi + kWordsPerSuper * S + 1);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            st.xa[nt] = live[nt] ? __ldg(xptr[nt] + 8 * S) : make_uint4(0, 0, 0, 0);
            st.xb[nt] = live[nt] ? __ldg(xptr[nt] + 8 * S + 1) : make_uint4(0, 0, 0, 0);
        }
    };
    const uint32_t smem_s = (uint32_t)__cvta_generic_to_shared(vq_smem);
    uint32_t book = 0;  // byte offset of the present codebook in the shared-memory buffers
    int in_book = 0;    // super-tiles of it already done
    auto consume = [&](const Stage& st) {
        while (in_book >= per_book) {  // the codebook of this super-tile
            in_book -= per_book;
            book += kBook;
        }
        // all eight centroids first (32-bit shared-space addresses; the loads keep their place before the products),
        // then the products
        const uint32_t bk = smem_s + book;
        uint32_t a[4][4];
        if (DIM == 4) {
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(a[s][0]), "=r"(a[s][2]) : "r"(bk + 8u * ((st.w_lo >> (8 * s)) & 255u)));
                asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(a[s][1]), "=r"(a[s][3]) : "r"(bk + 8u * ((st.w_hi >> (8 * s)) & 255u)));
            }
        } else {
            const int sh = (t & 1) * 16;
            const unsigned long long v_lo = (((unsigned long long)st.w_lo2 << 32) | st.w_lo) >> sh;
            const unsigned long long v_hi = (((unsigned long long)st.w_hi2 << 32) | st.w_hi) >> sh;
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(a[s][0]) : "r"(bk + 4u * ((uint32_t)(v_lo >> (12 * s)) & 63u)));
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(a[s][2]) : "r"(bk + 4u * ((uint32_t)(v_lo >> (12 * s + 6)) & 63u)));
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(a[s][1]) : "r"(bk + 4u * ((uint32_t)(v_hi >> (12 * s)) & 63u)));
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(a[s][3]) : "r"(bk + 4u * ((uint32_t)(v_hi >> (12 * s + 6)) & 63u)));
            }
        }
#pragma unroll
        for (int s = 0; s < 4; ++s)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const uint4& v = s < 2 ? st.xa[nt] : st.xb[nt];
                const uint32_t b0 = (s & 1) ? v.z : v.x, b1 = (s & 1) ? v.w : v.y;
                mma_bf16(acc[nt], a[s], b0, b1);
            }
        in_book += KS;
    };
    Stage stA, stB;
    const int per_section = per_book * p.section;  // super-tiles per section of codebooks
    for (int sec = 0; sec < n_sections; ++sec) {
        const int S_end = min(n_super, (sec + 1) * per_section);
        int S = sec * per_section + kq;
        if (S < S_end) fetch(stA, S);  // (in flight while the section's codebooks land)
        if (sec + 1 < n_sections) {
            copy_section(sec + 1);  // into the buffer whose last reader passed the barrier at the end of section sec - 1
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();  // section sec has landed for every warp
        book = (uint32_t)((sec & 1) * p.section * kBook);
        in_book = kq;
        for (; S + KS < S_end; S += 2 * KS) {
            fetch(stB, S + KS);
            consume(stA);
            if (S + 2 * KS < S_end) fetch(stA, S + 2 * KS);
            consume(stB);
        }
        if (S < S_end) consume(stA);  // an odd one at the end of the section: stage A holds it
        __syncthreads();  // every warp is done with section sec before its buffer is overwritten
    }
    if (KS > 1) {
        // the four shares of K meet in shared memory (the codebook buffers are free after the last barrier); warp w then
        // finishes token tile w
        float* part = reinterpret_cast<float*>(vq_smem);  // [KS][NT][4][32]
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) part[((warp * NT + nt) * 4 + e) * 32 + lane] = acc[nt][e];
        __syncthreads();
        if (warp >= NT) return;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
            if (nt == warp) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = 0.0f;
#pragma unroll
                    for (int w = 0; w < KS; ++w) v += part[((w * NT + nt) * 4 + e) * 32 + lane];
                    acc[nt][e] = v;
                }
            }
    }
    // low-rank term and store: the lane holds rows g, g + 8 and tokens 8 nt + 2 t, + 1
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (KS > 1 && nt != warp) continue;
            const int row = row0 + g + 8 * (e >> 1), tok = nt * 8 + 2 * t + (e & 1);
            if (tok >= p.T) continue;
            float v = acc[nt][e];
            if (p.r_pad > 0) {
                const uint4* ar = reinterpret_cast<const uint4*>(p.A + (size_t)row * p.r_pad);
                const uint4* tr = reinterpret_cast<const uint4*>(p.t + (size_t)tok * p.r_pad);
                float lr = 0.0f;
                for (int j = 0; j < p.r_pad / 8; ++j) {
                    const uint4 av = __ldg(ar + j), tv = __ldg(tr + j);
                    const __half2* ah = reinterpret_cast<const __half2*>(&av);
                    const __half2* th = reinterpret_cast<const __half2*>(&tv);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float2 fa = __half22float2(ah[q]), ft = __half22float2(th[q]);
                        lr = fmaf(fa.x, ft.x, lr);
                        lr = fmaf(fa.y, ft.y, lr);
                    }
                }
                v += lr;
            }
            if (p.out_f32) reinterpret_cast<float*>(p.y)[(size_t)tok * p.ldy + row] = v;
            else reinterpret_cast<__nv_bfloat16*>(p.y)[(size_t)tok * p.ldy + row] = __float2bfloat16_rn(v);
        }
}

template <int NT>
cudaError_t launch_vq_decode(const VqParams& p, int dim, cudaStream_t s) {
    // two sections of codebooks; at the end the same memory holds the four warps' partial sums [4][NT][4][32] fp32
    size_t smem = (size_t)2 * p.section * vq_book_bytes(dim);
    if (smem < (size_t)4 * NT * 4 * 32 * 4) smem = (size_t)4 * NT * 4 * 32 * 4;
    if (dim == 4) vq_decode_kernel<NT, 4, 4><<<p.m / 16, 128, smem, s>>>(p);
    else vq_decode_kernel<NT, 4, 2><<<p.m / 16, 128, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

}  // namespace lopro

using namespace lopro;

extern "C" {

size_t lopro_vq_packed_bytes(const lopro_vq_desc* desc) {
    if (vq_check(desc) != LOPRO_OK) return 0;
    return vq_layout(*desc).total;
}

size_t lopro_vq_workspace_bytes(const lopro_vq_desc* desc, int32_t T) {
    if (vq_check(desc) != LOPRO_OK || T < 0) return 0;
    return vq_workspace(*desc, T < 1 ? 1 : T).total;
}

lopro_status lopro_vq_pack(const lopro_vq_desc* desc, const uint8_t* idx, const uint16_t* codebooks_bf16, const int32_t* perm,
                           const uint16_t* A_f16, const uint16_t* B_f16, void* packed, size_t packed_bytes, void* stream) {
    lopro_status st = vq_check(desc);
    if (st != LOPRO_OK) return st;
    const lopro_vq_desc& d = *desc;
    if (!idx || !codebooks_bf16 || !perm || !packed || (d.rank > 0 && (!A_f16 || !B_f16))) return LOPRO_ERR_INVALID_ARG;
    if (!aligned_to(packed, 256)) return LOPRO_ERR_INVALID_ARG;
    const VqLayout L = vq_layout(d);
    if (packed_bytes < L.total) return LOPRO_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* blob = (uint8_t*)packed;
    const size_t m = d.d_out, n = d.d_in;
    // header: magic, the descriptor, and a word the permutation check raises
    uint32_t header[kVqHeader / 4] = {};
    header[0] = kVqMagic;
    memcpy(header + 1, &d, sizeof(d));
    if (cudaMemcpyAsync(blob, header, kVqHeader, cudaMemcpyHostToDevice, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    const int dim = vq_dim(d);
    int* flag = (int*)(blob + 128);  // inside the header, zero so far
    if (dim == 4) {
        if (cudaMemcpyAsync(blob + L.off_idx, idx, m * (n / 4), cudaMemcpyDeviceToDevice, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    } else {
        if (!aligned_to(idx, 4)) return LOPRO_ERR_INVALID_ARG;
        const size_t quads = m * (n / 2) / 4;  // n is a multiple of 64: whole quads per row
        vq_pack6_kernel<<<(unsigned)((quads + 255) / 256), 256, 0, s>>>(idx, quads, blob + L.off_idx, flag);
        if (cudaGetLastError() != cudaSuccess) return LOPRO_ERR_CUDA;
    }
    if (cudaMemcpyAsync(blob + L.off_books, codebooks_bf16, (size_t)L.n_rg * L.n_cg * vq_book_bytes(dim), cudaMemcpyDeviceToDevice,
                        s) != cudaSuccess)
        return LOPRO_ERR_CUDA;
    if (cudaMemcpyAsync(blob + L.off_perm, perm, n * 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (d.rank > 0) {
        const size_t na = m * (size_t)L.r_pad, nb = (size_t)L.r_pad * n;
        vq_copy_padded_kernel<<<(unsigned)((na + 255) / 256), 256, 0, s>>>((const __half*)A_f16, (int)m, d.rank, L.r_pad,
                                                                          (__half*)(blob + L.off_a));
        // B [r][n] -> [r_pad][n]: whole rows, then zero rows
        if (cudaMemcpyAsync(blob + L.off_b, B_f16, (size_t)d.rank * n * 2, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
            return LOPRO_ERR_CUDA;
        if (L.r_pad > d.rank &&
            cudaMemsetAsync(blob + L.off_b + (size_t)d.rank * n * 2, 0, (size_t)(L.r_pad - d.rank) * n * 2, s) != cudaSuccess)
            return LOPRO_ERR_CUDA;
        (void)nb;
    }
    if (cudaMemsetAsync(blob + L.off_bitmap, 0, (n + 31) / 32 * 4, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    vq_perm_check_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>((const int32_t*)(blob + L.off_perm), (int)n,
                                                                     (uint32_t*)(blob + L.off_bitmap), flag);
    if (cudaGetLastError() != cudaSuccess) return LOPRO_ERR_CUDA;
    int bad = 0;
    if (cudaMemcpyAsync(&bad, flag, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (bad) {
        // a caller that ignores the verdict and runs a forward on the record must still read in bounds: the identity
        // takes the place of the rejected index vector
        vq_identity_perm_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>((int32_t*)(blob + L.off_perm), (int)n);
        return LOPRO_ERR_INVALID_DATA;
    }
    return LOPRO_OK;
}

lopro_status lopro_vq_linear_fwd(const lopro_vq_desc* desc, const void* packed, const uint16_t* x_bf16, int64_t ldx, void* y,
                                 int64_t ldy, int32_t out_dtype, int32_t T, void* workspace, size_t workspace_bytes,
                                 void* stream) {
    lopro_status st = vq_check(desc);
    if (st != LOPRO_OK) return st;
    const lopro_vq_desc& d = *desc;
    if (T < 0 || (out_dtype != LOPRO_OUT_BF16 && out_dtype != LOPRO_OUT_F32)) return LOPRO_ERR_INVALID_ARG;
    if (T == 0) return LOPRO_OK;
    if (!packed || !x_bf16 || !y || !workspace) return LOPRO_ERR_INVALID_ARG;
    if (ldx < d.d_in || (ldx % 8) || ldy < d.d_out) return LOPRO_ERR_INVALID_ARG;
    if (!aligned_to(packed, 256) || !aligned_to(workspace, 256) || !aligned_to(x_bf16, 16) ||
        !aligned_to(y, out_dtype == LOPRO_OUT_F32 ? 4 : 2))
        return LOPRO_ERR_INVALID_ARG;
    const VqWorkspace W = vq_workspace(d, T);
    if (workspace_bytes < W.total) return LOPRO_ERR_BUFFER_TOO_SMALL;
    const VqLayout L = vq_layout(d);
    const lopro_desc sd = as_scalar_desc(d);
    cudaStream_t s = (cudaStream_t)stream;
    const uint8_t* blob = (const uint8_t*)packed;
    uint8_t* ws = (uint8_t*)workspace;
    __nv_bfloat16* xrot = (__nv_bfloat16*)(ws + W.off_xrot);
    __half* tbuf = (__half*)(ws + W.off_t);
    int* status = (int*)(ws + W.off_status);
    // the rotation kernels that write no column sums do not reset the status word themselves in every form: clear it here
    if (cudaMemsetAsync(status, 0, 4, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (launch_rotate(sd, (const int32_t*)(blob + L.off_perm), (const __nv_bfloat16*)x_bf16, ldx, xrot, d.d_in, nullptr,
                      status, T, s) != cudaSuccess)
        return LOPRO_ERR_CUDA;
    if (d.rank > 0) {
        const __half* B = (const __half*)(blob + L.off_b);
        cudaError_t e;
        if (T > kDecodeMaxT) {
            e = launch_lowrank_down_mma(sd, B, L.r_pad, (const __nv_bfloat16*)x_bf16, ldx, (float*)(ws + W.off_part), tbuf, T, s);
        } else {
            vq_lowrank_down_kernel<<<dim3(L.r_pad, (T + 7) / 8), 256, 0, s>>>(B, (const __nv_bfloat16*)x_bf16, ldx, tbuf, d.d_in,
                                                                            L.r_pad, T);
            e = cudaGetLastError();
        }
        if (e != cudaSuccess) return LOPRO_ERR_CUDA;
    }
    const size_t esz = out_dtype == LOPRO_OUT_F32 ? 4 : 2;
    for (int t0 = 0; t0 < T; t0 += kDecodeMaxT) {
        const int tc = T - t0 < kDecodeMaxT ? T - t0 : kDecodeMaxT;
        VqParams p;
        p.idx = blob + L.off_idx;
        p.books = blob + L.off_books;
        p.A = (const __half*)(blob + L.off_a);
        p.xrot = xrot + (size_t)t0 * d.d_in;
        p.t = tbuf + (size_t)t0 * L.r_pad;
        p.y = (uint8_t*)y + (size_t)t0 * ldy * esz;
        p.ldy = ldy;
        p.out_f32 = out_dtype == LOPRO_OUT_F32;
        p.m = d.d_out;
        p.n = d.d_in;
        p.T = tc;
        p.r_pad = d.rank > 0 ? L.r_pad : 0;
        p.cb_rows = d.cb_rows;
        p.cb_cols = d.cb_cols;
        p.n_cg = L.n_cg;
        const int dim = vq_dim(d);
        // dim 2: the books are an eighth the size -- 32 per section hold the row group's books of most layers at once
        p.section = dim == 4 ? (tc <= 8 ? 6 : kVqSectionMax) : (L.n_cg < 32 ? L.n_cg : 32);
        const cudaError_t e = tc <= 8 ? launch_vq_decode<1>(p, dim, s)
                                      : (tc <= 16 ? launch_vq_decode<2>(p, dim, s) : launch_vq_decode<4>(p, dim, s));
        if (e != cudaSuccess) return LOPRO_ERR_CUDA;
    }
    return LOPRO_OK;
}

}  // extern "C"
