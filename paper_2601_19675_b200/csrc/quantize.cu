// Offline side of the method (Algorithm 1 without its calibration inputs): the rank-1 randomized sketch with
// deflation (Sec. 3.3, Eq. 10-12), the residual against the stored low-rank factors, R' = R P Q (Eq. 5, Eq. 6) and
// the round-to-nearest group grid of Appendix A.2.  Everything here is a memory-bound pass over an fp32 matrix:
// plain coalesced loads, fp32 arithmetic, results independent of the launch shape (fixed summation orders, no atomics).
#include "common.cuh"
#include "ptx.cuh"

#include <cuda_fp16.h>

namespace lopro {

namespace {

constexpr int kGemvThreads = 256;  // 8 warps: one row of W per warp
constexpr int kSlabRows = 32;      // rows of W per CTA in the transposed product

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

__device__ __forceinline__ float inv_norm(float sumsq) {
    const float nrm = sqrtf(sumsq);
    return (nrm > 0.0f && isfinite(nrm)) ? 1.0f / nrm : 0.0f;
}

// y[i] = (sum_k W[i][k] v[k]) / |v|: one warp per row, 16-byte loads, lanes strided over the row, then a butterfly
// over the lanes.  Every warp reads all of v anyway, so each forms |v|^2 itself (same order, same bits) and no
// separate reduction launch is needed.
__global__ void __launch_bounds__(kGemvThreads) gemv_rows_kernel(const float* __restrict__ W, int m, int n,
                                                                  const float* __restrict__ v, float* __restrict__ y) {
    const int row = blockIdx.x * (kGemvThreads / 32) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= m) return;
    const float4* w4 = reinterpret_cast<const float4*>(W + (size_t)row * n);
    const float4* v4 = reinterpret_cast<const float4*>(v);
    float acc = 0.0f, vv = 0.0f;
#pragma unroll 4
    for (int c = lane; c < n / 4; c += 32) {
        const float4 a = __ldg(w4 + c), b = __ldg(v4 + c);
        acc = fmaf(a.x, b.x, acc);
        acc = fmaf(a.y, b.y, acc);
        acc = fmaf(a.z, b.z, acc);
        acc = fmaf(a.w, b.w, acc);
        vv = fmaf(b.x, b.x, vv);
        vv = fmaf(b.y, b.y, vv);
        vv = fmaf(b.z, b.z, vv);
        vv = fmaf(b.w, b.w, vv);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        acc += __shfl_xor_sync(0xffffffffu, acc, o);
        vv += __shfl_xor_sync(0xffffffffu, vv, o);
    }
    if (lane == 0) y[row] = acc * inv_norm(vv);
}

// partial[slab][k] = sum over the slab's rows i of W[i][k] y[i]: a CTA owns kSlabRows rows and 1024 columns, a
// thread four columns; rows in ascending order.
__global__ void __launch_bounds__(256) gemv_cols_kernel(const float* __restrict__ W, int m, int n,
                                                        const float* __restrict__ y, float* __restrict__ partial) {
    __shared__ float ys[kSlabRows];
    const int slab = blockIdx.y, r0 = slab * kSlabRows, rows = min(kSlabRows, m - r0);
    if ((int)threadIdx.x < rows) ys[threadIdx.x] = y[r0 + threadIdx.x];
    __syncthreads();
    const int c4 = blockIdx.x * 256 + threadIdx.x;
    if (c4 >= n / 4) return;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4* w4 = reinterpret_cast<const float4*>(W + (size_t)r0 * n) + c4;
#pragma unroll 8
    for (int i = 0; i < rows; ++i) {
        const float4 a = __ldg(w4 + (size_t)i * (n / 4));
        const float s = ys[i];
        acc.x = fmaf(a.x, s, acc.x);
        acc.y = fmaf(a.y, s, acc.y);
        acc.z = fmaf(a.z, s, acc.z);
        acc.w = fmaf(a.w, s, acc.w);
    }
    reinterpret_cast<float4*>(partial + (size_t)slab * n)[c4] = acc;
}

// p[k] = (sum over slabs of partial[slab][k]) / |y|.  A CTA owns 32 columns; warp w adds the slabs w, w + 8, ... of
// those columns (128-byte rows of the partial sums), the eight sums meet in shared memory in the order of w.  While
// the other warps start on the slabs, every warp also takes an eighth of |y|^2 (lanes strided, fixed order).
__global__ void __launch_bounds__(256) colsum_kernel(const float* __restrict__ partial, int slabs, int n,
                                                     const float* __restrict__ y, int m, float* __restrict__ p) {
    __shared__ float s_part[8][32];
    __shared__ float s_sq[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + lane;
    float acc = 0.0f;
    if (k < n)
        for (int s = warp; s < slabs; s += 8) acc += partial[(size_t)s * n + k];
    s_part[warp][lane] = acc;
    float sq = 0.0f;
    for (int i = warp * 32 + lane; i < m; i += 256) sq = fmaf(y[i], y[i], sq);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if (lane == 0) s_sq[warp] = sq;
    __syncthreads();
    if (warp == 0 && k < n) {
        float total = 0.0f, ss = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            total += s_part[w][lane];
            ss += s_sq[w];
        }
        p[k] = total * inv_norm(ss);
    }
}

// fp32 -> nearest fp8 e4m3 value (ties to even, saturating), returned as fp32; bits optionally kept.
__device__ __forceinline__ float round_e4m3(float x, unsigned char* bits) {
    unsigned short pair;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(0.0f), "f"(x));  // low byte = second operand
    if (bits) *bits = (unsigned char)(pair & 0xffu);
    const uint32_t h2 = e4m3x2_to_f16x2((unsigned short)(pair & 0xffu));
    return __half2float(__ushort_as_half((unsigned short)(h2 & 0xffffu)));
}

// Rank j is done: U[:, j] = y / |y|, V[j, :] = p / |p| (cast to fp8 values when asked), sigma[j] = |p| where
// p = W^T (y / |y|).  Every CTA forms the two norms itself (same order in every CTA, same bits).  A vanished y or p gives a zero triple.
__global__ void __launch_bounds__(256) finish_rank_kernel(const float* __restrict__ y, const float* __restrict__ p,
                                                          int m, int n, int r, int j, int cast, float* __restrict__ U,
                                                          float* __restrict__ sigma, float* __restrict__ V,
                                                          float* __restrict__ u1, float* __restrict__ v1) {
    __shared__ float s_sq[2][8];
    __shared__ float s_ny, s_np;
    {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        float a = 0.0f, b = 0.0f;
        for (int i = warp * 32 + lane; i < m; i += 256) a = fmaf(y[i], y[i], a);
        for (int i = warp * 32 + lane; i < n; i += 256) b = fmaf(p[i], p[i], b);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, o);
            b += __shfl_xor_sync(0xffffffffu, b, o);
        }
        if (lane == 0) {
            s_sq[0][warp] = a;
            s_sq[1][warp] = b;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float sa = 0.0f, sb = 0.0f;
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                sa += s_sq[0][w];
                sb += s_sq[1][w];
            }
            s_ny = sa;
            s_np = sb;
        }
    }
    __syncthreads();
    const float iy = inv_norm(s_ny), ip = inv_norm(s_np);
    const bool dead = iy == 0.0f || ip == 0.0f;
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i < m) {
        float u = dead ? 0.0f : y[i] * iy;
        if (cast) u = round_e4m3(u, nullptr);
        U[(size_t)i * r + j] = u;
        u1[i] = u;
    }
    if (i < n) {
        float v = dead ? 0.0f : p[i] * ip;
        if (cast) v = round_e4m3(v, nullptr);
        V[(size_t)j * n + i] = v;
        v1[i] = v;
    }
    if (i == 0) sigma[j] = dead ? 0.0f : sqrtf(s_np);
}

// W <- W - sigma_j u1 v1^T
__global__ void __launch_bounds__(256) deflate_kernel(float* __restrict__ W, int m, int n, const float* __restrict__ u1,
                                                      const float* __restrict__ v1, const float* __restrict__ sigma_j) {
    const int row = blockIdx.x;
    const int c4 = blockIdx.y * 256 + threadIdx.x;
    if (c4 >= n / 4) return;
    const float su = -(*sigma_j) * u1[row];
    float4* w4 = reinterpret_cast<float4*>(W + (size_t)row * n) + c4;
    float4 a = *w4;
    const float4 b = __ldg(reinterpret_cast<const float4*>(v1) + c4);
    a.x = fmaf(su, b.x, a.x);
    a.y = fmaf(su, b.y, a.y);
    a.z = fmaf(su, b.z, a.z);
    a.w = fmaf(su, b.w, a.w);
    *w4 = a;
}

struct R1Workspace {
    float *y, *p, *u1, *v1, *partial;
    int slabs;
    size_t total;
};

R1Workspace r1svd_workspace(int m, int n, uint8_t* base) {
    R1Workspace w;
    w.slabs = (m + kSlabRows - 1) / kSlabRows;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        float* p = reinterpret_cast<float*>(base + off);
        off += round_up_size(bytes, 256);
        return p;
    };
    w.y = take((size_t)m * 4);
    w.p = take((size_t)n * 4);
    w.u1 = take((size_t)m * 4);
    w.v1 = take((size_t)n * 4);
    w.partial = take((size_t)w.slabs * n * 4);
    w.total = off;
    return w;
}

cudaError_t run_r1svd(float* w, int m, int n, int r, int it, const float* sketches, int cast, float* U, float* sigma,
                      float* V, const R1Workspace& ws, cudaStream_t s) {
    const dim3 g_rows((m + kGemvThreads / 32 - 1) / (kGemvThreads / 32));
    const dim3 g_cols((n / 4 + 255) / 256, ws.slabs);
    const dim3 g_sum((n + 31) / 32);
    const dim3 g_fin((max(m, n) + 255) / 256);
    const dim3 g_def(m, (n / 4 + 255) / 256);
    auto cols = [&]() {  // p = W^T y / |y|
        gemv_cols_kernel<<<g_cols, 256, 0, s>>>(w, m, n, ws.y, ws.partial);
        colsum_kernel<<<g_sum, 256, 0, s>>>(ws.partial, ws.slabs, n, ws.y, m, ws.p);
    };
    for (int j = 0; j < r; ++j) {
        gemv_rows_kernel<<<g_rows, kGemvThreads, 0, s>>>(w, m, n, sketches + (size_t)j * n, ws.y);  // y = W v / |v|
        for (int k = 0; k < it; ++k) {
            cols();
            gemv_rows_kernel<<<g_rows, kGemvThreads, 0, s>>>(w, m, n, ws.p, ws.y);                  // y = W p / |p|
        }
        cols();  // |p| = sigma
        finish_rank_kernel<<<g_fin, 256, 0, s>>>(ws.y, ws.p, m, n, r, j, cast, U, sigma, V, ws.u1, ws.v1);
        deflate_kernel<<<g_def, 256, 0, s>>>(w, m, n, ws.u1, ws.v1, sigma + j);
    }
    return cudaGetLastError();
}


// ---- residual, R' = R P Q, group grid ------------------------------------------------------------

struct RowJob {
    const float* W;     // [m][n]
    const float* Af;    // [m][rank] stored low-rank factor values (may be null with rank 0)
    const float* Bf;    // [rank][n]
    const int32_t* perm;
    float* r_rot;       // [m][n] output of the unfused form
    uint8_t* codes;     // outputs of the fused form
    __half* scales;
    __half* zeros;
    int* status;
    int m, n, rank, b_i, b_h, g, bits;
    float inv_sqrt_bh;
};

// The group grid on one row held in shared memory: a warp per group, lanes strided over its columns.
// Every operation below is one IEEE single-precision operation, in the order of the definition.
__device__ __forceinline__ void quantize_row(const float* row, int n, int g, int bits, uint8_t* codes, __half* scales,
                                             __half* zeros, int* status) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const float qmax = (float)((1 << bits) - 1);
    for (int grp = warp; grp < n / g; grp += nwarps) {
        const float* v = row + grp * g;
        float lo = v[lane], hi = lo;
        bool bad = !isfinite(lo);
        for (int c = lane + 32; c < g; c += 32) {
            const float x = v[c];
            bad |= !isfinite(x);
            lo = fminf(lo, x);
            hi = fmaxf(hi, x);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        }
        bad = __any_sync(0xffffffffu, bad);
        const bool constant = hi == lo;
        const float step = constant ? (lo != 0.0f ? fabsf(lo) : 1.0f) : __fdiv_rn(__fsub_rn(hi, lo), qmax);
        const __half step_h = __float2half_rn(step);
        const float scale = __half2float(step_h);
        if (bad || scale == 0.0f) {
            // non-finite entry, or a range that underflows fp16: reported, the group stored as zeros
            if (lane == 0) {
                atomicCAS(status, LOPRO_OK, LOPRO_ERR_INVALID_DATA);
                scales[grp] = __float2half_rn(1.0f);
                zeros[grp] = __float2half_rn(0.0f);
            }
            for (int c = lane; c < g; c += 32) codes[grp * g + c] = 0;
            continue;
        }
        const __half zero_h = __float2half_rn(constant ? (lo < 0.0f ? 1.0f : 0.0f) : rintf(__fdiv_rn(-lo, scale)));
        const float zero = __half2float(zero_h);
        if (lane == 0) {
            scales[grp] = step_h;
            zeros[grp] = zero_h;
        }
        for (int c = lane; c < g; c += 32) {
            const float q = __fadd_rn(rintf(__fdiv_rn(v[c], scale)), zero);
            codes[grp * g + c] = (uint8_t)fminf(fmaxf(q, 0.0f), qmax);
        }
    }
}

// One row of the layer per CTA: residual against the stored factors (rank terms in ascending order), gather by
// perm, butterflies of the rotated blocks in shared memory, then either the row of R' or its quantized form.
template <bool FUSED>
__global__ void __launch_bounds__(256) residual_rotate_kernel(const RowJob p) {
    extern __shared__ __align__(16) float rowbuf[];  // [2][n]
    float* r0 = rowbuf;
    float* r1 = rowbuf + p.n;
    __shared__ float a_row[512];
    const int i = blockIdx.x, tid = threadIdx.x;
    for (int j = tid; j < p.rank; j += 256) a_row[j] = p.Af[(size_t)i * p.rank + j];
    __syncthreads();
    const float* wrow = p.W + (size_t)i * p.n;
    for (int k = tid; k < p.n; k += 256) {
        float acc = wrow[k];
        for (int j = 0; j < p.rank; ++j) acc = fmaf(-a_row[j], __ldg(p.Bf + (size_t)j * p.n + k), acc);
        r0[k] = acc;
    }
    __syncthreads();
    for (int k = tid; k < p.n; k += 256) {
        int src = p.perm[k];
        if ((unsigned)src >= (unsigned)p.n) {
            atomicCAS(p.status, LOPRO_OK, LOPRO_ERR_INVALID_DATA);
            src = 0;
        }
        r1[k] = r0[src];
    }
    __syncthreads();
    // Hadamard recursion of Eq. 2 on every block of b_h columns after the identity prefix: level h pairs
    // (c, c + h); pairs never leave their block because h < b_h and the blocks start at multiples of b_h.
    const int pairs = (p.n - p.b_i) / 2;
    float* rot = r1 + p.b_i;
    for (int h = 1; h < p.b_h; h <<= 1) {
        for (int q = tid; q < pairs; q += 256) {
            const int c = (q / h) * 2 * h + (q % h);
            const float a = rot[c], b = rot[c + h];
            rot[c] = a + b;
            rot[c + h] = a - b;
        }
        __syncthreads();
    }
    for (int k = p.b_i + tid; k < p.n; k += 256) r1[k] *= p.inv_sqrt_bh;
    __syncthreads();
    if (FUSED) {
        quantize_row(r1, p.n, p.g, p.bits, p.codes + (size_t)i * p.n, p.scales + (size_t)i * (p.n / p.g),
                     p.zeros + (size_t)i * (p.n / p.g), p.status);
    } else {
        float* out = p.r_rot + (size_t)i * p.n;
        for (int k = tid; k < p.n; k += 256) out[k] = r1[k];
    }
}

__global__ void __launch_bounds__(256) rtn_kernel(const float* __restrict__ r_rot, int n, int g, int bits,
                                                   uint8_t* __restrict__ codes, __half* __restrict__ scales,
                                                   __half* __restrict__ zeros, int* status) {
    extern __shared__ __align__(16) float rowbuf[];
    const int i = blockIdx.x;
    for (int k = threadIdx.x; k < n; k += 256) rowbuf[k] = r_rot[(size_t)i * n + k];
    __syncthreads();
    quantize_row(rowbuf, n, g, bits, codes + (size_t)i * n, scales + (size_t)i * (n / g), zeros + (size_t)i * (n / g), status);
}

constexpr int kQuantMaxDin = 24576;  // two fp32 rows of the layer in one CTA's shared memory

template <bool FUSED>
cudaError_t launch_residual_rotate(const RowJob& job, cudaStream_t s) {
    static unsigned long long attr_done = 0;
    const int smem = 2 * job.n * (int)sizeof(float);
    cudaError_t e = ensure_dynamic_smem(residual_rotate_kernel<FUSED>, 2 * kQuantMaxDin * (int)sizeof(float), &attr_done);
    if (e != cudaSuccess) return e;
    residual_rotate_kernel<FUSED><<<job.m, 256, smem, s>>>(job);
    return cudaGetLastError();
}

RowJob make_job(const lopro_desc& d, const float* W, const float* Af, const float* Bf, const int32_t* perm, int* status) {
    RowJob j = {};
    j.W = W;
    j.Af = Af;
    j.Bf = Bf;
    j.perm = perm;
    j.status = status;
    j.m = d.d_out;
    j.n = d.d_in;
    j.rank = d.rank;
    j.b_i = d.identity_cols;
    j.b_h = d.block_size;
    j.g = d.group_size;
    j.bits = d.bits;
    j.inv_sqrt_bh = (float)(1.0 / sqrt((double)d.block_size));
    return j;
}

}  // namespace

namespace {

// W_s = W diag(s_eff); s_eff = s, or s rounded to fp16 where the record stores it so (also written out as bits)
__global__ void __launch_bounds__(256) scale_columns_kernel(const float* __restrict__ W, const float* __restrict__ s,
                                                            int n, int round_s, float* __restrict__ Ws,
                                                            float* __restrict__ s_eff, __half* __restrict__ s16) {
    const int row = blockIdx.x;
    for (int k = threadIdx.x; k < n; k += 256) {
        float sv = s ? s[k] : 1.0f;
        if (round_s) sv = __half2float(__float2half_rn(sv));
        if (row == 0) {
            s_eff[k] = sv;
            if (s16) s16[k] = __float2half_rn(sv);
        }
        Ws[(size_t)row * n + k] = W[(size_t)row * n + k] * sv;
    }
}

// The record's factors from (U, sigma, V, s_eff), and their stored values as fp32 for the residual.
//   folded: A = fp16(U sigma), B = fp16(V / s);   fp8: U, V as e4m3 bytes, Sigma fp16; Af = U Sigma16, Bf = V / s.
__global__ void __launch_bounds__(256) factors_kernel(const float* __restrict__ U, const float* __restrict__ sigma,
                                                      const float* __restrict__ V, const float* __restrict__ s_eff,
                                                      int m, int n, int r, int fp8, void* lr0, void* lr1, void* lr2,
                                                      float* __restrict__ Af, float* __restrict__ Bf) {
    const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (idx < (size_t)m * r) {
        const int j = (int)(idx % r);
        if (fp8) {
            unsigned char b;
            const float u = round_e4m3(U[idx], &b);  // already an fp8 value: the conversion is exact
            reinterpret_cast<unsigned char*>(lr0)[idx] = b;
            Af[idx] = u * __half2float(__float2half_rn(sigma[j]));
        } else {
            const __half a = __float2half_rn(U[idx] * sigma[j]);
            reinterpret_cast<__half*>(lr0)[idx] = a;
            Af[idx] = __half2float(a);
        }
    }
    if (idx < (size_t)r * n) {
        const int k = (int)(idx % n);
        if (fp8) {
            unsigned char b;
            const float v = round_e4m3(V[idx], &b);
            reinterpret_cast<unsigned char*>(lr1)[idx] = b;
            Bf[idx] = __fdiv_rn(v, s_eff[k]);
        } else {
            const __half bb = __float2half_rn(__fdiv_rn(V[idx], s_eff[k]));
            reinterpret_cast<__half*>(lr1)[idx] = bb;
            Bf[idx] = __half2float(bb);
        }
    }
    if (fp8 && idx < (size_t)r) reinterpret_cast<__half*>(lr2)[idx] = __float2half_rn(sigma[idx]);
}

struct QuantWorkspace {
    int* status;
    float *Ws, *U, *V, *sigma, *Af, *Bf, *s_eff;
    uint8_t* r1;
    size_t total;
};

QuantWorkspace quant_workspace(const lopro_desc& d, uint8_t* base) {
    QuantWorkspace q;
    const size_t m = d.d_out, n = d.d_in, r = d.rank;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        uint8_t* p = base + off;
        off += round_up_size(bytes, 256);
        return p;
    };
    q.status = reinterpret_cast<int*>(take(256));
    q.Ws = reinterpret_cast<float*>(take(r ? m * n * 4 : 0));
    q.U = reinterpret_cast<float*>(take(m * r * 4));
    q.V = reinterpret_cast<float*>(take(r * n * 4));
    q.sigma = reinterpret_cast<float*>(take(r * 4));
    q.Af = reinterpret_cast<float*>(take(m * r * 4));
    q.Bf = reinterpret_cast<float*>(take(r * n * 4));
    q.s_eff = reinterpret_cast<float*>(take(n * 4));
    q.r1 = base + off;
    off += r ? r1svd_workspace((int)m, (int)n, nullptr).total : 0;
    q.total = off;
    return q;
}

lopro_status check_quant_desc(const lopro_desc* desc) {
    if (!desc) return LOPRO_ERR_INVALID_ARG;
    const lopro_status st = check_desc(*desc);
    if (st != LOPRO_OK) return st;
    if (desc->d_in > kQuantMaxDin) return LOPRO_ERR_UNSUPPORTED;
    return LOPRO_OK;
}

}  // namespace

}  // namespace lopro

using namespace lopro;

extern "C" {

size_t lopro_r1svd_workspace_bytes(int32_t m, int32_t n) {
    if (m <= 0 || n <= 0) return 0;
    return r1svd_workspace(m, n, nullptr).total;
}

lopro_status lopro_r1svd(float* w, int32_t m, int32_t n, int32_t r, int32_t it, const float* sketches, int32_t cast,
                         float* U, float* sigma, float* V, void* workspace, size_t workspace_bytes, void* stream) {
    if (m <= 0 || n <= 0 || (m % 4) || (n % 4) || r < 1 || r > 512 || it < 0 || it > 64) return LOPRO_ERR_INVALID_ARG;
    if (cast != 0 && cast != 1) return LOPRO_ERR_INVALID_ARG;
    if (!w || !sketches || !U || !sigma || !V || !workspace) return LOPRO_ERR_INVALID_ARG;
    if (!aligned_to(w, 16) || !aligned_to(sketches, 16) || !aligned_to(workspace, 256)) return LOPRO_ERR_INVALID_ARG;
    if (workspace_bytes < lopro_r1svd_workspace_bytes(m, n)) return LOPRO_ERR_BUFFER_TOO_SMALL;
    const R1Workspace ws = r1svd_workspace(m, n, (uint8_t*)workspace);
    return run_r1svd(w, m, n, r, it, sketches, cast, U, sigma, V, ws, (cudaStream_t)stream) == cudaSuccess ? LOPRO_OK
                                                                                                           : LOPRO_ERR_CUDA;
}

lopro_status lopro_residual_rotate(const lopro_desc* desc, const float* W, const float* Af, const float* Bf,
                                   const int32_t* perm, float* r_rot, void* status_word, void* stream) {
    const lopro_status st = check_quant_desc(desc);
    if (st != LOPRO_OK) return st;
    if (!W || !perm || !r_rot || !status_word || (desc->rank > 0 && (!Af || !Bf))) return LOPRO_ERR_INVALID_ARG;
    RowJob job = make_job(*desc, W, Af, Bf, perm, (int*)status_word);
    job.r_rot = r_rot;
    return launch_residual_rotate<false>(job, (cudaStream_t)stream) == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

lopro_status lopro_rtn_quantize(const lopro_desc* desc, const float* r_rot, uint8_t* codes, uint16_t* scales,
                                uint16_t* zeros, void* status_word, void* stream) {
    const lopro_status st = check_quant_desc(desc);
    if (st != LOPRO_OK) return st;
    if (!r_rot || !codes || !scales || !zeros || !status_word) return LOPRO_ERR_INVALID_ARG;
    static unsigned long long attr_done = 0;
    if (ensure_dynamic_smem(rtn_kernel, kQuantMaxDin * (int)sizeof(float), &attr_done) != cudaSuccess) return LOPRO_ERR_CUDA;
    rtn_kernel<<<desc->d_out, 256, desc->d_in * sizeof(float), (cudaStream_t)stream>>>(
        r_rot, desc->d_in, desc->group_size, desc->bits, codes, reinterpret_cast<__half*>(scales),
        reinterpret_cast<__half*>(zeros), (int*)status_word);
    return cudaGetLastError() == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

size_t lopro_quantize_workspace_bytes(const lopro_desc* desc) {
    if (check_quant_desc(desc) != LOPRO_OK) return 0;
    return quant_workspace(*desc, nullptr).total;
}

lopro_status lopro_quantize_layer(const lopro_desc* desc, const float* W, const float* s, const int32_t* perm,
                                  const float* sketches, int32_t it, uint8_t* codes, uint16_t* scales, uint16_t* zeros,
                                  void* lr0, void* lr1, void* lr2, void* lr3, void* workspace, size_t workspace_bytes,
                                  void* stream) {
    const lopro_status st = check_quant_desc(desc);
    if (st != LOPRO_OK) return st;
    const lopro_desc& d = *desc;
    const bool fp8 = d.lowrank_format == LOPRO_LOWRANK_FP8;
    if (!W || !perm || !codes || !scales || !zeros || !workspace || it < 0 || it > 64) return LOPRO_ERR_INVALID_ARG;
    if (d.rank > 0 && (!sketches || !lr0 || !lr1 || (fp8 && (!lr2 || !lr3)))) return LOPRO_ERR_INVALID_ARG;
    if (!aligned_to(W, 16) || !aligned_to(workspace, 256) || (sketches && !aligned_to(sketches, 16))) return LOPRO_ERR_INVALID_ARG;
    if (workspace_bytes < lopro_quantize_workspace_bytes(desc)) return LOPRO_ERR_BUFFER_TOO_SMALL;
    cudaStream_t cs = (cudaStream_t)stream;
    const QuantWorkspace q = quant_workspace(d, (uint8_t*)workspace);
    const int m = d.d_out, n = d.d_in, r = d.rank;
    if (cudaMemsetAsync(q.status, 0, 4, cs) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (r > 0) {
        scale_columns_kernel<<<m, 256, 0, cs>>>(W, s, n, fp8 ? 1 : 0, q.Ws, q.s_eff, fp8 ? (__half*)lr3 : nullptr);
        const R1Workspace ws = r1svd_workspace(m, n, q.r1);
        if (run_r1svd(q.Ws, m, n, r, it, sketches, fp8 ? 1 : 0, q.U, q.sigma, q.V, ws, cs) != cudaSuccess) return LOPRO_ERR_CUDA;
        const size_t items = (size_t)r * (size_t)(m > n ? m : n);
        factors_kernel<<<(unsigned)((items + 255) / 256), 256, 0, cs>>>(q.U, q.sigma, q.V, q.s_eff, m, n, r, fp8 ? 1 : 0, lr0,
                                                                        lr1, lr2, q.Af, q.Bf);
    }
    RowJob job = make_job(d, W, r > 0 ? q.Af : nullptr, r > 0 ? q.Bf : nullptr, perm, q.status);
    job.codes = codes;
    job.scales = reinterpret_cast<__half*>(scales);
    job.zeros = reinterpret_cast<__half*>(zeros);
    if (launch_residual_rotate<true>(job, cs) != cudaSuccess) return LOPRO_ERR_CUDA;
    return LOPRO_OK;
}

}  // extern "C"
