// Activation-side transform x~ = Q^T P^T x (Eq. 8; Eq. 5 permutation, Eq. 6 partial block
// Walsh-Hadamard rotation with the Sylvester recursion of Eq. 2), and the low-rank
// down-projection t = B x (Appendix A.3, "Y = V X").
#include <math.h>

#include "common.cuh"

namespace lopro {

namespace {

constexpr int kRotThreads = 256;

// One CTA per token row.  The row is staged in shared memory with coalesced 16-byte loads, the
// gather through `perm` reads shared memory (a 2-byte gather from global memory would use 1/16 of
// every sector), each warp transforms runs of 32*E consecutive rotated columns: lane l holds E
// consecutive entries, the first log2(E) butterfly stages stay in registers, the next five go
// through warp shuffles.  Results are rounded to bf16 once, collected in shared memory and stored
// with coalesced 16-byte stores.  E = 8 covers b_H <= 256, E = 16 and 32 cover 512 and 1024.
template <int E>
__global__ void __launch_bounds__(kRotThreads)
rotate_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, const int32_t* __restrict__ perm,
              __nv_bfloat16* __restrict__ xrot, int64_t ldo, float* __restrict__ s64, int n, int b_i, int b_h,
              float inv_sqrt_bh) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* xin = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* xout = xin + n;
    const int t = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = kRotThreads / 32;
    constexpr int kRun = 32 * E;

    const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t * ldx);
    for (int i = tid; i < n / 8; i += kRotThreads) reinterpret_cast<uint4*>(xin)[i] = __ldg(src + i);
    __syncthreads();

    // identity prefix: permuted only
    for (int k = tid; k < b_i; k += kRotThreads) xout[k] = xin[__ldg(perm + k)];

    const int nrot = n - b_i;
    const int nruns = (nrot + kRun - 1) / kRun;
    for (int run = warp; run < nruns; run += kWarps) {
        const int rel = run * kRun + lane * E;  // offset inside the rotated region
        float v[E];
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int idx = rel + e;
            v[e] = idx < nrot ? __bfloat162float(xin[__ldg(perm + b_i + idx)]) : 0.0f;
        }
        // stages inside the lane: distance h = 1, 2, ..., E/2
#pragma unroll
        for (int h = 1; h < E; h <<= 1) {
            if (h < b_h) {
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if ((e & h) == 0) {
                        const float a = v[e], b = v[e + h];
                        v[e] = a + b;
                        v[e + h] = a - b;
                    }
                }
            }
        }
        // stages across lanes: distance h = E, 2E, ..., 16E  (lane distance h / E)
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            if (d * E < b_h) {
                const bool upper = (lane & d) != 0;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const float other = __shfl_xor_sync(0xffffffffu, v[e], d);
                    v[e] = upper ? other - v[e] : v[e] + other;
                }
            }
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int idx = rel + e;
            if (idx < nrot) xout[b_i + idx] = __float2bfloat16_rn(v[e] * inv_sqrt_bh);
        }
    }
    __syncthreads();

    uint4* dst = reinterpret_cast<uint4*>(xrot + (size_t)t * ldo);
    for (int i = tid; i < n / 8; i += kRotThreads) dst[i] = reinterpret_cast<const uint4*>(xout)[i];
    if (s64 != nullptr) {
        const int nsteps = n / 64;
        for (int st = warp; st < nsteps; st += kWarps) {
            const __nv_bfloat162 p = reinterpret_cast<const __nv_bfloat162*>(xout)[st * 32 + lane];
            float s = __low2float(p) + __high2float(p);
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
            if (lane == 0) s64[(size_t)t * nsteps + st] = s;
        }
    }
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

template <int E>
cudaError_t launch_rotate_e(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                            __nv_bfloat16* xrot, int64_t ldo, float* s64, int T, cudaStream_t s) {
    const size_t smem = (size_t)d.d_in * 4;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(rotate_kernel<E>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const float inv = (float)(1.0 / sqrt((double)d.block_size));
    rotate_kernel<E><<<T, kRotThreads, smem, s>>>(x, ldx, perm, xrot, ldo, s64, d.d_in, d.identity_cols,
                                                  d.block_size, inv);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_rotate(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                          __nv_bfloat16* xrot, int64_t ldo, float* s64, int T, cudaStream_t s) {
    if (d.block_size <= 256) return launch_rotate_e<8>(d, perm, x, ldx, xrot, ldo, s64, T, s);
    if (d.block_size == 512) return launch_rotate_e<16>(d, perm, x, ldx, xrot, ldo, s64, T, s);
    return launch_rotate_e<32>(d, perm, x, ldx, xrot, ldo, s64, T, s);
}

cudaError_t launch_lowrank_down(const lopro_desc& d, const __half* B, int r_pad, const __nv_bfloat16* x,
                                int64_t ldx, __half* t, int T, cudaStream_t s) {
    dim3 grid((r_pad + 7) / 8, (T + 7) / 8);
    lowrank_down_kernel<<<grid, 256, 0, s>>>(B, x, ldx, t, d.d_in, r_pad, T);
    return cudaGetLastError();
}

}  // namespace lopro
