// Body of the rotation kernel (Eq. 5 permutation, Eq. 6 partial block Walsh-Hadamard rotation), shared by
// the stand-alone kernel and the launch that runs it side by side with the low-rank down-projection.
#pragma once

#include "common.cuh"

namespace lopro {

constexpr int kRotThreads = 256;

// One CTA per TOK token rows.  The rows are staged in shared memory with coalesced 16-byte loads,
// the gather through `perm` reads shared memory (a 2-byte gather from global memory would use 1/16
// of every sector; with TOK > 1 each index of perm is fetched once for all rows), each warp transforms
// runs of 32*E consecutive rotated columns: lane l holds E consecutive entries, the first log2(E)
// butterfly stages stay in registers, the next five go through warp shuffles.  Results are rounded to
// bf16 once, collected in shared memory and stored with coalesced 16-byte stores.  E = 8 covers
// b_H <= 256, E = 16 and 32 cover 512 and 1024.
template <int E, int TOK, bool DIRECT>
__device__ __forceinline__ void rotate_body(unsigned char* smem_raw, int block, const __nv_bfloat16* __restrict__ x,
                                            int64_t ldx, const int32_t* __restrict__ perm,
                                            __nv_bfloat16* __restrict__ xrot, int64_t ldo, float* __restrict__ s64,
                                            int s64_ld, int* __restrict__ status, int n, int b_i, int b_h,
                                            float inv_sqrt_bh, int T) {
    __nv_bfloat16* xin = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [TOK][n]
    __nv_bfloat16* xout = xin + (size_t)TOK * n;                       // [TOK][n], staged variant only
    const int t0 = block * TOK;
    const int nt = min(TOK, T - t0);  // live rows of this CTA
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = kRotThreads / 32;
    constexpr int kRun = 32 * E;
    if (status != nullptr && block == 0 && tid == 0) *status = LOPRO_OK;

    for (int r = 0; r < nt; ++r) {
        const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)(t0 + r) * ldx);
        for (int i = tid; i < n / 8; i += kRotThreads) reinterpret_cast<uint4*>(xin + (size_t)r * n)[i] = __ldg(src + i);
    }
    __syncthreads();

    if constexpr (DIRECT) {
        // identity prefix, b_I a multiple of 64: lane l of a warp gathers eight consecutive columns and stores
        // them as one 16-byte piece; eight lanes cover one 64-column step and add up its sum
        const int n8 = b_i >> 3;
        for (int base = warp * 32; base < n8; base += kWarps * 32) {
            const int k8 = base + lane;
            const bool on = k8 < n8;
            int pk[8];
            if (on) {
                const int4 p0 = __ldg(reinterpret_cast<const int4*>(perm + k8 * 8));
                const int4 p1 = __ldg(reinterpret_cast<const int4*>(perm + k8 * 8 + 4));
                pk[0] = p0.x; pk[1] = p0.y; pk[2] = p0.z; pk[3] = p0.w;
                pk[4] = p1.x; pk[5] = p1.y; pk[6] = p1.z; pk[7] = p1.w;
            }
            for (int r = 0; r < nt; ++r) {
                const __nv_bfloat16* row = xin + (size_t)r * n;
                __nv_bfloat16 o[8];
                float sum = 0.0f;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    o[e] = on ? row[pk[e]] : __float2bfloat16_rn(0.0f);
                    sum += __bfloat162float(o[e]);
                }
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                sum += __shfl_xor_sync(0xffffffffu, sum, 4);
                if (on) {
                    *reinterpret_cast<uint4*>(xrot + (size_t)(t0 + r) * ldo + k8 * 8) = *reinterpret_cast<const uint4*>(o);
                    if (s64 != nullptr && (lane & 7) == 0) s64[(size_t)(t0 + r) * s64_ld + (k8 >> 3)] = sum;
                }
            }
        }
    } else {
        // identity prefix: permuted only
        for (int k = tid; k < b_i; k += kRotThreads) {
            const int pk = __ldg(perm + k);
#pragma unroll
            for (int r = 0; r < TOK; ++r)
                if (r < nt) xout[(size_t)r * n + k] = xin[(size_t)r * n + pk];
        }
    }

    const int nrot = n - b_i;
    const int nruns = (nrot + kRun - 1) / kRun;
    for (int run = warp; run < nruns; run += kWarps) {
        const int rel = run * kRun + lane * E;  // offset inside the rotated region
        int pidx[E];
#pragma unroll
        for (int e = 0; e < E; ++e) pidx[e] = rel + e < nrot ? __ldg(perm + b_i + rel + e) : 0;
        for (int r = 0; r < nt; ++r) {
            const __nv_bfloat16* row = xin + (size_t)r * n;
            float v[E];
#pragma unroll
            for (int e = 0; e < E; ++e) v[e] = rel + e < nrot ? __bfloat162float(row[pidx[e]]) : 0.0f;
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
            if constexpr (DIRECT) {
                // rounded results leave from registers: 16-byte stores, contiguous across the warp; the lanes of a
                // 64-column step add up its sum
                __nv_bfloat16 o[E];
                float sum = 0.0f;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    o[e] = __float2bfloat16_rn(v[e] * inv_sqrt_bh);
                    sum += __bfloat162float(o[e]);
                }
#pragma unroll
                for (int d = 1; d < 64 / E; d <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
                if (rel < nrot) {
                    uint4* dst = reinterpret_cast<uint4*>(xrot + (size_t)(t0 + r) * ldo + b_i + rel);
#pragma unroll
                    for (int q = 0; q < E / 8; ++q) dst[q] = reinterpret_cast<const uint4*>(o)[q];
                    if (s64 != nullptr && (lane & (64 / E - 1)) == 0)
                        s64[(size_t)(t0 + r) * s64_ld + ((b_i + rel) >> 6)] = sum;
                }
            } else {
#pragma unroll
                for (int e = 0; e < E; ++e)
                    if (rel + e < nrot) xout[(size_t)r * n + b_i + rel + e] = __float2bfloat16_rn(v[e] * inv_sqrt_bh);
            }
        }
    }
    if constexpr (DIRECT) return;
    __syncthreads();

    for (int r = 0; r < nt; ++r) {
        const __nv_bfloat16* out_row = xout + (size_t)r * n;
        uint4* dst = reinterpret_cast<uint4*>(xrot + (size_t)(t0 + r) * ldo);
        for (int i = tid; i < n / 8; i += kRotThreads) dst[i] = reinterpret_cast<const uint4*>(out_row)[i];
        if (s64 != nullptr) {
            const int nsteps = n / 64;
            for (int st = warp; st < nsteps; st += kWarps) {
                const __nv_bfloat162 p = reinterpret_cast<const __nv_bfloat162*>(out_row)[st * 32 + lane];
                float s = __low2float(p) + __high2float(p);
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
                if (lane == 0) s64[(size_t)(t0 + r) * s64_ld + st] = s;
            }
        }
    }
}

}  // namespace lopro
