// Decoder-block operations between the quantized linear layers of a LLaMA-style stack at decode time (one new token
// per sequence): residual sum + RMS normalisation, rotary embedding + append to the key/value cache, attention of the
// new token over the cache (split over the keys, merged by a second launch), SiLU gating.  Not part of the
// quantization method: plain kernels, fp32 arithmetic, bf16 in and out, every read and write coalesced.
#include "lopro_block.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace {

constexpr int kSplitKeys = 256;   // keys per attention CTA (128 when that is needed to fill the GPU)
constexpr int kHeadDim = 128;     // the attention kernels are written for this head size
constexpr int kPartial = kHeadDim + 2;  // per (token, head, split): running max, sum of weights, weighted values

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    if ((threadIdx.x & 31) == 0) red[warp] = v;
    __syncthreads();
    float t = 0.0f;
    for (int w = 0; w < nw; ++w) t += red[w];
    __syncthreads();
    return t;
}
__device__ __forceinline__ float block_max(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    if ((threadIdx.x & 31) == 0) red[warp] = v;
    __syncthreads();
    float t = red[0];
    for (int w = 1; w < nw; ++w) t = fmaxf(t, red[w]);
    __syncthreads();
    return t;
}

// One token per CTA: h += y (rounded to bf16, stored), out = h * w / rms(h).
__global__ void __launch_bounds__(256) add_rmsnorm_kernel(__nv_bfloat16* __restrict__ h, int64_t ldh,
                                                          const __nv_bfloat16* __restrict__ y, int64_t ldy,
                                                          const __nv_bfloat16* __restrict__ w, float eps,
                                                          __nv_bfloat16* __restrict__ out, int64_t ldo, int d) {
    extern __shared__ float row[];  // [d]
    __shared__ float red[8];
    const int t = blockIdx.x;
    __nv_bfloat16* hr = h + (size_t)t * ldh;
    float ss = 0.0f;
    for (int i = threadIdx.x; i < d; i += 256) {
        float v = __bfloat162float(hr[i]);
        if (y != nullptr) {
            const __nv_bfloat16 s = __float2bfloat16_rn(v + __bfloat162float(y[(size_t)t * ldy + i]));
            hr[i] = s;
            v = __bfloat162float(s);
        }
        row[i] = v;
        ss = fmaf(v, v, ss);
    }
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += 256)
        out[(size_t)t * ldo + i] = __float2bfloat16_rn(row[i] * inv * __bfloat162float(w[i]));
}

// grid (n_heads, T), one thread per pair of dimensions.
__global__ void rope_append_kernel(__nv_bfloat16* __restrict__ q, int64_t ldq, const __nv_bfloat16* __restrict__ k,
                                   int64_t ldk, const __nv_bfloat16* __restrict__ v, int64_t ldv,
                                   const int32_t* __restrict__ pos, __nv_bfloat16* __restrict__ k_cache,
                                   __nv_bfloat16* __restrict__ v_cache, int n_heads, int head_dim, int ctx_max,
                                   double log2_theta, int* status) {
    const int hd = blockIdx.x, t = blockIdx.y, i = threadIdx.x;
    if (i >= head_dim / 2) return;
    const int p = pos[t];
    if (p < 0 || p >= ctx_max) {
        if (i == 0) atomicCAS(status, LOPRO_OK, LOPRO_ERR_INVALID_DATA);
        return;
    }
    double sn, cs;
    sincos((double)p * exp2(-2.0 * (double)i / (double)head_dim * log2_theta), &sn, &cs);
    const float c = (float)cs, s = (float)sn;
    const size_t col = (size_t)hd * head_dim + 2 * i;
    __nv_bfloat162* qp = reinterpret_cast<__nv_bfloat162*>(q + (size_t)t * ldq + col);
    const float2 qv = __bfloat1622float2(*qp);
    *qp = __floats2bfloat162_rn(qv.x * c - qv.y * s, qv.x * s + qv.y * c);
    const float2 kv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(k + (size_t)t * ldk + col));
    const size_t entry = (((size_t)t * n_heads + hd) * ctx_max + p) * head_dim + 2 * i;
    *reinterpret_cast<__nv_bfloat162*>(k_cache + entry) = __floats2bfloat162_rn(kv.x * c - kv.y * s, kv.x * s + kv.y * c);
    *reinterpret_cast<__nv_bfloat162*>(v_cache + entry) = *reinterpret_cast<const __nv_bfloat162*>(v + (size_t)t * ldv + col);
}

// grid (n_heads, T, splits), 128 threads.  A CTA takes split_keys (256 or 128) consecutive keys of one (sequence, head):
// scores with one key per thread (its 256-byte row in 16-byte loads), soft-max weights of the piece against the
// piece's own maximum, then the weighted values with two dimensions per thread and the keys split by parity.
__global__ void __launch_bounds__(128) attention_split_kernel(const __nv_bfloat16* __restrict__ q, int64_t ldq,
                                                              const __nv_bfloat16* __restrict__ k_cache,
                                                              const __nv_bfloat16* __restrict__ v_cache,
                                                              const int32_t* __restrict__ ctx, int n_heads, int ctx_max,
                                                              int splits, int split_keys, float scale,
                                                              float* __restrict__ partial, int* status) {
    __shared__ __align__(16) float qs[kHeadDim];
    __shared__ float ps[kSplitKeys];
    __shared__ float red[4];
    __shared__ float group_acc[8][kHeadDim];
    const int hd = blockIdx.x, t = blockIdx.y, z = blockIdx.z, tid = threadIdx.x;
    float* out = partial + (((size_t)t * n_heads + hd) * splits + z) * kPartial;
    const int n = ctx[t];
    if (n < 1 || n > ctx_max) {
        if (tid == 0 && hd == 0 && z == 0) atomicCAS(status, LOPRO_OK, LOPRO_ERR_INVALID_DATA);
        if (tid == 0) out[1] = 0.0f;  // an empty piece
        return;
    }
    const int j0 = z * split_keys, cnt = min(split_keys, n - j0);
    if (cnt <= 0) {
        if (tid == 0) out[1] = 0.0f;
        return;
    }
    qs[tid] = __bfloat162float(q[(size_t)t * ldq + (size_t)hd * kHeadDim + tid]) * scale;
    __syncthreads();
    const size_t base = ((size_t)t * n_heads + hd) * ctx_max;
    float mx = -INFINITY;
    for (int j = tid; j < cnt; j += 128) {
        const uint4* kr = reinterpret_cast<const uint4*>(k_cache + (base + j0 + j) * kHeadDim);
        float acc = 0.0f;
#pragma unroll
        for (int c = 0; c < kHeadDim / 8; ++c) {
            const uint4 u = __ldg(kr + c);
            const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 f = __bfloat1622float2(b[e]);
                acc = fmaf(f.x, qs[8 * c + 2 * e], acc);
                acc = fmaf(f.y, qs[8 * c + 2 * e + 1], acc);
            }
        }
        ps[j] = acc;
        mx = fmaxf(mx, acc);
    }
    mx = block_max(mx, red);
    float sum = 0.0f;
    for (int j = tid; j < cnt; j += 128) {
        const float p = __expf(ps[j] - mx);
        ps[j] = p;
        sum += p;
    }
    sum = block_sum(sum, red);  // also orders the writes of ps before the reads below
    // weighted values: sixteen threads cover a 256-byte row with 16-byte loads, the eight groups of sixteen take the
    // keys j = group, group + 8, ...; the groups' sums meet in shared memory in the order of the groups
    const int piece = tid & 15, group = tid >> 4;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
    const uint4* vr = reinterpret_cast<const uint4*>(v_cache + (base + j0) * kHeadDim) + piece;
#pragma unroll 8
    for (int j = group; j < cnt; j += 8) {
        const uint4 u = __ldg(vr + (size_t)j * (kHeadDim / 8));
        const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&u);
        const float p = ps[j];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(b[e]);
            acc[2 * e] = fmaf(p, f.x, acc[2 * e]);
            acc[2 * e + 1] = fmaf(p, f.y, acc[2 * e + 1]);
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) group_acc[group][8 * piece + e] = acc[e];
    __syncthreads();
    {
        float total = 0.0f;
#pragma unroll
        for (int g = 0; g < 8; ++g) total += group_acc[g][tid];
        out[2 + tid] = total;
    }
    if (tid == 0) {
        out[0] = mx;
        out[1] = sum;
    }
}

// grid (n_heads, T), 128 threads: merge the pieces of one (sequence, head).
__global__ void __launch_bounds__(128) attention_merge_kernel(const float* __restrict__ partial, int n_heads, int splits,
                                                              __nv_bfloat16* __restrict__ out, int64_t ldo) {
    const int hd = blockIdx.x, t = blockIdx.y, d = threadIdx.x;
    const float* p = partial + ((size_t)t * n_heads + hd) * splits * kPartial;
    float mx = -INFINITY;
    for (int s = 0; s < splits; ++s)
        if (p[s * kPartial + 1] > 0.0f) mx = fmaxf(mx, p[s * kPartial]);
    float num = 0.0f, den = 0.0f;
    for (int s = 0; s < splits; ++s) {
        const float sum = p[s * kPartial + 1];
        if (sum > 0.0f) {
            const float w = __expf(p[s * kPartial] - mx);
            num = fmaf(w, p[s * kPartial + 2 + d], num);
            den = fmaf(w, sum, den);
        }
    }
    out[(size_t)t * ldo + (size_t)hd * kHeadDim + d] = __float2bfloat16_rn(den > 0.0f ? num / den : 0.0f);
}

__global__ void __launch_bounds__(256) silu_mul_kernel(const __nv_bfloat16* __restrict__ gate, int64_t ldg,
                                                       const __nv_bfloat16* __restrict__ up, int64_t ldu,
                                                       __nv_bfloat16* __restrict__ out, int64_t ldo, int d) {
    const int t = blockIdx.y;
    const int i = (blockIdx.x * 256 + threadIdx.x) * 8;
    if (i >= d) return;
    const uint4 g4 = *reinterpret_cast<const uint4*>(gate + (size_t)t * ldg + i);
    const uint4 u4 = *reinterpret_cast<const uint4*>(up + (size_t)t * ldu + i);
    uint4 o4;
    const __nv_bfloat162* g = reinterpret_cast<const __nv_bfloat162*>(&g4);
    const __nv_bfloat162* u = reinterpret_cast<const __nv_bfloat162*>(&u4);
    __nv_bfloat162* o = reinterpret_cast<__nv_bfloat162*>(&o4);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 a = __bfloat1622float2(g[e]), b = __bfloat1622float2(u[e]);
        o[e] = __floats2bfloat162_rn(a.x / (1.0f + __expf(-a.x)) * b.x, a.y / (1.0f + __expf(-a.y)) * b.y);
    }
    *reinterpret_cast<uint4*>(out + (size_t)t * ldo + i) = o4;
}

}  // namespace

extern "C" {

lopro_status lopro_block_add_rmsnorm(uint16_t* h, int64_t ldh, const uint16_t* y, int64_t ldy, const uint16_t* w, float eps,
                                     uint16_t* out, int64_t ldo, int32_t T, int32_t d, void* stream) {
    if (T < 0 || d < 8 || (d % 8) || d > 12288 || !(eps >= 0.0f)) return LOPRO_ERR_INVALID_ARG;
    if (T == 0) return LOPRO_OK;
    if (!h || !w || !out || ldh < d || ldo < d || (y && ldy < d)) return LOPRO_ERR_INVALID_ARG;
    add_rmsnorm_kernel<<<T, 256, d * sizeof(float), (cudaStream_t)stream>>>(
        reinterpret_cast<__nv_bfloat16*>(h), ldh, reinterpret_cast<const __nv_bfloat16*>(y), ldy,
        reinterpret_cast<const __nv_bfloat16*>(w), eps, reinterpret_cast<__nv_bfloat16*>(out), ldo, d);
    return cudaGetLastError() == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

lopro_status lopro_block_rope_append(uint16_t* q, int64_t ldq, const uint16_t* k, int64_t ldk, const uint16_t* v, int64_t ldv,
                                     const int32_t* pos, uint16_t* k_cache, uint16_t* v_cache, int32_t T, int32_t n_heads,
                                     int32_t head_dim, int32_t ctx_max, float theta, void* status_word, void* stream) {
    if (T < 0 || n_heads < 1 || n_heads > 65535 || head_dim < 2 || (head_dim % 2) || head_dim > 256 || ctx_max < 1 ||
        !(theta > 1.0f))
        return LOPRO_ERR_INVALID_ARG;
    if (T == 0) return LOPRO_OK;
    const int64_t width = (int64_t)n_heads * head_dim;
    if (!q || !k || !v || !pos || !k_cache || !v_cache || !status_word || ldq < width || ldk < width || ldv < width ||
        (ldq % 2) || (ldk % 2) || (ldv % 2) || T > 65535)
        return LOPRO_ERR_INVALID_ARG;
    if (!aligned_to(q, 4) || !aligned_to(k, 4) || !aligned_to(v, 4) || !aligned_to(k_cache, 4) || !aligned_to(v_cache, 4))
        return LOPRO_ERR_INVALID_ARG;
    rope_append_kernel<<<dim3(n_heads, T), (head_dim / 2 + 31) / 32 * 32, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<__nv_bfloat16*>(q), ldq, reinterpret_cast<const __nv_bfloat16*>(k), ldk,
        reinterpret_cast<const __nv_bfloat16*>(v), ldv, pos, reinterpret_cast<__nv_bfloat16*>(k_cache),
        reinterpret_cast<__nv_bfloat16*>(v_cache), n_heads, head_dim, ctx_max, log2((double)theta), (int*)status_word);
    return cudaGetLastError() == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

size_t lopro_block_attention_workspace_bytes(int32_t T, int32_t n_heads, int32_t head_dim, int32_t ctx_max) {
    if (T < 0 || n_heads < 1 || head_dim != kHeadDim || ctx_max < 1) return 0;
    const size_t splits = ((size_t)ctx_max + kSplitKeys / 2 - 1) / (kSplitKeys / 2);  // the finer of the two splits
    return ((size_t)T * n_heads * splits * kPartial * sizeof(float) + 255) / 256 * 256 + 256;
}

lopro_status lopro_block_attention_decode(const uint16_t* q, int64_t ldq, const uint16_t* k_cache, const uint16_t* v_cache,
                                          const int32_t* ctx, uint16_t* out, int64_t ldo, int32_t T, int32_t n_heads,
                                          int32_t head_dim, int32_t ctx_max, float scale, void* workspace,
                                          size_t workspace_bytes, void* status_word, void* stream) {
    if (T < 0 || n_heads < 1 || n_heads > 65535 || ctx_max < 1) return LOPRO_ERR_INVALID_ARG;
    if (head_dim != kHeadDim) return LOPRO_ERR_UNSUPPORTED;
    if (T == 0) return LOPRO_OK;
    const int64_t width = (int64_t)n_heads * head_dim;
    // pieces of 256 keys, or of 128 when there would be too few CTAs for the GPU otherwise
    const int split_keys = (int64_t)T * n_heads * ((ctx_max + kSplitKeys - 1) / kSplitKeys) < 1024 ? kSplitKeys / 2 : kSplitKeys;
    const int splits = (ctx_max + split_keys - 1) / split_keys;
    if (!q || !k_cache || !v_cache || !ctx || !out || !workspace || !status_word || ldq < width || ldo < width || T > 65535 ||
        splits > 65535)
        return LOPRO_ERR_INVALID_ARG;
    if (!aligned_to(k_cache, 16) || !aligned_to(v_cache, 4) || !aligned_to(workspace, 256)) return LOPRO_ERR_INVALID_ARG;
    if (workspace_bytes < lopro_block_attention_workspace_bytes(T, n_heads, head_dim, ctx_max)) return LOPRO_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)stream;
    float* partial = reinterpret_cast<float*>(workspace);
    attention_split_kernel<<<dim3(n_heads, T, splits), 128, 0, s>>>(
        reinterpret_cast<const __nv_bfloat16*>(q), ldq, reinterpret_cast<const __nv_bfloat16*>(k_cache),
        reinterpret_cast<const __nv_bfloat16*>(v_cache), ctx, n_heads, ctx_max, splits, split_keys, scale, partial, (int*)status_word);
    attention_merge_kernel<<<dim3(n_heads, T), 128, 0, s>>>(partial, n_heads, splits, reinterpret_cast<__nv_bfloat16*>(out), ldo);
    return cudaGetLastError() == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

lopro_status lopro_block_silu_mul(const uint16_t* gate, int64_t ldg, const uint16_t* up, int64_t ldu, uint16_t* out,
                                  int64_t ldo, int32_t T, int32_t d, void* stream) {
    if (T < 0 || d < 8 || (d % 8) || T > 65535) return LOPRO_ERR_INVALID_ARG;
    if (T == 0) return LOPRO_OK;
    if (!gate || !up || !out || ldg < d || ldu < d || ldo < d || (ldg % 8) || (ldu % 8) || (ldo % 8)) return LOPRO_ERR_INVALID_ARG;
    if (!aligned_to(gate, 16) || !aligned_to(up, 16) || !aligned_to(out, 16)) return LOPRO_ERR_INVALID_ARG;
    silu_mul_kernel<<<dim3((d / 8 + 255) / 256, T), 256, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const __nv_bfloat16*>(gate), ldg, reinterpret_cast<const __nv_bfloat16*>(up), ldu,
        reinterpret_cast<__nv_bfloat16*>(out), ldo, d);
    return cudaGetLastError() == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

}  // extern "C"
