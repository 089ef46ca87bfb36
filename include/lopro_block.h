/* Decoder-block operations that sit BETWEEN the quantized linear layers when the library runs a whole LLaMA-style
 * decoder stack at decode time (one new token per sequence): RMS normalisation with the residual sum, rotary position
 * embedding with the append to the key/value cache, attention of the new token over the cache, SiLU gating.
 *
 * None of this is part of the quantization method -- the paper's forward (Eq. 8, Appendix A.3) is the linear layer
 * alone; its inference-latency table measures that layer inside such a decoder.  These are the textbook operations of
 * the architecture as plain CUDA kernels, so that the stack workload can be timed end to end with nothing but this
 * library's kernels in the timed region.  Same conventions as lopro.h: C ABI, device pointers, caller-owned buffers,
 * asynchronous on `stream`, host-side argument checks returning a status, no allocation, no synchronisation.
 * All activations are bf16 bit patterns, one token per row with a leading dimension in elements. */
#ifndef LOPRO_BLOCK_H_
#define LOPRO_BLOCK_H_

#include "lopro.h"

#ifdef __cplusplus
extern "C" {
#endif

/* h[t] <- bf16(h[t] + y[t]) (skipped when y is null), then out[t, i] = bf16(h[t, i] * w[i] / sqrt(mean_i h[t, i]^2 + eps)).
 * h [T][d] (ldh), y [T][d] (ldy), w [d], out [T][d] (ldo); fp32 arithmetic; d a multiple of 8, d <= 12288. */
LOPRO_API lopro_status lopro_block_add_rmsnorm(uint16_t* h, int64_t ldh, const uint16_t* y, int64_t ldy, const uint16_t* w,
                                               float eps, uint16_t* out, int64_t ldo, int32_t T, int32_t d, void* stream);

/* Rotary embedding of the new token's query and key, and the append of its key and value to the cache.
 *   q, k, v [T][n_heads * head_dim] (ldq, ldk, ldv): token t belongs to sequence t and sits at position pos[t];
 *   q is rotated in place; rotated k and v are written to k_cache / v_cache [T][n_heads][ctx_max][head_dim] at
 *   entry pos[t] (0 <= pos[t] < ctx_max, checked on the device: a bad position writes nothing and stores
 *   LOPRO_ERR_INVALID_DATA in *status_word).
 *   Pairs (2i, 2i+1) of every head turn by pos * theta^(-2i / head_dim) (angles in double precision).
 *   head_dim even, <= 256. */
LOPRO_API lopro_status lopro_block_rope_append(uint16_t* q, int64_t ldq, const uint16_t* k, int64_t ldk, const uint16_t* v,
                                               int64_t ldv, const int32_t* pos, uint16_t* k_cache, uint16_t* v_cache,
                                               int32_t T, int32_t n_heads, int32_t head_dim, int32_t ctx_max, float theta,
                                               void* status_word, void* stream);

/* out[t, h] = sum_j softmax_j(q[t, h] . K[t, h, j] * scale) V[t, h, j] over j < ctx[t] (1 <= ctx[t] <= ctx_max, else
 * LOPRO_ERR_INVALID_DATA in *status_word and zeros).  The keys are split into pieces of 256 (128 for small batches); a second launch merges the
 * pieces' partial soft-max sums.  head_dim = 128.  workspace: lopro_block_attention_workspace_bytes(...) bytes of
 * device memory, 256-byte aligned.  out [T][n_heads * head_dim] (ldo). */
LOPRO_API size_t lopro_block_attention_workspace_bytes(int32_t T, int32_t n_heads, int32_t head_dim, int32_t ctx_max);
LOPRO_API lopro_status lopro_block_attention_decode(const uint16_t* q, int64_t ldq, const uint16_t* k_cache,
                                                    const uint16_t* v_cache, const int32_t* ctx, uint16_t* out, int64_t ldo,
                                                    int32_t T, int32_t n_heads, int32_t head_dim, int32_t ctx_max, float scale,
                                                    void* workspace, size_t workspace_bytes, void* status_word, void* stream);

/* out[t, i] = bf16(silu(gate[t, i]) * up[t, i]), silu(x) = x / (1 + exp(-x)); d a multiple of 8. */
LOPRO_API lopro_status lopro_block_silu_mul(const uint16_t* gate, int64_t ldg, const uint16_t* up, int64_t ldu, uint16_t* out,
                                            int64_t ldo, int32_t T, int32_t d, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LOPRO_BLOCK_H_ */
