/* Vector-quantized residual: the forward of a layer whose rotated residual R' is stored as indices into codebooks
 * instead of scalar codes -- the "LoPRo_v" variant of the paper (implementation details: a randomly initialised
 * codebook, 4-D at 2 bits per weight, no block-wise scaling, no learned codebooks; the results tables list it beside
 * the scalar form).  Same forward, Eq. 8:  y = A (B x) + W^_vq (Q^T P^T x), with
 *     W^_vq[i, 4 v + e] = C[i / cb_rows][(4 v) / cb_cols][idx[i, v]][e],   e = 0..3,
 * one codebook C[.][.] of 256 four-dimensional bf16 centroids per group of cb_rows rows x cb_cols rotated columns, one
 * 8-bit index per four consecutive rotated columns of a row, no scale.  The paper fixes only the codebook dimension
 * and its random initialisation; granularity and entry format are this library's reading: 512 x 256 with bf16 entries
 * costs 0.125 bit per weight, the figure its average-bit column implies.
 * The 3-bit form (same passage: 2-D codebooks at 3 bits) is desc.dim = 2: 64 two-dimensional centroids per group, one
 * 6-bit index per two consecutive rotated columns,
 *     W^_vq[i, 2 v + e] = C[i / cb_rows][(2 v) / cb_cols][idx[i, v]][e],   e = 0, 1,
 * stored packed: the indices of a row are a little-endian bit stream, vector v in bits [6 v, 6 v + 6) (3 bits per
 * weight; a group of 512 x 256 adds 64 * 2 * 16 / (512 * 256) = 0.016 bit).
 * Conventions as in lopro.h (C ABI, device pointers, caller-owned buffers, asynchronous on `stream`). */
#ifndef LOPRO_VQ_H_
#define LOPRO_VQ_H_

#include "lopro.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lopro_vq_desc {
    int32_t d_in;           /* n, multiple of 64 */
    int32_t d_out;          /* m, multiple of 64 */
    int32_t cb_rows;        /* rows per codebook group, multiple of 64 */
    int32_t cb_cols;        /* rotated columns per codebook group, multiple of 64, divides d_in */
    int32_t block_size;     /* b_H of the rotation, as in lopro_desc */
    int32_t identity_cols;  /* b_I */
    int32_t rank;           /* r of the folded fp16 factors A [m][r], B [r][n]; 0: none */
    int32_t dim;            /* dimension of a centroid: 4 (256 centroids, 8-bit indices; 0 means 4) or 2 (64 centroids, 6-bit) */
} lopro_vq_desc;

/* Bytes of the packed record / of the forward's workspace for up to T tokens (0 on a bad descriptor). */
LOPRO_API size_t lopro_vq_packed_bytes(const lopro_vq_desc* desc);
LOPRO_API size_t lopro_vq_workspace_bytes(const lopro_vq_desc* desc, int32_t T);

/* Packs the record: idx [m][n / dim] one index per byte (the call packs them to 6 bits where dim = 2); codebooks
 * [ceil(m / cb_rows)][n / cb_cols][K][dim] bf16 bits, K = 256 (dim 4) or 64 (dim 2); perm [n]; A [m][r], B [r][n] fp16
 * bits (null with rank 0).  Checks that perm is a permutation of [0, n) and that every index is below K, and returns
 * LOPRO_ERR_INVALID_DATA otherwise (the call synchronises the stream to read the verdict; the record then holds the
 * identity permutation and indices reduced modulo K, so that a forward on it reads in bounds). */
LOPRO_API lopro_status lopro_vq_pack(const lopro_vq_desc* desc, const uint8_t* idx, const uint16_t* codebooks_bf16,
                                     const int32_t* perm, const uint16_t* A_f16, const uint16_t* B_f16, void* packed,
                                     size_t packed_bytes, void* stream);

/* y[t] = A (B x[t]) + W^_vq (Q^T P^T x[t]) for T token rows; x bf16 [T][d_in] (ldx), y [T][d_out] (ldy) bf16 or fp32
 * (LOPRO_OUT_BF16 / LOPRO_OUT_F32).  Rotation and t = B x by the kernels of lopro.h's forward; the product streams the
 * indices once per group of up to 32 tokens, looks the centroids up in shared memory and multiplies on the tensor
 * cores (bf16 x bf16, fp32 accumulation over all of K).  The first word of the workspace is the status word. */
LOPRO_API lopro_status lopro_vq_linear_fwd(const lopro_vq_desc* desc, const void* packed, const uint16_t* x_bf16, int64_t ldx,
                                           void* y, int64_t ldy, int32_t out_dtype, int32_t T, void* workspace,
                                           size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LOPRO_VQ_H_ */
