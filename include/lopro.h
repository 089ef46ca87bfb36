/*
 * lopro.h -- C ABI of the LoPRo quantized-linear forward for NVIDIA B200 (sm_100a).
 *
 * The library evaluates, for a linear layer W in R^{m x n} (m = d_out, n = d_in) that was
 * quantized with LoPRo, the forward of Eq. 8 of the paper,
 *
 *        y = W_r x + Qz(R') Q^T P^T x ,        W_r = A B ,   R' = (W - W_r) P Q ,
 *
 * where P is the column permutation built from the index vector `perm` (Eq. 5), Q the partial
 * block-wise Walsh-Hadamard matrix diag(I_{b_I}, H_wal, ..., H_wal) with blocks of size b_H
 * (Eq. 6, Hadamard recursion of Eq. 2), Qz(R') the group-quantized residual stored as d_q-bit
 * codes with one fp16 scale and one fp16 zero-point per group of g consecutive rotated columns
 * (Appendix A.2), and A = U Sigma [m][r], B = V alpha^-1 [r][n] the folded rank-r factors
 * (Eq. 4).  The steps are those of Appendix A.3: permutation, fast Walsh-Hadamard transform,
 * dequantize-and-multiply, the two skinny low-rank products, and the sum.
 *
 * Conventions
 *   - Activations hold one token per row: x[T][ldx] bf16 (the paper writes tokens as the
 *     columns of X in R^{n x b}).  Outputs y[T][ldy], bf16 or fp32.
 *   - Permutation is a gather: (P^T x)[k] = x[perm[k]].
 *   - Dequantization: W^[i][k] = scale[i][k / g] * (code[i][k] - zero[i][k / g]); column k
 *     is a column of the permuted and rotated basis.
 *   - 16-bit floats cross the ABI as their bit patterns (uint16_t).
 *   - Unless a parameter says "host", every array pointer is a DEVICE pointer that the caller
 *     owns.  The library allocates no memory, frees nothing and never synchronises the
 *     stream, except where an entry point says so.  `stream` is a cudaStream_t passed as
 *     void* (NULL = the default stream).  All work is enqueued on the current device.
 *   - Every entry point validates its arguments on the host and returns a status; none
 *     aborts, exits or traps the GPU.  Asynchronous device-side conditions are reported
 *     through the status word at the start of the workspace (see lopro_linear_fwd).
 *   - There is no CPU fallback: without a usable CUDA device the calls return
 *     LOPRO_ERR_CUDA.
 */
#ifndef LOPRO_H_
#define LOPRO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define LOPRO_API __attribute__((visibility("default")))
#else
#define LOPRO_API
#endif

typedef enum {
    LOPRO_OK = 0,
    LOPRO_ERR_INVALID_ARG = 1,      /* null pointer, bad size, misaligned pointer, bad descriptor  */
    LOPRO_ERR_UNSUPPORTED = 2,      /* legal by the method but outside what the kernels cover     */
    LOPRO_ERR_BUFFER_TOO_SMALL = 3, /* packed blob or workspace smaller than required             */
    LOPRO_ERR_CUDA = 4,             /* a CUDA runtime call failed (no device, launch failure ...)  */
    LOPRO_ERR_TIMEOUT = 5,          /* a bounded device-side wait expired (status word only)      */
    LOPRO_ERR_INVALID_DATA = 6      /* lopro_pack: perm is no permutation, code out of range,
                                       non-finite or zero scale, non-finite zero-point           */
} lopro_status;

/* Output element types of lopro_linear_fwd. */
enum { LOPRO_OUT_BF16 = 0, LOPRO_OUT_F32 = 1 };

/* Code layouts inside the packed blob. */
enum {
    LOPRO_LAYOUT_CANONICAL = 0, /* per row, code k occupies bits [k q, (k+1) q) of a little-endian
                                   bit stream stored as uint32 words (4-bit: 8 codes per word, low
                                   nibble first); interchange format, not accepted by the forward */
    LOPRO_LAYOUT_FRAGMENT = 1,  /* register-fragment order of the warp-level tensor-core kernels   */
    LOPRO_LAYOUT_ROWBLOCK = 2   /* blocks of 128 rows x 64 columns, a row's codes together: the order
                                   the tcgen05 kernels expand into shared-memory operand tiles    */
};

/* Descriptor of one quantized layer (plain data, host memory).
 *   d_in  = n, multiple of 64;  d_out = m, multiple of 16;
 *   bits  = d_q in {2, 3, 4};   group_size = g = 64 * 2^k (64, 128, 256, ...) dividing d_in;
 *   block_size = b_H, a power of two in [2, 1024];
 *   identity_cols = b_I >= 0 with (d_in - b_I) a multiple of b_H (Eq. 6); b_I = d_in disables
 *   the rotation;  rank = r in [0, 512] (stored padded with zeros to a multiple of 16). */
typedef struct {
    int32_t d_in;
    int32_t d_out;
    int32_t bits;
    int32_t group_size;
    int32_t block_size;
    int32_t identity_cols;
    int32_t rank;
    int32_t layout;
    int32_t lowrank_format; /* LOPRO_LOWRANK_FOLDED_F16 or LOPRO_LOWRANK_FP8 */
} lopro_desc;

/* Storage of the rank-r term W_r.
 *   FOLDED_F16: A = U Sigma [m][r] and B = V diag(s)^-1 [r][n] in fp16, the W_L W_R of Eq. 4; y_lr = A (B x).
 *   FP8: the record Algorithm 1 saves, (U, V, Sigma, s): U [m][r] and V [r][n] in fp8 e4m3 (Sec. 3.3 casts the unit
 *   vectors of every R1SVD step to fp8), Sigma [r] and the activation scale s [n] in fp16;
 *   y_lr = U (Sigma (V (x / s))).  Half the bytes per factor entry (Appendix A.2: about 0.05 bit per weight at r = 16).
 *   Served by the small-batch kernels of LOPRO_LAYOUT_FRAGMENT; with more than 32 tokens either as chunks of 32 through
 *   them or, where the tensor-core path is estimated faster, by that path after the record has been folded into fp16
 *   factors in the workspace (A = fp16(U Sigma), B = fp16(V / s): one more rounding per factor entry, one more launch). */
enum { LOPRO_LOWRANK_FOLDED_F16 = 0, LOPRO_LOWRANK_FP8 = 1 };

/* Sections of the packed blob, for lopro_packed_section. */
enum {
    LOPRO_SEC_HEADER = 0,
    LOPRO_SEC_CODES = 1,  /* packed codes in the descriptor's layout                               */
    LOPRO_SEC_SCALEZERO = 2, /* (scale, zero) fp16 pairs: canonical [m][n/g]; fragment layout
                                [m/16][n/g][16]                                                    */
    LOPRO_SEC_PERM = 3,   /* int32 [n]                                                             */
    LOPRO_SEC_A = 4,      /* fp16 [m][r_pad]  (FP8 format: U, e4m3 [m][r_pad])                      */
    LOPRO_SEC_B = 5,      /* fp16 [r_pad][n]  (FP8 format: V, e4m3 [r_pad][n])                      */
    LOPRO_SEC_SIGMA = 6,  /* FP8 format only: fp16 [r_pad]                                         */
    LOPRO_SEC_S = 7,      /* FP8 format only: fp16 [n]                                             */
    LOPRO_SEC_COUNT = 8
};

/* Tuning switches of lopro_configure.  They change which kernels a forward runs, never what it computes; they
 * exist for A/B timing and for tests that must reach a particular kernel (the paper has no counterpart).  The
 * initial value of each is read once per process from the environment variable of the same name
 * (LOPRO_NO_WIDE=1, ...); 0 = default behaviour. */
enum {
    LOPRO_OPT_NO_WIDE = 0,       /* 1: never the 32-warp variant of the streaming kernel                       */
    LOPRO_OPT_NO_TALL = 1,       /* 1: never the persistent streaming kernel for layers with many rows         */
    LOPRO_OPT_NO_CHUNKS = 2,     /* 1: token counts above 32 always take the tensor-core (prefill) kernel      */
    LOPRO_OPT_NO_TCGEN05 = 3,    /* 1: never the tcgen05 prefill kernel (general register-ring product)        */
    LOPRO_OPT_PREFILL_PAIRS = 4, /* >= 0: number of two-block row tiles of the prefill grid; where two CTAs share a
                                     tile (512 tokens and more): number of K parts of the last wave's tiles, 0 or 1
                                     = none, at most 4; -1: chosen by the library                              */
    LOPRO_OPT_ONE_KERNEL_SET = 5, /* 1: single-layer forwards launch the same kernel variants as grouped ones
                                      (lopro_linear_fwd_group / _experts), which carry a table of sibling layers in
                                      their parameters.  By default a single-layer forward launches variants without
                                      that table (0.15-0.4 us less per launch of a small layer); a caller that
                                      alternates single and grouped forwards -- a decoder stack -- then alternates
                                      between two copies of every kernel, which costs more than the table does
                                      (measured: 4 % of a 224-layer decode step).  Such callers set this switch. */
    LOPRO_OPT_NO_CTA_PAIRS = 6,  /* 1: the prefill kernel never pairs two CTAs on a tile (tcgen05 cta_group::2)   */
    LOPRO_OPT_COUNT = 7
};
/* Sets one switch for the whole process (not thread-safe against forwards running on other host threads).
 * Returns LOPRO_ERR_INVALID_ARG for an unknown option. */
LOPRO_API lopro_status lopro_configure(int32_t option, int32_t value);

/* Library version (major * 10000 + minor * 100 + patch). */
LOPRO_API int lopro_version(void);

/* Static, human-readable name of a status code. */
LOPRO_API const char* lopro_status_str(lopro_status s);

/* LOPRO_OK if the descriptor is inside the domain stated above, else the reason class. */
LOPRO_API lopro_status lopro_check_desc(const lopro_desc* desc);

/* Size in bytes of the packed blob of a layer (0 for an invalid descriptor).  The blob is a
 * flat, relocatable byte buffer: a 256-byte header followed by 256-byte aligned sections;
 * copying it (device to device, to the host, to a file) copies the layer.  Its size follows
 * the storage accounting of Eq. 13 with this library's widths: d_q bits per code, 2 x 16 bits
 * per group (scale and zero-point), 16 bits per factor entry (8 in the FP8 low-rank format, plus 16 bits per entry of
 * Sigma and s), 32 bits per permutation entry. */
LOPRO_API size_t lopro_packed_bytes(const lopro_desc* desc);

/* Offset and size in bytes of one section of the blob.  Returns LOPRO_ERR_INVALID_ARG for a
 * bad descriptor or section id. */
LOPRO_API lopro_status lopro_packed_section(const lopro_desc* desc, int32_t section, size_t* offset, size_t* bytes);

/* Bytes of device workspace lopro_linear_fwd needs for up to T tokens (0 on bad arguments).  Non-decreasing
 * in T: a workspace sized for the largest batch serves every smaller one. */
LOPRO_API size_t lopro_workspace_bytes(const lopro_desc* desc, int32_t T);

/* Build the packed blob from plain arrays -- the record (W_q, U, V, Sigma, p, s) that
 * Algorithm 1 saves, with U Sigma and V diag(s)^-1 folded into A and B (Eq. 4).
 *   codes      uint8 [m][n], one code per byte, columns in permuted-and-rotated order
 *   scales_f16 fp16  [m][n/g]        zeros_f16  fp16 [m][n/g] (code units, any finite value)
 *   perm       int32 [n]             A_f16 fp16 [m][r]        B_f16 fp16 [r][n]  (NULL if r = 0)
 *   packed     output blob of packed_bytes >= lopro_packed_bytes(desc), 256-byte aligned
 * The inputs are validated on the device: perm must be a bijection of [0, n), every code
 * < 2^bits, every scale finite and non-zero, every zero-point finite; otherwise
 * LOPRO_ERR_INVALID_DATA is returned and the blob content is unspecified.  This entry point
 * SYNCHRONISES the stream once (to read the validation result); it is a one-time set-up step. */
LOPRO_API lopro_status lopro_pack(const lopro_desc* desc, const uint8_t* codes, const uint16_t* scales_f16,
                        const uint16_t* zeros_f16, const int32_t* perm, const uint16_t* A_f16,
                        const uint16_t* B_f16, void* packed, size_t packed_bytes, void* stream);

/* The same for a layer whose descriptor says LOPRO_LOWRANK_FP8: the saved record (W_q, U, V, Sigma, p, s) of
 * Algorithm 1 as it is, nothing folded.
 *   U_e4m3 uint8 [m][r]   V_e4m3 uint8 [r][n]   (fp8 e4m3 bit patterns; NaN patterns are rejected)
 *   sigma_f16 fp16 [r]    s_f16 fp16 [n]        (finite; s non-zero)
 * Everything else as lopro_pack (which returns LOPRO_ERR_INVALID_ARG for such a descriptor, as this call does for
 * a LOPRO_LOWRANK_FOLDED_F16 one).  rank must be > 0. */
LOPRO_API lopro_status lopro_pack_lr8(const lopro_desc* desc, const uint8_t* codes, const uint16_t* scales_f16,
                                      const uint16_t* zeros_f16, const int32_t* perm, const uint8_t* U_e4m3,
                                      const uint8_t* V_e4m3, const uint16_t* sigma_f16, const uint16_t* s_f16, void* packed,
                                      size_t packed_bytes, void* stream);
/* Reads the low-rank record of an FP8-format blob back, bit for bit (any pointer may be NULL).  For such a blob
 * lopro_unpack returns the codes, scales, zero-points and perm; its A and B pointers must be NULL. */
LOPRO_API lopro_status lopro_unpack_lr8(const lopro_desc* desc, const void* packed, uint8_t* U_e4m3, uint8_t* V_e4m3,
                                        uint16_t* sigma_f16, uint16_t* s_f16, void* stream);

/* Exact inverse of lopro_pack for either layout: writes the arrays lopro_pack was given, bit
 * for bit.  Any output pointer may be NULL to skip that array.  `words` (optional) receives
 * the codes as the canonical uint32 bit stream [m][n*bits/32] regardless of the blob's layout.
 * Checks the blob header against `desc` (one small synchronous device-to-host copy) and returns
 * LOPRO_ERR_INVALID_DATA on a mismatch. */
LOPRO_API lopro_status lopro_unpack(const lopro_desc* desc, const void* packed, uint8_t* codes, uint32_t* words,
                          uint16_t* scales_f16, uint16_t* zeros_f16, int32_t* perm, uint16_t* A_f16,
                          uint16_t* B_f16, void* stream);

/* Activation-side transform of Eq. 8: xrot[t] = Q^T P^T x[t] for T token rows (Appendix A.3:
 * O(n) gather, then log2(b_H) butterfly stages per Hadamard block; Hadamard matrix in the
 * natural order of the recursion of Eq. 2, normalised by 1/sqrt(b_H); the first b_I entries
 * are only permuted).  Butterflies run in fp32, the result is rounded once to bf16.
 *   perm int32 [n] (a section of the blob or any other device array);
 *   x bf16 [T][ldx], xrot bf16 [T][ldo], ldx, ldo >= n; x and xrot 16-byte aligned with ldx
 *   and ldo multiples of 8; x and xrot must not overlap.  Uses d_in, block_size and
 *   identity_cols of the descriptor only.  T = 0 is a no-op. */
LOPRO_API lopro_status lopro_rotate(const lopro_desc* desc, const int32_t* perm, const uint16_t* x_bf16, int64_t ldx,
                          uint16_t* xrot_bf16, int64_t ldo, int32_t T, void* stream);

/* Forward of the quantized layer (Eq. 8; steps of Appendix A.3):
 *        y[t] = A (B x[t]) + W^ (Q^T P^T x[t])           for t in [0, T).
 *   packed    blob written by lopro_pack with LOPRO_LAYOUT_FRAGMENT, 256-byte aligned
 *   x         bf16 [T][ldx], 16-byte aligned, ldx >= n and a multiple of 8
 *   y         bf16 or fp32 [T][ldy] per out_dtype, ldy >= m; must not overlap x
 *   workspace at least lopro_workspace_bytes(desc, T) bytes, 256-byte aligned; scratch for the
 *             rotated activations, the low-rank intermediate and split-K partial sums.  Its
 *             first 4 bytes are a status word: it is set to LOPRO_OK when the call starts and a
 *             kernel that gives up on a bounded wait stores LOPRO_ERR_TIMEOUT there (read it
 *             after synchronising).  Calls that share a workspace must be ordered on one stream.
 * Arithmetic: rotated activations rounded to bf16; B x accumulated in fp32 and rounded to fp16; A
 * times that accumulated in fp32 into the same sum as the quantized part; one final rounding to the
 * output type.  Quantized part, T <= 32: code-times-activation products accumulated in fp32 on the
 * tensor cores, scales and zero-points applied in fp32 (the weights are never rounded).  T > 32:
 * weights dequantized in fp32 and rounded once to bf16, bf16 x bf16 products accumulated in fp32.
 * T = 0 is a no-op. */
LOPRO_API lopro_status lopro_linear_fwd(const lopro_desc* desc, const void* packed, const uint16_t* x_bf16, int64_t ldx,
                              void* y, int64_t ldy, int32_t out_dtype, int32_t T, void* workspace,
                              size_t workspace_bytes, void* stream);

/* Which kernels lopro_linear_fwd runs for this layer and token count on the current device (an
 * implementation detail of this library, exposed so that tests and benchmarks can name what they
 * measure; the paper's Appendix A.3 lists the steps, not their grouping into launches).
 *   LOPRO_PATH_STREAM   2 launches: prologue (permutation, rotation, B x) + streaming product, T <= 32
 *   LOPRO_PATH_WIDE     the same with the 32-warp variant of the streaming kernel (T <= 8, all of K in the ring)
 *   LOPRO_PATH_TALL     the same with the persistent streaming kernel for layers with many output rows
 *   LOPRO_PATH_GENERAL  rotation, B x, register-ring product (any shape the descriptor allows)
 *   LOPRO_PATH_PREFILL  rotation, B x (2 launches), tcgen05 product (one CTA per tile, or two with a launch more
 *                       where the last wave's tiles are cut along K), T > 32
 * For T a little above 32, where the library estimates it to be faster than the tensor-core path (layers with
 * few output rows; e.g. up to 64 tokens for 4096 x 4096), the forward runs as chunks of 32 tokens through the
 * small-batch kernels: STREAM or TALL with one prologue launch and one launch per chunk.
 * Returns the path (> 0) and stores the number of kernel launches in *launches (may be NULL), or
 * returns 0 for a bad descriptor or T < 1. */
typedef enum {
    LOPRO_PATH_STREAM = 2,
    LOPRO_PATH_GENERAL = 3,
    LOPRO_PATH_PREFILL = 4,
    LOPRO_PATH_TALL = 5,
    LOPRO_PATH_WIDE = 6,
    LOPRO_PATH_ROWBLOCK = 7  /* row-block layout: operand image (1 launch; 2-3 for descriptors the prologue kernel
                                does not take) + one tcgen05 small-batch launch per group of up to 32 tokens   */
} lopro_path;
LOPRO_API int32_t lopro_linear_fwd_path(const lopro_desc* desc, int32_t T, int32_t* launches);

/* Forward of several SIBLING layers that read the same activations -- the q/k/v projections of an attention block,
 * the gate/up projections of an MLP: y_i[t] = A_i (B_i x[t]) + W^_i (Q^T P_i^T x[t]), each layer with its own
 * permutation (Eq. 5 depends on the layer's residual and Hessian), low-rank factors and codes.  The paper names the
 * fusion of these steps as future work; its inference-latency table measures exactly this workload, layer by layer.
 *   n_layers >= 1; descs[i], packed[i], y[i], ldy[i] per layer (host arrays of n_layers entries); all layers have
 *   the same d_in; x, out_dtype, T as for lopro_linear_fwd; workspace of lopro_group_workspace_bytes(...) bytes,
 *   256-byte aligned.  The status word of the group is the first word of the workspace.
 * When the layers differ in nothing but d_out and their data, are in LOPRO_LAYOUT_FRAGMENT, n_layers <= 8, T <= 32 and
 * each would run as prologue + small-batch kernel of the same kind (all per-row-group, or all persistent: the
 * persistent CTAs are then shared out in proportion to the layers' rows), the group runs as TWO launches: one
 * prologue that writes every layer's rotated activations and B_i x, and one product launch over the row tiles of
 * all layers.  Otherwise the
 * layers run one after the other (same results, one lopro_linear_fwd each).  lopro_linear_fwd_group_path returns 2
 * in the first case, 1 in the second (0 on bad arguments) and the number of launches in *launches. */
LOPRO_API size_t lopro_group_workspace_bytes(int32_t n_layers, const lopro_desc* const* descs, int32_t T);
LOPRO_API int32_t lopro_linear_fwd_group_path(int32_t n_layers, const lopro_desc* const* descs, int32_t T, int32_t* launches);
LOPRO_API lopro_status lopro_linear_fwd_group(int32_t n_layers, const lopro_desc* const* descs, const void* const* packed,
                                              const uint16_t* x_bf16, int64_t ldx, void* const* y, const int64_t* ldy,
                                              int32_t out_dtype, int32_t T, void* workspace, size_t workspace_bytes,
                                              void* stream);

/* The same forward for callers whose activations live in HOST memory (Eq. 8 end to end):
 * copies x_host [T][n] (dense, bf16; pinned memory makes the copy asynchronous) to the device,
 * runs lopro_linear_fwd and copies y [T][m] back to y_host.  `workspace` must hold
 * lopro_workspace_bytes(desc, T) + lopro_host_staging_bytes(desc, T, out_dtype) bytes.  The call
 * enqueues everything on `stream` and does not synchronise; y_host is valid after the caller
 * synchronises the stream. */
LOPRO_API size_t lopro_host_staging_bytes(const lopro_desc* desc, int32_t T, int32_t out_dtype);
LOPRO_API lopro_status lopro_linear_fwd_host(const lopro_desc* desc, const void* packed, const uint16_t* x_host,
                                   void* y_host, int32_t out_dtype, int32_t T, void* workspace,
                                   size_t workspace_bytes, void* stream);

/* Forward for callers that cannot allocate device memory (the paper has no counterpart of this entry
 * point; it is a deployment convenience of this library).  Meant for code that runs where asking the
 * driver for memory is not an option: a plug-in inside a host program that owns the whole device
 * heap and hands out none of it, a latency-critical serving loop in which cudaMalloc's implicit
 * device synchronisation would stall every other stream, or a process started with a fixed memory
 * budget.  It computes exactly what lopro_linear_fwd computes, with the same arguments minus the
 * workspace: the scratch is a fixed array of LOPRO_NOALLOC_SCRATCH_BYTES inside the library itself
 * (every GPU that loads the library holds that memory until the process ends).
 *   - Accepted sizes: lopro_workspace_bytes(desc, T) <= LOPRO_NOALLOC_SCRATCH_BYTES, which covers
 *     the small-batch (decode) range of ordinary layers, e.g. d_in = 8192 with T <= 32.  Anything
 *     larger returns LOPRO_ERR_BUFFER_TOO_SMALL and does nothing.
 *   - The call allocates and frees nothing and does not synchronise.  The first call on each device
 *     looks up the array's device address (once per device, with that device current); make that
 *     first call before any stream capture begins.
 *   - All calls on one device share the one array and it keeps what the last call left in it.  No
 *     part of it needs clearing between calls (each forward rewrites what it reads), but two calls
 *     whose kernels overlap on the GPU -- different streams, or concurrent host threads -- race on
 *     it: order every use of this entry point on a device through one stream.
 *   - The workspace status word of lopro_linear_fwd is not visible here; use lopro_linear_fwd when
 *     the device-side status matters. */
#define LOPRO_NOALLOC_SCRATCH_BYTES (8 * 1024 * 1024)
LOPRO_API lopro_status lopro_linear_fwd_noalloc(const lopro_desc* desc, const void* packed, const uint16_t* x_bf16,
                                                int64_t ldx, void* y, int64_t ldy, int32_t out_dtype, int32_t T,
                                                void* stream);

/* Self-test of the library's failure detection (the paper has no counterpart).  Every wait of the forward
 * kernels on a shared-memory barrier is bounded: when the limit runs out the kernel stores LOPRO_ERR_TIMEOUT in
 * the workspace status word and returns normally instead of hanging.  This call exercises exactly that code path
 * without any fault: it launches one thread block that initialises a barrier, announces bytes that no copy will
 * ever deliver (nothing is in flight when the block exits), waits on it with the library's bounded wait under a
 * short limit (4096 polls), and on expiry stores LOPRO_ERR_TIMEOUT in *status_word (device memory, 4 bytes,
 * 4-byte aligned; the kernel first stores LOPRO_OK there).  Asynchronous: read the word after synchronising. */
LOPRO_API lopro_status lopro_selftest_wait(void* status_word, void* stream);

/* Forward of the EXPERTS of a mixture-of-experts layer (the paper quantizes Mixtral-8x7B expert by expert and lists
 * MoE models among its evaluations): n_experts layers of one shape (`desc`), each with its own packed record, and a
 * batch of token rows already grouped by expert, as a router's sort leaves them: expert e owns rows
 * [row_offsets[e], row_offsets[e+1]) of x and of y (row_offsets: HOST array of n_experts + 1 non-decreasing entries,
 * row_offsets[0] = 0; an expert without rows is skipped).  y[t] = A_e (B_e x[t]) + W^_e (Q^T P_e^T x[t]) for the rows
 * t of expert e (Eq. 8 per expert).
 *   x [rows][d_in] bf16 (ldx), y [rows][d_out] (ldy, out_dtype); workspace of
 *   lopro_experts_workspace_bytes(desc, n_experts, max_rows) bytes, max_rows >= the largest row count of an expert,
 *   256-byte aligned.
 * When no expert has more than 32 rows and the layer runs through the small-batch kernels (LOPRO_LAYOUT_FRAGMENT,
 * folded fp16 record), every 8 experts with rows run as TWO launches: one prologue (each expert its own permutation,
 * B and rows) and one product launch over the row tiles of all of them, both shaped for the largest row count.
 * Otherwise the experts run one after the other.  Status words: the first word of the workspace for the first 8
 * experts with rows, the first word of the k-th such expert's region (workspace_bytes / n_experts each) for the
 * next 8, and so on; in the one-after-the-other case every expert's region starts with its own.
 * lopro_linear_fwd_experts_path returns 2 / 1 for the two cases (0 on bad arguments) and the number of launches. */
LOPRO_API size_t lopro_experts_workspace_bytes(const lopro_desc* desc, int32_t n_experts, int32_t max_rows);
LOPRO_API int32_t lopro_linear_fwd_experts_path(const lopro_desc* desc, int32_t n_experts, const int32_t* row_offsets,
                                                int32_t* launches);
LOPRO_API lopro_status lopro_linear_fwd_experts(const lopro_desc* desc, int32_t n_experts, const void* const* packed,
                                                const int32_t* row_offsets, const uint16_t* x_bf16, int64_t ldx, void* y,
                                                int64_t ldy, int32_t out_dtype, void* workspace, size_t workspace_bytes,
                                                void* stream);

/* ---------------------------------------------------------------------------------------------------
 * Offline side of the method on the GPU (Algorithm 1 without its calibration inputs): the step BEFORE the forward
 * path.  All matrices are fp32 device memory, row-major; every call is asynchronous on `stream`.
 *
 * lopro_r1svd -- rank-1 randomized sketch with deflation (Sec. 3.3, Eq. 10-12; inner loop of Algorithm 1).  Per rank
 *   j: y = (W W^T)^it W v_j, p = W^T y, U_j = y / |y|, V_j = p / |p|, sigma_j = |p| / |y|, optionally U_j, V_j
 *   rounded to fp8 e4m3 (cast = 1; the values are then those fp8 numbers, held in fp32), then W <- W - sigma_j U_j V_j^T.
 *   The vector is renormalised after every product (a scaling that cancels in U_j, V_j and sigma_j), so no power of
 *   W overflows.  A rank whose y or p vanishes (matrix exhausted) and all later ones come out as zeros.
 *     w        [m][n], IN: the matrix to decompose (W diag(s)); OUT: the deflated remainder
 *     sketches [r][n] Gaussian test vectors v_j (the call draws nothing)
 *     U [m][r], sigma [r], V [r][n] outputs; workspace of lopro_r1svd_workspace_bytes(m, n) bytes, 256-byte aligned
 *   m, n multiples of 4, 1 <= r <= 512, 0 <= it <= 64.  The work is 2 it + 2 matrix-vector products and one
 *   rank-1 update per rank: memory-bound passes over w.
 *
 * lopro_residual_rotate -- R' = (W - Af Bf) P Q (Eq. 3 form ii, Eq. 5, Eq. 6), one row of W at a time: the residual
 *   against the STORED low-rank factors (Af [m][rank], Bf [rank][n] hold the stored values, e.g. fp16 numbers or
 *   U Sigma and V diag(s)^-1 formed from the fp8 / fp16 record; rank = desc->rank, may be 0 with null factors), the
 *   column gather R[:, perm[k]] and the partial block Walsh-Hadamard rotation of every row (the same transform the
 *   forward applies to an activation row), in fp32.  r_rot [m][n].  d_in <= 24576.
 *   An index of perm outside [0, n) stores LOPRO_ERR_INVALID_DATA in *status_word (device, 4 bytes) and reads column 0.
 *
 * lopro_rtn_quantize -- the group grid of Appendix A.2 by round-to-nearest (ablation row 'RTN'): per row and group of
 *   g consecutive columns of r_rot, lo = min, hi = max, scale = fp16((hi - lo) / (2^q - 1)),
 *   zero = fp16(rne(-lo / scale)), code = clamp(rne(v / scale) + zero, 0, 2^q - 1); a constant group v stores scale |v|
 *   (1 if v = 0), zero 1 if v < 0 else 0, code 1 if v > 0 else 0.  Every operation is an IEEE single-precision operation
 *   rounded to nearest-even, in this order.  Outputs in the input formats of lopro_pack: codes [m][n] one per byte,
 *   scales, zeros [m][n/g] fp16 bits.  A non-finite input or a group whose step rounds to zero in fp16 stores
 *   LOPRO_ERR_INVALID_DATA in *status_word.
 *
 * lopro_quantize_layer -- the three steps in sequence for one layer: W_s = W diag(s) (s null: ones; with
 *   LOPRO_LOWRANK_FP8 s is first rounded to fp16, as stored), R1SVD of W_s (fp8 cast inside the loop for
 *   LOPRO_LOWRANK_FP8), the record's factors, the residual against them, rotation and quantization.
 *     lr0..lr3: LOPRO_LOWRANK_FOLDED_F16: lr0 = A [m][r] fp16 = fp16(U Sigma), lr1 = B [r][n] fp16 = fp16(V diag(s)^-1);
 *               LOPRO_LOWRANK_FP8: lr0 = U [m][r] e4m3, lr1 = V [r][n] e4m3, lr2 = Sigma [r] fp16, lr3 = s [n] fp16
 *     -- exactly the arguments of lopro_pack / lopro_pack_lr8.  rank = 0: no factors, R = W.
 *   The first word of the workspace is the status word; workspace of lopro_quantize_workspace_bytes(desc) bytes
 *   (a copy of W among other things). */
LOPRO_API size_t lopro_r1svd_workspace_bytes(int32_t m, int32_t n);
LOPRO_API lopro_status lopro_r1svd(float* w, int32_t m, int32_t n, int32_t r, int32_t it, const float* sketches,
                                   int32_t cast, float* U, float* sigma, float* V, void* workspace,
                                   size_t workspace_bytes, void* stream);
LOPRO_API lopro_status lopro_residual_rotate(const lopro_desc* desc, const float* W, const float* Af, const float* Bf,
                                             const int32_t* perm, float* r_rot, void* status_word, void* stream);
LOPRO_API lopro_status lopro_rtn_quantize(const lopro_desc* desc, const float* r_rot, uint8_t* codes, uint16_t* scales,
                                          uint16_t* zeros, void* status_word, void* stream);
LOPRO_API size_t lopro_quantize_workspace_bytes(const lopro_desc* desc);
LOPRO_API lopro_status lopro_quantize_layer(const lopro_desc* desc, const float* W, const float* s, const int32_t* perm,
                                            const float* sketches, int32_t it, uint8_t* codes, uint16_t* scales,
                                            uint16_t* zeros, void* lr0, void* lr1, void* lr2, void* lr3, void* workspace,
                                            size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LOPRO_H_ */
