// Internal declarations shared by the translation units of liblopro (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lopro.h"

namespace lopro {

constexpr uint32_t kBlobMagic = 0x4F52504Cu;  // "LPRO"
constexpr uint32_t kBlobVersion = 1;
constexpr int kHeaderBytes = 256;
constexpr int kSectionAlign = 256;

// Header at offset 0 of the packed blob (256 bytes reserved).
struct BlobHeader {
    uint32_t magic;
    uint32_t version;
    lopro_desc desc;
    uint64_t total_bytes;
    uint64_t sec_off[LOPRO_SEC_COUNT];
    uint64_t sec_bytes[LOPRO_SEC_COUNT];
    uint32_t invalid;  // validation flags written by lopro_pack's check kernels (0 = clean)
    uint32_t reserved[3];
};
static_assert(sizeof(BlobHeader) <= kHeaderBytes, "header must fit its slot");

enum : uint32_t {
    kInvalidPermRange = 1u,
    kInvalidPermDuplicate = 2u,
    kInvalidCode = 4u,
    kInvalidScale = 8u,
    kInvalidZero = 16u,
    kInvalidLowrank = 32u,  // FP8 record: NaN pattern in U or V, non-finite Sigma, non-finite or zero s
};

struct BlobLayout {
    size_t off[LOPRO_SEC_COUNT];
    size_t bytes[LOPRO_SEC_COUNT];
    size_t total;
    int r_pad;
};

// Host: validates the descriptor and fills the section table.
lopro_status check_desc(const lopro_desc& d);
lopro_status blob_layout(const lopro_desc& d, BlobLayout* out);

// Raises a kernel's dynamic shared-memory limit once per device (function attributes are per device);
// later calls, e.g. during stream capture, make no CUDA call.  `done` is a per-kernel bit mask.
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, int bytes, unsigned long long* done) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = 1ull << (dev & 63);
    if (__atomic_load_n(done, __ATOMIC_ACQUIRE) & bit) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) __atomic_fetch_or(done, bit, __ATOMIC_RELEASE);
    return e;
}

// Tuning switches (lopro_configure; initial values from the environment, read once per process).
int option(int id);
// Multiprocessors of the current device (cached per device; 148 if the query fails).
int sm_count();

inline int round_up_int(int v, int a) { return (v + a - 1) / a * a; }
inline size_t round_up_size(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Workspace of lopro_linear_fwd: status word, rotated activations, 64-column sums of the rotated
// activations, low-rank intermediate (fp16, general path), per-chunk partial sums of the low-rank
// intermediate (fp32, small-batch path).
struct WorkspaceLayout {
    size_t off_status, off_xrot, off_s64, off_t, off_lrpart, off_kparts, off_fold_a, off_fold_b, total;
    int t_pad;  // tokens padded to a multiple of 8
    // row-block layout only: the operand image of the tcgen05 small-batch kernel (see ImageOut)
    size_t off_counters, off_ximg, off_sums, off_timg, off_partial;
    int np;        // tokens per image tile: 16 (T <= 16) or 32
    int n_tgroups; // token groups of np tokens
};
constexpr int kDecodeMaxT = 32;               // tokens per CTA of the streaming kernels
constexpr int kStreamMaxSmem = 220 * 1024;    // dynamic shared memory the small-batch kernel may use
// Row stride of the 64-column sums: a whole number of 16-step stages, so that a stage's sums of one
// token are one aligned 64-byte piece.
inline int s64_stride(int n) { return ((n / 64 + 15) / 16) * 16; }
// Small-batch path: the prologue stores the rotated activations as the shared-memory image of the
// streaming kernel's stages, [stage of 1024 columns][token][kActRecord bytes]: 1024 bf16 entries, the
// sixteen 64-column sums (fp32), 16 bytes of padding (the odd multiple of 16 bytes keeps ldmatrix
// reads of eight tokens conflict-free).  One bulk copy then brings a stage's activations.
constexpr int kActRecord = 2048 + 64 + 16;
inline size_t act_image_bytes(int n, int t_pad) { return (size_t)((n + 1023) / 1024) * t_pad * kActRecord; }
lopro_status workspace_layout(const lopro_desc& d, int T, WorkspaceLayout* out);

// Operand image of the tcgen05 small-batch kernel, written by the prologue (or converted from the plain rotated
// activations): per group of NP tokens and 64-column step one K-major tile [NP tokens][64 columns] of bf16 with the
// 128-byte swizzle the MMA reads (token row tl, 16-byte piece c at byte tl * 128 + ((c ^ (tl & 7)) << 4)), so that a
// plain bulk copy brings a tile; sums of the rotated (bf16-rounded) activations over runs of gs = min(g, 256) columns,
// [token group][run][NP] fp32; the low-rank intermediate t = B x as fp16 tiles of the same shape over the rank; and
// the per-row-block arrival counters of the split-K reduction, cleared by whoever writes the image.
constexpr int kRbMaxGrid = 160;  // CTAs of the tcgen05 small-batch kernel (one per SM), bound used to size the partial sums
struct ImageOut {
    unsigned char* ximg;  // nullptr: the record format of the warp-level kernels is written instead
    float* sums;
    unsigned char* timg;
    int* counters;
    int n_counters;
    int np, np_shift;   // tokens per tile (16 or 32) and its log2
    int nsteps;         // 64-column steps of K
    int gs_shift;       // log2(gs / 64): 0, 1 or 2
    int n_sums;         // d_in / gs
    int lr_steps;       // 64-column steps of the padded rank
};
inline size_t ximg_bytes(int n, int np) { return (size_t)(n / 64) * np * 128; }
inline int sum_run(const lopro_desc& d) { return d.group_size < 256 ? d.group_size : 256; }
ImageOut image_out(const lopro_desc& d, uint8_t* ws, const WorkspaceLayout& W);

// ---- launchers (each returns the CUDA status of its launches) -------------------------------
cudaError_t launch_validate(const lopro_desc& d, const uint8_t* codes, const uint16_t* scales,
                            const uint16_t* zeros, const int32_t* perm, void* blob, const BlobLayout& L,
                            cudaStream_t s);
cudaError_t launch_pack(const lopro_desc& d, const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros,
                        const int32_t* perm, const uint16_t* A, const uint16_t* B, void* blob,
                        const BlobLayout& L, cudaStream_t s);
// FP8 low-rank record: validation (flags in the header) and the copy into / out of the blob.
cudaError_t launch_pack_lr8(const lopro_desc& d, const uint8_t* U, const uint8_t* V, const uint16_t* sigma, const uint16_t* svec,
                            void* blob, const BlobLayout& L, cudaStream_t s);
cudaError_t launch_unpack_lr8(const lopro_desc& d, const void* blob, const BlobLayout& L, uint8_t* U, uint8_t* V,
                              uint16_t* sigma, uint16_t* svec, cudaStream_t s);
cudaError_t launch_unpack(const lopro_desc& d, const void* blob, const BlobLayout& L, uint8_t* codes,
                          uint32_t* words, uint16_t* scales, uint16_t* zeros, int32_t* perm, uint16_t* A,
                          uint16_t* B, cudaStream_t s);
// Rotation; s64 (optional) receives the sums of each aligned run of 64 rotated (bf16-rounded)
// entries, [T][n/64] fp32.
cudaError_t launch_rotate(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                          __nv_bfloat16* xrot, int64_t ldo, float* s64, int* status, int T, cudaStream_t s);
// Small-batch prologue: rotation, 64-column sums and t = B x in one launch.
bool prologue_supported(const lopro_desc& d, int T);
// Sibling layers of a grouped forward: they read the same x and differ only in their rows (d_out) and data.
constexpr int kMaxSiblings = 8;
struct PrologueSiblings {  // siblings 1 .. n of a grouped prologue (sibling 0 travels in the ordinary arguments)
    int n;
    const int32_t* perm[kMaxSiblings - 1];
    const __half* B[kMaxSiblings - 1];
    unsigned char* act[kMaxSiblings - 1];
    __half* t[kMaxSiblings - 1];
    // own_rows != 0 (experts of a mixture layer): sibling z = 0 .. n reads its own rows x_of[z] and has T_of[z] of
    // them; the launch is shaped for the largest count and the siblings with fewer rows leave the rest idle
    int own_rows;
    const __nv_bfloat16* x_of[kMaxSiblings];
    int T_of[kMaxSiblings];
};
// FP8 low-rank record: t = Sigma (V (x / s)) instead of t = B x (V null: folded fp16 format).
struct Lr8Args {
    const uint8_t* V;      // e4m3 [r_pad][n]
    const __half* sigma;   // [r_pad]
    const __half* svec;    // [n]
};
cudaError_t launch_prologue(const lopro_desc& d, const int32_t* perm, const __half* B, int r_pad,
                            const __nv_bfloat16* x, int64_t ldx, unsigned char* act_image, __half* t, int t_pad,
                            int* status, int T, cudaStream_t s, const ImageOut* img = nullptr,
                            const PrologueSiblings* siblings = nullptr, const Lr8Args* lr8 = nullptr);
// Plain rotated activations, 64-column sums and t (the general path's outputs) -> operand image.
cudaError_t launch_image_convert(const lopro_desc& d, const __nv_bfloat16* xrot, const float* s64, int s64_ld,
                                 const __half* t, int r_pad, const ImageOut& img, int T, cudaStream_t s);
// tcgen05 small-batch forward over the row-block layout, one launch per group of up to 32 tokens.
bool rowblock_supported(const lopro_desc& d);
int rowblock_launches(const lopro_desc& d);  // launches per group of up to 32 tokens (1 unless the layer is very large)
cudaError_t launch_rowblock(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, uint8_t* ws,
                            const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int tgroup, int t_live,
                            cudaStream_t s);
// t[T][r_pad] (fp16) = B x, fp32 accumulation.
cudaError_t launch_lowrank_down(const lopro_desc& d, const __half* B, int r_pad, const __nv_bfloat16* x,
                                int64_t ldx, __half* t, int T, cudaStream_t s);
// General forward over the fragment layout: any T, after launch_rotate and launch_lowrank_down.
cudaError_t launch_decode(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, const uint8_t* ws,
                          const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int T, cudaStream_t s);
// Small-batch forward (T <= 32) after launch_prologue: bulk-copy ring, one CTA per 32 output rows.
bool stream_supported(const lopro_desc& d, int T);
bool stream_uses_wide(const lopro_desc& d, int T);  // the 32-warp variant of the kernel will run
// `more`: sibling layers of a grouped launch (same descriptor but for d_out; each with its own blob, workspace
// region laid out like W, and output) whose row tiles are appended to the grid.
struct StreamSiblingArgs {
    int n;
    const uint8_t* blob[kMaxSiblings - 1];
    BlobLayout L[kMaxSiblings - 1];
    const uint8_t* ws[kMaxSiblings - 1];
    void* y[kMaxSiblings - 1];
    int64_t ldy[kMaxSiblings - 1];
    int d_out[kMaxSiblings - 1];
    // own_rows != 0: token counts per sibling, T_of[0] for the layer of the ordinary arguments (whose T then only
    // shapes the launch: the largest of the counts)
    int own_rows;
    int T_of[kMaxSiblings];
};
cudaError_t launch_stream(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, const uint8_t* ws,
                          const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int T, cudaStream_t s, int t0 = 0,
                          const StreamSiblingArgs* more = nullptr);

// Small-batch forward for tall layers after launch_prologue: persistent CTAs, one ring across tile groups.
bool tall_supported(const lopro_desc& d, int T, long long total_rows = 0);  // total_rows: of all siblings sharing the launch
cudaError_t launch_tall(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, const uint8_t* ws,
                        const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int T, cudaStream_t s, int t0 = 0,
                        const StreamSiblingArgs* more = nullptr);

// t = B x on the tensor cores for many tokens; `partial` holds lowrank_mma_scratch_bytes of fp32 K-slice sums.
size_t lowrank_mma_scratch_bytes(const lopro_desc& d, int T);
cudaError_t launch_lowrank_down_mma(const lopro_desc& d, const __half* B, int r_pad, const __nv_bfloat16* x, int64_t ldx,
                                    float* partial, __half* t, int T, cudaStream_t s);
// Rotation and t = B x of a many-token forward in one grid (plus the dependent launch that adds the K slices).
bool rotate_lowrank_supported(const lopro_desc& d, int T);
cudaError_t launch_rotate_lowrank(const lopro_desc& d, const int32_t* perm, const __nv_bfloat16* x, int64_t ldx,
                                  __nv_bfloat16* xrot, int64_t ldo, float* s64, int* status, const __half* B, int r_pad,
                                  float* partial, __half* t, int T, cudaStream_t s);
// Prefill forward (T > 32) on tcgen05 / TMEM, after launch_rotate and launch_lowrank_down.
bool prefill_supported(const lopro_desc& d, int T);
// Tiling of the prefill kernel that puts two CTAs on a tile (large batches): n_tiles tiles of 256 rows x 512 tokens, the
// last split_tiles of them cut along K into k_parts units whose fp32 partial sums meet in the workspace.
struct PairPlan {
    int use, row_tiles, n_tiles, split_tiles, k_parts;
};
PairPlan pair_plan(const lopro_desc& d, int T);
size_t prefill_kparts_bytes(const lopro_desc& d, int T);
// Estimated duration (microseconds) of the tensor-core product for T > 32 tokens and whether it runs two CTAs per tile
double prefill_estimate_us(const lopro_desc& d, int T, bool* use_pairs);
// FP8 low-rank record -> fp16 factors A = U Sigma [m][r_pad], B = V / s [r_pad][n] in the workspace (tensor-core path)
cudaError_t launch_lr8_fold(const lopro_desc& d, int r_pad, const uint8_t* U, const uint8_t* V, const __half* sigma,
                            const __half* svec, __half* A, __half* B, cudaStream_t s);
cudaError_t launch_prefill(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, const uint8_t* ws,
                           const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int T, cudaStream_t s,
                           const void* a_f16 = nullptr);  // a_f16: the up factor where it is not the blob's section

// ---- fragment layout ----------------------------------------------------------------------
// Codes are stored per tile of 16 rows x 64 columns as [32 lanes][q words].  Lane l = 4 gq + tg
// owns, for each of the four 16-column sub-steps j, the four register pairs rho = 0..3 of the
// A operand of mma.m16n8k16:  row = gq + 8 (rho & 1),  column = 16 j + 8 (rho >> 1) + 2 tg + h,
// h = 0 (low half) or 1 (high half).  Pair index pi = 4 j + rho.
//   4-bit: word j;      low code at bit 4 rho,       high code at bit 16 + 4 rho
//   2-bit: word pi / 8; low code at bit 2 (pi % 8),  high code at bit 16 + 2 (pi % 8)
//   3-bit: pi < 15: word pi / 5, low at bit 3 (pi % 5), high at bit 16 + 3 (pi % 5);
//          pi = 15: bit b of the low code is bit 15 of word b, of the high code bit 31 of word b.
struct FragPos {
    size_t word;     // index of the uint32 inside the blob's code section
    uint32_t shift;  // bit position of the code's bit 0 (2- and 4-bit, 3-bit with pi < 15)
    bool scattered;  // 3-bit pi = 15: bit b lives at bit `shift` of word + b
};

__host__ __device__ inline FragPos frag_pos(int bits, int n, int row, int k) {
    const int rt = row >> 4, rr = row & 15, gq = rr & 7, hi8 = rr >> 3;
    const int ks = k >> 6, kk = k & 63, j = kk >> 4, c = kk & 15;
    const int rho = hi8 + 2 * (c >> 3), c8 = c & 7, tg = c8 >> 1, h = c8 & 1;
    const int lane = 4 * gq + tg, pi = 4 * j + rho;
    const size_t base = (((size_t)rt * (size_t)(n >> 6) + (size_t)ks) * 32u + (size_t)lane) * (size_t)bits;
    FragPos p;
    p.scattered = false;
    if (bits == 4) {
        p.word = base + j;
        p.shift = 4 * rho + 16 * h;
    } else if (bits == 2) {
        p.word = base + (pi >> 3);
        p.shift = 2 * (pi & 7) + 16 * h;
    } else {
        if (pi < 15) {
            p.word = base + pi / 5;
            p.shift = 3 * (pi % 5) + 16 * h;
        } else {
            p.word = base;
            p.shift = 15 + 16 * h;
            p.scattered = true;
        }
    }
    return p;
}

// ---- row-block layout -------------------------------------------------------------------------
// Codes are stored per block of up to 128 rows (the last block holds the remaining rows, a multiple of 16) and
// 64-column step: R rows x 2 q words, the steps of a block one after the other, so that any run of steps of a block
// is one contiguous piece.  A row's 2 q words of a step are its two 32-column half-steps, each q words in the bit
// order of expand_codes with pair pi = columns (2 pi, 2 pi + 1) of the half-step: expanding a half-step yields the
// row's 32 columns as sixteen bf16 pairs in memory order, i.e. four 16-byte pieces of a K-major operand tile.  Inside
// a (block, step) the words are kept as planes of 4 words per row (the last plane of a 3-bit step has 2), [plane][row],
// so that thread r of a warp reads its row's plane with one conflict-free 16-byte (8-byte) load.
constexpr int kRbRows = 128;

__host__ __device__ inline int rb_rows(int m, int rb) { return m - rb * kRbRows < kRbRows ? m - rb * kRbRows : kRbRows; }
// word offset of the (block, step) piece inside the code section
__host__ __device__ inline size_t rb_step_word(int bits, int nsteps, int m, int rb, int ks) {
    return ((size_t)rb * kRbRows * (size_t)nsteps + (size_t)ks * (size_t)rb_rows(m, rb)) * (size_t)(2 * bits);
}
// word offset of word w (0 .. 2 q - 1) of row r inside a (block, step) piece of R rows
__host__ __device__ inline int rb_word_in_step(int bits, int R, int r, int w) {
    const int plane = w >> 2, len = (2 * bits - 4 * plane) < 4 ? (2 * bits - 4 * plane) : 4;
    return 4 * plane * R + r * len + (w & 3);
}
__host__ __device__ inline FragPos rb_pos(int bits, int n, int m, int row, int k) {
    const int rb = row >> 7, r = row & 127, ks = k >> 6, kk = k & 63, hs = kk >> 5, c = kk & 31, pi = c >> 1, h = c & 1;
    const int R = rb_rows(m, rb);
    const size_t base = rb_step_word(bits, n >> 6, m, rb, ks);
    FragPos p;
    p.scattered = false;
    int wi;
    if (bits == 4) {
        wi = pi >> 2;
        p.shift = 4 * (pi & 3) + 16 * h;
    } else if (bits == 2) {
        wi = pi >> 3;
        p.shift = 2 * (pi & 7) + 16 * h;
    } else if (pi < 15) {
        wi = pi / 5;
        p.shift = 3 * (pi % 5) + 16 * h;
    } else {
        wi = 0;  // bit b of the code sits at bit `shift` of half-step word b
        p.shift = 15 + 16 * h;
        p.scattered = true;
    }
    p.word = base + (size_t)rb_word_in_step(bits, R, r, hs * bits + wi);
    return p;
}
// word index of half-step word b (scattered 3-bit codes): words of one half-step may straddle two planes
__host__ __device__ inline size_t rb_halfstep_word(int bits, int n, int m, int row, int k, int b) {
    const int rb = row >> 7, r = row & 127, ks = k >> 6, hs = (k & 63) >> 5;
    return rb_step_word(bits, n >> 6, m, rb, ks) + (size_t)rb_word_in_step(bits, rb_rows(m, rb), r, hs * bits + b);
}
// (scale, zero) pairs in the row-block layout: [block][group][R rows] half2.
__host__ __device__ inline size_t sz_rb_index(int n_groups, int m, int row, int grp) {
    const int rb = row >> 7;
    return (size_t)rb * kRbRows * (size_t)n_groups + (size_t)grp * (size_t)rb_rows(m, rb) + (size_t)(row & 127);
}

// (scale, zero) pairs in the fragment layout: [m/16][n/g][16 rows] half2.
__host__ __device__ inline size_t sz_frag_index(int n_groups, int row, int grp) {
    return ((size_t)(row >> 4) * (size_t)n_groups + (size_t)grp) * 16u + (size_t)(row & 15);
}

}  // namespace lopro
