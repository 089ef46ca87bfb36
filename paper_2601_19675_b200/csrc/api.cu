// Host side of the C ABI: argument validation, blob and workspace layout, dispatch.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace lopro {

lopro_status check_desc(const lopro_desc& d) {
    if (d.d_in <= 0 || d.d_out <= 0) return LOPRO_ERR_INVALID_ARG;
    if (d.bits != 2 && d.bits != 3 && d.bits != 4) return LOPRO_ERR_INVALID_ARG;
    if (d.group_size <= 0 || d.d_in % d.group_size != 0) return LOPRO_ERR_INVALID_ARG;
    if (d.block_size < 2 || d.block_size > 1024 || (d.block_size & (d.block_size - 1))) return LOPRO_ERR_INVALID_ARG;
    if (d.identity_cols < 0 || d.identity_cols > d.d_in) return LOPRO_ERR_INVALID_ARG;
    if ((d.d_in - d.identity_cols) % d.block_size != 0) return LOPRO_ERR_INVALID_ARG;
    if (d.rank < 0 || d.rank > 512) return LOPRO_ERR_INVALID_ARG;
    if (d.lowrank_format != LOPRO_LOWRANK_FOLDED_F16 && d.lowrank_format != LOPRO_LOWRANK_FP8) return LOPRO_ERR_INVALID_ARG;
    if (d.lowrank_format == LOPRO_LOWRANK_FP8 && d.rank == 0) return LOPRO_ERR_INVALID_ARG;
    if (d.layout != LOPRO_LAYOUT_CANONICAL && d.layout != LOPRO_LAYOUT_FRAGMENT && d.layout != LOPRO_LAYOUT_ROWBLOCK)
        return LOPRO_ERR_INVALID_ARG;
    // Kernel coverage: 64-column steps, 16-row tiles, rows short enough for one CTA's shared memory.
    if (d.d_in % 64 != 0 || d.d_out % 16 != 0 || d.group_size % 64 != 0) return LOPRO_ERR_UNSUPPORTED;
    if ((d.group_size / 64) & (d.group_size / 64 - 1)) return LOPRO_ERR_UNSUPPORTED;  // g = 64 * 2^k
    if (d.d_in > 32768 || d.d_out > (1 << 20)) return LOPRO_ERR_UNSUPPORTED;
    return LOPRO_OK;
}

lopro_status blob_layout(const lopro_desc& d, BlobLayout* out) {
    lopro_status st = check_desc(d);
    if (st != LOPRO_OK) return st;
    const size_t m = d.d_out, n = d.d_in, ng = d.d_in / d.group_size;
    const int r_pad = round_up_int(d.rank, 16);
    size_t bytes[LOPRO_SEC_COUNT];
    bytes[LOPRO_SEC_HEADER] = kHeaderBytes;
    bytes[LOPRO_SEC_CODES] = m * n * (size_t)d.bits / 8;
    bytes[LOPRO_SEC_SCALEZERO] = m * ng * 4;
    bytes[LOPRO_SEC_PERM] = n * 4;
    const size_t esz = d.lowrank_format == LOPRO_LOWRANK_FP8 ? 1 : 2;
    bytes[LOPRO_SEC_A] = m * (size_t)r_pad * esz;
    bytes[LOPRO_SEC_B] = (size_t)r_pad * n * esz;
    bytes[LOPRO_SEC_SIGMA] = d.lowrank_format == LOPRO_LOWRANK_FP8 ? (size_t)r_pad * 2 : 0;
    bytes[LOPRO_SEC_S] = d.lowrank_format == LOPRO_LOWRANK_FP8 ? n * 2 : 0;
    size_t off = 0;
    for (int s = 0; s < LOPRO_SEC_COUNT; ++s) {
        out->off[s] = off;
        out->bytes[s] = bytes[s];
        off = round_up_size(off + bytes[s], kSectionAlign);
    }
    out->total = off;
    out->r_pad = r_pad;
    return LOPRO_OK;
}

lopro_status workspace_layout(const lopro_desc& d, int T, WorkspaceLayout* W) {
    lopro_status st = check_desc(d);
    if (st != LOPRO_OK) return st;
    if (T < 0) return LOPRO_ERR_INVALID_ARG;
    const int t_pad = round_up_int(T > 0 ? T : 1, 8);
    const int r_pad = round_up_int(d.rank, 16);
    size_t off = 0;
    W->t_pad = t_pad;
    W->off_status = off;
    off += 256;
    W->off_xrot = off;
    {
        // rotated activations, or the activation image of the small-batch kernels (a little larger)
        size_t xb = (size_t)t_pad * d.d_in * 2;
        if (act_image_bytes(d.d_in, t_pad) > xb) xb = act_image_bytes(d.d_in, t_pad);
        off += round_up_size(xb, 256);
    }
    W->off_s64 = off;
    off += round_up_size((size_t)t_pad * s64_stride(d.d_in) * 4, 256);
    W->off_t = off;
    off += round_up_size((size_t)t_pad * (r_pad > 0 ? r_pad : 16) * 2, 256);
    W->off_lrpart = off;
    if (T > kDecodeMaxT && d.rank > 0) off += round_up_size(lowrank_mma_scratch_bytes(d, T), 256);
    W->off_kparts = off;
    off += round_up_size(prefill_kparts_bytes(d, T), 256);
    // FP8 low-rank record on the tensor-core path: the fp16 factors it is folded into
    W->off_fold_a = W->off_fold_b = off;
    if (d.lowrank_format == LOPRO_LOWRANK_FP8 && T > kDecodeMaxT) {
        W->off_fold_a = off;
        off += round_up_size((size_t)d.d_out * r_pad * 2, 256);
        W->off_fold_b = off;
        off += round_up_size((size_t)r_pad * d.d_in * 2, 256);
    }
    // operand image of the tcgen05 small-batch kernel (row-block layout)
    W->np = T <= 16 ? 16 : 32;
    W->n_tgroups = T <= 16 ? 1 : (T + 31) / 32;
    W->off_counters = W->off_ximg = W->off_sums = W->off_timg = W->off_partial = off;
    if (d.layout == LOPRO_LAYOUT_ROWBLOCK) {
        const size_t tg = (size_t)W->n_tgroups;
        W->off_counters = off;
        off += round_up_size((size_t)((d.d_out + kRbRows - 1) / kRbRows) * 4, 256);
        W->off_ximg = round_up_size(off, 1024);
        off = W->off_ximg + tg * ximg_bytes(d.d_in, W->np);
        W->off_sums = off;
        off += round_up_size(tg * (size_t)(d.d_in / sum_run(d)) * W->np * 4, 1024);
        W->off_timg = off;
        off += tg * (size_t)((r_pad + 63) / 64) * W->np * 128;
        W->off_partial = off;
        off += (size_t)2 * kRbMaxGrid * W->np * kRbRows * 4;
    }
    W->total = off;
    return LOPRO_OK;
}

ImageOut image_out(const lopro_desc& d, uint8_t* ws, const WorkspaceLayout& W) {
    ImageOut o;
    o.ximg = ws + W.off_ximg;
    o.sums = reinterpret_cast<float*>(ws + W.off_sums);
    o.timg = ws + W.off_timg;
    o.counters = reinterpret_cast<int*>(ws + W.off_counters);
    o.n_counters = (d.d_out + kRbRows - 1) / kRbRows;
    o.np = W.np;
    o.np_shift = W.np == 16 ? 4 : 5;
    o.nsteps = d.d_in / 64;
    const int gs = sum_run(d);
    o.gs_shift = gs == 64 ? 0 : (gs == 128 ? 1 : 2);
    o.n_sums = d.d_in / gs;
    o.lr_steps = (round_up_int(d.rank, 16) + 63) / 64;
    return o;
}

static bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

namespace {
int g_options[LOPRO_OPT_COUNT];
int g_options_ready = 0;  // 0 = not read yet, 1 = being read, 2 = ready

void read_options_once() {
    int expected = 0;
    if (__atomic_compare_exchange_n(&g_options_ready, &expected, 1, false, __ATOMIC_ACQ_REL, __ATOMIC_ACQUIRE)) {
        static const char* const names[LOPRO_OPT_COUNT] = {"LOPRO_NO_WIDE", "LOPRO_NO_TALL", "LOPRO_NO_CHUNKS",
                                                           "LOPRO_NO_TCGEN05", "LOPRO_PREFILL_PAIRS",
                                                           "LOPRO_ONE_KERNEL_SET", "LOPRO_NO_CTA_PAIRS"};
        for (int i = 0; i < LOPRO_OPT_COUNT; ++i) {
            const char* e = getenv(names[i]);
            g_options[i] = e ? atoi(e) : (i == LOPRO_OPT_PREFILL_PAIRS ? -1 : 0);
        }
        __atomic_store_n(&g_options_ready, 2, __ATOMIC_RELEASE);
    } else {
        while (__atomic_load_n(&g_options_ready, __ATOMIC_ACQUIRE) != 2) {
        }
    }
}
}  // namespace

int option(int id) {
    if (__atomic_load_n(&g_options_ready, __ATOMIC_ACQUIRE) != 2) read_options_once();
    return __atomic_load_n(&g_options[id], __ATOMIC_RELAXED);
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    int& c = cached[dev & 63];
    if (c == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        c = v;
    }
    return c;
}

}  // namespace lopro

using namespace lopro;

extern "C" {

int lopro_version(void) { return 100; }

const char* lopro_status_str(lopro_status s) {
    switch (s) {
        case LOPRO_OK: return "ok";
        case LOPRO_ERR_INVALID_ARG: return "invalid argument";
        case LOPRO_ERR_UNSUPPORTED: return "unsupported configuration";
        case LOPRO_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case LOPRO_ERR_CUDA: return "CUDA error";
        case LOPRO_ERR_TIMEOUT: return "device-side wait timed out";
        case LOPRO_ERR_INVALID_DATA: return "invalid layer data";
    }
    return "unknown status";
}

lopro_status lopro_check_desc(const lopro_desc* desc) {
    if (!desc) return LOPRO_ERR_INVALID_ARG;
    return check_desc(*desc);
}

size_t lopro_packed_bytes(const lopro_desc* desc) {
    BlobLayout L;
    if (!desc || blob_layout(*desc, &L) != LOPRO_OK) return 0;
    return L.total;
}

lopro_status lopro_packed_section(const lopro_desc* desc, int32_t section, size_t* offset, size_t* bytes) {
    BlobLayout L;
    if (!desc || section < 0 || section >= LOPRO_SEC_COUNT) return LOPRO_ERR_INVALID_ARG;
    lopro_status st = blob_layout(*desc, &L);
    if (st != LOPRO_OK) return st;
    if (offset) *offset = L.off[section];
    if (bytes) *bytes = L.bytes[section];
    return LOPRO_OK;
}

size_t lopro_workspace_bytes(const lopro_desc* desc, int32_t T) {
    WorkspaceLayout W;
    if (!desc || workspace_layout(*desc, T, &W) != LOPRO_OK) return 0;
    return W.total;
}

static lopro_status pack_any(const lopro_desc* desc, const uint8_t* codes, const uint16_t* scales_f16,
                             const uint16_t* zeros_f16, const int32_t* perm, const uint16_t* A_f16, const uint16_t* B_f16,
                             const uint8_t* U8, const uint8_t* V8, const uint16_t* sigma, const uint16_t* svec, void* packed,
                             size_t packed_bytes, void* stream) {
    BlobLayout L;
    lopro_status st = blob_layout(*desc, &L);
    if (st != LOPRO_OK) return st;
    const bool lr8 = desc->lowrank_format == LOPRO_LOWRANK_FP8;
    if (!codes || !scales_f16 || !zeros_f16 || !perm || !packed) return LOPRO_ERR_INVALID_ARG;
    if (!lr8 && desc->rank > 0 && (!A_f16 || !B_f16)) return LOPRO_ERR_INVALID_ARG;
    if (lr8 && (!U8 || !V8 || !sigma || !svec)) return LOPRO_ERR_INVALID_ARG;
    if (!aligned(packed, 256)) return LOPRO_ERR_INVALID_ARG;
    if (packed_bytes < L.total) return LOPRO_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)stream;

    BlobHeader h;
    memset(&h, 0, sizeof(h));
    h.magic = kBlobMagic;
    h.version = kBlobVersion;
    h.desc = *desc;
    h.total_bytes = L.total;
    for (int i = 0; i < LOPRO_SEC_COUNT; ++i) {
        h.sec_off[i] = L.off[i];
        h.sec_bytes[i] = L.bytes[i];
    }
    // Zero the whole blob (padding bytes included, so that equal layers give equal blobs), then
    // the header.  The header source is on this stack frame: the copy below is synchronous with
    // respect to the host for pageable memory, and the stream is synchronised before returning.
    if (cudaMemsetAsync(packed, 0, L.total, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (cudaMemcpyAsync(packed, &h, sizeof(h), cudaMemcpyHostToDevice, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (launch_validate(*desc, codes, scales_f16, zeros_f16, perm, packed, L, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (launch_pack(*desc, codes, scales_f16, zeros_f16, perm, lr8 ? nullptr : A_f16, lr8 ? nullptr : B_f16, packed, L, s) !=
        cudaSuccess)
        return LOPRO_ERR_CUDA;
    if (lr8 && launch_pack_lr8(*desc, U8, V8, sigma, svec, packed, L, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    BlobHeader back;
    if (cudaMemcpyAsync(&back, packed, sizeof(back), cudaMemcpyDeviceToHost, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (back.magic != kBlobMagic) return LOPRO_ERR_CUDA;
    if (back.invalid != 0) {
        // A rejected blob must stay harmless if a caller ignores the status and runs a forward on it: the kernels
        // gather x[perm[k]] without a range check, so the permutation section is cleared (every entry 0, in range;
        // codes were masked to their width while packing).  The header keeps the validation flags.
        if (cudaMemsetAsync((uint8_t*)packed + L.off[LOPRO_SEC_PERM], 0, L.bytes[LOPRO_SEC_PERM], s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess)
            return LOPRO_ERR_CUDA;
        return LOPRO_ERR_INVALID_DATA;
    }
    return LOPRO_OK;
}

lopro_status lopro_pack(const lopro_desc* desc, const uint8_t* codes, const uint16_t* scales_f16,
                        const uint16_t* zeros_f16, const int32_t* perm, const uint16_t* A_f16,
                        const uint16_t* B_f16, void* packed, size_t packed_bytes, void* stream) {
    if (!desc) return LOPRO_ERR_INVALID_ARG;
    if (check_desc(*desc) == LOPRO_OK && desc->lowrank_format != LOPRO_LOWRANK_FOLDED_F16) return LOPRO_ERR_INVALID_ARG;
    return pack_any(desc, codes, scales_f16, zeros_f16, perm, A_f16, B_f16, nullptr, nullptr, nullptr, nullptr, packed,
                    packed_bytes, stream);
}

lopro_status lopro_pack_lr8(const lopro_desc* desc, const uint8_t* codes, const uint16_t* scales_f16,
                            const uint16_t* zeros_f16, const int32_t* perm, const uint8_t* U_e4m3, const uint8_t* V_e4m3,
                            const uint16_t* sigma_f16, const uint16_t* s_f16, void* packed, size_t packed_bytes, void* stream) {
    if (!desc) return LOPRO_ERR_INVALID_ARG;
    if (check_desc(*desc) == LOPRO_OK && desc->lowrank_format != LOPRO_LOWRANK_FP8) return LOPRO_ERR_INVALID_ARG;
    return pack_any(desc, codes, scales_f16, zeros_f16, perm, nullptr, nullptr, U_e4m3, V_e4m3, sigma_f16, s_f16, packed,
                    packed_bytes, stream);
}

static lopro_status read_header(const lopro_desc* desc, const void* packed, const BlobLayout& L, cudaStream_t s) {
    BlobHeader h;
    if (cudaMemcpyAsync(&h, packed, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (h.magic != kBlobMagic || h.version != kBlobVersion || memcmp(&h.desc, desc, sizeof(lopro_desc)) != 0 ||
        h.total_bytes != L.total || h.invalid != 0)
        return LOPRO_ERR_INVALID_DATA;
    return LOPRO_OK;
}

lopro_status lopro_unpack_lr8(const lopro_desc* desc, const void* packed, uint8_t* U_e4m3, uint8_t* V_e4m3,
                              uint16_t* sigma_f16, uint16_t* s_f16, void* stream) {
    if (!desc || !packed) return LOPRO_ERR_INVALID_ARG;
    BlobLayout L;
    lopro_status st = blob_layout(*desc, &L);
    if (st != LOPRO_OK) return st;
    if (desc->lowrank_format != LOPRO_LOWRANK_FP8) return LOPRO_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    st = read_header(desc, packed, L, s);
    if (st != LOPRO_OK) return st;
    return launch_unpack_lr8(*desc, packed, L, U_e4m3, V_e4m3, sigma_f16, s_f16, s) == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

lopro_status lopro_unpack(const lopro_desc* desc, const void* packed, uint8_t* codes, uint32_t* words,
                          uint16_t* scales_f16, uint16_t* zeros_f16, int32_t* perm, uint16_t* A_f16,
                          uint16_t* B_f16, void* stream) {
    if (!desc || !packed) return LOPRO_ERR_INVALID_ARG;
    BlobLayout L;
    lopro_status st = blob_layout(*desc, &L);
    if (st != LOPRO_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    if (desc->lowrank_format == LOPRO_LOWRANK_FP8 && (A_f16 || B_f16)) return LOPRO_ERR_INVALID_ARG;
    st = read_header(desc, packed, L, s);
    if (st != LOPRO_OK) return st;
    if (launch_unpack(*desc, packed, L, codes, words, scales_f16, zeros_f16, perm, A_f16, B_f16, s) != cudaSuccess)
        return LOPRO_ERR_CUDA;
    return LOPRO_OK;
}

lopro_status lopro_rotate(const lopro_desc* desc, const int32_t* perm, const uint16_t* x_bf16, int64_t ldx,
                          uint16_t* xrot_bf16, int64_t ldo, int32_t T, void* stream) {
    if (!desc) return LOPRO_ERR_INVALID_ARG;
    lopro_status st = check_desc(*desc);
    if (st != LOPRO_OK) return st;
    if (T < 0) return LOPRO_ERR_INVALID_ARG;
    if (T == 0) return LOPRO_OK;
    if (!perm || !x_bf16 || !xrot_bf16) return LOPRO_ERR_INVALID_ARG;
    if (ldx < desc->d_in || ldo < desc->d_in || (ldx % 8) || (ldo % 8)) return LOPRO_ERR_INVALID_ARG;
    if (!aligned(x_bf16, 16) || !aligned(xrot_bf16, 16) || !aligned(perm, 4)) return LOPRO_ERR_INVALID_ARG;
    cudaError_t e = launch_rotate(*desc, perm, (const __nv_bfloat16*)x_bf16, ldx, (__nv_bfloat16*)xrot_bf16, ldo,
                                  nullptr, nullptr, T, (cudaStream_t)stream);
    return e == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

// LOPRO_OPT_NO_TALL keeps the persistent kernel for tall layers off (A/B comparison and tests of the other kernel).
static bool use_tall(const lopro_desc& d, int T, long long total_rows = 0) {
    if (option(LOPRO_OPT_NO_TALL) == 1) return false;
    return tall_supported(d, T, total_rows);
}
// Sibling layers that share their launches: the persistent kernel when their rows together make more than one wave of
// the per-group kernel (three 4096-row projections do, each alone does not).
static bool group_uses_tall(int32_t n, const lopro_desc* const* descs, int32_t T) {
    long long rows = 0;
    for (int i = 0; i < n; ++i) rows += descs[i]->d_out;
    return use_tall(*descs[0], T, rows);
}

// Token counts a little above the small-batch range run as ONE prologue plus chunks of kDecodeMaxT tokens through
// the small-batch kernels when that costs less than the tensor-core path: a prefill CTA walks all of K for its
// 128 or 256 rows whatever the token count, and a layer with few rows fills few SMs.  Both sides are estimated from
// timings on B200 (microseconds, beyond a common 8 for the first launches): a chunk 3 + 0.45e-6 d_out d_in (10.9 for
// 4096 x 4096, 23.4 for 4096 x 11008 either way round), the tensor-core product by prefill_estimate_us plus 0.0015 d_in
// for the longer launches in front of it (4096 x 4096: chunks up to 64 tokens, 25.0 against 29.8; 11008 -> 4096: up to
// 96, 77 against 84).  LOPRO_OPT_NO_CHUNKS turns this off (A/B runs, tests of the prefill kernels on small layers).
static int small_batch_chunks(const lopro_desc& d, int T) {
    if (T <= kDecodeMaxT) return 0;
    // the FP8 low-rank record has no general path: chunks wherever the tensor-core kernels cannot take the layer
    if (d.lowrank_format == LOPRO_LOWRANK_FP8 && !prefill_supported(d, T))
        return (prologue_supported(d, kDecodeMaxT) && stream_supported(d, kDecodeMaxT)) ? (T + kDecodeMaxT - 1) / kDecodeMaxT : 0;
    if (option(LOPRO_OPT_NO_CHUNKS) == 1) return 0;
    if (!prefill_supported(d, T)) return 0;  // keep the general path's behaviour where there is no prefill kernel
    const int chunks = (T + kDecodeMaxT - 1) / kDecodeMaxT;
    const double chunk_us = 3.0 + 0.45e-6 * (double)d.d_out * (double)d.d_in;
    const double prefill_us = prefill_estimate_us(d, T, nullptr) + 0.0015 * (double)d.d_in;  // + its longer launches in front
    if ((double)chunks * chunk_us >= prefill_us) return 0;
    if (!prologue_supported(d, kDecodeMaxT) || !stream_supported(d, kDecodeMaxT)) return 0;
    return chunks;
}

// Row-block layout: launches before the product (the prologue, or rotation + B x + image conversion).
static int rowblock_pre_launches(const lopro_desc& d, int T) {
    if (prologue_supported(d, 1)) return 1;
    return 2 + (d.rank > 0 ? 1 : 0);
}

// The FP8 low-rank record is served by the prologue + small-batch kernels of the fragment layout.
static bool lr8_unsupported(const lopro_desc& d) {
    return d.lowrank_format == LOPRO_LOWRANK_FP8 &&
           (d.layout != LOPRO_LAYOUT_FRAGMENT || !prologue_supported(d, 1) || !stream_supported(d, kDecodeMaxT));
}

int32_t lopro_linear_fwd_path(const lopro_desc* desc, int32_t T, int32_t* launches) {
    if (!desc || check_desc(*desc) != LOPRO_OK || desc->layout == LOPRO_LAYOUT_CANONICAL || T < 1) return 0;
    if (lr8_unsupported(*desc)) return 0;
    if (desc->layout == LOPRO_LAYOUT_ROWBLOCK) {
        if (!rowblock_supported(*desc)) return 0;
        if (launches) *launches = rowblock_pre_launches(*desc, T) + rowblock_launches(*desc) * (T <= 16 ? 1 : (T + 31) / 32);
        return LOPRO_PATH_ROWBLOCK;
    }
    int32_t path, n;
    if (const int chunks = small_batch_chunks(*desc, T)) {
        path = use_tall(*desc, kDecodeMaxT) ? LOPRO_PATH_TALL : LOPRO_PATH_STREAM;
        n = 1 + chunks;
    } else if (prologue_supported(*desc, T) && stream_supported(*desc, T)) {
        path = use_tall(*desc, T) ? LOPRO_PATH_TALL : (stream_uses_wide(*desc, T) ? LOPRO_PATH_WIDE : LOPRO_PATH_STREAM);
        n = 2;
    } else {
        const int pre = (T > kDecodeMaxT && rotate_lowrank_supported(*desc, T))
                            ? 2
                            : 1 + (desc->rank > 0 ? (T > kDecodeMaxT ? 2 : 1) : 0);
        path = prefill_supported(*desc, T) ? LOPRO_PATH_PREFILL : LOPRO_PATH_GENERAL;
        n = pre + 1;
        if (desc->lowrank_format == LOPRO_LOWRANK_FP8) ++n;  // the record folded into fp16 factors
        if (path == LOPRO_PATH_PREFILL) {
            bool use_pairs = false;
            (void)prefill_estimate_us(*desc, T, &use_pairs);
            if (use_pairs && pair_plan(*desc, T).split_tiles > 0) ++n;  // the sum of the K parts of the last wave's tiles
        }
    }
    if (launches) *launches = n;
    return path;
}

lopro_status lopro_linear_fwd(const lopro_desc* desc, const void* packed, const uint16_t* x_bf16, int64_t ldx,
                              void* y, int64_t ldy, int32_t out_dtype, int32_t T, void* workspace,
                              size_t workspace_bytes, void* stream) {
    if (!desc) return LOPRO_ERR_INVALID_ARG;
    BlobLayout L;
    lopro_status st = blob_layout(*desc, &L);
    if (st != LOPRO_OK) return st;
    if (desc->layout == LOPRO_LAYOUT_CANONICAL) return LOPRO_ERR_UNSUPPORTED;
    if (desc->layout == LOPRO_LAYOUT_ROWBLOCK && !rowblock_supported(*desc)) return LOPRO_ERR_UNSUPPORTED;
    if (lr8_unsupported(*desc)) return LOPRO_ERR_UNSUPPORTED;
    if (T < 0 || (out_dtype != LOPRO_OUT_BF16 && out_dtype != LOPRO_OUT_F32)) return LOPRO_ERR_INVALID_ARG;
    if (T == 0) return LOPRO_OK;
    if (!packed || !x_bf16 || !y || !workspace) return LOPRO_ERR_INVALID_ARG;
    if (ldx < desc->d_in || (ldx % 8) || ldy < desc->d_out) return LOPRO_ERR_INVALID_ARG;
    if (!aligned(packed, 256) || !aligned(workspace, 256) || !aligned(x_bf16, 16) ||
        !aligned(y, out_dtype == LOPRO_OUT_F32 ? 4 : 2))
        return LOPRO_ERR_INVALID_ARG;
    WorkspaceLayout W;
    st = workspace_layout(*desc, T, &W);
    if (st != LOPRO_OK) return st;
    if (workspace_bytes < W.total) return LOPRO_ERR_BUFFER_TOO_SMALL;

    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)workspace;
    const uint8_t* blob = (const uint8_t*)packed;
    const int32_t* perm = (const int32_t*)(blob + L.off[LOPRO_SEC_PERM]);
    const __half* B = (const __half*)(blob + L.off[LOPRO_SEC_B]);
    __nv_bfloat16* xrot = (__nv_bfloat16*)(ws + W.off_xrot);
    float* s64 = (float*)(ws + W.off_s64);
    int* status = (int*)(ws + W.off_status);
    Lr8Args lr8 = {};
    if (desc->lowrank_format == LOPRO_LOWRANK_FP8) {
        lr8.V = blob + L.off[LOPRO_SEC_B];
        lr8.sigma = (const __half*)(blob + L.off[LOPRO_SEC_SIGMA]);
        lr8.svec = (const __half*)(blob + L.off[LOPRO_SEC_S]);
    }
    if (desc->layout == LOPRO_LAYOUT_ROWBLOCK) {
        // operand image (one launch where the prologue kernel takes the descriptor), then one tcgen05 launch per
        // group of up to 32 tokens
        const ImageOut img = image_out(*desc, ws, W);
        if (prologue_supported(*desc, 1)) {
            if (launch_prologue(*desc, perm, B, L.r_pad, (const __nv_bfloat16*)x_bf16, ldx, nullptr, nullptr, W.t_pad, status,
                                T, s, &img) != cudaSuccess)
                return LOPRO_ERR_CUDA;
        } else {
            if (launch_rotate(*desc, perm, (const __nv_bfloat16*)x_bf16, ldx, xrot, desc->d_in, s64, status, T, s) !=
                cudaSuccess)
                return LOPRO_ERR_CUDA;
            if (desc->rank > 0 && launch_lowrank_down(*desc, B, L.r_pad, (const __nv_bfloat16*)x_bf16, ldx,
                                                      (__half*)(ws + W.off_t), T, s) != cudaSuccess)
                return LOPRO_ERR_CUDA;
            if (launch_image_convert(*desc, xrot, s64, s64_stride(desc->d_in), (const __half*)(ws + W.off_t), L.r_pad, img, T,
                                     s) != cudaSuccess)
                return LOPRO_ERR_CUDA;
        }
        for (int tg = 0; tg < W.n_tgroups; ++tg) {
            const int live = T - tg * W.np < W.np ? T - tg * W.np : W.np;
            if (launch_rowblock(*desc, blob, L, ws, W, y, ldy, out_dtype, tg, live, s) != cudaSuccess) return LOPRO_ERR_CUDA;
        }
        return LOPRO_OK;
    }
    if (const int chunks = small_batch_chunks(*desc, T)) {
        // one prologue for all tokens, then chunks of kDecodeMaxT tokens through the small-batch kernels, each
        // reading its tokens' records of the activation image and rows of t
        if (launch_prologue(*desc, perm, B, L.r_pad, (const __nv_bfloat16*)x_bf16, ldx, ws + W.off_xrot,
                            (__half*)(ws + W.off_t), W.t_pad, status, T, s, nullptr, nullptr, &lr8) != cudaSuccess)
            return LOPRO_ERR_CUDA;
        const size_t esz = out_dtype == LOPRO_OUT_F32 ? 4 : 2;
        for (int c = 0; c < chunks; ++c) {
            const int t0 = c * kDecodeMaxT, tc = T - t0 < kDecodeMaxT ? T - t0 : kDecodeMaxT;
            void* yc = (uint8_t*)y + (size_t)t0 * ldy * esz;
            const cudaError_t e = use_tall(*desc, tc) ? launch_tall(*desc, blob, L, ws, W, yc, ldy, out_dtype, tc, s, t0)
                                                      : launch_stream(*desc, blob, L, ws, W, yc, ldy, out_dtype, tc, s, t0);
            if (e != cudaSuccess) return LOPRO_ERR_CUDA;
        }
        return LOPRO_OK;
    }
    if (prologue_supported(*desc, T) && stream_supported(*desc, T)) {
        // small batch: prologue + streaming kernel, chained by programmatic launches
        if (launch_prologue(*desc, perm, B, L.r_pad, (const __nv_bfloat16*)x_bf16, ldx, ws + W.off_xrot,
                            (__half*)(ws + W.off_t), W.t_pad, status, T, s, nullptr, nullptr, &lr8) != cudaSuccess)
            return LOPRO_ERR_CUDA;
        const cudaError_t e = use_tall(*desc, T) ? launch_tall(*desc, blob, L, ws, W, y, ldy, out_dtype, T, s)
                                                 : launch_stream(*desc, blob, L, ws, W, y, ldy, out_dtype, T, s);
        if (e != cudaSuccess) return LOPRO_ERR_CUDA;
        return LOPRO_OK;
    }
    const void* a_f16 = nullptr;  // the up factor where it is not the blob's section
    if (desc->lowrank_format == LOPRO_LOWRANK_FP8) {
        // More than 32 tokens on the tensor-core path (small_batch_chunks has sent every other case to the small-batch
        // kernels): the record is folded into fp16 factors in the workspace, A = U Sigma and B = V / s, one rounding each.
        if (!(T > kDecodeMaxT && prefill_supported(*desc, T))) return LOPRO_ERR_UNSUPPORTED;
        __half* fa = (__half*)(ws + W.off_fold_a);
        __half* fb = (__half*)(ws + W.off_fold_b);
        if (launch_lr8_fold(*desc, L.r_pad, blob + L.off[LOPRO_SEC_A], lr8.V, lr8.sigma, lr8.svec, fa, fb, s) != cudaSuccess)
            return LOPRO_ERR_CUDA;
        B = fb;
        a_f16 = fa;
    }
    if (T > kDecodeMaxT && rotate_lowrank_supported(*desc, T)) {
        // many tokens: rotation and B x side by side in one grid, then the sum over K slices
        if (launch_rotate_lowrank(*desc, perm, (const __nv_bfloat16*)x_bf16, ldx, xrot, desc->d_in, s64, status, B, L.r_pad,
                                  (float*)(ws + W.off_lrpart), (__half*)(ws + W.off_t), T, s) != cudaSuccess)
            return LOPRO_ERR_CUDA;
    } else {
    if (launch_rotate(*desc, perm, (const __nv_bfloat16*)x_bf16, ldx, xrot, desc->d_in, s64, status, T, s) !=
        cudaSuccess)
        return LOPRO_ERR_CUDA;
    if (desc->rank > 0) {
        cudaError_t e = T > kDecodeMaxT
                            ? launch_lowrank_down_mma(*desc, B, L.r_pad, (const __nv_bfloat16*)x_bf16, ldx,
                                                      (float*)(ws + W.off_lrpart), (__half*)(ws + W.off_t), T, s)
                            : launch_lowrank_down(*desc, B, L.r_pad, (const __nv_bfloat16*)x_bf16, ldx,
                                                  (__half*)(ws + W.off_t), T, s);
        if (e != cudaSuccess) return LOPRO_ERR_CUDA;
    }
    }
    if (prefill_supported(*desc, T)) {
        if (launch_prefill(*desc, blob, L, ws, W, y, ldy, out_dtype, T, s, a_f16) != cudaSuccess) return LOPRO_ERR_CUDA;
        return LOPRO_OK;
    }
    if (launch_decode(*desc, blob, L, ws, W, y, ldy, out_dtype, T, s) != cudaSuccess) return LOPRO_ERR_CUDA;
    return LOPRO_OK;
}

lopro_status lopro_configure(int32_t opt, int32_t value) {
    if (opt < 0 || opt >= LOPRO_OPT_COUNT) return LOPRO_ERR_INVALID_ARG;
    (void)option(opt);  // make sure the environment has been read, so that it cannot overwrite this value later
    __atomic_store_n(&g_options[opt], (int)value, __ATOMIC_RELAXED);
    return LOPRO_OK;
}

// Sibling layers can share launches when they differ in nothing but their rows and data, the batch is small and
// the per-layer path would be prologue + streaming kernel for each of them.
static bool group_shares_launches(int32_t n, const lopro_desc* const* descs, int32_t T) {
    if (n < 2 || n > kMaxSiblings || T < 1 || T > kDecodeMaxT) return false;
    const lopro_desc& d0 = *descs[0];
    if (d0.layout != LOPRO_LAYOUT_FRAGMENT) return false;
    for (int i = 0; i < n; ++i) {
        const lopro_desc& d = *descs[i];
        if (d.d_in != d0.d_in || d.bits != d0.bits || d.group_size != d0.group_size || d.block_size != d0.block_size ||
            d.identity_cols != d0.identity_cols || d.rank != d0.rank || d.layout != d0.layout ||
            d.lowrank_format != LOPRO_LOWRANK_FOLDED_F16)
            return false;
        if (!prologue_supported(d, T)) return false;
    }
    // all siblings through the persistent kernel (by their rows together) or all through the per-group kernel
    if (!group_uses_tall(n, descs, T))
        for (int i = 0; i < n; ++i)
            if (!stream_supported(*descs[i], T)) return false;
    return true;
}

static size_t group_region_bytes(const lopro_desc& d, int32_t T) {
    WorkspaceLayout W;
    if (workspace_layout(d, T, &W) != LOPRO_OK) return 0;
    return round_up_size(W.total, 1024);
}

size_t lopro_group_workspace_bytes(int32_t n_layers, const lopro_desc* const* descs, int32_t T) {
    if (n_layers < 1 || !descs || T < 0) return 0;
    size_t total = 0;
    for (int i = 0; i < n_layers; ++i) {
        if (!descs[i]) return 0;
        const size_t r = group_region_bytes(*descs[i], T);
        if (r == 0) return 0;
        total += r;
    }
    return total;
}

int32_t lopro_linear_fwd_group_path(int32_t n_layers, const lopro_desc* const* descs, int32_t T, int32_t* launches) {
    if (n_layers < 1 || !descs || T < 1) return 0;
    for (int i = 0; i < n_layers; ++i)
        if (!descs[i] || check_desc(*descs[i]) != LOPRO_OK) return 0;
    if (group_shares_launches(n_layers, descs, T)) {
        if (launches) *launches = 2;
        return 2;
    }
    int32_t total = 0;
    for (int i = 0; i < n_layers; ++i) {
        int32_t one = 0;
        if (lopro_linear_fwd_path(descs[i], T, &one) == 0) return 0;
        total += one;
    }
    if (launches) *launches = total;
    return 1;
}

lopro_status lopro_linear_fwd_group(int32_t n_layers, const lopro_desc* const* descs, const void* const* packed,
                                    const uint16_t* x_bf16, int64_t ldx, void* const* y, const int64_t* ldy, int32_t out_dtype,
                                    int32_t T, void* workspace, size_t workspace_bytes, void* stream) {
    if (n_layers < 1 || !descs || !packed || !y || !ldy) return LOPRO_ERR_INVALID_ARG;
    if (T < 0 || (out_dtype != LOPRO_OUT_BF16 && out_dtype != LOPRO_OUT_F32)) return LOPRO_ERR_INVALID_ARG;
    for (int i = 0; i < n_layers; ++i) {
        if (!descs[i]) return LOPRO_ERR_INVALID_ARG;
        const lopro_status st = check_desc(*descs[i]);
        if (st != LOPRO_OK) return st;
        if (descs[i]->d_in != descs[0]->d_in) return LOPRO_ERR_INVALID_ARG;  // siblings read the same x
    }
    if (T == 0) return LOPRO_OK;
    if (!workspace || !aligned(workspace, 256)) return LOPRO_ERR_INVALID_ARG;
    if (workspace_bytes < lopro_group_workspace_bytes(n_layers, descs, T)) return LOPRO_ERR_BUFFER_TOO_SMALL;
    uint8_t* ws = (uint8_t*)workspace;
    if (!group_shares_launches(n_layers, descs, T)) {
        // layer by layer, each in its own region of the workspace
        for (int i = 0; i < n_layers; ++i) {
            const size_t region = group_region_bytes(*descs[i], T);
            const lopro_status st =
                lopro_linear_fwd(descs[i], packed[i], x_bf16, ldx, y[i], ldy[i], out_dtype, T, ws, region, stream);
            if (st != LOPRO_OK) return st;
            ws += region;
        }
        return LOPRO_OK;
    }
    // one prologue for all siblings (one read of x per rotation CTA set, every layer its own permutation, Eq. 5),
    // one product launch over the row tiles of all of them
    const lopro_desc& d0 = *descs[0];
    if (!x_bf16 || ldx < d0.d_in || (ldx % 8) || !aligned(x_bf16, 16)) return LOPRO_ERR_INVALID_ARG;
    WorkspaceLayout W;
    lopro_status st = workspace_layout(d0, T, &W);
    if (st != LOPRO_OK) return st;
    const size_t region = group_region_bytes(d0, T);
    BlobLayout L[kMaxSiblings];
    for (int i = 0; i < n_layers; ++i) {
        if (!packed[i] || !y[i] || !aligned(packed[i], 256) || ldy[i] < descs[i]->d_out ||
            !aligned(y[i], out_dtype == LOPRO_OUT_F32 ? 4 : 2))
            return LOPRO_ERR_INVALID_ARG;
        st = blob_layout(*descs[i], &L[i]);
        if (st != LOPRO_OK) return st;
    }
    cudaStream_t s = (cudaStream_t)stream;
    PrologueSiblings ps = {};
    StreamSiblingArgs ss = {};
    ps.n = ss.n = n_layers - 1;
    for (int i = 1; i < n_layers; ++i) {
        const uint8_t* blob = (const uint8_t*)packed[i];
        uint8_t* wsi = ws + (size_t)i * region;
        ps.perm[i - 1] = (const int32_t*)(blob + L[i].off[LOPRO_SEC_PERM]);
        ps.B[i - 1] = (const __half*)(blob + L[i].off[LOPRO_SEC_B]);
        ps.act[i - 1] = wsi + W.off_xrot;
        ps.t[i - 1] = (__half*)(wsi + W.off_t);
        ss.blob[i - 1] = blob;
        ss.L[i - 1] = L[i];
        ss.ws[i - 1] = wsi;
        ss.y[i - 1] = y[i];
        ss.ldy[i - 1] = ldy[i];
        ss.d_out[i - 1] = descs[i]->d_out;
    }
    const uint8_t* blob0 = (const uint8_t*)packed[0];
    if (launch_prologue(d0, (const int32_t*)(blob0 + L[0].off[LOPRO_SEC_PERM]), (const __half*)(blob0 + L[0].off[LOPRO_SEC_B]),
                        L[0].r_pad, (const __nv_bfloat16*)x_bf16, ldx, ws + W.off_xrot, (__half*)(ws + W.off_t), W.t_pad,
                        (int*)(ws + W.off_status), T, s, nullptr, &ps) != cudaSuccess)
        return LOPRO_ERR_CUDA;
    const cudaError_t e = group_uses_tall(n_layers, descs, T)
                              ? launch_tall(d0, blob0, L[0], ws, W, y[0], ldy[0], out_dtype, T, s, 0, &ss)
                              : launch_stream(d0, blob0, L[0], ws, W, y[0], ldy[0], out_dtype, T, s, 0, &ss);
    return e == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}

// ---- experts of a mixture layer: the same layer shape, each expert its own rows of x and y -----------------------

static bool experts_share_launches(const lopro_desc& d, int max_rows) {
    if (max_rows < 1 || max_rows > kDecodeMaxT) return false;
    if (d.layout != LOPRO_LAYOUT_FRAGMENT || d.lowrank_format != LOPRO_LOWRANK_FOLDED_F16) return false;
    if (!prologue_supported(d, max_rows)) return false;
    return use_tall(d, max_rows) || stream_supported(d, max_rows);
}

static lopro_status check_expert_rows(int32_t n_experts, const int32_t* row_offsets, int* max_rows, int* active) {
    if (n_experts < 1 || !row_offsets || row_offsets[0] != 0) return LOPRO_ERR_INVALID_ARG;
    int mx = 0, act = 0;
    for (int e = 0; e < n_experts; ++e) {
        const int cnt = row_offsets[e + 1] - row_offsets[e];
        if (cnt < 0) return LOPRO_ERR_INVALID_ARG;
        if (cnt > mx) mx = cnt;
        if (cnt > 0) ++act;
    }
    *max_rows = mx;
    *active = act;
    return LOPRO_OK;
}

size_t lopro_experts_workspace_bytes(const lopro_desc* desc, int32_t n_experts, int32_t max_rows) {
    if (!desc || n_experts < 1 || max_rows < 0 || check_desc(*desc) != LOPRO_OK) return 0;
    const size_t region = group_region_bytes(*desc, max_rows < 1 ? 1 : max_rows);
    return region == 0 ? 0 : region * (size_t)n_experts;
}

int32_t lopro_linear_fwd_experts_path(const lopro_desc* desc, int32_t n_experts, const int32_t* row_offsets, int32_t* launches) {
    int max_rows = 0, active = 0;
    if (!desc || check_desc(*desc) != LOPRO_OK || check_expert_rows(n_experts, row_offsets, &max_rows, &active) != LOPRO_OK)
        return 0;
    if (active == 0) {
        if (launches) *launches = 0;
        return 1;
    }
    if (experts_share_launches(*desc, max_rows)) {
        if (launches) *launches = 2 * ((active + kMaxSiblings - 1) / kMaxSiblings);
        return 2;
    }
    int32_t total = 0;
    for (int e = 0; e < n_experts; ++e) {
        const int cnt = row_offsets[e + 1] - row_offsets[e];
        int32_t one = 0;
        if (cnt > 0 && lopro_linear_fwd_path(desc, cnt, &one) == 0) return 0;
        total += cnt > 0 ? one : 0;
    }
    if (launches) *launches = total;
    return 1;
}

lopro_status lopro_linear_fwd_experts(const lopro_desc* desc, int32_t n_experts, const void* const* packed,
                                      const int32_t* row_offsets, const uint16_t* x_bf16, int64_t ldx, void* y, int64_t ldy,
                                      int32_t out_dtype, void* workspace, size_t workspace_bytes, void* stream) {
    if (!desc || !packed) return LOPRO_ERR_INVALID_ARG;
    if (out_dtype != LOPRO_OUT_BF16 && out_dtype != LOPRO_OUT_F32) return LOPRO_ERR_INVALID_ARG;
    lopro_status st = check_desc(*desc);
    if (st != LOPRO_OK) return st;
    const lopro_desc& d = *desc;
    int max_rows = 0, active = 0;
    st = check_expert_rows(n_experts, row_offsets, &max_rows, &active);
    if (st != LOPRO_OK) return st;
    if (active == 0) return LOPRO_OK;
    const size_t esz = out_dtype == LOPRO_OUT_F32 ? 4 : 2;
    if (!x_bf16 || !y || !workspace || ldx < d.d_in || (ldx % 8) || ldy < d.d_out || !aligned(x_bf16, 16) ||
        !aligned(y, esz) || !aligned(workspace, 256))
        return LOPRO_ERR_INVALID_ARG;
    if (workspace_bytes < lopro_experts_workspace_bytes(desc, n_experts, max_rows)) return LOPRO_ERR_BUFFER_TOO_SMALL;
    for (int e = 0; e < n_experts; ++e)
        if (row_offsets[e + 1] > row_offsets[e] && (!packed[e] || !aligned(packed[e], 256))) return LOPRO_ERR_INVALID_ARG;
    const size_t region = group_region_bytes(d, max_rows);
    uint8_t* ws = (uint8_t*)workspace;
    const __nv_bfloat16* x = (const __nv_bfloat16*)x_bf16;
    auto rows_of_y = [&](int row) { return (void*)((uint8_t*)y + (size_t)row * (size_t)ldy * esz); };
    if (!experts_share_launches(d, max_rows)) {
        // expert by expert, each in its own region of the workspace
        for (int e = 0; e < n_experts; ++e) {
            const int r0 = row_offsets[e], cnt = row_offsets[e + 1] - r0;
            if (cnt == 0) continue;
            st = lopro_linear_fwd(desc, packed[e], x_bf16 + (size_t)r0 * ldx, ldx, rows_of_y(r0), ldy, out_dtype, cnt,
                                  ws + (size_t)e * region, region, stream);
            if (st != LOPRO_OK) return st;
        }
        return LOPRO_OK;
    }
    // up to kMaxSiblings experts per pair of launches: one prologue (every expert its own permutation, B and rows of
    // x), one product launch over the row tiles of all of them; the launches are shaped for the largest row count
    WorkspaceLayout W;
    st = workspace_layout(d, max_rows, &W);
    if (st != LOPRO_OK) return st;
    BlobLayout L;
    st = blob_layout(d, &L);
    if (st != LOPRO_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    int e = 0;
    while (e < n_experts) {
        int ids[kMaxSiblings], n = 0;
        for (; e < n_experts && n < kMaxSiblings; ++e)
            if (row_offsets[e + 1] > row_offsets[e]) ids[n++] = e;
        if (n == 0) break;
        PrologueSiblings ps = {};
        StreamSiblingArgs ss = {};
        ps.n = ss.n = n - 1;
        ps.own_rows = ss.own_rows = 1;
        for (int i = 0; i < n; ++i) {
            const int r0 = row_offsets[ids[i]], cnt = row_offsets[ids[i] + 1] - r0;
            const uint8_t* blob = (const uint8_t*)packed[ids[i]];
            uint8_t* wsi = ws + (size_t)ids[i] * region;
            ps.x_of[i] = x + (size_t)r0 * ldx;
            ps.T_of[i] = ss.T_of[i] = cnt;
            if (i == 0) continue;
            ps.perm[i - 1] = (const int32_t*)(blob + L.off[LOPRO_SEC_PERM]);
            ps.B[i - 1] = (const __half*)(blob + L.off[LOPRO_SEC_B]);
            ps.act[i - 1] = wsi + W.off_xrot;
            ps.t[i - 1] = (__half*)(wsi + W.off_t);
            ss.blob[i - 1] = blob;
            ss.L[i - 1] = L;
            ss.ws[i - 1] = wsi;
            ss.y[i - 1] = rows_of_y(r0);
            ss.ldy[i - 1] = ldy;
            ss.d_out[i - 1] = d.d_out;
        }
        const uint8_t* blob0 = (const uint8_t*)packed[ids[0]];
        uint8_t* ws0 = ws + (size_t)ids[0] * region;
        if (launch_prologue(d, (const int32_t*)(blob0 + L.off[LOPRO_SEC_PERM]), (const __half*)(blob0 + L.off[LOPRO_SEC_B]),
                            L.r_pad, ps.x_of[0], ldx, ws0 + W.off_xrot, (__half*)(ws0 + W.off_t), W.t_pad,
                            (int*)(ws0 + W.off_status), max_rows, s, nullptr, &ps) != cudaSuccess)
            return LOPRO_ERR_CUDA;
        void* y0 = rows_of_y(row_offsets[ids[0]]);
        const cudaError_t err = use_tall(d, max_rows) ? launch_tall(d, blob0, L, ws0, W, y0, ldy, out_dtype, max_rows, s, 0, &ss)
                                                      : launch_stream(d, blob0, L, ws0, W, y0, ldy, out_dtype, max_rows, s, 0, &ss);
        if (err != cudaSuccess) return LOPRO_ERR_CUDA;
    }
    return LOPRO_OK;
}

size_t lopro_host_staging_bytes(const lopro_desc* desc, int32_t T, int32_t out_dtype) {
    if (!desc || check_desc(*desc) != LOPRO_OK || T < 0) return 0;
    const size_t esz = out_dtype == LOPRO_OUT_F32 ? 4 : 2;
    return round_up_size((size_t)T * desc->d_in * 2, 256) + round_up_size((size_t)T * desc->d_out * esz, 256);
}

lopro_status lopro_linear_fwd_host(const lopro_desc* desc, const void* packed, const uint16_t* x_host,
                                   void* y_host, int32_t out_dtype, int32_t T, void* workspace,
                                   size_t workspace_bytes, void* stream) {
    if (!desc) return LOPRO_ERR_INVALID_ARG;
    if (out_dtype != LOPRO_OUT_BF16 && out_dtype != LOPRO_OUT_F32) return LOPRO_ERR_INVALID_ARG;
    WorkspaceLayout W;
    lopro_status st = workspace_layout(*desc, T, &W);
    if (st != LOPRO_OK) return st;
    if (T == 0) return LOPRO_OK;
    if (!x_host || !y_host || !workspace) return LOPRO_ERR_INVALID_ARG;
    const size_t stage = lopro_host_staging_bytes(desc, T, out_dtype);
    if (workspace_bytes < W.total + stage) return LOPRO_ERR_BUFFER_TOO_SMALL;
    if (!aligned(workspace, 256)) return LOPRO_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t esz = out_dtype == LOPRO_OUT_F32 ? 4 : 2;
    uint8_t* xd = (uint8_t*)workspace + W.total;
    uint8_t* yd = xd + round_up_size((size_t)T * desc->d_in * 2, 256);
    if (cudaMemcpyAsync(xd, x_host, (size_t)T * desc->d_in * 2, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return LOPRO_ERR_CUDA;
    st = lopro_linear_fwd(desc, packed, (const uint16_t*)xd, desc->d_in, yd, desc->d_out, out_dtype, T, workspace,
                          W.total, stream);
    if (st != LOPRO_OK) return st;
    if (cudaMemcpyAsync(y_host, yd, (size_t)T * desc->d_out * esz, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return LOPRO_ERR_CUDA;
    return LOPRO_OK;
}

}  // extern "C"
