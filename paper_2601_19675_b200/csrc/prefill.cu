// Prefill forward (T > 32): y = W^ x~ + A t as one tensor-core GEMM on tcgen05 / TMEM
// (steps "Dequant(W_q) X" and "U (Sigma Y)" of Appendix A.3, summed as in Eq. 8).
//
// CTA tile: one or two blocks of 128 weight rows (the M side of the MMA, one TMEM lane per row, one
// accumulator per block) x N tokens (N = 64, 128 or 256 TMEM columns, fp32) x 64 columns of K per
// pipeline stage.  Two row blocks share every activation tile, which halves the traffic of the
// activation operand from L2 (each CTA streams all K columns of its tokens).
//   * warps 0-15 (dequant): one per 16-row tile of the fragment layout (with a single row block: two
//     per tile, taking turns by pairs of stages);
//     each reads the tile's packed codes from global memory (registers, two visits ahead), turns them
//     into bf16(s (c - z)) -- fp32 arithmetic, one rounding -- and writes them into the stages' A tiles
//     in the K-major 128-byte-swizzled layout the MMA reads;
//   * warp 16 (loader): one thread brings the stage's tile of rotated activations (B operand) with a
//     tiled TMA copy, and for the low-rank stages the tiles of A (fp16) and t (fp16);
//   * warps 17, 18 (MMA): one thread per accumulator issues four tcgen05.mma (K = 16 each) per stage into its
//     TMEM accumulator and commits the stage back to the producers; the rank-r term A t runs as extra K
//     stages with fp16 operands into the same accumulator, so the sum of Eq. 8 costs no extra pass;
//   * warps 16-19 (epilogue): tcgen05.ld the accumulator, round once, store y[token][row].
// All mbarrier waits are bounded; a wait that runs out sets LOPRO_ERR_TIMEOUT in the workspace status
// word, the CTA stops waiting, still frees its TMEM and returns (outputs then unspecified).
#include <stdlib.h>

#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"
#include "tc5.cuh"

namespace lopro {

namespace {

constexpr int kDequantWarps = 16;  // two warps per 16-row tile, eight register pairs (32 columns) each
constexpr int kThreads = (kDequantWarps + 4) * 32;
constexpr int kTileM = 128;      // weight rows per CTA
constexpr int kMaxTileN = 256;   // tokens per CTA
constexpr int kStageK = 64;      // K columns per stage = 128 bytes of bf16 = one swizzle atom
constexpr int kAStages = 4;      // ring of weight tiles (two row blocks of 16 KB each)
constexpr int kBStages = 3;      // ring of activation tiles (32 KB each)
constexpr int kABlock = kTileM * 128;           // 16 KB: one row block of one stage
constexpr int kABytes = 2 * kABlock;            // 32 KB
constexpr int kBBytes = kMaxTileN * 128;        // 32 KB: one 256-token tile
constexpr double kPairCost = 1.4;  // duration of a two-block CTA relative to a one-block CTA (scheduling estimate)
constexpr int kSmemBytes = kAStages * kABytes + kBStages * kBBytes + 1024;  // + slack for 1024-byte alignment
constexpr uint32_t kPrefillSpin = 1u << 24;  // polls of one wait: a CTA's stages are milliseconds apart at most

struct PrefillParams {
    const uint32_t* codes;
    const uint32_t* sz;
    int* status;
    void* y;
    int64_t ldy;
    int out_f32;
    int y_vec;       // bf16 output whose rows allow 16-byte stores (y 16-byte aligned, ldy a multiple of 8)
    int m, n, T;
    int nsteps, gshift, ng, r_pad;
    int tile_n;      // tokens per accumulator: 64, 128 or 256
    int pair_tiles;    // row tiles of two blocks (256 rows, two accumulators)
    int single_tiles;  // row tiles of one block
    int units;         // token tiles
    int lr_stages;   // ceil(r_pad / 64)
};

template <int BITS>
__global__ void __launch_bounds__(kThreads, 1)
prefill_kernel(const PrefillParams p, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_a,
               const __grid_constant__ CUtensorMap map_t) {
    extern __shared__ unsigned char smem_raw[];
    // full_a, empty_a per A slot; full_b, empty_b per B slot; accumulator ready
    __shared__ __align__(8) uint64_t bars[2 * kAStages + 2 * kBStages + 1];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_timeout;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The grid is one-dimensional and lists every two-block CTA (256 rows, two accumulators) before the
    // one-block CTAs, so that the cheaper tiles fill the last wave: pair_tiles two-block row tiles and
    // single_tiles one-block row tiles per token tile.
    const int n_pair_ctas = p.pair_tiles * p.units;
    const bool is_pair = (int)blockIdx.x < n_pair_ctas;
    const int n_acc = is_pair ? 2 : 1;
    const int rest = (int)blockIdx.x - n_pair_ctas;
    const int tile_x = is_pair ? (int)blockIdx.x % p.pair_tiles : p.pair_tiles + rest % p.single_tiles;
    const int tile_y = is_pair ? (int)blockIdx.x / p.pair_tiles : rest / p.single_tiles;
    const int row_base = (is_pair ? tile_x * 2 : p.pair_tiles + tile_x) * kTileM;
    const int tok_base = tile_y * p.tile_n;
    const int total = p.nsteps + p.lr_stages;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzle atoms are 1024-byte aligned
    unsigned char* base_ptr = smem_raw + (base - raw);
    const uint32_t b_ring = base + kAStages * kABytes;  // B slots follow the A slots
    const uint32_t bar0 = smem_u32(bars);
    auto full_a = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty_a = [&](int s) { return bar0 + 8u * (uint32_t)(kAStages + s); };
    auto full_b = [&](int s) { return bar0 + 8u * (uint32_t)(2 * kAStages + s); };
    auto empty_b = [&](int s) { return bar0 + 8u * (uint32_t)(2 * kAStages + kBStages + s); };
    const uint32_t acc_ready = bar0 + 8u * (uint32_t)(2 * kAStages + 2 * kBStages);
    auto time_out = [&]() {
        s_timeout = 1;
        atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
    };
    // one lane polls, the warp follows (bar.warp.sync orders the other lanes' accesses after the wait)
    // A wait on a phase that is already complete costs one shared-memory round trip; the time-out flag (another
    // round trip) is read only when the first poll fails.
    auto wait_phase = [&](uint32_t bar, uint32_t parity) {
        if (mbar_try_wait(bar, parity)) return;
        if (!*reinterpret_cast<volatile int*>(&s_timeout) && !mbar_wait(bar, parity, kPrefillSpin)) time_out();
    };
    auto warp_wait = [&](uint32_t bar, uint32_t parity) {
        if (lane == 0) wait_phase(bar, parity);
        __syncwarp();
    };
    const uint32_t tmem_cols = n_acc == 2 ? 512u : 256u;

    if (tid == 0) {
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(full_a(s), (n_acc == 2 ? kDequantWarps : kDequantWarps / 2) + 1);  // the slot's dequant warps and the loader
            mbar_init(empty_a(s), n_acc);  // one commit per MMA-issuing thread
        }
        for (int s = 0; s < kBStages; ++s) {
            mbar_init(full_b(s), 1);
            mbar_init(empty_b(s), n_acc);
        }
        mbar_init(acc_ready, n_acc);
        s_timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kDequantWarps + 1) {  // one warp allocates the accumulator columns and later frees them
        tmem_alloc(smem_u32(&s_tmem_base), tmem_cols);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;

    if (warp < kDequantWarps) {
        // ---------------- dequant warps: fill the A tile of every weight stage ----------------
        // A visit converts two consecutive stages of one 16-row tile (2 x 64 columns, 32 register pairs per
        // lane) between one pair of waits and one proxy fence.  Two row blocks: warp w owns tile w and visits
        // every pair of stages.  One row block: warps w and w + 8 share tile w, group g = w >> 3 takes the
        // stages 4 v + 2 g and 4 v + 2 g + 1, so the two groups work on different stages at the same time.
        static_assert(kAStages == 4, "the visit schedule assumes four weight slots");
        const int gq = lane >> 2, tg = lane & 3;
        const int g = n_acc == 2 ? 0 : warp >> 3;
        const int vstride = n_acc == 2 ? 2 : 4;  // stages between the visits of this warp
        const int rt = row_base / 16 + (n_acc == 2 ? warp : (warp & 7));
        const bool valid = rt * 16 < p.m;
        uint32_t wbuf[2][2][BITS];
        uint32_t szbuf[2][2][2];
        const uint32_t* wbase = p.codes + ((size_t)rt * p.nsteps * 32 + lane) * BITS;
        const uint32_t* szbase = p.sz + (size_t)rt * p.ng * 16 + gq;
        auto load_visit = [&](int buf, int v) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int s = vstride * v + 2 * g + j;
                if (valid && s < p.nsteps) {
#pragma unroll
                    for (int q = 0; q < BITS; ++q) wbuf[buf][j][q] = __ldg(wbase + (size_t)s * 32 * BITS + q);
                    const uint32_t* z = szbase + (size_t)(s >> p.gshift) * 16;
                    szbuf[buf][j][0] = __ldg(z);
                    szbuf[buf][j][1] = __ldg(z + 8);
                }
            }
        };
        load_visit(0, 0);
        load_visit(1, 1);
        // byte offset of this lane's 4-byte slot in 16-byte chunk c of its row (row & 7 == gq, 128-byte swizzle)
        uint32_t off[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) off[c] = (uint32_t)(((warp & 7) * 16 + gq) * 128 + ((c ^ gq) << 4) + tg * 4);
        // all sixteen register pairs of the tile and stage: 64 columns of rows gq and gq + 8
        auto convert = [&](const uint32_t (&w)[BITS], uint32_t sz_lo, uint32_t sz_hi, unsigned char* a_tile) {
            uint32_t a[16];
            expand_codes<BITS>(a, w);
            const float2 f_lo = __half22float2(*reinterpret_cast<const __half2*>(&sz_lo));
            const float2 f_hi = __half22float2(*reinterpret_cast<const __half2*>(&sz_hi));
            const float sc[2] = {f_lo.x, f_hi.x};
            const float zs[2] = {128.0f + f_lo.y, 128.0f + f_hi.y};  // exact in fp32
#pragma unroll
            for (int pi = 0; pi < 16; ++pi) {
                const int j = pi >> 2, rho = pi & 3, hi8 = rho & 1;
                const uint32_t av = a[pi];
                const float lo_f = __uint_as_float(av << 16), hi_f = __uint_as_float(av & 0xFFFF0000u);
                // (128 + c) - (128 + z) is exact, so s (c - z) is rounded once to fp32, once to bf16
                const __nv_bfloat162 wv = __floats2bfloat162_rn((lo_f - zs[hi8]) * sc[hi8], (hi_f - zs[hi8]) * sc[hi8]);
                *reinterpret_cast<__nv_bfloat162*>(a_tile + off[2 * j + (rho >> 1)] + hi8 * 1024) = wv;
            }
        };
        unsigned char* const blk_ptr = base_ptr + (n_acc == 2 ? (warp >> 3) * kABlock : 0);
        const int n_visits = total > 2 * g ? (total - 2 * g + vstride - 1) / vstride : 0;
        for (int v0 = 0; v0 < n_visits; v0 += 2) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {  // u = register buffer of the visit
                const int v = v0 + u;
                if (v < n_visits) {
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const int s = vstride * v + 2 * g + j;
                        if (s < total) {
                            const int slot = s & 3, use = s >> 2;
                            if (use >= 1) warp_wait(empty_a(slot), (uint32_t)(use - 1) & 1u);
                            if (valid && s < p.nsteps)
                                convert(wbuf[u][j], szbuf[u][j][0], szbuf[u][j][1], blk_ptr + slot * kABytes);
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> async proxy (MMA)
                    __syncwarp();
                    if (lane == 0) {
                        const int s0 = vstride * v + 2 * g;
                        mbar_arrive(full_a(s0 & 3));
                        if (s0 + 1 < total) mbar_arrive(full_a((s0 + 1) & 3));
                    }
                    // after the fence and the releasing arrivals, which would wait for these loads to land
                    load_visit(u, v + 2);
                }
            }
        }
    } else if (warp == kDequantWarps) {
        // ---------------- loader: activation tiles, and the fp16 tiles of the low-rank stages ----------------
        if (lane == 0) {
            // under a programmatic launch the rotated activations and t of the preceding kernels are complete
            // only after this wait; the dequant warps start on the layer's own data right away
            asm volatile("griddepcontrol.wait;" ::: "memory");
            const uint32_t b_bytes = (uint32_t)(p.tile_n * 128);
            for (int s = 0; s < total; ++s) {
                const int sa = s % kAStages, sb = s % kBStages;
                if (s >= kAStages) wait_phase(empty_a(sa), (uint32_t)((s / kAStages) - 1) & 1u);
                if (s >= kBStages) wait_phase(empty_b(sb), (uint32_t)((s / kBStages) - 1) & 1u);
                const uint32_t a_tile = base + sa * kABytes, b_tile = b_ring + sb * kBBytes;
                mbar_expect_tx(full_b(sb), b_bytes);
                if (s < p.nsteps) {
                    tma_load_2d(b_tile, &map_x, s * kStageK, tok_base, full_b(sb));
                    mbar_arrive(full_a(sa));
                } else {
                    const int lr = s - p.nsteps;
                    tma_load_2d(b_tile, &map_t, lr * kStageK, tok_base, full_b(sb));
                    mbar_expect_tx(full_a(sa), (uint32_t)(n_acc * kABlock));
                    for (int acc = 0; acc < n_acc; ++acc)
                        tma_load_2d(a_tile + acc * kABlock, &map_a, lr * kStageK, row_base + acc * kTileM, full_a(sa));
                }
            }
        }
    } else if (warp == kDequantWarps + 1 || warp == kDequantWarps + 2) {
        // ---------------- MMA issuers ----------------
        // One thread per accumulator: a thread spends several hundred cycles per stage on its two barrier waits,
        // the descriptors and the commits, during which the tensor pipe would idle (an issued MMA occupies the
        // thread until the pipe takes it); with two row blocks the second thread's MMAs fill those gaps.  Each
        // accumulator receives its MMAs from one thread only, in program order, so results do not depend on timing.
        const int acc = warp - (kDequantWarps + 1);
        if (lane == 0 && acc < n_acc) {
            const uint32_t idesc_w = make_idesc(p.tile_n, 1u), idesc_lr = make_idesc(p.tile_n, 0u);
            const uint32_t d = tmem + (uint32_t)(acc * 256);
            // The next stage's barriers are polled (without suspending) before this stage's MMAs are issued, so
            // that the answers arrive while the MMAs queue up: every barrier operation is a shared-memory round
            // trip behind the dequant warps' traffic, and the tensor pipe idles while this thread waits.
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            bool ready_a = mbar_test_wait(full_a(0), 0u), ready_b = mbar_test_wait(full_b(0), 0u);
            for (int s = 0; s < total; ++s) {
                if (!ready_a) wait_phase(full_a(sa), pa);
                if (!ready_b) wait_phase(full_b(sb), pb);
                tc_fence_after();
                const uint64_t da = make_desc_sw128(base + sa * kABytes + acc * kABlock);
                const uint64_t db = make_desc_sw128(b_ring + sb * kBBytes);
                const uint32_t commit_a = empty_a(sa), commit_b = empty_b(sb);
                if (++sa == kAStages) {
                    sa = 0;
                    pa ^= 1u;
                }
                if (++sb == kBStages) {
                    sb = 0;
                    pb ^= 1u;
                }
                if (s + 1 < total) {
                    ready_a = mbar_test_wait(full_a(sa), pa);
                    ready_b = mbar_test_wait(full_b(sb), pb);
                }
                const bool lowrank = s >= p.nsteps;
                const int ksub = lowrank ? min(4, (p.r_pad - (s - p.nsteps) * kStageK) / 16) : 4;
                const uint32_t idesc = lowrank ? idesc_lr : idesc_w;
                for (int k = 0; k < ksub; ++k)  // 16 columns = 32 bytes = 2 descriptor address units
                    umma_f16(d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (s > 0 || k > 0) ? 1u : 0u);
                umma_commit(commit_a);  // the slots may be refilled once these MMAs have read them
                umma_commit(commit_b);
            }
            umma_commit(acc_ready);
        }
    }

    if (warp >= kDequantWarps) {
        // ---------------- epilogue: TMEM -> registers -> y[token][row] ----------------
        __syncwarp();
        if (lane == 0) wait_phase(acc_ready, 0u);
        __syncwarp();
        tc_fence_after();
        const int lane_base = (warp & 3) * 32;  // a warp may read the 32 TMEM lanes of its quarter
        for (int acc = 0; acc < n_acc; ++acc) {
            const int row = row_base + acc * kTileM + lane_base + lane;
            for (int c0 = 0; c0 < p.tile_n; c0 += 32) {
                uint32_t v[32];
                const uint32_t taddr = tmem + ((uint32_t)lane_base << 16) + (uint32_t)(acc * 256 + c0);
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                      "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                      "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                      "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(taddr)
                    : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (p.y_vec) {
                    // bf16 rows of 32 tokens meet in shared memory (the rings are idle now), [token][32 rows], and
                    // leave as 16-byte pieces of eight consecutive rows
                    __nv_bfloat16* stg = reinterpret_cast<__nv_bfloat16*>(base_ptr + (warp - kDequantWarps) * 2048);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 32; ++i) stg[i * 32 + lane] = __float2bfloat16_rn(__uint_as_float(v[i]));
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int piece = q * 32 + lane, ti = piece >> 2, r8 = (piece & 3) * 8;
                        const int tok = tok_base + c0 + ti, prow = row_base + acc * kTileM + lane_base + r8;
                        if (tok < p.T && prow < p.m)
                            *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.y) + (size_t)tok * p.ldy + prow) =
                                *reinterpret_cast<const uint4*>(stg + ti * 32 + r8);
                    }
                } else if (row < p.m) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int tok = tok_base + c0 + i;
                        if (tok < p.T) {
                            const size_t o = (size_t)tok * p.ldy + row;
                            if (p.out_f32) reinterpret_cast<float*>(p.y)[o] = __uint_as_float(v[i]);
                            else reinterpret_cast<__nv_bfloat16*>(p.y)[o] = __float2bfloat16_rn(__uint_as_float(v[i]));
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kDequantWarps + 1) {
        tc_fence_after();
        tmem_dealloc(tmem, tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------------------------
// The same GEMM with the two CTAs of a cluster on one tile (tcgen05 cta_group::2): 256 weight rows (128 per CTA)
// x 512 or 256 tokens (two accumulators or one, N = 256 each) x 64 columns of K per stage.  Every dequantized weight
// tile now meets 512 tokens instead of 256 -- half the conversion work per multiply-add -- while each CTA still
// streams the activations of only 256 tokens per stage (its half of each accumulator's B operand).
//   * both CTAs: 16 dequant warps (two per 16-row tile, taking turns by pairs of stages), a loader thread (its own
//     halves of the activation tiles; its own 128 rows of A in the low-rank stages), 4 epilogue warps (own 128 rows);
//   * the pair's first CTA alone: the MMA issuers, one thread per accumulator.  All "full" barriers are the first
//     CTA's (the second CTA's warps arrive on them through the cluster's shared-memory window, its TMA copies count
//     their bytes there); the "empty" and "accumulator ready" barriers exist in both CTAs and take the commits of
//     the first CTA's issuers by multicast.
// A wait that runs out stops all further waits of both CTAs; both still reach the final cluster barrier, free the
// tensor memory and return.
constexpr int kPairABytes = kABlock;                 // 16 KB: 128 rows of one stage
constexpr int kPairBHalf = 128 * 128;                // 16 KB: this CTA's 128 tokens of one accumulator's stage
constexpr int kPairBBytes = 2 * kPairBHalf;          // 32 KB: both accumulators
#ifndef LOPRO_PAIR_A_STAGES
#define LOPRO_PAIR_A_STAGES 8
#endif
#ifndef LOPRO_PAIR_B_STAGES
#define LOPRO_PAIR_B_STAGES 3
#endif
constexpr int kPairAStages = LOPRO_PAIR_A_STAGES;  // even: a visit fills two neighbouring slots
constexpr int kPairBStages = LOPRO_PAIR_B_STAGES;
static_assert(kPairBStages <= kPairAStages, "one 'empty' barrier per weight slot serves both rings");
constexpr int kPairSmemBytes = kPairAStages * kPairABytes + kPairBStages * kPairBBytes + 1024;
#ifndef LOPRO_PAIR_MIN_T
#define LOPRO_PAIR_MIN_T 512
#endif
constexpr int kPairMinT = LOPRO_PAIR_MIN_T;   // from here on always two CTAs per tile; below, by prefill_estimate_us
constexpr int kMaxKParts = 4;    // K parts of a tile of the last wave

struct PairParams {
    const uint32_t* codes;
    const uint32_t* sz;
    int* status;
    void* y;
    int64_t ldy;
    int out_f32;
    int y_vec;
    int m, n, T;
    int nsteps, gshift, ng, r_pad;
    int row_tiles;    // tiles of 256 rows
    int split_first;  // tiles from this index on are split along K into k_parts units each (the last wave)
    int k_parts;
    float* kparts;    // their fp32 partial sums, [unit][kp_tokens][256 rows]
    int kp_tokens;    // token rows per unit there: min(512, T rounded up to 32)
    int lr_stages;
};

template <int BITS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
prefill_pair_kernel(const PairParams p, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_a,
                    const __grid_constant__ CUtensorMap map_t) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * kPairAStages + kPairBStages + 1];  // full_a, empty, full_b, accumulators ready
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_timeout;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_cta_rank();  // 0: the CTA that issues the MMAs
    // Units in grid order: whole tiles first, then the tiles of the last wave cut along K into k_parts units, which
    // leave fp32 partial sums for prefill_kparts_kernel (so that the last wave fills the machine too).
    const int unit = (int)(blockIdx.x >> 1);
    const bool whole = unit < p.split_first;
    const int tile = whole ? unit : p.split_first + (unit - p.split_first) / p.k_parts;
    const int part = whole ? 0 : (unit - p.split_first) % p.k_parts;
    const int parts = whole ? 1 : p.k_parts;
    const int tile_x = tile % p.row_tiles, tile_y = tile / p.row_tiles;
    const int row_base = tile_x * 2 * kTileM + (int)rank * kTileM;  // this CTA's 128 rows
    const int tok_base = tile_y * 512;
    const int n_acc = p.T - tok_base > 256 ? 2 : 1;
    // the unit's stages [s_begin, s_begin + total) of the layer's nsteps weight stages and lr_stages low-rank stages
    const int all_stages = p.nsteps + p.lr_stages;
    const int s_begin = (all_stages * part / parts) & ~1;
    const int total = (part == parts - 1 ? all_stages : ((all_stages * (part + 1) / parts) & ~1)) - s_begin;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - raw);
    const uint32_t b_ring = base + kPairAStages * kPairABytes;
    const uint32_t bar0 = smem_u32(bars);
    auto full_a = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty_a = [&](int s) { return bar0 + 8u * (uint32_t)(kPairAStages + s); };
    auto full_b = [&](int s) { return bar0 + 8u * (uint32_t)(2 * kPairAStages + s); };
    const uint32_t acc_ready = bar0 + 8u * (uint32_t)(2 * kPairAStages + kPairBStages);
    const uint32_t peer_timeout = map_to_cta(smem_u32(&s_timeout), rank ^ 1u);
    auto time_out = [&]() {
        s_timeout = 1;
        st_cluster_u32(peer_timeout, 1u);
        atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
    };
    auto timed_out = [&]() { return *reinterpret_cast<volatile int*>(&s_timeout) != 0; };
    // A wait on a phase that is already complete costs one shared-memory round trip; the time-out flag (another
    // round trip) is read only when the first poll fails.
    auto wait_phase = [&](uint32_t bar, uint32_t parity) {
        if (mbar_try_wait(bar, parity)) return;
        if (!timed_out() && !mbar_wait(bar, parity, kPrefillSpin)) time_out();
    };
    // Waits of the warps that run ahead of the MMAs or behind them: a failed poll sleeps before the next one.  Every
    // poll is a shared-memory operation, and the MMA-issuing threads' own barrier operations queue behind them.
    auto wait_relaxed = [&](uint32_t bar, uint32_t parity, unsigned sleep_ns) {
        if (mbar_try_wait(bar, parity)) return;
        if (timed_out()) return;
        for (uint32_t it = 0; it < kPrefillSpin; ++it) {
            __nanosleep(sleep_ns);
            if (mbar_try_wait(bar, parity)) return;
        }
        time_out();
    };
    auto warp_wait = [&](uint32_t bar, uint32_t parity) {
        if (lane == 0) wait_relaxed(bar, parity, 128u);
        __syncwarp();
    };
    const uint32_t tmem_cols = n_acc == 2 ? 512u : 256u;

    if (tid == 0) {
        for (int s = 0; s < kPairAStages; ++s) {
            mbar_init(full_a(s), kDequantWarps + 1);  // eight dequant warps of each CTA, and the first CTA's loader
            mbar_init(empty_a(s), n_acc);
        }
        for (int s = 0; s < kPairBStages; ++s) mbar_init(full_b(s), 1);
        mbar_init(acc_ready, n_acc);
        s_timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kDequantWarps + 1) tmem_alloc_pair(smem_u32(&s_tmem_base), tmem_cols);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the other CTA's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;

    if (warp < kDequantWarps) {
        // ---------------- dequant warps: warps w and w + 8 share tile w; group g = w >> 3 converts the stages
        // 4 v + 2 g and 4 v + 2 g + 1 of visit v ----------------
        static_assert(kPairAStages % 2 == 0 && kPairAStages >= 4, "a visit fills two neighbouring weight slots");
        const int gq = lane >> 2, tg = lane & 3;
        const int g = warp >> 3;
        const int rt = row_base / 16 + (warp & 7);
        const bool valid = rt * 16 < p.m;
        uint32_t wbuf[2][2][BITS];
        uint32_t szbuf[2][2][2];
        const uint32_t* wbase = p.codes + ((size_t)rt * p.nsteps * 32 + lane) * BITS;
        const uint32_t* szbase = p.sz + (size_t)rt * p.ng * 16 + gq;
        auto load_visit = [&](int buf, int v) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int i = 4 * v + 2 * g + j, s = s_begin + i;
                if (valid && i < total && s < p.nsteps) {
#pragma unroll
                    for (int q = 0; q < BITS; ++q) wbuf[buf][j][q] = __ldg(wbase + (size_t)s * 32 * BITS + q);
                    const uint32_t* z = szbase + (size_t)(s >> p.gshift) * 16;
                    szbuf[buf][j][0] = __ldg(z);
                    szbuf[buf][j][1] = __ldg(z + 8);
                }
            }
        };
        load_visit(0, 0);
        load_visit(1, 1);
        uint32_t off[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) off[c] = (uint32_t)(((warp & 7) * 16 + gq) * 128 + ((c ^ gq) << 4) + tg * 4);
        auto convert = [&](const uint32_t (&w)[BITS], uint32_t sz_lo, uint32_t sz_hi, unsigned char* a_tile) {
            uint32_t a[16];
            expand_codes<BITS>(a, w);
            const float2 f_lo = __half22float2(*reinterpret_cast<const __half2*>(&sz_lo));
            const float2 f_hi = __half22float2(*reinterpret_cast<const __half2*>(&sz_hi));
            const float sc[2] = {f_lo.x, f_hi.x};
            const float zs[2] = {128.0f + f_lo.y, 128.0f + f_hi.y};  // exact in fp32
#pragma unroll
            for (int pi = 0; pi < 16; ++pi) {
                const int j = pi >> 2, rho = pi & 3, hi8 = rho & 1;
                const uint32_t av = a[pi];
                const float lo_f = __uint_as_float(av << 16), hi_f = __uint_as_float(av & 0xFFFF0000u);
                // (128 + c) - (128 + z) is exact, so s (c - z) is rounded once to fp32, once to bf16
                const __nv_bfloat162 wv = __floats2bfloat162_rn((lo_f - zs[hi8]) * sc[hi8], (hi_f - zs[hi8]) * sc[hi8]);
                *reinterpret_cast<__nv_bfloat162*>(a_tile + off[2 * j + (rho >> 1)] + hi8 * 1024) = wv;
            }
        };
        const uint32_t full_a0 = map_to_cta(full_a(0), 0u);  // the first CTA's barriers, 8 bytes apart
        const int n_visits = total > 2 * g ? (total - 2 * g + 3) / 4 : 0;
        for (int v0 = 0; v0 < n_visits; v0 += 2) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int v = v0 + u;
                if (v < n_visits) {
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const int i = 4 * v + 2 * g + j;
                        if (i < total) {
                            const int slot = i % kPairAStages, use = i / kPairAStages;
                            if (use >= 1) warp_wait(empty_a(slot), (uint32_t)(use - 1) & 1u);
                            if (valid && s_begin + i < p.nsteps)
                                convert(wbuf[u][j], szbuf[u][j][0], szbuf[u][j][1], base_ptr + slot * kPairABytes);
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> async proxy (MMA)
                    __syncwarp();
                    if (lane == 0) {
                        const int s0 = 4 * v + 2 * g;
                        mbar_arrive_cluster(full_a0 + 8u * (uint32_t)(s0 % kPairAStages));
                        if (s0 + 1 < total) mbar_arrive_cluster(full_a0 + 8u * (uint32_t)(s0 % kPairAStages + 1));
                    }
                    // after the fence and the releasing arrivals, which would wait for these loads to land
                    load_visit(u, v + 2);
                }
            }
        }
    } else if (warp == kDequantWarps) {
        // ---------------- loader: this CTA's halves of the activation tiles; its rows of A in the low-rank stages ----------------
        if (lane == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            const uint32_t full_a0 = map_to_cta(full_a(0), 0u), full_b0 = map_to_cta(full_b(0), 0u);
            const uint32_t b_bytes = (uint32_t)(2 * n_acc * kPairBHalf);  // both CTAs' copies of a stage
            int sa = 0, sb = 0;
            uint32_t pa = 1;  // parity of the phase of the weight slot's previous use
            for (int i = 0; i < total; ++i) {
                const int s = s_begin + i;  // stage of the layer; i counts the unit's stages (rings, parities)
                // Weight stages: the first CTA's loader is one of the arrivals of full_a (so that the low-rank stages
                // can count their A tiles there); it may arrive for this use of the slot once the previous use's
                // phase is complete, which does not wait for the MMAs.  Low-rank stages write the slot: empty_a.
                if (i >= kPairAStages) {
                    if (s >= p.nsteps) wait_relaxed(empty_a(sa), pa, 64u);
                    else if (rank == 0) wait_relaxed(full_a(sa), pa, 64u);
                }
                // the commit that frees weight slot (i - kPairBStages) % kPairAStages frees this activation slot too
                if (i >= kPairBStages)
                    wait_relaxed(empty_a((i - kPairBStages) % kPairAStages), (uint32_t)((i - kPairBStages) / kPairAStages) & 1u, 64u);
                const uint32_t a_tile = base + sa * kPairABytes, b_tile = b_ring + sb * kPairBBytes;
                const uint32_t fb = full_b0 + 8u * (uint32_t)sb, fa = full_a0 + 8u * (uint32_t)sa;
                if (rank == 0) mbar_expect_tx(full_b(sb), b_bytes);
                const CUtensorMap* bmap = s < p.nsteps ? &map_x : &map_t;
                const int kcol = (s < p.nsteps ? s : s - p.nsteps) * kStageK;
                for (int acc = 0; acc < n_acc; ++acc)
                    tma_load_2d_pair(b_tile + acc * kPairBHalf, bmap, kcol, tok_base + acc * 256 + (int)rank * 128, fb);
                if (s < p.nsteps) {
                    if (rank == 0) mbar_arrive(full_a(sa));
                } else {
                    if (rank == 0) mbar_expect_tx(full_a(sa), (uint32_t)(2 * kPairABytes));
                    tma_load_2d_pair(a_tile, &map_a, kcol, row_base, fa);
                }
                if (++sa == kPairAStages) {
                    sa = 0;
                    pa ^= 1u;
                }
                if (++sb == kPairBStages) sb = 0;
            }
        }
    } else if ((warp == kDequantWarps + 1 || warp == kDequantWarps + 2) && rank == 0) {
        // ---------------- MMA issuers (first CTA): one thread per accumulator ----------------
        const int acc = warp - (kDequantWarps + 1);
        if (lane == 0 && acc < n_acc) {
            const uint32_t idesc_w = make_idesc_pair(256, 1u), idesc_lr = make_idesc_pair(256, 0u);
            const uint32_t d = tmem + (uint32_t)(acc * 256);
            // The thread's time per stage bounds the kernel: the tensor pipe holds a few MMAs in its queue and idles
            // once the thread falls behind, and every barrier operation is a shared-memory round trip behind the
            // dequant warps' traffic.  So the next stage's barriers are polled (without suspending) right after
            // this stage's MMAs and commit are queued, and a stage whose tiles were ready by then waits for nothing.
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            bool ready_a = mbar_test_wait(full_a(0), 0u), ready_b = mbar_test_wait(full_b(0), 0u);
            for (int i = 0; i < total; ++i) {
                const int s = s_begin + i;
                if (!ready_a) wait_phase(full_a(sa), pa);
                if (!ready_b) wait_phase(full_b(sb), pb);
                tc_fence_after();
                const uint64_t da = make_desc_sw128(base + sa * kPairABytes);
                const uint64_t db = make_desc_sw128(b_ring + sb * kPairBBytes + acc * kPairBHalf);
                const uint32_t commit_a = empty_a(sa);
                if (++sa == kPairAStages) {
                    sa = 0;
                    pa ^= 1u;
                }
                if (++sb == kPairBStages) {
                    sb = 0;
                    pb ^= 1u;
                }
                const bool lowrank = s >= p.nsteps;
                const int ksub = lowrank ? min(4, (p.r_pad - (s - p.nsteps) * kStageK) / 16) : 4;
                const uint32_t idesc = lowrank ? idesc_lr : idesc_w;
                for (int k = 0; k < ksub; ++k)
                    umma_f16_pair(d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (i > 0 || k > 0) ? 1u : 0u);
                umma_commit_pair(commit_a);  // one commit per stage: the stage's weight and activation slots
                if (i + 1 < total) {  // answered while the tensor pipe works through the MMAs just queued
                    ready_a = mbar_test_wait(full_a(sa), pa);
                    ready_b = mbar_test_wait(full_b(sb), pb);
                }
            }
            umma_commit_pair(acc_ready);
        }
    }

    {
        // ---------------- epilogue: this CTA's 128 rows of every accumulator, by all twenty warps ----------------
        // A warp may read the 32 tensor-memory lanes of its quarter (warp & 3); the five warps of a quarter take the
        // accumulators' 32-column pieces in turn, so the tensor pipe idles a fifth as long as with four warps.
        __syncwarp();
        if (lane == 0) wait_relaxed(acc_ready, 0u, warp < kDequantWarps ? 256u : 512u);
        __syncwarp();
        tc_fence_after();
        const int lane_base = (warp & 3) * 32;
        const int row = row_base + lane_base + lane;
        for (int piece32 = warp >> 2; piece32 < n_acc * 8; piece32 += (kDequantWarps + 4) / 4) {
            {
                const int acc = piece32 >> 3, c0 = (piece32 & 7) * 32;
                if (tok_base + acc * 256 + c0 >= p.T) break;  // uniform over the warp
                uint32_t v[32];
                const uint32_t taddr = tmem + ((uint32_t)lane_base << 16) + (uint32_t)(acc * 256 + c0);
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                      "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                      "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                      "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(taddr)
                    : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int tok0 = tok_base + acc * 256 + c0;
                if (!whole) {
                    // fp32 partial sums of this K part: [unit][token of the tile][row of the tile]
                    float* dst = p.kparts + ((size_t)(unit - p.split_first) * p.kp_tokens + (size_t)(acc * 256 + c0)) * 256 +
                                 (int)rank * kTileM + lane_base + lane;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (tok0 + i < p.T) dst[(size_t)i * 256] = __uint_as_float(v[i]);
                } else if (p.y_vec) {
                    __nv_bfloat16* stg = reinterpret_cast<__nv_bfloat16*>(base_ptr + warp * 2048);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 32; ++i) stg[i * 32 + lane] = __float2bfloat16_rn(__uint_as_float(v[i]));
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int piece = q * 32 + lane, ti = piece >> 2, r8 = (piece & 3) * 8;
                        const int tok = tok0 + ti, prow = row_base + lane_base + r8;
                        if (tok < p.T && prow < p.m)
                            *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.y) + (size_t)tok * p.ldy + prow) =
                                *reinterpret_cast<const uint4*>(stg + ti * 32 + r8);
                    }
                } else if (row < p.m) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int tok = tok0 + i;
                        if (tok < p.T) {
                            const size_t o = (size_t)tok * p.ldy + row;
                            if (p.out_f32) reinterpret_cast<float*>(p.y)[o] = __uint_as_float(v[i]);
                            else reinterpret_cast<__nv_bfloat16*>(p.y)[o] = __float2bfloat16_rn(__uint_as_float(v[i]));
                        }
                    }
                }
            }
        }
    }
    // neither CTA leaves, or frees tensor memory, while the other may still read its shared memory, arrive on its
    // barriers or read the accumulators
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == kDequantWarps + 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem, tmem_cols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime so that the library does not link
// against the driver library (it must load on machines without one).
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D row-major tensor [rows][cols] of 2-byte elements, box {64 columns, box_rows}, 128-byte swizzle,
// out-of-range elements read as zero.
bool make_map(CUtensorMap* map, CUtensorMapDataType dt, const void* ptr, uint64_t cols, uint64_t rows, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kStageK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BITS>
cudaError_t launch_prefill_bits(const PrefillParams& p, const CUtensorMap& mx, const CUtensorMap& ma, const CUtensorMap& mt,
                                dim3 grid, cudaStream_t s) {
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(prefill_kernel<BITS>, kSmemBytes, &attr_done);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, prefill_kernel<BITS>, p, mx, ma, mt);
}

// The partial sums of the units cut along K, added in a fixed order: y[token][row] = sum over parts.  One thread per
// token and four rows.
__global__ void __launch_bounds__(256)
prefill_kparts_kernel(const float* __restrict__ kparts, void* __restrict__ y, int64_t ldy, int out_f32, int m, int T,
                      int row_tiles, int first_tile, int k_parts, int kp_tokens) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int blocks_per_tile = kp_tokens >> 2;                  // blocks of 4 tokens x 256 rows
    const int split_tile = (int)blockIdx.x / blocks_per_tile;
    const int tok_l = (((int)blockIdx.x % blocks_per_tile) << 2) + ((int)threadIdx.x >> 6);
    const int row_l = ((int)threadIdx.x & 63) << 2;
    const int tile = first_tile + split_tile;
    const int tok = (tile / row_tiles) * 512 + tok_l, row = (tile % row_tiles) * 256 + row_l;
    if (tok >= T || row >= m) return;
    const float* src = kparts + (((size_t)split_tile * k_parts) * kp_tokens + tok_l) * 256 + row_l;
    float4 acc = *reinterpret_cast<const float4*>(src);
    for (int part = 1; part < k_parts; ++part) {
        const float4 v = *reinterpret_cast<const float4*>(src + (size_t)part * kp_tokens * 256);
        acc.x += v.x;
        acc.y += v.y;
        acc.z += v.z;
        acc.w += v.w;
    }
    const float r[4] = {acc.x, acc.y, acc.z, acc.w};
    const size_t o = (size_t)tok * ldy + row;
    for (int e = 0; e < 4; ++e)
        if (row + e < m) {  // d_out is a multiple of 64 today; the check keeps the kernel right for any m
            if (out_f32) reinterpret_cast<float*>(y)[o + e] = r[e];
            else reinterpret_cast<__nv_bfloat16*>(y)[o + e] = __float2bfloat16_rn(r[e]);
        }
}

template <int BITS>
cudaError_t launch_pair_bits(PairParams p, const CUtensorMap& mx, const CUtensorMap& ma, const CUtensorMap& mt,
                             const PairPlan& plan, cudaStream_t s) {
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(prefill_pair_kernel<BITS>, kPairSmemBytes, &attr_done);
    if (e != cudaSuccess) return e;
    const long long n_ctas = 2LL * (plan.n_tiles - plan.split_tiles + (long long)plan.split_tiles * plan.k_parts);
    if (n_ctas > 0x7fffffffLL) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kPairSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, prefill_pair_kernel<BITS>, p, mx, ma, mt);
    if (e != cudaSuccess || plan.split_tiles == 0) return e;
    cfg.gridDim = dim3((unsigned)plan.split_tiles * (unsigned)(p.kp_tokens / 4));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    return cudaLaunchKernelEx(&cfg, prefill_kparts_kernel, (const float*)p.kparts, p.y, p.ldy, p.out_f32, p.m, p.T, p.row_tiles,
                              plan.n_tiles - plan.split_tiles, plan.k_parts, p.kp_tokens);
}

}  // namespace

bool prefill_supported(const lopro_desc& d, int T) {
    const int off = option(LOPRO_OPT_NO_TCGEN05) == 1 ? 1 : 0;  // tuning / A-B comparison only
    return off == 0 && T > kDecodeMaxT && encode_tiled_fn() != nullptr && (d.d_in % 64) == 0;
}

// Tiling of the two-CTA kernel: tiles of 256 rows x 512 tokens over the CTA pairs the device holds at once (one CTA
// fills a multiprocessor).  The tiles of the last, partial wave are cut along K into as many parts as fill the idle
// pairs (at most kMaxKParts, at least eight stages each), so that the wave ends early instead of running a full
// tile's length on a few pairs.
PairPlan pair_plan(const lopro_desc& d, int T) {
    PairPlan plan = {};
    if (T <= kDecodeMaxT) return plan;
    plan.use = 1;
    plan.row_tiles = (d.d_out + 2 * kTileM - 1) / (2 * kTileM);
    const long long n_tiles = (long long)plan.row_tiles * ((T + 511) / 512);
    if (n_tiles > 0x3fffffffLL) {
        plan.use = 0;
        return plan;
    }
    plan.n_tiles = (int)n_tiles;
    const int slots = sm_count() / 2 > 0 ? sm_count() / 2 : 1;
    const int rem = plan.n_tiles % slots;
    const int stages = d.d_in / kStageK + (round_up_int(d.rank, 16) + kStageK - 1) / kStageK;
    int parts = rem > 0 ? slots / rem : 1;
    if (parts > kMaxKParts) parts = kMaxKParts;
    if (parts > stages / 8) parts = stages / 8;
    const int forced = option(LOPRO_OPT_PREFILL_PAIRS);  // tuning and tests: K parts of the last wave, 0 or 1 = none
    if (forced >= 0 && rem > 0) parts = forced < kMaxKParts ? forced : kMaxKParts;
    if (rem > 0 && parts > slots / rem) parts = slots / rem;  // the units of the last wave fit the resident pairs
    if (parts > stages / 2) parts = stages / 2;  // every part holds at least two stages
    if (parts >= 2) {
        plan.split_tiles = rem;
        plan.k_parts = parts;
    } else {
        plan.split_tiles = 0;
        plan.k_parts = 1;
    }
    return plan;
}

// fp32 partial sums of the tiles cut along K: room for the most units any plan may use (one per resident pair, four
// per tile), whatever the switches say -- a bound that does not decrease as T grows, unlike the plan's own count
static int kparts_tokens(int T) { return T >= 512 ? 512 : round_up_int(T, 32); }
size_t prefill_kparts_bytes(const lopro_desc& d, int T) {
    const PairPlan plan = pair_plan(d, T);
    if (!plan.use) return 0;
    const long long slots = sm_count() / 2 > 0 ? sm_count() / 2 : 1;
    const long long by_tiles = (long long)plan.n_tiles * kMaxKParts;
    return (size_t)(by_tiles < slots ? by_tiles : slots) * kparts_tokens(T) * 256 * sizeof(float);
}

// Which of the two tensor-core kernels serves T tokens, and an estimate of its duration in microseconds (beyond the
// launches in front of it), from timings on B200 per 64-column stage of one CTA: two CTAs on a tile 0.95 (two
// accumulators) or 0.80 (one, T <= 256), one CTA per tile 0.78 (one 128-row block) or 1.03 (two); a tile cut along K
// costs its share plus 9 (start-up of the shorter units and the kernel that adds them).  From 512 tokens on the
// two-CTA kernel always; below, whichever is estimated faster: few row tiles favour the two-CTA kernel (its K parts
// fill the machine), many row tiles and at most 256 tokens the other (twice the rows per CTA for the same conversion).
double prefill_estimate_us(const lopro_desc& d, int T, bool* use_pairs) {
    const int stages = d.d_in / kStageK + (round_up_int(d.rank, 16) + kStageK - 1) / kStageK;
    // one CTA per tile
    const int tile_n = T <= 64 ? 64 : (T <= 128 ? 128 : 256);
    const int units = (T + tile_n - 1) / tile_n, m_tiles = (d.d_out + kTileM - 1) / kTileM;
    const int n_sm = sm_count() > 0 ? sm_count() : 1;
    const long long two_block = (long long)(m_tiles / 2) * units, one_block = (long long)(m_tiles % 2) * units;
    const long long waves2 = (two_block + n_sm - 1) / n_sm, all_single_waves = ((long long)m_tiles * units + n_sm - 1) / n_sm;
    double single_us = (double)stages * 0.78 * (double)all_single_waves;
    const double mixed_us = (double)stages * (1.03 * (double)waves2 + (one_block > 0 && two_block % n_sm == 0 ? 0.78 : 0.0));
    if (two_block > 0 && mixed_us < single_us) single_us = mixed_us;
    single_us += 4.0;  // start-up and read-out of a CTA
    // two CTAs per tile
    const PairPlan plan = pair_plan(d, T);
    double pair_us = 1e30;
    if (plan.use && option(LOPRO_OPT_NO_CTA_PAIRS) != 1) {
        const int slots = n_sm / 2 > 0 ? n_sm / 2 : 1;
        const double tile_us = (double)stages * (T > 256 ? 0.95 : 0.80) + 4.0;
        const int whole_waves = (plan.n_tiles - plan.split_tiles + slots - 1) / slots;
        pair_us = tile_us * (double)whole_waves + (plan.split_tiles > 0 ? tile_us / (double)plan.k_parts + 9.0 : 0.0);
    }
    const bool pairs = T >= kPairMinT ? pair_us < 1e29 : (T > 256 ? pair_us <= single_us * 1.05 : pair_us < single_us);
    if (use_pairs) *use_pairs = pairs;
    return pairs ? pair_us : single_us;
}

cudaError_t launch_prefill(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, const uint8_t* ws,
                           const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int T, cudaStream_t s,
                           const void* a_f16) {
    const void* const a_src = a_f16 != nullptr ? a_f16 : (const void*)(blob + L.off[LOPRO_SEC_A]);
    PrefillParams p;
    p.codes = reinterpret_cast<const uint32_t*>(blob + L.off[LOPRO_SEC_CODES]);
    p.sz = reinterpret_cast<const uint32_t*>(blob + L.off[LOPRO_SEC_SCALEZERO]);
    p.status = reinterpret_cast<int*>(const_cast<uint8_t*>(ws) + W.off_status);
    p.y = y;
    p.ldy = ldy;
    p.out_f32 = out_dtype == LOPRO_OUT_F32;
    p.y_vec = !p.out_f32 && (ldy % 8) == 0 && (reinterpret_cast<uintptr_t>(y) % 16) == 0 && (d.d_out % 8) == 0;
    p.m = d.d_out;
    p.n = d.d_in;
    p.T = T;
    p.nsteps = d.d_in / 64;
    int gs = d.group_size / 64, gshift = 0;
    while ((1 << gshift) < gs) ++gshift;
    p.gshift = gshift;
    p.ng = d.d_in / d.group_size;
    p.r_pad = d.rank > 0 ? L.r_pad : 0;
    p.tile_n = T <= 64 ? 64 : (T <= 128 ? 128 : 256);
    p.lr_stages = (p.r_pad + kStageK - 1) / kStageK;
    const PairPlan plan = pair_plan(d, T);
    bool use_pairs = false;
    (void)prefill_estimate_us(d, T, &use_pairs);
    if (use_pairs) {
        // two CTAs per tile (each loads boxes of 128 tokens)
        PairParams q;
        q.codes = p.codes;
        q.sz = p.sz;
        q.status = p.status;
        q.y = y;
        q.ldy = ldy;
        q.out_f32 = p.out_f32;
        q.y_vec = p.y_vec;
        q.m = p.m;
        q.n = p.n;
        q.T = T;
        q.nsteps = p.nsteps;
        q.gshift = p.gshift;
        q.ng = p.ng;
        q.r_pad = p.r_pad;
        q.lr_stages = p.lr_stages;
        q.row_tiles = plan.row_tiles;
        q.split_first = plan.n_tiles - plan.split_tiles;
        q.k_parts = plan.k_parts;
        q.kparts = reinterpret_cast<float*>(const_cast<uint8_t*>(ws) + W.off_kparts);
        q.kp_tokens = kparts_tokens(T);
        CUtensorMap qx, qa, qt;
        if (!make_map(&qx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, ws + W.off_xrot, (uint64_t)d.d_in, (uint64_t)T, 128u))
            return cudaErrorInvalidValue;
        qa = qx;
        qt = qx;
        if (q.r_pad > 0) {
            if (!make_map(&qa, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, a_src, (uint64_t)q.r_pad, (uint64_t)d.d_out,
                          (uint32_t)kTileM) ||
                !make_map(&qt, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, ws + W.off_t, (uint64_t)q.r_pad, (uint64_t)T, 128u))
                return cudaErrorInvalidValue;
        }
        switch (d.bits) {
            case 2: return launch_pair_bits<2>(q, qx, qa, qt, plan, s);
            case 3: return launch_pair_bits<3>(q, qx, qa, qt, plan, s);
            default: return launch_pair_bits<4>(q, qx, qa, qt, plan, s);
        }
    }
    CUtensorMap mx, ma, mt;
    if (!make_map(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, ws + W.off_xrot, (uint64_t)d.d_in, (uint64_t)T, (uint32_t)p.tile_n))
        return cudaErrorInvalidValue;
    ma = mx;
    mt = mx;
    if (p.r_pad > 0) {
        if (!make_map(&ma, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, a_src, (uint64_t)p.r_pad, (uint64_t)d.d_out,
                      (uint32_t)kTileM) ||
            !make_map(&mt, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, ws + W.off_t, (uint64_t)p.r_pad, (uint64_t)T, (uint32_t)p.tile_n))
            return cudaErrorInvalidValue;
    }
    // Row tiling: R blocks of 128 rows.  A CTA with two blocks streams its activations once for both (the
    // kernel is bound by that stream, so it costs little more than a CTA with one block), but coarser
    // tiles waste more of the last wave; pick the number of two-block CTAs that minimises the makespan of a
    // greedy schedule over the SMs (two-block CTAs are dispatched first, then the single blocks).
    const int units = (T + p.tile_n - 1) / p.tile_n;
    const int m_tiles = (d.d_out + kTileM - 1) / kTileM;
    int best_pairs = m_tiles / 2;
    const int n_sm = sm_count() > 0 ? sm_count() : 1;
    {
        // Makespan of the greedy schedule in closed form (the search runs on the host at every launch): the two-block
        // CTAs leave the SMs on at most two levels, and the one-block CTAs then fill the lower level a round at a time.
        auto makespan = [&](long long n_pairs, long long n_singles) {
            const long long q = n_pairs / n_sm, rem = n_pairs % n_sm;
            double level[2] = {(double)q * kPairCost, (double)(q + 1) * kPairCost};
            long long count[2] = {n_sm - rem, rem};
            double span = n_pairs > 0 ? (rem > 0 ? level[1] : level[0]) : 0.0;
            while (n_singles > 0) {
                const int g = (count[1] == 0 || level[0] <= level[1]) ? 0 : 1;
                level[g] += 1.0;
                if (level[g] > span) span = level[g];
                n_singles -= count[g];
            }
            return span;
        };
        double best_cost = 1e30;
        // (many waves: the mix hardly matters, and the search is not worth its host time)
        for (int pairs = m_tiles / 2; pairs >= ((long long)m_tiles * units <= 20000 ? 0 : m_tiles / 2); --pairs) {
            const double cost = makespan((long long)pairs * units, (long long)(m_tiles - 2 * pairs) * units);
            if (cost < best_cost - 1e-9) {
                best_cost = cost;
                best_pairs = pairs;
            }
        }
    }
    {
        const int forced = option(LOPRO_OPT_PREFILL_PAIRS);  // overrides the choice (tuning only)
        if (forced >= 0 && forced <= m_tiles / 2) best_pairs = forced;
    }
    p.pair_tiles = best_pairs;
    p.single_tiles = m_tiles - 2 * best_pairs;
    p.units = units;
    const long long n_ctas = (long long)(p.pair_tiles + p.single_tiles) * units;
    if (n_ctas > 0x7fffffffLL) return cudaErrorInvalidValue;
    dim3 grid((unsigned)n_ctas);
    switch (d.bits) {
        case 2: return launch_prefill_bits<2>(p, mx, ma, mt, grid, s);
        case 3: return launch_prefill_bits<3>(p, mx, ma, mt, grid, s);
        default: return launch_prefill_bits<4>(p, mx, ma, mt, grid, s);
    }
}

}  // namespace lopro
