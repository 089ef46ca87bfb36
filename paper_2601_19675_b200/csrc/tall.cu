// Small-batch forward (decode, T <= 32) for TALL layers -- more 16-row tiles than one wave of the
// per-tile-group kernel in stream.cu can hold: y = W^ x~ + A t  (steps "Dequant(W_q) X" and
// "U (Sigma Y)" of Appendix A.3, summed as in Eq. 8), after the prologue kernel that writes the
// rotated activations x~ (as the stage image), their 64-column sums and t = B x.
//
// Persistent: one CTA per SM, each owning a contiguous run of 16-row tiles (the runs differ by at
// most one tile) and walking it in groups of up to four tiles (two with 32 tokens).  A producer warp keeps one ring of
// shared-memory stages full ACROSS the groups (16 steps of 64 columns per stage: the packed codes
// and the (scale, zero) pairs of the group's tiles, and the activation records of those columns),
// so the start-up latency of a tile group and the wave tail of a plain grid are paid once per
// kernel, not once per group.  The rows of A of the next group are fetched into the other half of
// a double buffer while the current group is multiplied.
//
// Sixteen consumer warps split a group by (tile, K phase): with R = 1, 2 or 4 tile slots, warp w
// takes tile w mod R and the steps kq, kq + 16/R, ... of every stage, kq = w div R.  A warp
// therefore keeps the sums of ONE tile in registers; at the end of a group the warps kq > 0 pass
// theirs through a small shared-memory buffer to the warp kq = 0 of the tile, which adds them in a
// fixed order and stores the rows.  That warp also starts its sums from the low-rank term A t.  Two
// named barriers (arrive on one side, sync on the other) guard the buffer; the producer never
// takes part in them.
//
// Arithmetic as in stream.cu: sum_k s (c_k - z) x~_k = s (sum_k (128 + c_k) x~_k - (128 + z) sum_k x~_k),
// exact bf16 operands 128 + c_k on the tensor cores, fp32 accumulation, scale and zero-point
// applied in fp32 once per 64 columns.
//
// Every mbarrier wait is bounded; a wait that runs out stores LOPRO_ERR_TIMEOUT in the workspace
// status word and the CTA stops waiting (its outputs are then unspecified).
#include "common.cuh"
#include "ptx.cuh"

namespace lopro {

namespace {

constexpr int kConsumerWarps = 16;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;  // + one producer warp
constexpr int kStageSteps = 16;                  // 64-column steps per stage
constexpr int kMaxGroupTiles = 4;                // 16-row tiles per group (2 when 32 tokens fill the stages)
constexpr int kMaxStages = 8;
constexpr int kSzTile = kStageSteps * 64;        // bytes reserved per tile and stage for (scale, zero) pairs

struct TallParams {
    const unsigned char* codes;
    const uint32_t* sz;
    const __half* A;
    const unsigned char* act;  // activation image [stage][t_pad][kActRecord]
    const __half* t;           // [T][r_pad] low-rank intermediate
    int* status;
    void* y;
    int64_t ldy;
    int out_f32;
    int m, n, T, t_pad;
    int nsteps, gshift, ng, r_pad;
    int gt;            // 16-row tiles per group: 4 or 2
    int n_stages;      // ring depth (<= stages per group)
    int total_stages;  // stages per group = ceil(nsteps / 16)
    int lr8;           // the up-projection factor is fp8 e4m3 (U of the FP8 low-rank record), one byte per entry
    // shared-memory layout (bytes from the dynamic base)
    int off_a, a_bytes, off_t, off_red, off_ring, stage_bytes, off_stage_sz, off_stage_x;
};

// Sibling layers of a grouped launch: the grid's CTAs from cta0[i] on work on sibling i (the layer of TallParams
// owns the CTAs before cta0[0]); each sibling walks its own rows with its own share of the persistent CTAs.
struct TallSiblings {
    int n;
    int cta0[kMaxSiblings - 1];
    const unsigned char* codes[kMaxSiblings - 1];
    const uint32_t* sz[kMaxSiblings - 1];
    const __half* A[kMaxSiblings - 1];
    const unsigned char* act[kMaxSiblings - 1];
    const __half* t[kMaxSiblings - 1];
    void* y[kMaxSiblings - 1];
    int64_t ldy[kMaxSiblings - 1];
    int m[kMaxSiblings - 1];
    int T[kMaxSiblings - 1];  // token rows of the sibling
};

// A launch of a single layer carries no table (several hundred bytes of kernel parameters less).
struct NoTallSiblings {};
__device__ __forceinline__ int2 select_sibling(TallParams&, const NoTallSiblings&) {
    return make_int2((int)blockIdx.x, (int)gridDim.x);
}

// The layer a CTA works on: patches the per-layer fields, returns the CTA's index among the layer's CTAs and
// their number.
__device__ __forceinline__ int2 select_sibling(TallParams& p, const TallSiblings& sibs) {
    int idx = -1;
#pragma unroll
    for (int i = 0; i < kMaxSiblings - 1; ++i)
        if (i < sibs.n && (int)blockIdx.x >= sibs.cta0[i]) idx = i;
    if (idx < 0) return make_int2((int)blockIdx.x, sibs.n > 0 ? sibs.cta0[0] : (int)gridDim.x);
    // (a __grid_constant__ parameter: one constant-bank load per field at a computed index)
    const int first = sibs.cta0[idx], end = idx + 1 < sibs.n ? sibs.cta0[idx + 1] : (int)gridDim.x;
    p.codes = sibs.codes[idx];
    p.sz = sibs.sz[idx];
    p.A = sibs.A[idx];
    p.act = sibs.act[idx];
    p.t = sibs.t[idx];
    p.y = sibs.y[idx];
    p.ldy = sibs.ldy[idx];
    p.m = sibs.m[idx];
    p.T = sibs.T[idx];
    return make_int2((int)blockIdx.x - first, end - first);
}

__device__ __forceinline__ void named_sync(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(kConsumerThreads) : "memory");
}
__device__ __forceinline__ void named_arrive(int id) {
    __threadfence_block();
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(kConsumerThreads) : "memory");
}

// One 16-row tile times one 64-column step: expand the packed codes to bf16 operands 128 + c, four
// m16n8k16 products per token tile, then scale and zero-point in fp32 against the 64-column sums.
// wp: the lane's words of the step; xaddr: the lane's ldmatrix row of the step (shared-space address);
// sxp: the step's 64-column sum of token 2 * tg; szp: the (scale, zero) pair of row gq in the step's group.
template <int BITS, int NT>
__device__ __forceinline__ void tile_step(const uint32_t* wp, uint32_t xaddr, const float* sxp, const uint32_t* szp,
                                          float (&yacc)[NT][4]) {
    uint32_t b[NT][8];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        ldmatrix_x4(*reinterpret_cast<uint32_t(*)[4]>(&b[nt][0]), xaddr + (uint32_t)(nt * 8 * kActRecord));
        ldmatrix_x4(*reinterpret_cast<uint32_t(*)[4]>(&b[nt][4]), xaddr + (uint32_t)(nt * 8 * kActRecord) + 64u);
    }
    float sx[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        sx[nt][0] = sxp[nt * 8 * (kActRecord / 4)];
        sx[nt][1] = sxp[(nt * 8 + 1) * (kActRecord / 4)];
    }
    uint32_t w[BITS];
    if constexpr (BITS == 4) {
        const uint4 v = *reinterpret_cast<const uint4*>(wp);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    } else if constexpr (BITS == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(wp);
        w[0] = v.x; w[1] = v.y;
    } else {
#pragma unroll
        for (int q = 0; q < BITS; ++q) w[q] = wp[q];
    }
    uint32_t a[16];
    expand_codes<BITS>(a, w);
    const uint32_t sz_lo = szp[0], sz_hi = szp[8];
    const float2 f_lo = __half22float2(*reinterpret_cast<const __half2*>(&sz_lo));
    const float2 f_hi = __half22float2(*reinterpret_cast<const __half2*>(&sz_hi));
    const float nsz_lo = -f_lo.x * (128.0f + f_lo.y), nsz_hi = -f_hi.x * (128.0f + f_hi.y);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float acc[4];
        mma_bf16_first(acc, &a[0], b[nt][0], b[nt][1]);
        mma_bf16(acc, &a[4], b[nt][2], b[nt][3]);
        mma_bf16(acc, &a[8], b[nt][4], b[nt][5]);
        mma_bf16(acc, &a[12], b[nt][6], b[nt][7]);
        yacc[nt][0] = fmaf(f_lo.x, acc[0], fmaf(nsz_lo, sx[nt][0], yacc[nt][0]));
        yacc[nt][1] = fmaf(f_lo.x, acc[1], fmaf(nsz_lo, sx[nt][1], yacc[nt][1]));
        yacc[nt][2] = fmaf(f_hi.x, acc[2], fmaf(nsz_hi, sx[nt][0], yacc[nt][2]));
        yacc[nt][3] = fmaf(f_hi.x, acc[3], fmaf(nsz_hi, sx[nt][1], yacc[nt][3]));
    }
}

// Byte offsets, from the start of a stage, of what a warp reads in its first step (step kq of tile slot r); they
// change only when the split of the warps changes, i.e. once per group of tiles.
struct WarpOffsets {
    uint32_t w, x, sx, sz;
};

// The steps kq, kq + KQ, ... of one stage for tile slot r (KQ = 16 >> RBITS phases), unrolled with constant
// strides; gs = min(gshift, 4): a stage starts on a group boundary or lies inside one group, so the group of
// step st within the stage's (scale, zero) block is st >> gs.
template <int BITS, int NT, int RBITS>
__device__ __forceinline__ void consume_stage(const unsigned char* stage, uint32_t stage_u32, const WarpOffsets& o, int kq,
                                              int gs, int steps, float (&yacc)[NT][4]) {
    constexpr int KQ = kConsumerWarps >> RBITS, PER = kStageSteps / KQ;
    constexpr int kStepBytes = 128 * BITS;
    const unsigned char* wbase = stage + o.w;
    const float* sxbase = reinterpret_cast<const float*>(stage + o.sx);
    const uint32_t* szbase = reinterpret_cast<const uint32_t*>(stage + o.sz);
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int st = kq + i * KQ;
        if (st < steps)
            tile_step<BITS, NT>(reinterpret_cast<const uint32_t*>(wbase + i * KQ * kStepBytes),
                                stage_u32 + o.x + (uint32_t)(i * KQ * 128), sxbase + i * KQ, szbase + (st >> gs) * 16,
                                yacc);
    }
}

template <int BITS, int NT, typename SIBS>
__global__ void __launch_bounds__(kThreads, 1)
tall_kernel(const TallParams p_in, const __grid_constant__ SIBS sibs) {
    TallParams p = p_in;
    const int2 cta = select_sibling(p, sibs);  // x: index among the layer's CTAs, y: their number
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bars[2 * kMaxStages + 3];  // full, empty per stage; A buffers; t
    __shared__ int s_timeout;
    constexpr int kTok = NT * 8;
    constexpr int kStepBytes = 128 * BITS;  // codes of one 16-row tile and one 64-column step

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, tg = lane & 3;
    // this CTA's run of 16-row tiles: the first `extra` CTAs hold one tile more
    const int tiles = p.m >> 4;
    const int base = tiles / cta.y, extra = tiles - base * cta.y;
    const int my_cnt = base + (cta.x < extra ? 1 : 0);
    const int my_start = cta.x * base + min(cta.x, extra);
    const int n_groups = (my_cnt + p.gt - 1) / p.gt;
    const int TS = p.total_stages;
    const int tc = min(kTok, p.T);  // live tokens
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty = [&](int s) { return bar0 + 8u * (uint32_t)(kMaxStages + s); };
    auto afull = [&](int b) { return bar0 + 8u * (uint32_t)(2 * kMaxStages + b); };
    const uint32_t tbar = bar0 + 8u * (uint32_t)(2 * kMaxStages + 2);
    const uint32_t smem0 = smem_u32(smem);

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < p.n_stages; ++s) {
            mbar_init(full(s), 2);  // one arrival with the layer data, one with the activations
            mbar_init(empty(s), kConsumerWarps);
        }
        mbar_init(afull(0), 1);
        mbar_init(afull(1), 1);
        mbar_init(tbar, 1);
        s_timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto steps_of = [&](int s) { return min(kStageSteps, p.nsteps - s * kStageSteps); };

    if (warp == kConsumerWarps) {
        // ---------------- producer warp ----------------
        // layer data of global stage S = (group, stage): codes and (scale, zero) pairs of the group's
        // tiles; with a group's first stage, its rows of A into the buffer of the group's parity
        auto issue_w = [&](int S) {
            const int gi = S / TS, s = S - gi * TS, slot = S % p.n_stages;
            const int tile0 = my_start + gi * p.gt;
            const int n_rt = min(p.gt, my_cnt - gi * p.gt);
            const int steps = steps_of(s);
            const int g0 = (s * kStageSteps) >> p.gshift, g1 = (s * kStageSteps + steps - 1) >> p.gshift;
            const uint32_t b_codes = (uint32_t)(steps * kStepBytes), b_sz = (uint32_t)((g1 - g0 + 1) * 64);
            const uint32_t dst = smem0 + p.off_ring + slot * p.stage_bytes;
            mbar_expect_tx(full(slot), (b_codes + b_sz) * (uint32_t)n_rt);
            for (int r = 0; r < n_rt; ++r) {
                bulk_g2s(dst + r * kStageSteps * kStepBytes,
                         p.codes + ((size_t)(tile0 + r) * p.nsteps + (size_t)s * kStageSteps) * kStepBytes, b_codes,
                         full(slot));
                bulk_g2s(dst + p.off_stage_sz + r * kSzTile, p.sz + ((size_t)(tile0 + r) * p.ng + g0) * 16, b_sz,
                         full(slot));
            }
            if (s == 0 && p.r_pad > 0) {
                const uint32_t b_a = (uint32_t)(n_rt * 16 * p.r_pad * (p.lr8 ? 1 : 2));
                mbar_expect_tx(afull(gi & 1), b_a);
                bulk_g2s(smem0 + p.off_a + (gi & 1) * p.a_bytes,
                         reinterpret_cast<const unsigned char*>(p.A) + (size_t)tile0 * 16 * p.r_pad * (p.lr8 ? 1 : 2), b_a, afull(gi & 1));
            }
        };
        // activations of the stage: the records of the live tokens, one contiguous piece of the image
        auto issue_x = [&](int S) {
            const int s = S % TS, slot = S % p.n_stages;
            const uint32_t bytes = (uint32_t)(tc * kActRecord);
            mbar_expect_tx(full(slot), bytes);
            bulk_g2s(smem0 + p.off_ring + slot * p.stage_bytes + p.off_stage_x,
                     p.act + (size_t)s * p.t_pad * kActRecord, bytes, full(slot));
        };
        const int total = n_groups * TS;
        const int first = min(p.n_stages, total);
        if (lane == 0)
            for (int S = 0; S < first; ++S) issue_w(S);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (lane == 0 && total > 0) {
            for (int S = 0; S < first; ++S) issue_x(S);
            if (p.r_pad > 0) {  // low-rank intermediate of the live tokens
                const uint32_t t_bytes = (uint32_t)(tc * p.r_pad * 2);
                mbar_expect_tx(tbar, t_bytes);
                bulk_g2s(smem0 + p.off_t, p.t, t_bytes, tbar);
            }
            for (int S = first; S < total; ++S) {
                const int slot = S % p.n_stages;
                const uint32_t parity = (uint32_t)((S / p.n_stages) - 1) & 1u;
                if (!s_timeout && !mbar_wait(empty(slot), parity)) {
                    s_timeout = 1;
                    atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
                }
                issue_w(S);
                issue_x(S);
            }
        }
        return;
    }

    // ---------------- consumer warps ----------------
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t ldm_off = (uint32_t)((lane & 7) * kActRecord + (lane >> 3) * 16);
    float* red = reinterpret_cast<float*>(smem + p.off_red);  // [writer][NT * 4][32 lanes]
    bool wrote_red = false;  // this warp handed sums over in an earlier group
    bool dead = false;       // a wait of this warp ran out
    const int gs = min(p.gshift, 4);
    // the ring slot of the next stage, its parity and its address
    int slot = 0;
    uint32_t phase = 0;
    const unsigned char* stage = smem + p.off_ring;
    uint32_t stage_u32 = smem0 + (uint32_t)p.off_ring;
    for (int gi = 0; gi < n_groups; ++gi) {
        const int tile0 = my_start + gi * p.gt;
        const int n_rt = min(p.gt, my_cnt - gi * p.gt);
        const int rbits = n_rt == 1 ? 0 : (n_rt == 2 ? 1 : 2);
        const int R = 1 << rbits, KQ = kConsumerWarps >> rbits;
        const int r = warp & (R - 1), kq = warp >> rbits;
        const bool active = r < n_rt;

        // a change of the split (last, shorter group): warps that turn from reading the hand-over buffer
        // to writing it must not overtake the other readers of the previous group
        if (gi > 0 && (1 << rbits) < p.gt) named_sync(3);

        float yacc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) yacc[nt][i] = 0.0f;
        if (kq == 0 && p.r_pad > 0) {
            // low-rank term A t of the tile (f16 tensor-core product) starts the sums
            bool ok = mbar_wait(afull(gi & 1), (uint32_t)(gi >> 1) & 1u);
            if (gi == 0) ok = mbar_wait(tbar, 0) && ok;
            if (!ok) {
                s_timeout = 1;
                if (lane == 0) atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
            }
            if (active) {
                const unsigned char* as = smem + p.off_a + (gi & 1) * p.a_bytes + (size_t)r * 16 * p.r_pad * (p.lr8 ? 1 : 2);
                const __half* ts = reinterpret_cast<const __half*>(smem + p.off_t);
                for (int jj = 0; jj < p.r_pad; jj += 16) {
                    uint32_t a[4];
                    load_up_fragment(a, as, p.r_pad, gq, tg, jj, p.lr8 != 0);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const __half* trow = ts + (nt * 8 + gq) * p.r_pad + jj + 2 * tg;
                        mma_f16(yacc[nt], a, *reinterpret_cast<const uint32_t*>(trow),
                                *reinterpret_cast<const uint32_t*>(trow + 8));
                    }
                }
            }
        }

        WarpOffsets wo;
        wo.w = (uint32_t)((r * kStageSteps + kq) * kStepBytes + lane * (BITS * 4));
        wo.x = (uint32_t)p.off_stage_x + ldm_off + (uint32_t)(kq * 128);
        wo.sx = (uint32_t)(p.off_stage_x + 2048 + 2 * tg * kActRecord + kq * 4);
        wo.sz = (uint32_t)(p.off_stage_sz + r * kSzTile + gq * 4);
        for (int s = 0; s < TS; ++s) {
            if (!dead && !mbar_wait(full(slot), phase)) {
                dead = true;  // this warp stops waiting; its outputs are unspecified
                s_timeout = 1;
                if (lane == 0) atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
            }
            if (active) {
                const int steps = steps_of(s);
                if (rbits == 2) consume_stage<BITS, NT, 2>(stage, stage_u32, wo, kq, gs, steps, yacc);
                else if (rbits == 1) consume_stage<BITS, NT, 1>(stage, stage_u32, wo, kq, gs, steps, yacc);
                else consume_stage<BITS, NT, 0>(stage, stage_u32, wo, kq, gs, steps, yacc);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty(slot));
            // next slot of the ring
            ++slot;
            stage += p.stage_bytes;
            stage_u32 += (uint32_t)p.stage_bytes;
            if (slot == p.n_stages) {
                slot = 0;
                phase ^= 1u;
                stage = smem + p.off_ring;
                stage_u32 = smem0 + (uint32_t)p.off_ring;
            }
        }

        // ---- end of the group: the K phases of a tile meet in the warp kq = 0, which stores the rows ----
        if (kq > 0) {
            if (wrote_red) named_sync(2);  // the previous group's sums have been read
            float* mine = red + (size_t)((kq - 1) * R + r) * (NT * 4 * 32);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) mine[(nt * 4 + i) * 32 + lane] = yacc[nt][i];
            named_arrive(1);
            wrote_red = true;
        } else {
            if (KQ > 1) named_sync(1);
            for (int k = 1; k < KQ; ++k) {
                const float* theirs = red + (size_t)((k - 1) * R + r) * (NT * 4 * 32);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) yacc[nt][i] += theirs[(nt * 4 + i) * 32 + lane];
            }
            if (KQ > 1) named_arrive(2);
            if (active) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int tk = nt * 8 + 2 * tg + (i & 1);
                        if (tk < p.T) {
                            const size_t o = (size_t)tk * p.ldy + (size_t)(tile0 + r) * 16 + gq + 8 * (i >> 1);
                            if (p.out_f32) reinterpret_cast<float*>(p.y)[o] = yacc[nt][i];
                            else reinterpret_cast<__nv_bfloat16*>(p.y)[o] = __float2bfloat16_rn(yacc[nt][i]);
                        }
                    }
            }
        }
    }
}

struct TallPlan {
    int nt, gt, grid, n_stages, total_stages;
    int off_a, a_bytes, off_t, off_red, off_ring, stage_bytes, off_stage_sz, off_stage_x, smem_bytes;
};

// total_rows: rows of the layer, or of all the sibling layers that share the launch
bool plan_tall(const lopro_desc& d, int T, TallPlan* pl, long long total_rows = 0) {
    if (T < 1 || T > kDecodeMaxT) return false;
    const int n_sm = sm_count();
    const long long tiles = (total_rows > 0 ? total_rows : (long long)d.d_out) / 16;
    // Up to two 16-row tiles per SM one wave of the per-group kernel holds the layer and is faster (4096 rows at 1 and 8
    // tokens: 5.7 and 6.2 us against 7.4 and 8.4); with more than 16 tokens the persistent kernel wins from one tile
    // per SM on (4096 rows 12.8 -> 12.5 us, 11008 -> 4096 27.6 -> 25.6).
    if (tiles <= (T > 16 ? 1LL : 2LL) * n_sm) return false;
    const int r_pad = d.rank > 0 ? round_up_int(d.rank, 16) : 0;
    pl->nt = T <= 8 ? 1 : (T <= 16 ? 2 : 4);
    const int ktok = pl->nt * 8;
    pl->gt = pl->nt == 4 ? 2 : kMaxGroupTiles;
    pl->grid = n_sm;
    pl->total_stages = (d.d_in / 64 + kStageSteps - 1) / kStageSteps;
    int off = 0;
    pl->off_a = off;
    pl->a_bytes = round_up_int(pl->gt * 16 * r_pad * 2, 128);
    off += 2 * pl->a_bytes;
    pl->off_t = off;
    off += round_up_int(ktok * r_pad * 2, 128);
    pl->off_red = off;
    off += (kConsumerWarps - 1) * pl->nt * 4 * 32 * 4;
    pl->off_ring = off;
    pl->off_stage_sz = pl->gt * kStageSteps * 128 * d.bits;
    pl->off_stage_x = pl->off_stage_sz + pl->gt * kSzTile;
    pl->stage_bytes = round_up_int(pl->off_stage_x + ktok * kActRecord, 128);
    int stages = (kStreamMaxSmem - off) / pl->stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages > pl->total_stages) stages = pl->total_stages;  // the ring never spans more than one group
    if (stages < 1 || (stages < 2 && pl->total_stages > 1)) return false;
    pl->n_stages = stages;
    pl->smem_bytes = off + stages * pl->stage_bytes;
    return true;
}

template <int BITS, int NT, typename SIBS>
cudaError_t launch_tall_ks(const TallParams& p, const SIBS& sibs, int grid, int smem_bytes, cudaStream_t s) {
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(tall_kernel<BITS, NT, SIBS>, kStreamMaxSmem, &attr_done);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tall_kernel<BITS, NT, SIBS>, p, sibs);
}

template <int BITS, int NT>
cudaError_t launch_tall_k(const TallParams& p, const TallSiblings& sibs, int grid, int smem_bytes, cudaStream_t s) {
    return sibs.n == 0 && option(LOPRO_OPT_ONE_KERNEL_SET) != 1 ? launch_tall_ks<BITS, NT, NoTallSiblings>(p, NoTallSiblings{}, grid, smem_bytes, s)
                       : launch_tall_ks<BITS, NT, TallSiblings>(p, sibs, grid, smem_bytes, s);
}

template <int BITS>
cudaError_t launch_tall_bits(const TallParams& p, const TallSiblings& sibs, int nt, int grid, int smem_bytes, cudaStream_t s) {
    if (nt == 1) return launch_tall_k<BITS, 1>(p, sibs, grid, smem_bytes, s);
    if (nt == 2) return launch_tall_k<BITS, 2>(p, sibs, grid, smem_bytes, s);
    return launch_tall_k<BITS, 4>(p, sibs, grid, smem_bytes, s);
}

}  // namespace

bool tall_supported(const lopro_desc& d, int T, long long total_rows) {
    TallPlan pl;
    return plan_tall(d, T, &pl, total_rows);
}

cudaError_t launch_tall(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, const uint8_t* ws,
                        const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int T, cudaStream_t s, int t0,
                        const StreamSiblingArgs* more) {
    TallPlan pl;
    long long total_rows = d.d_out;
    if (more != nullptr)
        for (int i = 0; i < more->n; ++i) total_rows += more->d_out[i];
    if (!plan_tall(d, T, &pl, total_rows)) return cudaErrorInvalidValue;
    TallParams p;
    p.codes = blob + L.off[LOPRO_SEC_CODES];
    p.sz = reinterpret_cast<const uint32_t*>(blob + L.off[LOPRO_SEC_SCALEZERO]);
    p.A = reinterpret_cast<const __half*>(blob + L.off[LOPRO_SEC_A]);
    // t0: first token of this launch within the activation image and t (a chunk of a longer batch)
    p.act = ws + W.off_xrot + (size_t)t0 * kActRecord;
    p.t = reinterpret_cast<const __half*>(ws + W.off_t) + (size_t)t0 * (d.rank > 0 ? L.r_pad : 0);
    p.status = reinterpret_cast<int*>(const_cast<uint8_t*>(ws) + W.off_status);
    p.y = y;
    p.ldy = ldy;
    p.out_f32 = out_dtype == LOPRO_OUT_F32;
    p.m = d.d_out;
    p.n = d.d_in;
    p.T = T;
    p.t_pad = W.t_pad;
    p.nsteps = d.d_in / 64;
    int gs = d.group_size / 64, gshift = 0;
    while ((1 << gshift) < gs) ++gshift;
    p.gshift = gshift;
    p.ng = d.d_in / d.group_size;
    p.r_pad = d.rank > 0 ? L.r_pad : 0;
    p.lr8 = d.lowrank_format == LOPRO_LOWRANK_FP8 ? 1 : 0;
    p.gt = pl.gt;
    p.n_stages = pl.n_stages;
    p.total_stages = pl.total_stages;
    p.off_a = pl.off_a;
    p.a_bytes = pl.a_bytes;
    p.off_t = pl.off_t;
    p.off_red = pl.off_red;
    p.off_ring = pl.off_ring;
    p.stage_bytes = pl.stage_bytes;
    p.off_stage_sz = pl.off_stage_sz;
    p.off_stage_x = pl.off_stage_x;
    TallSiblings sibs = {};
    if (more != nullptr && more->n > 0) {
        // the persistent CTAs are shared out in proportion to the layers' row tiles (at least one CTA each)
        long long tiles_all = d.d_out / 16;
        for (int i = 0; i < more->n; ++i) tiles_all += more->d_out[i] / 16;
        sibs.n = more->n;
        long long tiles_before = d.d_out / 16;
        for (int i = 0; i < more->n; ++i) {
            int c0 = (int)((tiles_before * pl.grid + tiles_all / 2) / tiles_all);
            const int lo = (i == 0 ? 0 : sibs.cta0[i - 1]) + 1, hi = pl.grid - (more->n - i);
            if (c0 < lo) c0 = lo;
            if (c0 > hi) c0 = hi;
            sibs.cta0[i] = c0;
            tiles_before += more->d_out[i] / 16;
            const uint8_t* b = more->blob[i];
            const BlobLayout& Li = more->L[i];
            const uint8_t* wsi = more->ws[i];
            sibs.codes[i] = b + Li.off[LOPRO_SEC_CODES];
            sibs.sz[i] = reinterpret_cast<const uint32_t*>(b + Li.off[LOPRO_SEC_SCALEZERO]);
            sibs.A[i] = reinterpret_cast<const __half*>(b + Li.off[LOPRO_SEC_A]);
            sibs.act[i] = wsi + W.off_xrot + (size_t)t0 * kActRecord;
            sibs.t[i] = reinterpret_cast<const __half*>(wsi + W.off_t) + (size_t)t0 * (d.rank > 0 ? L.r_pad : 0);
            sibs.y[i] = more->y[i];
            sibs.ldy[i] = more->ldy[i];
            sibs.m[i] = more->d_out[i];
            sibs.T[i] = more->own_rows ? more->T_of[i + 1] : T;
        }
        if (more->own_rows) p.T = more->T_of[0];
    }
    switch (d.bits) {
        case 2: return launch_tall_bits<2>(p, sibs, pl.nt, pl.grid, pl.smem_bytes, s);
        case 3: return launch_tall_bits<3>(p, sibs, pl.nt, pl.grid, pl.smem_bytes, s);
        default: return launch_tall_bits<4>(p, sibs, pl.nt, pl.grid, pl.smem_bytes, s);
    }
}

}  // namespace lopro
