// Small-batch forward (decode, T <= 32): y = W^ x~ + A t, the packed codes streamed once from HBM
// by bulk asynchronous copies (steps "Dequant(W_q) X" and "U (Sigma Y)" of Appendix A.3, summed as
// in Eq. 8).
//
// One CTA owns 32 or 64 output rows (two or four 16-row tiles of the fragment layout) over the WHOLE K range, so
// no partial sums ever cross CTAs.  A producer warp fills a ring of shared-memory stages with
// cp.async.bulk copies (16 steps of 64 columns per stage): the layer's own data -- codes,
// (scale, zero) pairs, the rows of A -- is requested before griddepcontrol.wait, i.e. while the
// prologue kernel of the same forward still runs; the rotated activations and their 64-column
// sums follow after the wait.  Sixteen consumer warps split each stage by K step (warp w takes
// step w), multiply with mma.sync and keep their sums in registers (the warps 0 .. RT-1 start theirs
// from the low-rank term A t); one shared-memory reduction over the warps at the end, then the store.
//
// Arithmetic: as in the general path, sum_k s (c_k - z) x~_k = s (sum_k (128 + c_k) x~_k
// - (128 + z) sum_k x~_k), the first sum on the tensor cores with exact bf16 operands 128 + c_k,
// fp32 accumulation, scale and zero-point applied in fp32 once per 64 columns.
//
// Every wait on an mbarrier is bounded; a wait that runs out stores LOPRO_ERR_TIMEOUT in the
// workspace status word and the CTA stops waiting (its outputs are then unspecified).
#include <stdlib.h>

#include "common.cuh"
#include "ptx.cuh"

namespace lopro {

namespace {

constexpr int kConsumerWarps = 16;
constexpr int kThreads = (kConsumerWarps + 1) * 32;  // + one producer warp
constexpr int kStageSteps = 16;                      // 64-column steps per stage = one per consumer warp
constexpr int kXsStride = kActRecord / 2;            // bf16 elements between the token rows of a stage
constexpr int kMaxStages = 8;
constexpr int kRedPad = 4;  // floats of padding per token row of the reduction buffer

struct StreamParams {
    const uint32_t* codes;
    const uint32_t* sz;
    const __half* A;
    const unsigned char* act;   // activation image [stage][t_pad][kActRecord]
    const __half* t;            // [T][r_pad] low-rank intermediate
    int* status;
    void* y;
    int64_t ldy;
    int out_f32;
    int m, n, T, t_pad;
    int nsteps, gshift, ng, r_pad;
    int n_stages;  // ring depth
    int total_stages;
    int lr8;       // the up-projection factor is fp8 e4m3 (U of the FP8 low-rank record), one byte per entry
    // shared-memory layout (bytes from the dynamic base)
    int off_sz, off_a, off_t, off_ring, stage_bytes, off_stage_x;
};

// Sibling layers 1 .. n of a grouped launch (sibling 0 travels in StreamParams): same shape of K, quantization and
// rank, each its own rows and data; CTAs [cta0[i], cta0[i + 1]) of the grid belong to sibling i + 1.
struct StreamSiblings {
    int n;
    int cta0[kMaxSiblings - 1];
    const uint32_t* codes[kMaxSiblings - 1];
    const uint32_t* sz[kMaxSiblings - 1];
    const __half* A[kMaxSiblings - 1];
    const unsigned char* act[kMaxSiblings - 1];
    const __half* t[kMaxSiblings - 1];
    void* y[kMaxSiblings - 1];
    int64_t ldy[kMaxSiblings - 1];
    int m[kMaxSiblings - 1];
    int T[kMaxSiblings - 1];  // token rows of the sibling (experts of a mixture layer differ; otherwise all alike)
};

// A launch of a single layer carries no table at all (the table is several hundred bytes of kernel parameters, and
// their mere presence was measured at 0.15 us per launch of the smallest layers).
struct NoSiblings {};
__device__ __forceinline__ int select_sibling(StreamParams&, const NoSiblings&) { return (int)blockIdx.x; }

// The layer a CTA works on: patches the per-layer fields of the parameters, returns the CTA's index within the layer.
// (The table is a __grid_constant__ parameter: its arrays are read from the constant bank with a computed index,
// one load per field, instead of a chain of selects over every entry.)
__device__ __forceinline__ int select_sibling(StreamParams& p, const StreamSiblings& sibs) {
    int idx = -1;
#pragma unroll
    for (int i = 0; i < kMaxSiblings - 1; ++i)
        if (i < sibs.n && (int)blockIdx.x >= sibs.cta0[i]) idx = i;
    if (idx < 0) return (int)blockIdx.x;
    p.codes = sibs.codes[idx];
    p.sz = sibs.sz[idx];
    p.A = sibs.A[idx];
    p.act = sibs.act[idx];
    p.t = sibs.t[idx];
    p.y = sibs.y[idx];
    p.ldy = sibs.ldy[idx];
    p.m = sibs.m[idx];
    p.T = sibs.T[idx];
    return (int)blockIdx.x - sibs.cta0[idx];
}

template <int BITS, int NT, int RT, typename SIBS>
__global__ void __launch_bounds__(kThreads, 1)
stream_kernel(const StreamParams p_in, const __grid_constant__ SIBS sibs) {
    StreamParams p = p_in;
    const int bx = select_sibling(p, sibs);
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bars[3 * kMaxStages + 2];  // wfull, xfull, empty per stage; sz + A; t
    __shared__ int s_timeout;
    constexpr int kTok = NT * 8;
    constexpr int kStepBytes = 128 * BITS;  // codes of one 16-row tile and one 64-column step

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, tg = lane & 3;
    const int rt0 = bx * RT;                             // first 16-row tile of this CTA
    const int n_rt = min(RT, (p.m >> 4) - rt0);          // live row tiles
    const int tc = min(kTok, p.T);                                  // live tokens
    const uint32_t bar0 = smem_u32(bars);
    auto wfull = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto xfull = [&](int s) { return bar0 + 8u * (uint32_t)(kMaxStages + s); };
    auto empty = [&](int s) { return bar0 + 8u * (uint32_t)(2 * kMaxStages + s); };
    const uint32_t cbar = bar0 + 8u * (uint32_t)(3 * kMaxStages);
    const uint32_t tbar = cbar + 8u;
    const uint32_t smem0 = smem_u32(smem);

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < p.n_stages; ++s) {
            mbar_init(wfull(s), 1);
            mbar_init(xfull(s), 1);
            mbar_init(empty(s), kConsumerWarps);
        }
        mbar_init(cbar, 1);
        mbar_init(tbar, 1);
        s_timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto steps_of = [&](int stage) { return min(kStageSteps, p.nsteps - stage * kStageSteps); };
    // weights of one stage: for each live row tile, `steps` consecutive steps of packed codes
    auto issue_w = [&](int stage, int slot) {
        const int steps = steps_of(stage);
        const uint32_t bytes = (uint32_t)(steps * kStepBytes);
        mbar_expect_tx(wfull(slot), bytes * (uint32_t)n_rt);
        for (int r = 0; r < n_rt; ++r) {
            const unsigned char* src = reinterpret_cast<const unsigned char*>(p.codes) +
                                       ((size_t)(rt0 + r) * p.nsteps + (size_t)stage * kStageSteps) * kStepBytes;
            bulk_g2s(smem0 + p.off_ring + slot * p.stage_bytes + r * kStageSteps * kStepBytes, src, bytes, wfull(slot));
        }
    };
    // activations of one stage: the records of the live tokens, one contiguous piece of the image
    auto issue_x = [&](int stage, int slot) {
        const uint32_t bytes = (uint32_t)(tc * kActRecord);
        mbar_expect_tx(xfull(slot), bytes);
        bulk_g2s(smem0 + p.off_ring + slot * p.stage_bytes + p.off_stage_x,
                 p.act + (size_t)stage * p.t_pad * kActRecord, bytes, xfull(slot));
    };

    float yacc[RT][NT][4];
#pragma unroll
    for (int r = 0; r < RT; ++r)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) yacc[r][nt][i] = 0.0f;

    // low-rank up-projection A t: warp r starts the sums of row tile r with it (fp16 tensor-core product
    // into the fp32 sums), before the first stage, so that nothing but the reduction follows the last one
    auto lowrank_up = [&](float (&acc)[NT][4], int r) {
        const unsigned char* as = smem + p.off_a + (size_t)r * 16 * p.r_pad * (p.lr8 ? 1 : 2);
        const __half* ts = reinterpret_cast<const __half*>(smem + p.off_t);
        for (int jj = 0; jj < p.r_pad; jj += 16) {
            uint32_t a[4];
            load_up_fragment(a, as, p.r_pad, gq, tg, jj, p.lr8 != 0);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const __half* trow = ts + (nt * 8 + gq) * p.r_pad + jj + 2 * tg;
                mma_f16(acc[nt], a, *reinterpret_cast<const uint32_t*>(trow), *reinterpret_cast<const uint32_t*>(trow + 8));
            }
        }
    };
    if (warp == kConsumerWarps) {
        // ---------------- producer warp ----------------
        const int first = min(p.n_stages, p.total_stages);
        if (lane == 0) {
            // layer data: (scale, zero) pairs and rows of A of the live row tiles, then the first stages of codes
            const uint32_t sz_bytes = (uint32_t)(n_rt * p.ng * 64);
            const uint32_t a_bytes = (uint32_t)(n_rt * 16 * p.r_pad * (p.lr8 ? 1 : 2));
            mbar_expect_tx(cbar, sz_bytes + a_bytes);
            bulk_g2s(smem0 + p.off_sz, p.sz + (size_t)rt0 * p.ng * 16, sz_bytes, cbar);
            if (a_bytes)
                bulk_g2s(smem0 + p.off_a, reinterpret_cast<const unsigned char*>(p.A) + (size_t)rt0 * 16 * p.r_pad * (p.lr8 ? 1 : 2),
                         a_bytes, cbar);
            for (int s = 0; s < first; ++s) issue_w(s, s);
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (lane == 0) {
            for (int s = 0; s < first; ++s) issue_x(s, s);
            if (p.r_pad > 0) {  // low-rank intermediate of the live tokens
                const uint32_t t_bytes = (uint32_t)(tc * p.r_pad * 2);
                mbar_expect_tx(tbar, t_bytes);
                bulk_g2s(smem0 + p.off_t, p.t, t_bytes, tbar);
            }
        }
        if (lane == 0) {
            for (int s = first; s < p.total_stages; ++s) {
                const int slot = s % p.n_stages;
                const uint32_t parity = (uint32_t)((s / p.n_stages) - 1) & 1u;
                if (!s_timeout && !mbar_wait(empty(slot), parity)) {
                    s_timeout = 1;
                    atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
                }
                issue_w(s, slot);
                issue_x(s, slot);
            }
        }
    } else {
        // ---------------- consumer warps ----------------
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (!mbar_wait(cbar, 0)) {
            s_timeout = 1;
            if (lane == 0) atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
        }
        if (p.r_pad > 0 && warp < n_rt) {
            if (!mbar_wait(tbar, 0) && lane == 0) atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
#pragma unroll
            for (int r = 0; r < RT; ++r)
                if (warp == r) lowrank_up(yacc[r], r);
        }
        // Offsets of what this warp (step `warp` of every stage) reads, from the start of a stage; the stage loop
        // keeps a running slot, parity and address instead of dividing by the ring depth.
        const uint32_t wofs = (uint32_t)(warp * kStepBytes + lane * (BITS * 4));
        const uint32_t xofs = (uint32_t)p.off_stage_x + (uint32_t)(warp * 64) * 2u +
                              (uint32_t)((lane & 7) * kXsStride + (lane >> 3) * 8) * 2u;
        const uint32_t sxofs = (uint32_t)(p.off_stage_x + 2048 + 2 * tg * kActRecord + warp * 4);
        const uint32_t* szs = reinterpret_cast<const uint32_t*>(smem + p.off_sz) + gq;
        const int sz_tile = p.ng * 16;  // (scale, zero) words between row tiles
        int kstep = warp;               // this warp's 64-column step of the current stage
        int slot = 0;
        uint32_t parity = 0;
        const unsigned char* stage = smem + p.off_ring;
        uint32_t stage_u32 = smem0 + (uint32_t)p.off_ring;
        bool dead = false;  // a wait of this warp ran out
        int steps_left = p.nsteps;
        for (int s = 0; s < p.total_stages; ++s) {
            if (!dead && !(mbar_wait(wfull(slot), parity) && mbar_wait(xfull(slot), parity))) {
                dead = true;
                s_timeout = 1;
                if (lane == 0) atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
            }
            if (warp < steps_left) {
                // B operand: the 64 columns of step `warp`, all token tiles
                uint32_t b[NT][8];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint32_t base = stage_u32 + xofs + (uint32_t)(nt * 8 * kXsStride) * 2u;
                    ldmatrix_x4(*reinterpret_cast<uint32_t(*)[4]>(&b[nt][0]), base);
                    ldmatrix_x4(*reinterpret_cast<uint32_t(*)[4]>(&b[nt][4]), base + 64u);
                }
                const float* sxp = reinterpret_cast<const float*>(stage + sxofs);
                const uint32_t* szp = szs + (kstep >> p.gshift) * 16;
                float sx[NT][2];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    sx[nt][0] = sxp[nt * 8 * (kActRecord / 4)];
                    sx[nt][1] = sxp[(nt * 8 + 1) * (kActRecord / 4)];
                }
#pragma unroll
                for (int r = 0; r < RT; ++r) {
                    if (r < n_rt) {
                        uint32_t w[BITS];
                        const uint32_t* wp = reinterpret_cast<const uint32_t*>(stage + wofs + r * kStageSteps * kStepBytes);
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
                        const uint32_t sz_lo = szp[r * sz_tile], sz_hi = szp[r * sz_tile + 8];
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
                            yacc[r][nt][0] = fmaf(f_lo.x, acc[0], fmaf(nsz_lo, sx[nt][0], yacc[r][nt][0]));
                            yacc[r][nt][1] = fmaf(f_lo.x, acc[1], fmaf(nsz_lo, sx[nt][1], yacc[r][nt][1]));
                            yacc[r][nt][2] = fmaf(f_hi.x, acc[2], fmaf(nsz_hi, sx[nt][0], yacc[r][nt][2]));
                            yacc[r][nt][3] = fmaf(f_hi.x, acc[3], fmaf(nsz_hi, sx[nt][1], yacc[r][nt][3]));
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty(slot));
            // next stage: its steps, its slot of the ring
            kstep += kStageSteps;
            steps_left -= kStageSteps;
            ++slot;
            stage += p.stage_bytes;
            stage_u32 += (uint32_t)p.stage_bytes;
            if (slot == p.n_stages) {
                slot = 0;
                parity ^= 1u;
                stage = smem + p.off_ring;
                stage_u32 = smem0 + (uint32_t)p.off_ring;
            }
        }
    }
    __syncthreads();  // every stage consumed: the ring can be reused for the reduction

    // reduction over the consumer warps: red[warp][token][RT * 16 rows + 4] -- the padding puts the four token
    // pairs of a warp's store into different banks
    constexpr int kRows = RT * 16, kRowsP = kRows + kRedPad;
    float* red = reinterpret_cast<float*>(smem + p.off_ring);
    if (warp < kConsumerWarps) {
#pragma unroll
        for (int r = 0; r < RT; ++r)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tk = nt * 8 + 2 * tg + (i & 1), rl = r * 16 + gq + 8 * (i >> 1);
                    red[(warp * kTok + tk) * kRowsP + rl] = yacc[r][nt][i];
                }
    }
    __syncthreads();
    const int rows_here = n_rt * 16;
    for (int i = tid; i < tc * kRows; i += kThreads) {
        const int tk = i / kRows, rl = i - tk * kRows;
        if (rl < rows_here) {
            // four independent partial sums, then their sum
            float s4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) s4[w & 3] += red[(w * kTok + tk) * kRowsP + rl];
            const float sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
            const size_t o = (size_t)tk * p.ldy + (size_t)rt0 * 16 + rl;
            if (p.out_f32) reinterpret_cast<float*>(p.y)[o] = sum;
            else reinterpret_cast<__nv_bfloat16*>(p.y)[o] = __float2bfloat16_rn(sum);
        }
    }
}

// Variant for up to 8 tokens when the whole K range fits the ring (no refills): 32 consumer warps and no
// producer warp.  Warp w takes step w & 15 of every stage for row tile w >> 4, i.e. ONE tile step per stage, so
// each scheduler has eight warps to hide the expand -> MMA -> FMA chains behind; lane 0 of warp 0 issues every
// copy (layer data before griddepcontrol.wait, activations and t after it).
constexpr int kWideWarps = 32;
constexpr int kWideThreads = kWideWarps * 32;

// Partial sums of the 16 step warps of a tile, red[step][token][row] with padded strides: the four token pairs of
// a warp's store fall into different banks, and so do the four partial sums that a thread adds afterwards.
constexpr int kRedTok = 36;                 // floats between tokens
constexpr int kRedStep = 8 * kRedTok + 8;   // floats between steps

template <int BITS, typename SIBS>
__global__ void __launch_bounds__(kWideThreads, 1)
stream_wide_kernel(const StreamParams p_in, const __grid_constant__ SIBS sibs) {
    StreamParams p = p_in;
    const int bx = select_sibling(p, sibs);
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bars[kMaxStages + 2];  // full per stage (codes and activations); sz + A; t
    constexpr int kTok = 8;
    constexpr int kStepBytes = 128 * BITS;
    // stage geometry of this variant (8 tokens, two row tiles) as compile-time constants: the unrolled stage loop
    // then addresses everything with immediates
    constexpr int kOffX = 2 * kStageSteps * kStepBytes;                             // activations after the codes
    constexpr int kStageBytes = (kOffX + kTok * kActRecord + 127) / 128 * 128;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, tg = lane & 3;
    const int step = warp & 15, r = warp >> 4;
    const int rt0 = bx * 2;
    const int n_rt = min(2, (p.m >> 4) - rt0);
    const int tc = min(kTok, p.T);
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    const uint32_t cbar = bar0 + 8u * (uint32_t)kMaxStages;
    const uint32_t tbar = cbar + 8u;
    const uint32_t smem0 = smem_u32(smem);

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < p.total_stages; ++s) mbar_init(full(s), 2);  // two arrivals: codes, activations
        mbar_init(cbar, 1);
        mbar_init(tbar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto steps_of = [&](int stage) { return min(kStageSteps, p.nsteps - stage * kStageSteps); };

    if (tid == 0) {
        // layer data: (scale, zero) pairs and rows of A of the live row tiles, the codes of every stage
        const uint32_t sz_bytes = (uint32_t)(n_rt * p.ng * 64);
        const uint32_t a_bytes = (uint32_t)(n_rt * 16 * p.r_pad * (p.lr8 ? 1 : 2));
        mbar_expect_tx(cbar, sz_bytes + a_bytes);
        bulk_g2s(smem0 + p.off_sz, p.sz + (size_t)rt0 * p.ng * 16, sz_bytes, cbar);
        if (a_bytes)
            bulk_g2s(smem0 + p.off_a, reinterpret_cast<const unsigned char*>(p.A) + (size_t)rt0 * 16 * p.r_pad * (p.lr8 ? 1 : 2),
                     a_bytes, cbar);
        for (int s = 0; s < p.total_stages; ++s) {
            const uint32_t bytes = (uint32_t)(steps_of(s) * kStepBytes);
            mbar_expect_tx(full(s), bytes * (uint32_t)n_rt);
            for (int q = 0; q < n_rt; ++q)
                bulk_g2s(smem0 + p.off_ring + s * kStageBytes + q * kStageSteps * kStepBytes,
                         reinterpret_cast<const unsigned char*>(p.codes) +
                             ((size_t)(rt0 + q) * p.nsteps + (size_t)s * kStageSteps) * kStepBytes,
                         bytes, full(s));
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (tid == 0) {
        const uint32_t bytes = (uint32_t)(tc * kActRecord);
        for (int s = 0; s < p.total_stages; ++s) {
            mbar_expect_tx(full(s), bytes);
            bulk_g2s(smem0 + p.off_ring + s * kStageBytes + kOffX, p.act + (size_t)s * p.t_pad * kActRecord, bytes,
                     full(s));
        }
        if (p.r_pad > 0) {
            const uint32_t t_bytes = (uint32_t)(tc * p.r_pad * 2);
            mbar_expect_tx(tbar, t_bytes);
            bulk_g2s(smem0 + p.off_t, p.t, t_bytes, tbar);
        }
    }

    // Everything a warp needs to address its tile steps, worked out while the copies are in flight: the stage
    // loop below adds compile-time offsets only.
    const bool live = r < n_rt;
    const int my_stages = live ? min(p.total_stages, (p.nsteps - step + kStageSteps - 1) / kStageSteps) : 0;
    const unsigned char* ring = smem + p.off_ring;
    const unsigned char* wptr = ring + (r * kStageSteps + step) * kStepBytes + lane * (BITS * 4);
    const uint32_t xaddr = smem0 + p.off_ring + kOffX + (uint32_t)(step * 64) * 2u +
                           (uint32_t)((lane & 7) * kXsStride + (lane >> 3) * 8) * 2u;
    const float* sxp = reinterpret_cast<const float*>(ring + kOffX + 2048 + (2 * tg) * kActRecord) + step;
    const uint32_t* szs = reinterpret_cast<const uint32_t*>(smem + p.off_sz) + r * p.ng * 16 + gq;
    bool timed_out = false;

    float yacc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (!mbar_wait(cbar, 0)) timed_out = true;
    if (p.r_pad > 0 && step == 0) {
        // low-rank term A t of row tile r starts the sums of its step-0 warp
        if (!mbar_wait(tbar, 0)) timed_out = true;
        if (live) {
            const unsigned char* as = smem + p.off_a + (size_t)r * 16 * p.r_pad * (p.lr8 ? 1 : 2);
            const __half* ts = reinterpret_cast<const __half*>(smem + p.off_t);
            for (int jj = 0; jj < p.r_pad; jj += 16) {
                uint32_t a[4];
                load_up_fragment(a, as, p.r_pad, gq, tg, jj, p.lr8 != 0);
                const __half* trow = ts + gq * p.r_pad + jj + 2 * tg;
                mma_f16(yacc, a, *reinterpret_cast<const uint32_t*>(trow), *reinterpret_cast<const uint32_t*>(trow + 8));
            }
        }
    }
#pragma unroll
    for (int s = 0; s < kMaxStages; ++s) {
        if (s >= my_stages) break;
        if (!mbar_wait(full(s), 0)) timed_out = true;
        uint32_t b[8];
        ldmatrix_x4(*reinterpret_cast<uint32_t(*)[4]>(&b[0]), xaddr + s * kStageBytes);
        ldmatrix_x4(*reinterpret_cast<uint32_t(*)[4]>(&b[4]), xaddr + s * kStageBytes + 64u);
        const float sx0 = sxp[s * (kStageBytes / 4)];
        const float sx1 = sxp[s * (kStageBytes / 4) + kActRecord / 4];
        uint32_t w[BITS];
        const uint32_t* wp = reinterpret_cast<const uint32_t*>(wptr + s * kStageBytes);
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
        const uint32_t* szp = szs + ((s * kStageSteps + step) >> p.gshift) * 16;  // the step's group
        const uint32_t sz_lo = szp[0], sz_hi = szp[8];
        const float2 f_lo = __half22float2(*reinterpret_cast<const __half2*>(&sz_lo));
        const float2 f_hi = __half22float2(*reinterpret_cast<const __half2*>(&sz_hi));
        const float nsz_lo = -f_lo.x * (128.0f + f_lo.y), nsz_hi = -f_hi.x * (128.0f + f_hi.y);
        float acc[4];
        mma_bf16_first(acc, &a[0], b[0], b[1]);
        mma_bf16(acc, &a[4], b[2], b[3]);
        mma_bf16(acc, &a[8], b[4], b[5]);
        mma_bf16(acc, &a[12], b[6], b[7]);
        yacc[0] = fmaf(f_lo.x, acc[0], fmaf(nsz_lo, sx0, yacc[0]));
        yacc[1] = fmaf(f_lo.x, acc[1], fmaf(nsz_lo, sx1, yacc[1]));
        yacc[2] = fmaf(f_hi.x, acc[2], fmaf(nsz_hi, sx0, yacc[2]));
        yacc[3] = fmaf(f_hi.x, acc[3], fmaf(nsz_hi, sx1, yacc[3]));
    }
    if (timed_out && lane == 0) atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
    // Every stage has a step-0 warp that waited for it, so after this barrier every copy has landed and the ring
    // can be reused for the reduction.
    __syncthreads();

    static_assert(kStageSteps * kRedStep * 4 <= kStageBytes, "the partial sums fit one stage of the ring");
    float* red = reinterpret_cast<float*>(smem + p.off_ring);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int tk = 2 * tg + (i & 1), rl = r * 16 + gq + 8 * (i >> 1);
        red[step * kRedStep + tk * kRedTok + rl] = yacc[i];
    }
    __syncthreads();
    // four threads per output: each adds four of the 16 partial sums, two shuffles finish
    {
        const int o = tid >> 2, part = tid & 3;
        const int tk = o >> 5, rl = o & 31;
        const float* src = red + part * kRedStep + tk * kRedTok + rl;
        float sum = (src[0] + src[4 * kRedStep]) + (src[8 * kRedStep] + src[12 * kRedStep]);
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        if (part == 0 && tk < tc && rl < n_rt * 16) {
            const size_t idx = (size_t)tk * p.ldy + (size_t)rt0 * 16 + rl;
            if (p.out_f32) reinterpret_cast<float*>(p.y)[idx] = sum;
            else reinterpret_cast<__nv_bfloat16*>(p.y)[idx] = __float2bfloat16_rn(sum);
        }
    }
}

template <int BITS, typename SIBS>
cudaError_t launch_stream_wide_s(const StreamParams& p, const SIBS& sibs, int grid, int smem_bytes, cudaStream_t s) {
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(stream_wide_kernel<BITS, SIBS>, kStreamMaxSmem, &attr_done);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kWideThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, stream_wide_kernel<BITS, SIBS>, p, sibs);
}

template <int BITS>
cudaError_t launch_stream_wide(const StreamParams& p, const StreamSiblings& sibs, int grid, int smem_bytes, cudaStream_t s) {
    return sibs.n == 0 && option(LOPRO_OPT_ONE_KERNEL_SET) != 1 ? launch_stream_wide_s<BITS, NoSiblings>(p, NoSiblings{}, grid, smem_bytes, s)
                       : launch_stream_wide_s<BITS, StreamSiblings>(p, sibs, grid, smem_bytes, s);
}

template <int BITS, int NT, int RT, typename SIBS>
cudaError_t launch_stream_ks(const StreamParams& p, const SIBS& sibs, int grid, int smem_bytes, cudaStream_t s) {
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(stream_kernel<BITS, NT, RT, SIBS>, kStreamMaxSmem, &attr_done);
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
    return cudaLaunchKernelEx(&cfg, stream_kernel<BITS, NT, RT, SIBS>, p, sibs);
}

template <int BITS, int NT, int RT>
cudaError_t launch_stream_k(const StreamParams& p, const StreamSiblings& sibs, int grid, int smem_bytes, cudaStream_t s) {
    return sibs.n == 0 && option(LOPRO_OPT_ONE_KERNEL_SET) != 1 ? launch_stream_ks<BITS, NT, RT, NoSiblings>(p, NoSiblings{}, grid, smem_bytes, s)
                       : launch_stream_ks<BITS, NT, RT, StreamSiblings>(p, sibs, grid, smem_bytes, s);
}

template <int BITS>
cudaError_t launch_stream_bits(const StreamParams& p, const StreamSiblings& sibs, int grid, int nt, int rt, int smem_bytes,
                               cudaStream_t s) {
    if (nt == 1)
        return rt == 4 ? launch_stream_k<BITS, 1, 4>(p, sibs, grid, smem_bytes, s) : launch_stream_k<BITS, 1, 2>(p, sibs, grid, smem_bytes, s);
    if (nt == 2)
        return rt == 4 ? launch_stream_k<BITS, 2, 4>(p, sibs, grid, smem_bytes, s) : launch_stream_k<BITS, 2, 2>(p, sibs, grid, smem_bytes, s);
    return launch_stream_k<BITS, 4, 2>(p, sibs, grid, smem_bytes, s);
}

struct StreamPlan {
    int nt, rt, n_stages, total_stages, smem_bytes;
    int off_sz, off_a, off_t, off_ring, stage_bytes, off_stage_x;
};

bool plan_layout(const lopro_desc& d, StreamPlan* pl, int r_pad, int ng, int ktok);

bool plan_stream(const lopro_desc& d, int T, StreamPlan* pl) {
    if (T < 1 || T > kDecodeMaxT) return false;
    const int r_pad = d.rank > 0 ? round_up_int(d.rank, 16) : 0;
    const int ng = d.d_in / d.group_size;
    pl->nt = T <= 8 ? 1 : (T <= 16 ? 2 : 4);
    const int ktok = pl->nt * 8;
    // Rows per CTA: 64 instead of 32 when the layer is tall enough to keep two CTAs per SM busy anyway --
    // every CTA reads all of x~ from L2, so taller CTAs halve that traffic.
    pl->rt = (pl->nt <= 2 && (d.d_out / 16) / 4 >= 296) ? 4 : 2;
    for (;;) {
        if (plan_layout(d, pl, r_pad, ng, ktok)) return true;
        if (pl->rt == 2) return false;
        pl->rt = 2;
    }
}

bool plan_layout(const lopro_desc& d, StreamPlan* pl, int r_pad, int ng, int ktok) {
    int off = 0;
    pl->off_sz = off;
    off += round_up_int(pl->rt * ng * 64, 128);
    pl->off_a = off;
    off += round_up_int(pl->rt * 16 * r_pad * 2, 128);
    pl->off_t = off;
    off += round_up_int(ktok * r_pad * 2, 128);
    pl->off_ring = off;
    const int w_bytes = pl->rt * kStageSteps * 128 * d.bits;
    pl->off_stage_x = w_bytes;
    pl->stage_bytes = round_up_int(w_bytes + ktok * kActRecord, 128);
    pl->total_stages = (d.d_in / 64 + kStageSteps - 1) / kStageSteps;
    const int red_bytes = kConsumerWarps * ktok * (pl->rt * 16 + kRedPad) * 4;
    int stages = (kStreamMaxSmem - off) / pl->stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages > pl->total_stages) stages = pl->total_stages;
    if (stages < 1) return false;
    if (pl->rt > 2 && stages < pl->total_stages && stages < 3) return false;  // too shallow a ring: fall back to 32 rows
    int ring = stages * pl->stage_bytes;
    if (ring < red_bytes) ring = red_bytes;
    pl->n_stages = stages;
    pl->smem_bytes = off + ring;
    return pl->smem_bytes <= kStreamMaxSmem;
}

}  // namespace

// The 32-warp variant runs for up to 8 tokens when all of K fits the ring; LOPRO_OPT_NO_WIDE keeps it off (A/B
// comparison and tests).
static bool wide_variant(const lopro_desc& d, const StreamPlan& pl) {
    const bool no_wide = option(LOPRO_OPT_NO_WIDE) == 1;
    return !no_wide && pl.nt == 1 && pl.rt == 2 && pl.n_stages == pl.total_stages &&
           pl.off_stage_x == 2 * kStageSteps * 128 * d.bits;  // the variant's compile-time stage geometry
}

bool stream_uses_wide(const lopro_desc& d, int T) {
    StreamPlan pl;
    return plan_stream(d, T, &pl) && wide_variant(d, pl);
}

bool stream_supported(const lopro_desc& d, int T) {
    StreamPlan pl;
    return plan_stream(d, T, &pl);
}

cudaError_t launch_stream(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, const uint8_t* ws,
                          const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int T, cudaStream_t s, int t0,
                          const StreamSiblingArgs* more) {
    StreamPlan pl;
    if (!plan_stream(d, T, &pl)) return cudaErrorInvalidValue;
    StreamParams p;
    p.codes = reinterpret_cast<const uint32_t*>(blob + L.off[LOPRO_SEC_CODES]);
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
    p.n_stages = pl.n_stages;
    p.total_stages = pl.total_stages;
    p.off_sz = pl.off_sz;
    p.off_a = pl.off_a;
    p.off_t = pl.off_t;
    p.off_ring = pl.off_ring;
    p.stage_bytes = pl.stage_bytes;
    p.off_stage_x = pl.off_stage_x;
    const bool wide = wide_variant(d, pl);
    const int rows_per_cta = wide ? 32 : pl.rt * 16;
    int grid = (d.d_out + rows_per_cta - 1) / rows_per_cta;
    // sibling layers: the CTAs of each follow those of the one before
    StreamSiblings sibs = {};
    if (more != nullptr) {
        sibs.n = more->n;
        if (more->own_rows) p.T = more->T_of[0];
        for (int i = 0; i < more->n; ++i) {
            const uint8_t* b = more->blob[i];
            const BlobLayout& Li = more->L[i];
            const uint8_t* wsi = more->ws[i];
            sibs.cta0[i] = grid;
            sibs.codes[i] = reinterpret_cast<const uint32_t*>(b + Li.off[LOPRO_SEC_CODES]);
            sibs.sz[i] = reinterpret_cast<const uint32_t*>(b + Li.off[LOPRO_SEC_SCALEZERO]);
            sibs.A[i] = reinterpret_cast<const __half*>(b + Li.off[LOPRO_SEC_A]);
            sibs.act[i] = wsi + W.off_xrot + (size_t)t0 * kActRecord;
            sibs.t[i] = reinterpret_cast<const __half*>(wsi + W.off_t) + (size_t)t0 * (d.rank > 0 ? L.r_pad : 0);
            sibs.y[i] = more->y[i];
            sibs.ldy[i] = more->ldy[i];
            sibs.m[i] = more->d_out[i];
            sibs.T[i] = more->own_rows ? more->T_of[i + 1] : T;
            grid += (more->d_out[i] + rows_per_cta - 1) / rows_per_cta;
        }
    }
    if (wide) {
        switch (d.bits) {
            case 2: return launch_stream_wide<2>(p, sibs, grid, pl.smem_bytes, s);
            case 3: return launch_stream_wide<3>(p, sibs, grid, pl.smem_bytes, s);
            default: return launch_stream_wide<4>(p, sibs, grid, pl.smem_bytes, s);
        }
    }
    switch (d.bits) {
        case 2: return launch_stream_bits<2>(p, sibs, grid, pl.nt, pl.rt, pl.smem_bytes, s);
        case 3: return launch_stream_bits<3>(p, sibs, grid, pl.nt, pl.rt, pl.smem_bytes, s);
        default: return launch_stream_bits<4>(p, sibs, grid, pl.nt, pl.rt, pl.smem_bytes, s);
    }
}

}  // namespace lopro
