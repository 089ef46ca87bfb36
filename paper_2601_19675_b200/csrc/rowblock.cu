// Small-batch forward (decode, up to 32 tokens per launch) on tcgen05 / TMEM over the row-block layout:
// y = W^ x~ + A t  (steps "Dequant(W_q) X" and "U (Sigma Y)" of Appendix A.3, summed as in Eq. 8), after the
// prologue that writes the operand image (rotated activations as K-major tiles, their column sums, t = B x).
//
// Arithmetic.  With w = s (c - z):  sum_k w_k x~_k = s (sum_k (128 + c_k) x~_k - (128 + z) sum_k x~_k).  The tensor
// cores multiply the bf16 activations with the EXACT bf16 numbers 128 + c (fp32 accumulation); the quantized
// weights are never rounded.  Each quantization group owns one accumulator slice of NP columns of tensor memory;
// when the group's last MMA has completed, the slice is read back and scale and zero-point enter once, in fp32,
// with the pre-computed column sums of x~.  The rank-r term A t runs as fp16 MMAs into a slice of its own (scale 1).
//
// The expanded weights never touch shared memory: a thread expands the 64 codes of one row and step into 32
// registers of bf16 pairs and stores them with one tcgen05.st into 32 columns of tensor memory, from where the MMA
// reads its A operand (row = lane).  Shared memory carries only what arrives by bulk copy: packed codes,
// (scale, zero) pairs, activation tiles and column sums.
//
// Work split ("stream-K").  A unit is one quantization group of one block of 128 rows; the units of the layer,
// ordered [block][group], are cut into one contiguous run per CTA.  A CTA whose run covers a whole block stores
// its rows; where a block is shared, every contributor writes its fp32 partial sums to the workspace and counts
// itself in; whoever arrives last adds the partial sums in the fixed order of the contributors (the result does
// not depend on who was last) and stores the rows.  Nobody waits for another CTA.
//
// A CTA walks its run in stages of up to four 64-column steps (a wait on a shared-memory barrier costs a thread
// about 125 cycles even when it is satisfied, so every role waits once per stage, not once per step).
// Roles (16 warps):
//   warps 0-3   epilogue: thread = row; per stage, the slices of the groups that end in it: tcgen05.ld,
//               scale / zero-point, running sums; at the end of a block's piece the output or the partial sums;
//   warps 4-11  expansion, two sets of four warps (one warp per 32-row quarter) taking turns by stage: thread = row;
//               reads the row's packed codes from the code ring, expands, tcgen05.st (for the low-rank steps:
//               the row's fp16 entries of A); the set's first warp also waits for the stage's activation tiles
//               and for the accumulator slices the stage opens, so that the MMA thread has a single wait;
//   warp 12     one thread streams packed codes and (scale, zero) pairs with bulk copies -- layer data, requested
//               before griddepcontrol.wait, i.e. while the prologue of the same forward still runs;
//   warp 13     one thread waits for the prologue and streams the activation tiles and column sums;
//   warps 14-15 one thread each issues tcgen05.mma (M 128, N = NP, K 16; A from tensor memory, B from shared memory)
//               and commits stages, tiles and slices back; the two take turns by stage.
// Every mbarrier wait is bounded; a wait that runs out stores LOPRO_ERR_TIMEOUT in the workspace status word, the
// CTA stops waiting, frees its tensor memory and returns (outputs then unspecified).
#include "common.cuh"
#include "ptx.cuh"
#include "tc5.cuh"

namespace lopro {

namespace {

constexpr int kEpiWarps = 4;
constexpr int kExpWarps = 8;
constexpr int kWarpW = kEpiWarps + kExpWarps, kWarpX = kWarpW + 1, kWarpMma = kWarpW + 2;  // two MMA warps
constexpr int kThreads = (kWarpMma + 2) * 32;
constexpr int kStageItems = 4;  // 64-column steps per stage
constexpr int kAStages = 2;     // stages of expanded weights in tensor memory (128 columns each)
constexpr int kXSlots = 4;      // ring of activation stages
constexpr int kGSlots = 6;      // ring of group records: (scale, zero) pairs and column sums of the groups a stage ends
constexpr int kGSlotBytes = 4096;
constexpr int kSlices = 8;      // accumulator slices in tensor memory
constexpr int kMaxCSlots = 16;  // ring of packed-code stages (depth chosen at launch)
constexpr int kSmemLimit = 200 * 1024;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSliceCol0 = kAStages * kStageItems * 32;  // tensor-memory column of slice 0

struct RbParams {
    const uint32_t* codes;
    const uint32_t* sz;
    const __half* A;
    const unsigned char* ximg;  // this token group's tiles [step][NP][128 B]
    const float* sums;          // [run][NP]
    const unsigned char* timg;  // [rank step][NP][128 B]
    float* partial;             // [2 * grid][NP][128] fp32
    int* counters;              // [blocks]
    int* status;
    void* y;
    int64_t ldy;
    int out_f32;
    int m, T;                   // T: live tokens of this launch (<= NP)
    int nsteps, ng, gshift;     // 64-column steps of K, groups per row, log2(steps per group)
    int r_pad, lr_steps;
    int units;                  // blocks of this launch * ng
    int rb_base;                // first block of rows of this launch
    int spg;                    // column-sum runs per group (1 unless g > 256)
    int c_slots;                // depth of the code ring
    int two_issuers;            // the two MMA threads take turns by stage (no group spans two stages)
};

// Ring position: slot and the parity of its current use.
struct Ring {
    int slot = 0;
    uint32_t phase = 0;
    bool wrapped = false;
    int n;
    __device__ explicit Ring(int n_) : n(n_) {}
    __device__ void next() {
        if (++slot == n) {
            slot = 0;
            phase ^= 1u;
            wrapped = true;
        }
    }
};

// One stage of a CTA's run: up to four consecutive 64-column steps of one block of rows -- either steps of the
// quantized part or (first in a piece that starts its block) steps of the low-rank term.
struct Stage {
    int rb;          // block of rows
    bool lr;         // low-rank steps (operands A and t) instead of quantized steps
    int i0, ni;      // first step (of the block's K range, or of the padded rank) and number of steps
    int first_mask, last_mask;  // bit i: step i0 + i is the first / the last of its group (lr: of the low-rank term)
    int n_open, n_close;        // groups that begin / end in the stage (popcounts of the masks)
    int close0;      // index of the first group that ends in the stage
    bool piece_end;  // last stage of this CTA's piece of the block
    bool piece_whole, piece_first;  // the piece covers the whole block / starts at the block's first unit
};

// The stages of a CTA's run of units [u0, u1), in the order every role follows, are worked out once, by all threads
// in parallel, into a table in shared memory (16 bytes per stage): walking the run costs a couple of hundred
// instructions per stage, which sixteen warps would otherwise each repeat.
constexpr int kMaxStagesPerCta = 512;

struct RunShape {  // pieces of the run: a first piece (possibly partial), whole blocks, a last partial piece
    int ng, gshift, lr_steps, nlr;
    int rb0, gb0, ge0, s0;     // first piece: block, groups [gb0, ge0), stages
    int full, s_full;          // whole blocks after it and the stages of each
    int tail, total;           // groups of the last piece (0: none), stages of the run
};

__device__ __forceinline__ int piece_stages(int gb, int ge, int gshift, int nlr) {
    return (gb == 0 ? nlr : 0) + ((((ge - gb) << gshift) + kStageItems - 1) / kStageItems);
}

__device__ __forceinline__ RunShape run_shape(int u0, int u1, int ng, int gshift, int lr_steps) {
    RunShape r;
    r.ng = ng;
    r.gshift = gshift;
    r.lr_steps = lr_steps;
    r.nlr = (lr_steps + kStageItems - 1) / kStageItems;
    r.rb0 = u0 / ng;
    r.gb0 = u0 - r.rb0 * ng;
    r.ge0 = min(ng, r.gb0 + (u1 - u0));
    r.s0 = u1 > u0 ? piece_stages(r.gb0, r.ge0, gshift, r.nlr) : 0;
    const int rem = (u1 - u0) - (r.ge0 - r.gb0);
    r.full = rem / ng;
    r.tail = rem - r.full * ng;
    r.s_full = piece_stages(0, ng, gshift, r.nlr);
    r.total = r.s0 + r.full * r.s_full + (r.tail > 0 ? piece_stages(0, r.tail, gshift, r.nlr) : 0);
    return r;
}

// Stage k of the run, packed: x = block | steps << 20 | low-rank << 23 | piece_end << 24 | piece_whole << 25 |
// piece_first << 26;  y = first step | first closing group << 16;  z = first_mask | last_mask << 4;  w = 0.
__device__ __forceinline__ uint4 stage_record(const RunShape& r, int k) {
    int rb, gb, ge, j;
    if (k < r.s0) {
        rb = r.rb0; gb = r.gb0; ge = r.ge0; j = k;
    } else {
        const int k1 = k - r.s0, f = min(k1 / r.s_full, r.full);
        rb = r.rb0 + 1 + f; gb = 0; ge = f < r.full ? r.ng : r.tail; j = k1 - f * r.s_full;
    }
    const int n_lr = gb == 0 ? r.nlr : 0;
    const int q_first = gb << r.gshift, q_last = ge << r.gshift;
    const int total = n_lr + (q_last - q_first + kStageItems - 1) / kStageItems;
    int lr = j < n_lr, i0, ni, first_mask, last_mask, close0 = 0;
    if (lr) {
        i0 = j * kStageItems;
        ni = min(kStageItems, r.lr_steps - i0);
        first_mask = j == 0 ? 1 : 0;
        last_mask = j == n_lr - 1 ? 1 << (ni - 1) : 0;
    } else {
        i0 = q_first + (j - n_lr) * kStageItems;
        ni = min(kStageItems, q_last - i0);
        const int gmask = (1 << r.gshift) - 1, live = (1 << ni) - 1;
        if (r.gshift == 0) {
            first_mask = last_mask = live;
        } else if (r.gshift == 1) {
            first_mask = 0x5 & live;  // stages start on even steps
            last_mask = 0xA & live;
        } else {  // groups of four steps or more: at most one begins and one ends in a stage
            first_mask = (i0 & gmask) == 0 ? 1 : 0;
            last_mask = ((i0 + ni) & gmask) == 0 ? 1 << (ni - 1) : 0;
        }
        close0 = ((i0 + gmask + 1) >> r.gshift) - 1;
    }
    const int piece_end = j == total - 1, piece_first = gb == 0, piece_whole = gb == 0 && ge == r.ng;
    return make_uint4((uint32_t)(rb | (ni << 20) | (lr << 23) | (piece_end << 24) | (piece_whole << 25) | (piece_first << 26)),
                      (uint32_t)(i0 | (close0 << 16)), (uint32_t)(first_mask | (last_mask << 4)), 0u);
}

__device__ __forceinline__ Stage unpack_stage(const uint4& v) {
    Stage s;
    s.rb = (int)(v.x & 0xFFFFFu);
    s.ni = (int)((v.x >> 20) & 7u);
    s.lr = ((v.x >> 23) & 1u) != 0;
    s.piece_end = ((v.x >> 24) & 1u) != 0;
    s.piece_whole = ((v.x >> 25) & 1u) != 0;
    s.piece_first = ((v.x >> 26) & 1u) != 0;
    s.i0 = (int)(v.y & 0xFFFFu);
    s.close0 = (int)(v.y >> 16);
    s.first_mask = (int)(v.z & 15u);
    s.last_mask = (int)((v.z >> 4) & 15u);
    s.n_open = __popc(s.first_mask);
    s.n_close = __popc(s.last_mask);
    return s;
}

// Out-of-line slow path of every wait of this file (one copy of the polling loop for all roles: the kernel is bound
// by instruction fetch as soon as its hot loops outgrow the instruction caches).  Polls with a suspend-time hint, so a
// waiting warp issues few instructions.  False if the limit ran out.
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait_hint(bar, parity, 2000u)) return true;
    return false;
}
__device__ __noinline__ void report_timeout(int* status, int* flag) {
    *flag = 1;
    atomicExch(status, (int)LOPRO_ERR_TIMEOUT);
}

template <int NP>
__device__ __forceinline__ void tmem_ld(uint32_t (&v)[NP], uint32_t taddr) {
    if constexpr (NP == 16) {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
              "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
            : "r"(taddr)
            : "memory");
    } else {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
              "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
              "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
              "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
            : "r"(taddr)
            : "memory");
    }
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 32 registers of one thread -> 32 consecutive columns of its lane of tensor memory
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
          "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
          "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem desc], 128 x N x 16, issued by one thread
__device__ __forceinline__ void umma_f16_ta(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"r"(kEpiWarps * 32) : "memory"); }

template <int BITS, int NP>
__global__ void __launch_bounds__(kThreads, 1)
rowblock_kernel(const RbParams p) {
    extern __shared__ unsigned char smem_raw[];
    // full / empty per slot: A stages, activation stages, group records, slices, code stages
    __shared__ __align__(8) uint64_t bars[2 * (kAStages + kXSlots + kGSlots + kSlices + kMaxCSlots)];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_timeout;
    __shared__ int s_last;
    // what the MMA thread needs to know about the stage in A slot k, written by the expansion warps that fill it:
    // x = first_mask | last_mask << 4 | steps << 8 | low-rank << 12 | end << 13 | MMAs of the last step << 16,
    // y = activation slot, z = slices opened before the stage
    __shared__ uint4 s_cmd[kAStages];
    __shared__ uint4 s_stage[kMaxStagesPerCta];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // operand tiles are 1024-byte aligned (swizzle atoms)
    unsigned char* base_ptr = smem_raw + (base - raw);
    constexpr int kXTile = NP * 128, kXStage = kStageItems * kXTile;
    constexpr int kStepBytes = kRbRows * 8 * BITS;  // packed codes of 128 rows x 64 columns
    constexpr int kCStage = kStageItems * kStepBytes;
    const uint32_t x_ring = base, g_ring = x_ring + kXSlots * kXStage, c_ring = g_ring + kGSlots * kGSlotBytes;
    const unsigned char* g_ring_ptr = base_ptr + kXSlots * kXStage;
    const unsigned char* c_ring_ptr = g_ring_ptr + kGSlots * kGSlotBytes;

    const uint32_t bar0 = smem_u32(bars);
    int bi = 0;
    const uint32_t full_a = bar0 + 8u * bi; bi += kAStages;
    const uint32_t empty_a = bar0 + 8u * bi; bi += kAStages;
    const uint32_t full_x = bar0 + 8u * bi; bi += kXSlots;
    const uint32_t empty_x = bar0 + 8u * bi; bi += kXSlots;
    const uint32_t full_g = bar0 + 8u * bi; bi += kGSlots;
    const uint32_t empty_g = bar0 + 8u * bi; bi += kGSlots;
    const uint32_t full_s = bar0 + 8u * bi; bi += kSlices;
    const uint32_t empty_s = bar0 + 8u * bi; bi += kSlices;
    const uint32_t full_c = bar0 + 8u * bi; bi += kMaxCSlots;
    const uint32_t empty_c = bar0 + 8u * bi;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(full_a + 8u * s, 4);   // the four expansion warps of the stage's set
            mbar_init(empty_a + 8u * s, 1);  // tcgen05.commit
        }
        for (int s = 0; s < kXSlots; ++s) {
            mbar_init(full_x + 8u * s, 1);
            mbar_init(empty_x + 8u * s, 1);
        }
        for (int s = 0; s < kGSlots; ++s) {
            mbar_init(full_g + 8u * s, 2);   // (scale, zero) pairs and column sums come from two threads
            mbar_init(empty_g + 8u * s, kEpiWarps);
        }
        for (int s = 0; s < kSlices; ++s) {
            mbar_init(full_s + 8u * s, 1);
            mbar_init(empty_s + 8u * s, kEpiWarps);
        }
        for (int s = 0; s < p.c_slots; ++s) {
            mbar_init(full_c + 8u * s, 1);
            mbar_init(empty_c + 8u * s, 4);
        }
        s_timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kWarpMma) tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
    // this CTA's run of units [u0, u1) and its table of stages
    const long long G = gridDim.x;
    const int u0 = (int)((long long)blockIdx.x * p.units / G), u1 = (int)(((long long)blockIdx.x + 1) * p.units / G);
    const RunShape shape = run_shape(u0, u1, p.ng, p.gshift, p.lr_steps);
    const int n_stages = min(shape.total, kMaxStagesPerCta);  // (the host splits a layer so that the table holds a run)
    for (int k = tid; k < n_stages; k += kThreads) s_stage[k] = stage_record(shape, k);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    Stage st;
    int stage_k = 0;
    auto next_stage = [&]() {
        if (stage_k >= n_stages) return false;
        st = unpack_stage(s_stage[stage_k++]);
        st.rb += p.rb_base;
        return true;
    };

    bool dead = false;  // a wait of this thread ran out: it stops waiting
    auto wait = [&](uint32_t bar, uint32_t parity) {
        if (dead || mbar_try_wait(bar, parity)) return;
        if (!wait_slow(bar, parity)) {
            dead = true;
            report_timeout(p.status, &s_timeout);
        }
    };

    if (warp == kWarpW) {
        // ---------------- layer-data producer: packed codes and (scale, zero) pairs ----------------
        if (lane == 0) {
            Ring rc(p.c_slots), rg(kGSlots);
            while (next_stage()) {
                if (st.lr) continue;
                const int R = rb_rows(p.m, st.rb);
                const uint32_t bytes = (uint32_t)(st.ni * R * 8 * BITS);
                if (rc.wrapped) wait(empty_c + 8u * rc.slot, rc.phase ^ 1u);
                mbar_expect_tx(full_c + 8u * rc.slot, bytes);
                bulk_g2s(c_ring + (uint32_t)(rc.slot * kCStage), p.codes + rb_step_word(BITS, p.nsteps, p.m, st.rb, st.i0), bytes,
                         full_c + 8u * rc.slot);
                rc.next();
                if (st.n_close > 0) {
                    const uint32_t sz_bytes = (uint32_t)(st.n_close * R * 4);
                    if (rg.wrapped) wait(empty_g + 8u * rg.slot, rg.phase ^ 1u);
                    mbar_expect_tx(full_g + 8u * rg.slot, sz_bytes);
                    bulk_g2s(g_ring + (uint32_t)(rg.slot * kGSlotBytes),
                             p.sz + (size_t)st.rb * kRbRows * p.ng + (size_t)st.close0 * R, sz_bytes, full_g + 8u * rg.slot);
                    rg.next();
                }
            }
        }
    } else if (warp == kWarpX) {
        // ---------------- activation producer: tiles of x~ (and of t), column sums ----------------
        if (lane == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");  // the prologue's image is complete
            Ring rx(kXSlots), rg(kGSlots);
            while (next_stage()) {
                const uint32_t bytes = (uint32_t)(st.ni * kXTile);
                if (rx.wrapped) wait(empty_x + 8u * rx.slot, rx.phase ^ 1u);
                mbar_expect_tx(full_x + 8u * rx.slot, bytes);
                bulk_g2s(x_ring + (uint32_t)(rx.slot * kXStage), (st.lr ? p.timg : p.ximg) + (size_t)st.i0 * kXTile, bytes,
                         full_x + 8u * rx.slot);
                rx.next();
                if (!st.lr && st.n_close > 0) {
                    const uint32_t sum_bytes = (uint32_t)(st.n_close * p.spg * NP * 4);
                    if (rg.wrapped) wait(empty_g + 8u * rg.slot, rg.phase ^ 1u);
                    mbar_expect_tx(full_g + 8u * rg.slot, sum_bytes);
                    bulk_g2s(g_ring + (uint32_t)(rg.slot * kGSlotBytes) + 2048u, p.sums + (size_t)st.close0 * p.spg * NP, sum_bytes,
                             full_g + 8u * rg.slot);
                    rg.next();
                }
            }
        }
    } else if (warp >= kWarpMma) {
        // ---------------- MMA issuers: one wait per stage, everything else comes ready-made ----------------
        // A single thread runs a few hundred cycles per stage on bookkeeping alone, about as long as the stage's MMAs
        // take in the tensor pipe; two issuing threads on two schedulers taking turns by stage hide that.  (Only when no
        // accumulator slice spans two stages -- otherwise the order of the MMAs into it would be open -- else the first
        // thread issues every stage.)
        const int k = warp - kWarpMma;
        if (lane == 0 && (k == 0 || p.two_issuers)) {
            const uint32_t idesc_w = make_idesc(NP, 1u), idesc_lr = make_idesc(NP, 0u);
            const uint64_t desc_x0 = make_desc_sw128(x_ring);
            int slot = k;
            uint32_t phase = 0;
            for (;;) {
                wait(full_a + 8u * slot, phase);  // expanded weights in tensor memory, tiles and slices ready
                tc_fence_after();
                const uint4 cmd = s_cmd[slot];
                if (dead || ((cmd.x >> 13) & 1u)) break;
                const uint32_t ni = (cmd.x >> 8) & 15u, lr = (cmd.x >> 12) & 1u, ksub_last = (cmd.x >> 16) & 7u;
                uint32_t first_mask = cmd.x & 15u, last_mask = (cmd.x >> 4) & 15u, spos = cmd.z;
                uint32_t a = tmem + (uint32_t)(slot * kStageItems * 32);
                uint64_t db = desc_x0 + (uint64_t)(cmd.y * (uint32_t)(kXStage >> 4));
                const uint32_t idesc = lr ? idesc_lr : idesc_w;
#pragma unroll
                for (int i = 0; i < kStageItems; ++i) {
                    if (i < (int)ni) {
                        const uint32_t first = first_mask & 1u;
                        spos += first;
                        const uint32_t sl = (spos - 1u) & (kSlices - 1);
                        const uint32_t d = tmem + kSliceCol0 + sl * NP;
                        if (i + 1 < (int)ni || ksub_last == 4u) {
                            // a whole step: four MMAs of 16 columns (8 columns of tensor memory, 32 bytes of the B tile)
                            umma_f16_ta(d, a, db, idesc, first ^ 1u);
                            umma_f16_ta(d, a + 8u, db + 2u, idesc, 1u);
                            umma_f16_ta(d, a + 16u, db + 4u, idesc, 1u);
                            umma_f16_ta(d, a + 24u, db + 6u, idesc, 1u);
                        } else {
                            // the last step of a padded rank that is not a multiple of 64
                            for (uint32_t kk = 0; kk < ksub_last; ++kk)
                                umma_f16_ta(d, a + 8u * kk, db + (uint64_t)(2u * kk), idesc, (first && kk == 0) ? 0u : 1u);
                        }
                        if (last_mask & 1u) umma_commit(full_s + 8u * sl);  // the group's slice is complete
                        first_mask >>= 1;
                        last_mask >>= 1;
                        a += 32u;
                        db += (uint64_t)(kXTile >> 4);
                    }
                }
                umma_commit(empty_a + 8u * slot);  // the stage may be refilled once these MMAs have read it
                umma_commit(empty_x + 8u * cmd.y);
                if (p.two_issuers) {
                    phase ^= 1u;
                } else {
                    slot ^= 1;
                    if (slot == 0) phase ^= 1u;
                }
            }
        }
    } else if (warp >= kEpiWarps) {
        // ---------------- expansion warps ----------------
        const int e = warp - kEpiWarps, quarter = e & 3, set = e >> 2;
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        Ring rc(p.c_slots), rx(kXSlots);
        int sidx = 0;   // stages seen so far: set `sidx & 1` expands stage sidx into A stage `sidx & 1`
        int spos = 0;   // slices opened so far
        for (; next_stage(); ++sidx) {
            const bool mine = (sidx & 1) == set;
            const int R = rb_rows(p.m, st.rb);
            const bool live = r < R;
            const int opened = st.n_open;
            if (mine) {
                const uint32_t a0 = tmem + lane_addr + (uint32_t)(set * kStageItems * 32);
                if (!st.lr) wait(full_c + 8u * rc.slot, rc.phase);
                if (sidx >= kAStages) wait(empty_a + 8u * set, (uint32_t)((sidx >> 1) - 1) & 1u);
                __syncwarp();
                tc_fence_after();
                if (st.lr) {
                    // low-rank steps: the row's fp16 entries of A, 64 columns of the rank per step
                    const __half* arow = p.A + (size_t)(st.rb * kRbRows + r) * p.r_pad;
#pragma unroll 1
                    for (int i = 0; i < st.ni; ++i) {
                        uint32_t a[32];
                        const int pieces = min(8, (p.r_pad - (st.i0 + i) * 64) / 8);
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            uint4 v = make_uint4(0, 0, 0, 0);
                            if (live && c < pieces) v = __ldg(reinterpret_cast<const uint4*>(arow + (st.i0 + i) * 64) + c);
                            a[4 * c] = v.x; a[4 * c + 1] = v.y; a[4 * c + 2] = v.z; a[4 * c + 3] = v.w;
                        }
                        tmem_st32(a0 + (uint32_t)(i * 32), a);
                    }
                } else {
                    const unsigned char* src = c_ring_ptr + rc.slot * kCStage;
#pragma unroll 1
                    for (int i = 0; i < st.ni; ++i, src += R * 8 * BITS) {
                        uint32_t w[2 * BITS];
#pragma unroll
                        for (int b = 0; b < 2 * BITS; ++b) w[b] = 0;
                        if (live) {
                            const uint4 v0 = *reinterpret_cast<const uint4*>(src + r * 16);
                            w[0] = v0.x; w[1] = v0.y; w[2] = v0.z; w[3] = v0.w;
                            if constexpr (BITS == 4) {
                                const uint4 v1 = *reinterpret_cast<const uint4*>(src + R * 16 + r * 16);
                                w[4] = v1.x; w[5] = v1.y; w[6] = v1.z; w[7] = v1.w;
                            } else if constexpr (BITS == 3) {
                                const uint2 v1 = *reinterpret_cast<const uint2*>(src + R * 16 + r * 8);
                                w[4] = v1.x; w[5] = v1.y;
                            }
                        }
                        uint32_t a[32];
#pragma unroll
                        for (int hs = 0; hs < 2; ++hs) {
                            uint32_t wh[BITS], ah[16];
#pragma unroll
                            for (int b = 0; b < BITS; ++b) wh[b] = w[hs * BITS + b];
                            expand_codes<BITS>(ah, wh);
#pragma unroll
                            for (int q = 0; q < 16; ++q) a[hs * 16 + q] = ah[q];
                        }
                        tmem_st32(a0 + (uint32_t)(i * 32), a);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_c + 8u * rc.slot);  // the words have been read
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                if (quarter == 0) {
                    // on behalf of the MMA thread: the stage's activation tiles have landed, and the slices the stage
                    // opens have been drained (the slices are opened and drained in order: the last one decides)
                    wait(full_x + 8u * rx.slot, rx.phase);
                    if (opened > 0 && spos + opened > kSlices) {
                        const int use = spos + opened - 1;  // running number of the last slice the stage opens
                        wait(empty_s + 8u * (use & (kSlices - 1)), (uint32_t)((use / kSlices) - 1) & 1u);
                    }
                    if (lane == 0) {
                        const int ksub_last = st.lr ? min(4, (p.r_pad - (st.i0 + st.ni - 1) * 64) / 16) : 4;
                        s_cmd[set] =
                            make_uint4((uint32_t)(st.first_mask | (st.last_mask << 4) | (st.ni << 8) | ((st.lr ? 1 : 0) << 12) |
                                                  (ksub_last << 16)),
                                       (uint32_t)rx.slot, (uint32_t)spos, 0u);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(full_a + 8u * set);  // (release: the command is visible to the MMA thread)
            }
            if (!st.lr) rc.next();
            rx.next();
            spos += opened;
        }
        // end of the run: one more (empty) stage per set tells its MMA thread to stop
        {
            const int send = sidx + (((sidx & 1) == set) ? 0 : 1);
            if (send >= kAStages) wait(empty_a + 8u * set, (uint32_t)((send >> 1) - 1) & 1u);
            if (quarter == 0 && lane == 0) s_cmd[set] = make_uint4(1u << 13, 0u, 0u, 0u);
            __syncwarp();
            if (lane == 0) mbar_arrive(full_a + 8u * set);
        }
    } else {
        // ---------------- epilogue warps: thread = row ----------------
        asm volatile("griddepcontrol.wait;" ::: "memory");  // y, the partial sums and the counters belong to this call only now
        const int r = warp * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        Ring rg(kGSlots);
        int spos = 0;  // slices closed so far
        float yacc[NP];
#pragma unroll
        for (int i = 0; i < NP; ++i) yacc[i] = 0.0f;
        while (next_stage()) {
            const int R = rb_rows(p.m, st.rb);
            const bool live = r < R;
            if (st.n_close > 0) {
                // the slices close in order: when the last one of the stage is complete, all are
                const int last_use = spos + st.n_close - 1;
                wait(full_s + 8u * (last_use & (kSlices - 1)), (uint32_t)(last_use / kSlices) & 1u);
                if (!st.lr) wait(full_g + 8u * rg.slot, rg.phase);
                __syncwarp();
                tc_fence_after();
                const unsigned char* rec = g_ring_ptr + rg.slot * kGSlotBytes;
#pragma unroll 1
                for (int c = 0; c < st.n_close; ++c, ++spos) {
                    uint32_t v[NP];
                    tmem_ld<NP>(v, tmem + lane_addr + kSliceCol0 + (uint32_t)((spos & (kSlices - 1)) * NP));
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_s + 8u * (spos & (kSlices - 1)));
                    if (st.lr) {
#pragma unroll
                        for (int i = 0; i < NP; ++i) yacc[i] += __uint_as_float(v[i]);
                    } else if (live) {
                        const uint32_t szw = *reinterpret_cast<const uint32_t*>(rec + (c * R + r) * 4);
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&szw));
                        const float sc = f.x, nsz = -f.x * (128.0f + f.y);
                        const float4* sp = reinterpret_cast<const float4*>(rec + 2048 + c * p.spg * NP * 4);
#pragma unroll
                        for (int i = 0; i < NP / 4; ++i) {
                            float4 sx = sp[i];
                            for (int q = 1; q < p.spg; ++q) {
                                const float4 o = sp[q * (NP / 4) + i];
                                sx.x += o.x; sx.y += o.y; sx.z += o.z; sx.w += o.w;
                            }
                            yacc[4 * i + 0] = fmaf(sc, __uint_as_float(v[4 * i + 0]), fmaf(nsz, sx.x, yacc[4 * i + 0]));
                            yacc[4 * i + 1] = fmaf(sc, __uint_as_float(v[4 * i + 1]), fmaf(nsz, sx.y, yacc[4 * i + 1]));
                            yacc[4 * i + 2] = fmaf(sc, __uint_as_float(v[4 * i + 2]), fmaf(nsz, sx.z, yacc[4 * i + 2]));
                            yacc[4 * i + 3] = fmaf(sc, __uint_as_float(v[4 * i + 3]), fmaf(nsz, sx.w, yacc[4 * i + 3]));
                        }
                    }
                }
                if (!st.lr) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_g + 8u * rg.slot);
                    rg.next();
                }
            }
            if (!st.piece_end) continue;

            // ---- the block's rows: stored directly, or handed over as partial sums ----
            const int row = st.rb * kRbRows + r;
            auto store_rows = [&](const float (&acc)[NP]) {
                if (!live) return;
#pragma unroll
                for (int i = 0; i < NP; ++i)
                    if (i < p.T) {
                        const size_t o = (size_t)i * p.ldy + row;
                        if (p.out_f32) reinterpret_cast<float*>(p.y)[o] = acc[i];
                        else reinterpret_cast<__nv_bfloat16*>(p.y)[o] = __float2bfloat16_rn(acc[i]);
                    }
            };
            if (st.piece_whole) {
                store_rows(yacc);
            } else {
                // contributors of this block: the CTAs whose runs meet its units, in grid order
                const long long ub = (long long)(st.rb - p.rb_base) * p.ng, ue = ub + p.ng - 1;
                const int c_first = (int)(((ub + 1) * G - 1) / p.units), c_last = (int)(((ue + 1) * G - 1) / p.units);
                float* mine = p.partial + (size_t)(2 * blockIdx.x + (st.piece_first ? 1 : 0)) * (NP * kRbRows);
#pragma unroll
                for (int i = 0; i < NP; ++i)
                    if (i < p.T) mine[i * kRbRows + r] = yacc[i];
                __threadfence();
                epi_sync();
                if (tid == 0) {
                    const int old = atomicAdd(p.counters + st.rb, 1);
                    const int last = old == c_last - c_first;
                    if (last) atomicExch(p.counters + st.rb, 0);  // ready for the next forward
                    s_last = last;
                }
                epi_sync();
                if (s_last) {
                    __threadfence();
                    float acc[NP];
#pragma unroll
                    for (int i = 0; i < NP; ++i) acc[i] = 0.0f;
                    for (int c = c_first; c <= c_last; ++c) {
                        // c_first's piece starts at the block's first unit (slot 1), the others continue it (slot 0)
                        const float* theirs = p.partial + (size_t)(2 * c + (c == c_first ? 1 : 0)) * (NP * kRbRows);
#pragma unroll
                        for (int i = 0; i < NP; ++i)
                            if (i < p.T) acc[i] += __ldcg(theirs + i * kRbRows + r);
                    }
                    store_rows(acc);
                }
                epi_sync();  // s_last is rewritten by the next shared block
            }
#pragma unroll
            for (int i = 0; i < NP; ++i) yacc[i] = 0.0f;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kWarpMma) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// Plain rotated activations [T][n], their 64-column sums [T][s64_ld] and t [T][r_pad] -> operand image (layer
// descriptors the prologue kernel does not take: long Hadamard blocks, identity prefixes off the block grid).
__global__ void __launch_bounds__(256)
image_convert_kernel(const __nv_bfloat16* __restrict__ xrot, int n, const float* __restrict__ s64, int s64_ld,
                     const __half* __restrict__ t, int r_pad, const ImageOut img, int T) {
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = tid; i < (size_t)img.n_counters; i += stride) img.counters[i] = 0;
    const size_t n8 = (size_t)n / 8;
    for (size_t i = tid; i < (size_t)T * n8; i += stride) {
        const int tok = (int)(i / n8), col0 = (int)(i % n8) * 8;
        const int tgp = tok >> img.np_shift, tl = tok & (img.np - 1);
        unsigned char* tile = img.ximg + ((size_t)tgp * img.nsteps + (col0 >> 6)) * img.np * 128;
        *reinterpret_cast<uint4*>(tile + tl * 128 + ((((col0 & 63) >> 3) ^ (tl & 7)) << 4)) =
            *reinterpret_cast<const uint4*>(xrot + (size_t)tok * n + col0);
    }
    const int per_run = 1 << img.gs_shift;
    for (size_t i = tid; i < (size_t)T * img.n_sums; i += stride) {
        const int tok = (int)(i / img.n_sums), run = (int)(i % img.n_sums);
        float sum = 0.0f;
        for (int q = 0; q < per_run; ++q) sum += s64[(size_t)tok * s64_ld + run * per_run + q];
        img.sums[((size_t)(tok >> img.np_shift) * img.n_sums + run) * img.np + (tok & (img.np - 1))] = sum;
    }
    for (size_t i = tid; i < (size_t)T * r_pad; i += stride) {
        const int tok = (int)(i / r_pad), j = (int)(i % r_pad);
        const int tgp = tok >> img.np_shift, tl = tok & (img.np - 1);
        unsigned char* tile = img.timg + ((size_t)tgp * img.lr_steps + (j >> 6)) * img.np * 128;
        *reinterpret_cast<__half*>(tile + tl * 128 + ((((j & 63) >> 3) ^ (tl & 7)) << 4) + (j & 7) * 2) = t[i];
    }
}

struct RbPlan {
    int c_slots, smem_bytes;
};

RbPlan plan_rowblock(const lopro_desc& d, int np) {
    RbPlan pl;
    const int fixed = 1024 + kXSlots * kStageItems * np * 128 + kGSlots * kGSlotBytes;
    const int c_stage = kStageItems * kRbRows * 8 * d.bits;
    int slots = (kSmemLimit - fixed) / c_stage;
    if (slots > kMaxCSlots) slots = kMaxCSlots;
    pl.c_slots = slots;
    pl.smem_bytes = fixed + slots * c_stage;
    return pl;
}

template <int BITS, int NP>
cudaError_t launch_rb(const RbParams& p, int grid, int smem_bytes, cudaStream_t s) {
    static unsigned long long attr_done = 0;
    cudaError_t e = ensure_dynamic_smem(rowblock_kernel<BITS, NP>, kSmemLimit, &attr_done);
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
    return cudaLaunchKernelEx(&cfg, rowblock_kernel<BITS, NP>, p);
}

template <int BITS>
cudaError_t launch_rb_bits(const RbParams& p, int np, int grid, int smem_bytes, cudaStream_t s) {
    return np == 16 ? launch_rb<BITS, 16>(p, grid, smem_bytes, s) : launch_rb<BITS, 32>(p, grid, smem_bytes, s);
}

}  // namespace

// Blocks of rows per launch such that no CTA's run exceeds its stage table (0: not even one block fits).
static int rowblock_blocks_per_launch(const lopro_desc& d) {
    int sms = sm_count();
    if (sms > kRbMaxGrid) sms = kRbMaxGrid;
    const int ng = d.d_in / d.group_size, r_pad = d.rank > 0 ? round_up_int(d.rank, 16) : 0;
    int gshift = 0;
    while ((64 << gshift) < d.group_size) ++gshift;
    const int nlr = ((r_pad + 63) / 64 + kStageItems - 1) / kStageItems;
    // bound on the stages of a run of `u` units: its steps in fours, plus per piece the low-rank stages and one stage
    // of rounding
    auto stages_bound = [&](int nblocks) {
        const long long units = (long long)nblocks * ng;
        const int grid = (int)(units < sms ? units : sms);
        const long long u = (units + grid - 1) / grid;
        return (long long)(((u << gshift) + kStageItems - 1) / kStageItems) + (u / ng + 3) * (nlr + 1);
    };
    int per_launch = (d.d_out + kRbRows - 1) / kRbRows;
    while (per_launch > 1 && stages_bound(per_launch) > kMaxStagesPerCta) per_launch = (per_launch + 1) / 2;
    return stages_bound(per_launch) > kMaxStagesPerCta ? 0 : per_launch;
}

int rowblock_launches(const lopro_desc& d) {
    const int per_launch = rowblock_blocks_per_launch(d), blocks = (d.d_out + kRbRows - 1) / kRbRows;
    return per_launch > 0 ? (blocks + per_launch - 1) / per_launch : 0;
}

bool rowblock_supported(const lopro_desc& d) {
    // a group record holds the (scale, zero) pairs and the column sums of up to 16 runs of 256 columns
    return d.layout == LOPRO_LAYOUT_ROWBLOCK && d.group_size <= 4096 && rowblock_blocks_per_launch(d) > 0;
}

cudaError_t launch_image_convert(const lopro_desc& d, const __nv_bfloat16* xrot, const float* s64, int s64_ld,
                                 const __half* t, int r_pad, const ImageOut& img, int T, cudaStream_t s) {
    const size_t work = (size_t)T * d.d_in / 8;
    const unsigned blocks = (unsigned)((work + 255) / 256 < 1184 ? (work + 255) / 256 : 1184);
    image_convert_kernel<<<blocks ? blocks : 1, 256, 0, s>>>(xrot, d.d_in, s64, s64_ld, t, d.rank > 0 ? r_pad : 0, img, T);
    return cudaGetLastError();
}

cudaError_t launch_rowblock(const lopro_desc& d, const uint8_t* blob, const BlobLayout& L, uint8_t* ws,
                            const WorkspaceLayout& W, void* y, int64_t ldy, int out_dtype, int tgroup, int t_live,
                            cudaStream_t s) {
    const int np = W.np;
    const RbPlan pl = plan_rowblock(d, np);
    const ImageOut img = image_out(d, ws, W);
    RbParams p;
    p.codes = reinterpret_cast<const uint32_t*>(blob + L.off[LOPRO_SEC_CODES]);
    p.sz = reinterpret_cast<const uint32_t*>(blob + L.off[LOPRO_SEC_SCALEZERO]);
    p.A = reinterpret_cast<const __half*>(blob + L.off[LOPRO_SEC_A]);
    p.r_pad = d.rank > 0 ? L.r_pad : 0;
    p.lr_steps = (p.r_pad + 63) / 64;
    p.nsteps = d.d_in / 64;
    p.ximg = img.ximg + (size_t)tgroup * ximg_bytes(d.d_in, np);
    p.sums = img.sums + (size_t)tgroup * img.n_sums * np;
    p.timg = img.timg + (size_t)tgroup * p.lr_steps * np * 128;
    p.partial = reinterpret_cast<float*>(ws + W.off_partial);
    p.counters = img.counters;
    p.status = reinterpret_cast<int*>(ws + W.off_status);
    const size_t esz = out_dtype == LOPRO_OUT_F32 ? 4 : 2;
    p.y = static_cast<uint8_t*>(y) + (size_t)tgroup * np * ldy * esz;
    p.ldy = ldy;
    p.out_f32 = out_dtype == LOPRO_OUT_F32;
    p.m = d.d_out;
    p.T = t_live;
    p.ng = d.d_in / d.group_size;
    p.gshift = 0;
    while ((64 << p.gshift) < d.group_size) ++p.gshift;
    const int blocks = (d.d_out + kRbRows - 1) / kRbRows;
    p.spg = d.group_size > 256 ? d.group_size / 256 : 1;
    p.c_slots = pl.c_slots;
    p.two_issuers = (p.gshift <= 2 && p.lr_steps <= kStageItems) ? 1 : 0;
    int sms = sm_count();
    if (sms > kRbMaxGrid) sms = kRbMaxGrid;
    // A CTA's table holds kMaxStagesPerCta stages: a layer with more work per CTA than that runs as several launches
    // over ranges of blocks.
    const int per_launch = rowblock_blocks_per_launch(d);
    if (per_launch == 0) return cudaErrorInvalidValue;
    for (int b0 = 0; b0 < blocks; b0 += per_launch) {
        const int nb = blocks - b0 < per_launch ? blocks - b0 : per_launch;
        p.rb_base = b0;
        p.units = nb * p.ng;
        const int grid = p.units < sms ? p.units : sms;
        cudaError_t e;
        switch (d.bits) {
            case 2: e = launch_rb_bits<2>(p, np, grid, pl.smem_bytes, s); break;
            case 3: e = launch_rb_bits<3>(p, np, grid, pl.smem_bytes, s); break;
            default: e = launch_rb_bits<4>(p, np, grid, pl.smem_bytes, s); break;
        }
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace lopro
