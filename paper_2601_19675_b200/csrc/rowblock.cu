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
// Work split ("stream-K").  A unit is one quantization group of one block of 128 rows; the units of the layer,
// ordered [block][group], are cut into one contiguous run per CTA.  A CTA whose run covers a whole block stores
// its rows; where a block is shared, every contributor writes its fp32 partial sums to the workspace and counts
// itself in; whoever arrives last adds the partial sums in the fixed order of the contributors (the result does
// not depend on who was last) and stores the rows.  Nobody waits for another CTA.
//
// Roles of a CTA (15 warps):
//   warps 0-3   epilogue: thread = row; tcgen05.ld of a finished slice, scale / zero-point, running sums, output;
//   warps 4-11  expansion: thread = row; reads the row's packed codes of a 64-column step from the code ring,
//               expands them to bf16 128 + c and stores eight 16-byte pieces into the step's K-major, 128-byte
//               swizzled A tile (for the low-rank steps: copies the row's fp16 entries of A);
//   warp 12     one thread streams packed codes and (scale, zero) pairs with bulk copies -- layer data, requested
//               before griddepcontrol.wait, i.e. while the prologue of the same forward still runs;
//   warp 13     one thread waits for the prologue and streams the activation tiles and column sums;
//   warp 14     one thread issues tcgen05.mma (M 128, N = NP, K 16) and commits stages, tiles and slices back.
// Every mbarrier wait is bounded; a wait that runs out stores LOPRO_ERR_TIMEOUT in the workspace status word, the
// CTA stops waiting, frees its tensor memory and returns (outputs then unspecified).
#include "common.cuh"
#include "ptx.cuh"
#include "tc5.cuh"

namespace lopro {

namespace {

constexpr int kEpiWarps = 4;
constexpr int kExpWarps = 8;  // two sets of four warps (one warp per 32-row quarter), alternating steps
constexpr int kWarpW = kEpiWarps + kExpWarps, kWarpX = kWarpW + 1, kWarpMma = kWarpW + 2;
constexpr int kThreads = (kWarpMma + 1) * 32;
#ifndef RB_XSLOTS
#define RB_XSLOTS 6
#endif
#ifndef RB_GSLOTS
#define RB_GSLOTS 8
#endif
#ifndef RB_POLL_ALL
#define RB_POLL_ALL 1
#endif
constexpr int kASlots = 4;             // ring of expanded A tiles
constexpr int kATile = kRbRows * 128;  // 16 KB: 128 rows x 64 columns of bf16
constexpr int kXSlots = RB_XSLOTS;     // ring of activation tiles
constexpr int kGSlots = RB_GSLOTS;     // ring of group records: (scale, zero) pairs and column sums
constexpr int kSlices = 8;             // accumulator slices in tensor memory
constexpr int kMaxCSlots = 32;         // ring of packed-code steps (depth chosen at launch)
constexpr int kSmemLimit = 200 * 1024;

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
    int nsteps, ng, gsteps;     // 64-column steps of K, groups per row, steps per group
    int r_pad, lr_steps;
    int units;                  // blocks * ng
    int spg;                    // column-sum runs per group (1 unless g > 256)
    int c_slots;                // depth of the code ring
    int g_slot_bytes;
    int bits;
};

// Ring position: slot and the parity of its current use.
struct Ring {
    int slot = 0;
    uint32_t phase = 0;
    int n;
    __device__ explicit Ring(int n_) : n(n_) {}
    __device__ void next() {
        if (++slot == n) {
            slot = 0;
            phase ^= 1u;
        }
    }
};

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

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"r"(kEpiWarps * 32) : "memory"); }

template <int BITS, int NP>
__global__ void __launch_bounds__(kThreads, 1)
rowblock_kernel(const RbParams p) {
    extern __shared__ unsigned char smem_raw[];
    // full / empty per slot of the five rings
    __shared__ __align__(8) uint64_t bars[2 * (kASlots + kXSlots + kGSlots + kSlices + kMaxCSlots)];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_timeout;
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // operand tiles are 1024-byte aligned (swizzle atoms)
    unsigned char* base_ptr = smem_raw + (base - raw);
    constexpr int kXTile = NP * 128;
    constexpr int kStepBytes = kRbRows * 8 * BITS;  // packed codes of 128 rows x 64 columns
    const uint32_t a_ring = base, x_ring = a_ring + kASlots * kATile, g_ring = x_ring + kXSlots * kXTile;
    const uint32_t c_ring = g_ring + (uint32_t)(kGSlots * p.g_slot_bytes);
    const unsigned char* g_ring_ptr = base_ptr + kASlots * kATile + kXSlots * kXTile;
    const unsigned char* c_ring_ptr = g_ring_ptr + kGSlots * p.g_slot_bytes;

    const uint32_t bar0 = smem_u32(bars);
    int bi = 0;
    const uint32_t full_a = bar0 + 8u * bi; bi += kASlots;
    const uint32_t empty_a = bar0 + 8u * bi; bi += kASlots;
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
        for (int s = 0; s < kASlots; ++s) {
            mbar_init(full_a + 8u * s, 4);   // the four expansion warps of a step
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
    constexpr uint32_t kTmemCols = kSlices * NP;  // 128 or 256: a power of two >= 32
    if (warp == kWarpMma) tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;

    // this CTA's run of units [u0, u1)
    const long long G = gridDim.x;
    const int u0 = (int)((long long)blockIdx.x * p.units / G), u1 = (int)(((long long)blockIdx.x + 1) * p.units / G);

    auto time_out = [&]() {
        s_timeout = 1;
        atomicExch(p.status, (int)LOPRO_ERR_TIMEOUT);
    };
    // bounded wait of one thread / of every lane of a warp (all lanes poll: they all read what the wait guards)
    auto wait = [&](uint32_t bar, uint32_t parity) {
        if (!*(volatile int*)&s_timeout && !mbar_wait(bar, parity)) time_out();
    };
    // wait of a whole warp: one lane polls, the warp follows (bar.warp.sync orders the other lanes' accesses after it)
    auto slow_wait = [&](uint32_t bar, uint32_t parity) {
        if (!*(volatile int*)&s_timeout && !mbar_wait_backoff(bar, parity)) time_out();
    };
    auto warp_wait = [&](uint32_t bar, uint32_t parity) {
#if RB_POLL_ALL
        slow_wait(bar, parity);
#else
        if (lane == 0) slow_wait(bar, parity);
        __syncwarp();
#endif
    };

    if (warp == kWarpW) {
        // ---------------- layer-data producer: packed codes and (scale, zero) pairs ----------------
        if (lane == 0) {
            Ring rc(p.c_slots), rg(kGSlots);
            bool c_wrapped = false, g_wrapped = false;
            for (int u = u0; u < u1;) {
                const int rb = u / p.ng, gb = u - rb * p.ng, ge = min(p.ng, gb + (u1 - u));
                const int R = rb_rows(p.m, rb);
                const uint32_t step_bytes = (uint32_t)(R * 8 * BITS), sz_bytes = (uint32_t)(R * 4);
                const uint32_t* cblock = p.codes + rb_step_word(BITS, p.nsteps, p.m, rb, 0);
                const uint32_t* szblock = p.sz + (size_t)rb * kRbRows * p.ng;
                for (int g = gb; g < ge; ++g) {
                    if (g_wrapped) slow_wait(empty_g + 8u * rg.slot, rg.phase ^ 1u);
                    mbar_expect_tx(full_g + 8u * rg.slot, sz_bytes);
                    bulk_g2s(g_ring + (uint32_t)(rg.slot * p.g_slot_bytes), szblock + (size_t)g * R, sz_bytes, full_g + 8u * rg.slot);
                    rg.next();
                    if (rg.slot == 0) g_wrapped = true;
                    for (int st = 0; st < p.gsteps; ++st) {
                        if (c_wrapped) slow_wait(empty_c + 8u * rc.slot, rc.phase ^ 1u);
                        mbar_expect_tx(full_c + 8u * rc.slot, step_bytes);
                        bulk_g2s(c_ring + (uint32_t)(rc.slot * kStepBytes),
                                 cblock + (size_t)(g * p.gsteps + st) * R * (2 * BITS), step_bytes, full_c + 8u * rc.slot);
                        rc.next();
                        if (rc.slot == 0) c_wrapped = true;
                    }
                }
                u += ge - gb;
            }
        }
    } else if (warp == kWarpX) {
        // ---------------- activation producer: tiles of x~ (and of t), column sums ----------------
        if (lane == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");  // the prologue's image is complete
            Ring rx(kXSlots), rg(kGSlots);
            bool x_wrapped = false, g_wrapped = false;
            const uint32_t sum_bytes = (uint32_t)(p.spg * NP * 4);
            auto issue_x = [&](const unsigned char* src) {
                if (x_wrapped) slow_wait(empty_x + 8u * rx.slot, rx.phase ^ 1u);
                mbar_expect_tx(full_x + 8u * rx.slot, kXTile);
                bulk_g2s(x_ring + (uint32_t)(rx.slot * kXTile), src, kXTile, full_x + 8u * rx.slot);
                rx.next();
                if (rx.slot == 0) x_wrapped = true;
            };
            for (int u = u0; u < u1;) {
                const int rb = u / p.ng, gb = u - rb * p.ng, ge = min(p.ng, gb + (u1 - u));
                if (gb == 0)
                    for (int j = 0; j < p.lr_steps; ++j) issue_x(p.timg + (size_t)j * kXTile);
                for (int g = gb; g < ge; ++g) {
                    if (g_wrapped) slow_wait(empty_g + 8u * rg.slot, rg.phase ^ 1u);
                    mbar_expect_tx(full_g + 8u * rg.slot, sum_bytes);
                    bulk_g2s(g_ring + (uint32_t)(rg.slot * p.g_slot_bytes) + 512u, p.sums + (size_t)g * p.spg * NP, sum_bytes,
                             full_g + 8u * rg.slot);
                    rg.next();
                    if (rg.slot == 0) g_wrapped = true;
                    for (int st = 0; st < p.gsteps; ++st) issue_x(p.ximg + (size_t)(g * p.gsteps + st) * kXTile);
                }
                u += ge - gb;
            }
        }
    } else if (warp == kWarpMma) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc_w = make_idesc(NP, 1u), idesc_lr = make_idesc(NP, 0u);
            Ring ra(kASlots), rx(kXSlots), rs(kSlices);
            bool s_wrapped = false;
            // one 64-column step: up to four MMAs of K = 16 into slice `d`
            auto step = [&](uint32_t d, uint32_t idesc, int ksub, bool first) {
                wait(full_a + 8u * ra.slot, ra.phase);
                wait(full_x + 8u * rx.slot, rx.phase);
                tc_fence_after();
                const uint64_t da = make_desc_sw128(a_ring + ra.slot * kATile), db = make_desc_sw128(x_ring + rx.slot * kXTile);
                for (int k = 0; k < ksub; ++k)  // 16 columns = 32 bytes = 2 descriptor address units
                    umma_f16(d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (first && k == 0) ? 0u : 1u);
                umma_commit(empty_a + 8u * ra.slot);  // the tiles may be refilled once these MMAs have read them
                umma_commit(empty_x + 8u * rx.slot);
                ra.next();
                rx.next();
            };
            auto open_slice = [&]() {
                if (s_wrapped) wait(empty_s + 8u * rs.slot, rs.phase ^ 1u);
                tc_fence_after();
                return tmem + (uint32_t)(rs.slot * NP);
            };
            auto close_slice = [&]() {
                umma_commit(full_s + 8u * rs.slot);
                rs.next();
                if (rs.slot == 0) s_wrapped = true;
            };
            for (int u = u0; u < u1;) {
                const int rb = u / p.ng, gb = u - rb * p.ng, ge = min(p.ng, gb + (u1 - u));
                if (gb == 0 && p.lr_steps > 0) {
                    const uint32_t d = open_slice();
                    for (int j = 0; j < p.lr_steps; ++j) step(d, idesc_lr, min(4, (p.r_pad - j * 64) / 16), j == 0);
                    close_slice();
                }
                for (int g = gb; g < ge; ++g) {
                    const uint32_t d = open_slice();
                    for (int st = 0; st < p.gsteps; ++st) step(d, idesc_w, 4, st == 0);
                    close_slice();
                }
                u += ge - gb;
            }
        }
    } else if (warp >= kEpiWarps) {
        // ---------------- expansion warps ----------------
        const int e = warp - kEpiWarps, quarter = e & 3, set = e >> 2;
        const int r = quarter * 32 + lane;
        // byte offset of 16-byte piece 0 of row r in an A tile; piece c sits at (off ^ (c << 4))
        const uint32_t row_off = (uint32_t)(r * 128 + ((r & 7) << 4));
        Ring rc(p.c_slots);
        int it = 0;  // steps seen so far by this CTA: set `it & 1` expands it into A slot `it & 3`
        auto a_slot_ready = [&](int item) {
            if (item >= kASlots) warp_wait(empty_a + 8u * (item & (kASlots - 1)), (uint32_t)((item / kASlots) - 1) & 1u);
        };
        auto publish = [&](int item) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> async proxy (MMA)
            __syncwarp();
            if (lane == 0) mbar_arrive(full_a + 8u * (item & (kASlots - 1)));
        };
        for (int u = u0; u < u1;) {
            const int rb = u / p.ng, gb = u - rb * p.ng, ge = min(p.ng, gb + (u1 - u));
            const int R = rb_rows(p.m, rb);
            const bool live = r < R;
            if (gb == 0) {
                // low-rank steps: the row's fp16 entries of A, 64 columns of the rank per step
                const __half* arow = p.A + (size_t)(rb * kRbRows + r) * p.r_pad;
                for (int j = 0; j < p.lr_steps; ++j, ++it) {
                    if ((it & 1) != set) continue;
                    a_slot_ready(it);
                    unsigned char* tile = base_ptr + (it & (kASlots - 1)) * kATile;
                    if (live) {
                        const int pieces = min(8, (p.r_pad - j * 64) / 8);
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            if (c < pieces)
                                *reinterpret_cast<uint4*>(tile + (row_off ^ (uint32_t)(c << 4))) =
                                    __ldg(reinterpret_cast<const uint4*>(arow + j * 64) + c);
                    }
                    publish(it);
                }
            }
            const int n_q = (ge - gb) * p.gsteps;
            for (int q = 0; q < n_q; ++q, ++it, rc.next()) {
                if ((it & 1) != set) continue;
                warp_wait(full_c + 8u * rc.slot, rc.phase);
                uint32_t w[2 * BITS];
                if (live) {
                    const unsigned char* src = c_ring_ptr + rc.slot * kStepBytes;
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
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_c + 8u * rc.slot);  // the words are in registers
                a_slot_ready(it);
                if (live) {
                    unsigned char* tile = base_ptr + (it & (kASlots - 1)) * kATile;
#pragma unroll
                    for (int hs = 0; hs < 2; ++hs) {
                        uint32_t wh[BITS], a[16];
#pragma unroll
                        for (int b = 0; b < BITS; ++b) wh[b] = w[hs * BITS + b];
                        expand_codes<BITS>(a, wh);
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4*>(tile + (row_off ^ (uint32_t)((hs * 4 + c) << 4))) =
                                make_uint4(a[4 * c], a[4 * c + 1], a[4 * c + 2], a[4 * c + 3]);
                    }
                }
                publish(it);
            }
            u += ge - gb;
        }
    } else {
        // ---------------- epilogue warps: thread = row ----------------
        asm volatile("griddepcontrol.wait;" ::: "memory");  // y, the partial sums and the counters belong to this call only now
        const int r = warp * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        Ring rs(kSlices), rg(kGSlots);
        for (int u = u0; u < u1;) {
            const int rb = u / p.ng, gb = u - rb * p.ng, ge = min(p.ng, gb + (u1 - u));
            const int R = rb_rows(p.m, rb);
            const bool live = r < R;
            float yacc[NP];
#pragma unroll
            for (int i = 0; i < NP; ++i) yacc[i] = 0.0f;
            uint32_t v[NP];
            auto take_slice = [&]() {
                warp_wait(full_s + 8u * rs.slot, rs.phase);
                __syncwarp();
                tc_fence_after();
                tmem_ld<NP>(v, tmem + lane_addr + (uint32_t)(rs.slot * NP));
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_s + 8u * rs.slot);
                rs.next();
            };
            if (gb == 0 && p.lr_steps > 0) {
                take_slice();
#pragma unroll
                for (int i = 0; i < NP; ++i) yacc[i] += __uint_as_float(v[i]);
            }
            for (int g = gb; g < ge; ++g) {
                take_slice();
                warp_wait(full_g + 8u * rg.slot, rg.phase);
                const unsigned char* rec = g_ring_ptr + rg.slot * p.g_slot_bytes;
                if (live) {
                    const uint32_t szw = *reinterpret_cast<const uint32_t*>(rec + r * 4);
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&szw));
                    const float sc = f.x, nsz = -f.x * (128.0f + f.y);
                    const float4* sp = reinterpret_cast<const float4*>(rec + 512);
                    if (p.spg == 1) {
#pragma unroll
                        for (int i = 0; i < NP / 4; ++i) {
                            const float4 sx = sp[i];
                            yacc[4 * i + 0] = fmaf(sc, __uint_as_float(v[4 * i + 0]), fmaf(nsz, sx.x, yacc[4 * i + 0]));
                            yacc[4 * i + 1] = fmaf(sc, __uint_as_float(v[4 * i + 1]), fmaf(nsz, sx.y, yacc[4 * i + 1]));
                            yacc[4 * i + 2] = fmaf(sc, __uint_as_float(v[4 * i + 2]), fmaf(nsz, sx.z, yacc[4 * i + 2]));
                            yacc[4 * i + 3] = fmaf(sc, __uint_as_float(v[4 * i + 3]), fmaf(nsz, sx.w, yacc[4 * i + 3]));
                        }
                    } else {
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
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_g + 8u * rg.slot);
                rg.next();
            }

            // ---- the block's rows: stored directly, or handed over as partial sums ----
            const int row = rb * kRbRows + r;
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
            if (gb == 0 && ge == p.ng) {
                store_rows(yacc);
            } else {
                // contributors of this block: the CTAs whose runs meet its units, in grid order
                const long long ub = (long long)rb * p.ng, ue = ub + p.ng - 1;
                const int c_first = (int)(((ub + 1) * G - 1) / p.units), c_last = (int)(((ue + 1) * G - 1) / p.units);
                float* mine = p.partial + (size_t)(2 * blockIdx.x + (gb > 0 ? 0 : 1)) * (NP * kRbRows);
#pragma unroll
                for (int i = 0; i < NP; ++i)
                    if (i < p.T) mine[i * kRbRows + r] = yacc[i];
                __threadfence();
                epi_sync();
                if (tid == 0) {
                    const int old = atomicAdd(p.counters + rb, 1);
                    const int last = old == c_last - c_first;
                    if (last) atomicExch(p.counters + rb, 0);  // ready for the next forward
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
            u += ge - gb;
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
    int c_slots, g_slot_bytes, smem_bytes;
};

RbPlan plan_rowblock(const lopro_desc& d, int np) {
    RbPlan pl;
    const int spg = d.group_size > 256 ? d.group_size / 256 : 1;
    pl.g_slot_bytes = round_up_int(512 + spg * np * 4, 128);
    const int fixed = 1024 + kASlots * kATile + kXSlots * np * 128 + kGSlots * pl.g_slot_bytes;
    int slots = (kSmemLimit - fixed) / (kRbRows * 8 * d.bits);
    if (slots > kMaxCSlots) slots = kMaxCSlots;
    pl.c_slots = slots;
    pl.smem_bytes = fixed + slots * kRbRows * 8 * d.bits;
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

bool rowblock_supported(const lopro_desc& d) {
    // a group record holds 512 bytes of (scale, zero) pairs and the column sums of the group's runs
    return d.layout == LOPRO_LAYOUT_ROWBLOCK && d.group_size <= 4096;
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
    p.gsteps = d.group_size / 64;
    const int blocks = (d.d_out + kRbRows - 1) / kRbRows;
    p.units = blocks * p.ng;
    p.spg = d.group_size > 256 ? d.group_size / 256 : 1;
    p.c_slots = pl.c_slots;
    p.g_slot_bytes = pl.g_slot_bytes;
    p.bits = d.bits;
    int grid = sm_count();
    if (grid > kRbMaxGrid) grid = kRbMaxGrid;
    if (grid > p.units) grid = p.units;
    switch (d.bits) {
        case 2: return launch_rb_bits<2>(p, np, grid, pl.smem_bytes, s);
        case 3: return launch_rb_bits<3>(p, np, grid, pl.smem_bytes, s);
        default: return launch_rb_bits<4>(p, np, grid, pl.smem_bytes, s);
    }
}

}  // namespace lopro
