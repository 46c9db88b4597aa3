// BitDelta fused GEMM, streaming decode schedule (few token rows per unit) on tcgen05 tensor cores.
//
//   Y[b,t,n] = sum_k X[b,t,k] W[n,k] + alpha[b] sum_k X[b,t,k] S[b,n,k]
//
// Same orientation as the tiled kernel (weight rows on the MMA's M side, tokens on its N side, decoded signs
// written to tensor memory as the A operand, e5m2 signs x four exact e5m2 pieces of every activation), but
// laid out so that a thread block needs at most HALF of a multiprocessor:
//   * 14 warps: one TMA producer, one MMA issuer, eight sign-decode warps, four epilogue / activation-split
//     warps; at most 113 KB of shared memory; tensor memory is allocated only after the grid this launch
//     depends on has completed.
//   * A launch queued behind another one with an early start therefore becomes RESIDENT next to the running
//     launch's blocks and fills its shared-memory rings with weights (which no kernel writes) while the
//     running launch finishes its tiles, its split-K fix-up and its teardown: the next launch's start-up and
//     first DRAM round trip are hidden behind the previous launch's tail.
//   * Per 128-k step the eight decode warps fill two operand SETS in tensor memory (all the unit's tenants x
//     64 k, 128 columns; two sets in flight) and hand each one to the single MMA issuer through a named barrier
//     on which they only arrive; the issuer sleeps on it.  Nothing in the decode warps' loop waits for
//     another role except for a free set (released by tcgen05.commit, several sets ahead) and for the sign
//     words (TMA, several steps ahead).
//   * Data paths.  On B200 a bulk-tensor copy costs the copy engine several hundred cycles whatever its size, and
//     rows of 16 bytes go through it at about one per cycle, so the sign words of a step (1024 rows) alone keep
//     it busy for half of the step's DRAM time.  A step therefore costs it exactly two operations: the W_base
//     tile (both 64-k atoms, 32 KB) and the sign words of all the unit's tenants (16 KB).  The few activation
//     rows are read straight from global memory by the threads that split them.
// Work split, partial results of tiles cut across blocks and their fixed-order sum are those of the tiled
// kernel.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <type_traits>

#include "gemm_common.cuh"
#include "gemm_tc.h"
#include "ptx.cuh"

namespace bd {

constexpr int kSWarpProducer = 0;
constexpr int kSWarpMma = 1;
constexpr int kSWarpDecode0 = 2;                 // warps 2 .. 9 decode
constexpr int kSEpiWarps = 4;                    // the four warps after them
__host__ __device__ constexpr int stream_threads(int /*kG*/) { return (kSWarpDecode0 + 8 + kSEpiWarps) * 32; }   // 448
constexpr int kSBarSet0 = 2;                     // named barrier of operand set s: id 2 + s
constexpr int kSBarDep = 15;                     // named barrier the decode and epilogue warps sleep on until the grid
                                                 // dependency is resolved (the issuer warp arrives on it)
constexpr uint32_t kSAtomBytes = kTileN * 128;   // one W_base atom: 128 rows x 64 k of 16-bit values

#ifdef BD_TRACE
// Trace build (build.py --trace, a separate library): every thread block stamps the global nanosecond timer at
// the main events of each role into 128 words of a buffer set with bitdelta_debug_set_trace.  Layout: 0 start,
// 1 set-up done, 2 dependency resolved, 3 tensor memory allocated, 4 multiprocessor id, 5 producer done,
// 8+2p / 9+2p issuer: step p's activations and first atom / pieces ready, 30+s issuer: set s handed over,
// 60+s decode warp 0: set s free, 90+p decode warp 0: step p's sign words landed, 100+3g epilogue: segment g's
// accumulators complete, drained, fix-up done, 110 teardown, 111..117 decode warp 0: cycles spent in the decode
// arithmetic, waiting for its stores + hand-over, waiting for a free set, issuing stores, per-step sign-word wait
// and loads, end-of-step flush; sets done.
__device__ unsigned long long* g_stream_trace;
#define ST_DECL unsigned long long* const st_buf = g_stream_trace ? g_stream_trace + ((size_t)(a.hold_prefetch & 1) * 256 + blockIdx.x) * 256 : nullptr
#define ST(idx) do { if (st_buf && lane == 0 && (idx) < 256) st_buf[idx] = global_timer_ns(); } while (0)
#define ST_VAL(idx, v) do { if (st_buf && lane == 0) st_buf[idx] = (v); } while (0)
#define ST_CLK(name) const long long name = clock64()
#else
#define ST_CLK(name) do { } while (0)
#define ST_DECL do { } while (0)
#define ST(idx) do { } while (0)
#define ST_VAL(idx, v) do { } while (0)
#endif

struct SCtl {
    uint64_t wfull[kMaxStages];     // W_base atom landed
    uint64_t wempty[kMaxStages];    // ... and was read by its base MMAs
    uint64_t bfull[4];              // sign words of a 128-k step landed
    uint64_t bempty[4];             // ... and are in the decode warps' registers (8 arrivals)
    uint64_t pfull[4];              // the step's activation tile and e5m2 pieces are in place (128 splitter threads)
    uint64_t pempty[4];             // ... and were read by the step's MMAs
    uint64_t opfree[kStreamMaxSets];// operand set in tensor memory free again
    uint64_t accfull;               // all MMAs of a segment have completed
    uint64_t accempty;              // the accumulators were drained (4 epilogue warps)
    uint64_t depready;              // the grid this launch depends on has completed
    uint64_t tmemready;             // tensor memory is allocated (its base address is in tmem_base)
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t is_last;
};
static_assert(sizeof(SCtl) <= kSmemCtrlBytes, "control block too large");

// Activation split of one 128-k step straight from global memory (few token rows per unit): writes the step's
// 16-bit activation tile (two swizzled 64-k atoms, the base MMAs' B operand) and its four e5m2 piece rows per
// token (the delta MMAs' B operand).  Same task layout and piece arithmetic as split_activations: task
// (r, q4, h, pc) owns, of token row r and 32-k group q4, the k pairs 8i + 4h + 2pc (i = 0..3).  `xg`: row 0,
// first k of the step.
template <bool kF16>
__device__ __forceinline__ void split_from_global(const GemmArgs& a, int am, const uint16_t* __restrict__ xg, uint8_t* xt,
                                                  uint8_t* x8t, int ntok, int tid, int nthreads) {
    const int ntasks = ntok * 16;
    bool out_of_range = false;
    for (int task = tid; task < ntasks; task += nthreads) {
        const int r = task >> 4, q4 = (task >> 2) & 3, h = (task >> 1) & 1, pc = task & 1;
        const int j = r / am, t = r - j * am;
        const uint32_t* src = reinterpret_cast<const uint32_t*>(xg + (size_t)r * a.K + q4 * 32 + h * 4 + pc * 2);
        uint8_t* xrow = xt + (q4 >> 1) * a.x_atom_bytes + r * 128 + h * 8 + pc * 4;
        uint32_t v[4], y[4];   // v[i]: the pair k = 8i + 4h + 2pc, +1 as stored; y[i]: as an f16 pair
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = __ldcg(src + 4 * i);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int chunk = ((q4 & 1) * 4 + i) ^ (r & 7);
            *reinterpret_cast<uint32_t*>(xrow + chunk * 16) = v[i];
            if constexpr (kF16) {
                y[i] = v[i];
            } else {
                if (((v[i] & 0x7FFFu) >= 0x4780u) || (((v[i] >> 16) & 0x7FFFu) >= 0x4780u)) out_of_range = true;
                const __half2 lim = __floats2half2_rn(65504.f, 65504.f);
                const __half2 hv = __hmax2(__hmin2(__floats2half2_rn(__uint_as_float(v[i] << 16), __uint_as_float(v[i] & 0xFFFF0000u)), lim), __hneg2(lim));
                y[i] = *reinterpret_cast<const uint32_t*>(&hv);
            }
        }
#pragma unroll
        for (int q = 0; q < kPieces; ++q) {
            uint32_t pq[4];   // byte 1 / byte 3: the e5m2 piece of k / k+1
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                pq[i] = y[i] & 0xFF00FF00u;
                if (q + 1 < kPieces) {
                    const __half2 d = __hsub2(*reinterpret_cast<const __half2*>(&y[i]), *reinterpret_cast<const __half2*>(&pq[i]));
                    y[i] = *reinterpret_cast<const uint32_t*>(&d);
                }
            }
            const uint32_t t01 = __byte_perm(pq[0], pq[1], 0x7351);
            const uint32_t t23 = __byte_perm(pq[2], pq[3], 0x7351);
            const uint2 w = make_uint2(__byte_perm(t01, t23, 0x5410), __byte_perm(t01, t23, 0x7632));
            const int r8 = j * (kPieces * am) + q * am + t;
            *reinterpret_cast<uint2*>(x8t + r8 * 128 + (((2 * q4 + h) ^ (r8 & 7)) * 16) + pc * 8) = w;
        }
    }
    if (out_of_range) atomicCAS(&g_device_status[0], 0u, kStatusRange);
}

// The same split for more than eight token rows per unit: a task is a whole 32-k group of one row (64 bytes, four
// 16-byte loads requested together, so a step costs one round trip to L2 per thread), 16-byte shared stores.
template <bool kF16>
__device__ __forceinline__ void split_from_global_wide(const GemmArgs& a, int am, const uint16_t* __restrict__ xg, uint8_t* xt,
                                                       uint8_t* x8t, int ntok, int tid, int nthreads) {
    const int ntasks = ntok * 4;
    bool out_of_range = false;
    for (int task = tid; task < ntasks; task += nthreads) {
        const int r = task >> 2, q4 = task & 3;
        const int j = r / am, t = r - j * am;
        const uint4* src = reinterpret_cast<const uint4*>(xg + (size_t)r * a.K + q4 * 32);
        uint4 L[4];   // L[i]: k = 8i .. 8i+7 of the group as four pairs
#pragma unroll
        for (int i = 0; i < 4; ++i) L[i] = __ldcg(src + i);
        uint8_t* xrow = xt + (q4 >> 1) * a.x_atom_bytes + r * 128;
#pragma unroll
        for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(xrow + ((((q4 & 1) * 4 + i) ^ (r & 7)) * 16)) = L[i];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint2 w[kPieces][2];   // [piece][pc]
#pragma unroll
            for (int pc = 0; pc < 2; ++pc) {
                uint32_t y[4];   // the pair k = 8i + 4h + 2pc as an f16 pair
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t v = (h == 0) ? (pc == 0 ? L[i].x : L[i].y) : (pc == 0 ? L[i].z : L[i].w);
                    if constexpr (kF16) {
                        y[i] = v;
                    } else {
                        if (((v & 0x7FFFu) >= 0x4780u) || (((v >> 16) & 0x7FFFu) >= 0x4780u)) out_of_range = true;
                        const __half2 lim = __floats2half2_rn(65504.f, 65504.f);
                        const __half2 hv = __hmax2(__hmin2(__floats2half2_rn(__uint_as_float(v << 16), __uint_as_float(v & 0xFFFF0000u)), lim), __hneg2(lim));
                        y[i] = *reinterpret_cast<const uint32_t*>(&hv);
                    }
                }
#pragma unroll
                for (int q = 0; q < kPieces; ++q) {
                    uint32_t pq[4];   // byte 1 / byte 3: the e5m2 piece of k / k+1
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        pq[i] = y[i] & 0xFF00FF00u;
                        if (q + 1 < kPieces) {
                            const __half2 d = __hsub2(*reinterpret_cast<const __half2*>(&y[i]), *reinterpret_cast<const __half2*>(&pq[i]));
                            y[i] = *reinterpret_cast<const uint32_t*>(&d);
                        }
                    }
                    const uint32_t t01 = __byte_perm(pq[0], pq[1], 0x7351);
                    const uint32_t t23 = __byte_perm(pq[2], pq[3], 0x7351);
                    w[q][pc] = make_uint2(__byte_perm(t01, t23, 0x5410), __byte_perm(t01, t23, 0x7632));
                }
            }
#pragma unroll
            for (int q = 0; q < kPieces; ++q) {
                const int r8 = j * (kPieces * am) + q * am + t;
                *reinterpret_cast<uint4*>(x8t + r8 * 128 + (((2 * q4 + h) ^ (r8 & 7)) * 16)) = make_uint4(w[q][0].x, w[q][0].y, w[q][1].x, w[q][1].y);
            }
        }
    }
    if (out_of_range) atomicCAS(&g_device_status[0], 0u, kStatusRange);
}

// Cluster form: where a block's partial sums go (its own shared memory, [token][128 weight rows] floats).
struct ClusterPartOut {
    float* part_row;   // &part[0][this thread's weight row]
    __device__ __forceinline__ void put(int tok, float v) const { part_row[tok * kTileN] = v; }
};

// epilogue_decode for a run-time m of 5..16.
template <bool kG, class Out>
__device__ __forceinline__ void epilogue_decode_any_m(const GemmArgs& a, const Unit& u, uint32_t lane_taddr, const Out& out,
                                                      const float* alv, float al_lane, int am) {
    switch (am) {
        case 5: epilogue_decode<5, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 6: epilogue_decode<6, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 7: epilogue_decode<7, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 8: epilogue_decode<8, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 9: epilogue_decode<9, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 10: epilogue_decode<10, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 11: epilogue_decode<11, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 12: epilogue_decode<12, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 13: epilogue_decode<13, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 14: epilogue_decode<14, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        case 15: epilogue_decode<15, kG>(a, u, lane_taddr, out, alv, al_lane); break;
        default: epilogue_decode<16, kG>(a, u, lane_taddr, out, alv, al_lane); break;
    }
}

// kMode 1..4: m = kMode tokens per tenant; 5: any m up to 16.  kGen: binary16 I/O, bias, activation.
// kG = 1: at most half a multiprocessor per block (72 registers per thread), units of up to 16 token rows; kG = 2: a
// whole multiprocessor per block (its rings need more than half of the shared memory), units of up to 32 token rows.
template <int kMode, bool kGen, int kG>
__global__ void __launch_bounds__(stream_threads(kG), kG == 1 ? 2 : 1)
bitdelta_gemm_stream_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmBits,
                            const GemmArgs a) {
    constexpr int kSDecodeWarps = 8;
    constexpr int kSWarpEpi0 = kSWarpDecode0 + kSDecodeWarps;
    constexpr int kSThreads = stream_threads(kG);
    constexpr int kSHandover = kSDecodeWarps * 32 + 32;   // decode threads arrive, the issuer warp syncs
    constexpr int kTenPerWarp = 4;                        // tenants of a unit a decode warp owns (of up to eight)
    constexpr int kTenStride = 2;                         // ... tenant j = kTenStride * i + h for warp half h
    constexpr int kWarpCols = 64;                         // ... and its columns of an operand set
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t w_addr = base;                                          // ring of W_base atoms
    const uint32_t bits_off = a.n_w * (2 * kSAtomBytes);                   // sign-word slots
    const uint32_t bits_addr = base + bits_off;
    const uint32_t x_off = bits_off + a.n_bits * a.bslot_bytes;            // ring of activation tiles
    const uint32_t x_addr = base + x_off;
    const uint32_t x8_off = x_off + a.n_x * a.x_tile_bytes;                // ring of e5m2 piece tiles
    const uint32_t x8_addr = base + x8_off;
    // (the last tenant's delta window runs up to 2 KB past the last piece tile, in whole 8-row swizzle atoms: the
    // control block and the pad behind it are there to be read as ignored accumulator columns)
    SCtl* ctl = reinterpret_cast<SCtl*>(smem + x8_off + a.n_x8 * a.x8_atom_bytes);
    volatile uint32_t* abort_flag = &ctl->abort_flag;

    const int am = (kMode <= 4) ? kMode : a.m;
    const bool io_f16 = kGen && a.f16 != 0;
    auto unit_info = [&](const GemmArgs& aa, int un) { return unit_info_t<true, false, false>(aa, un, am, 0); };
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    ST_DECL;
    if (warp == 0) ST(0);
    if (threadIdx.x == 32) {
        prefetch_tensormap(&tmW);
        prefetch_tensormap(&tmBits);
    }

    // Work: an even share of the flat (unit, k-step) list (or whole units round-robin), or, in the cluster form,
    // this block's share of the k-steps of its cluster's unit.
    const int crank = (a.cluster > 1) ? (int)cluster_ctarank() : 0;
    int lo, hi;
    if (a.cluster > 1) {
        const int cunit = (int)blockIdx.x / a.cluster;
        lo = cunit * a.P + (crank * a.P) / a.cluster;
        hi = cunit * a.P + ((crank + 1) * a.P) / a.cluster;
    } else {
        lo = a.whole_units ? (int)blockIdx.x * a.P : cta_first_item(a, (int)blockIdx.x);
        hi = a.whole_units ? (int)a.T : cta_first_item(a, (int)blockIdx.x + 1);
    }
    SegIter it{lo, hi, a.P, (a.whole_units && a.cluster <= 1) ? (int)gridDim.x : 0};
    int unit, p0, p1;

    // Weight loads of one 128-k step: sub 0 / 1 = its two W_base atoms, sub 2 = its sign words.  One thread.
    // The W_base tile of a step (128 rows x 128 k: both 64-k atoms) in ONE bulk-tensor copy.  One thread.
    auto issue_w = [&](const Unit& u, int p, int stage) {
        const uint32_t bar = smem_u32(&ctl->wfull[stage]);
        mbar_arrive_expect_tx(bar, 2 * kSAtomBytes);
        tma_load_3d(w_addr + stage * (2 * kSAtomBytes), &tmW, bar, 0, u.n0, p * (kPairK / kAtomK));
    };
    // The sign words of a step for all the unit's tenants: one bulk-tensor copy.  One thread.
    auto issue_bits = [&](const Unit& u, int p, int bslot) {
        const uint32_t bar = smem_u32(&ctl->bfull[bslot]);
        mbar_arrive_expect_tx(bar, a.bslot_bytes);
        tma_load_3d(bits_addr + bslot * a.bslot_bytes, &tmBits, bar, p * 4, u.n0, u.tenant0);
    };
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&ctl->wfull[s]), 1);
            mbar_init(smem_u32(&ctl->wempty[s]), 1);
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_u32(&ctl->bfull[s]), 1);
            mbar_init(smem_u32(&ctl->bempty[s]), kSDecodeWarps);
            mbar_init(smem_u32(&ctl->pfull[s]), kSEpiWarps * 32);
            mbar_init(smem_u32(&ctl->pempty[s]), 1);
        }
        for (int s = 0; s < kStreamMaxSets; ++s) mbar_init(smem_u32(&ctl->opfree[s]), 1);
        mbar_init(smem_u32(&ctl->accfull), 1);
        mbar_init(smem_u32(&ctl->accempty), kSEpiWarps);
        mbar_init(smem_u32(&ctl->depready), 1);
        mbar_init(smem_u32(&ctl->tmemready), 1);
        ctl->abort_flag = 0;
        ctl->is_last = 0;
        fence_barrier_init();
        // The first step's sign words are requested right here: every cycle until the first load is queued
        // is added to the launch's latency.
        if (lo < hi && a.early_weights) {
            const int unit0 = (int)((unsigned)lo / (unsigned)a.P);
            const Unit u0 = unit_info(a, unit0);
            const int pfirst = a.whole_units ? 0 : lo - unit0 * a.P;
            issue_bits(u0, pfirst, 0);
            issue_w(u0, pfirst, 0);
        }
    }
    __syncthreads();
    if (warp == 0) {
        ST(1);
#ifdef BD_TRACE
        unsigned int smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        ST_VAL(4, smid);
#endif
    }
    // (a.trigger_early, experiments: let the kernel queued behind this one become resident right away)
    if (threadIdx.x == 0 && a.trigger_early) grid_launch_dependents();

    const uint32_t tmemready = smem_u32(&ctl->tmemready);

    if (warp == kSWarpProducer) {
        // ------------------------------------------------------------ weight producer
        // Walks the block's steps in order and queues each step's two loads (sign words, W_base tile) as soon as
        // their rings have a free place.  Weights are never written by another kernel, so this runs before the
        // grid dependency is resolved, as far as the rings allow.  Two operations per step and no more: the copy
        // engine's time is what bounds this kernel.
        ItemIter wi(it), bi(it);
        Ring wr{0, 0u, a.n_w}, br{0, 0u, a.n_bits};
        Unit uw{}, ub{};
        bool more_w = wi.next(), more_b = bi.next();
        if (!a.early_weights) {
            // (experiment: no weight loads before the grid dependency is resolved)
            (void)wait_bar(smem_u32(&ctl->depready), 0u, abort_flag, 21);
            if (more_w) { uw = unit_info(a, wi.unit); ub = uw; }
        } else if (more_w) {
            // the first step's loads were queued by thread 0 in the prologue
            wr.step();
            br.step();
            more_w = wi.next();
            more_b = bi.next();
            if (more_w) { uw = unit_info(a, wi.unit); ub = uw; }
        }
        long long t_idle = 0;
        int idle = 0;
        int n_w_queued = more_w || a.early_weights ? 1 : 0;   // W_base tiles queued so far (the prologue's included)
        bool dep_done = false;
        while (more_w || more_b) {
            bool did = false;
            if (more_b && warp_all(mbar_test_wait(smem_u32(&ctl->bempty[br.idx]), br.par ^ 1))) {
                if (elect_one()) issue_bits(ub, bi.p, br.idx);
                __syncwarp();
                br.step();
                more_b = bi.next();
                if (more_b && bi.first) ub = unit_info(a, bi.unit);
                did = true;
            }
            if (more_w && warp_all(mbar_test_wait(smem_u32(&ctl->wempty[wr.idx]), wr.par ^ 1))) {
                if (elect_one()) issue_w(uw, wi.p, wr.idx);
                __syncwarp();
                wr.step();
                if (++n_w_queued == a.trigger_step && lane == 0) grid_launch_dependents();
                more_w = wi.next();
                if (more_w && wi.first) uw = unit_info(a, wi.unit);
                did = true;
            }
            if (did) {
                idle = 0;
                continue;
            }
            // Nothing can advance.  Before the grid dependency is resolved that means the rings are full and stay
            // full (nothing is consumed before then): sleep in the hardware until it is, rather than poll next to
            // the running launch's warps.  Afterwards: a short suspended wait on a ring that blocks, then look again.
            if (!dep_done) {
                dep_done = warp_all(mbar_try_wait_hint(smem_u32(&ctl->depready), 0u, 20000u));
                continue;
            }
            if (more_b) (void)mbar_try_wait_hint(smem_u32(&ctl->bempty[br.idx]), br.par ^ 1, 64u);
            else (void)mbar_try_wait_hint(smem_u32(&ctl->wempty[wr.idx]), wr.par ^ 1, 64u);
            if (idle == 0) t_idle = clock64();
            if ((++idle & 255) == 0) {
                if (*abort_flag) break;
                if (clock64() - t_idle > kWaitLimitCycles) {
                    *abort_flag = 1;
                    if (atomicCAS(&g_device_status[0], 0u, kStatusTimeout) == 0u) g_device_status[1] = 2u;
                    break;
                }
            }
        }
        ST(5);
        // All of this block's loads are queued: a kernel queued behind this one with an early start may become
        // resident now (this block leaves it half of the multiprocessor) and fill its rings while this block works
        // through its last steps, its epilogue and its fix-up, when the copy engine and DRAM have nothing else to do.
        // (Not earlier: a block of a new grid arriving on the multiprocessor costs the running block several
        // microseconds in its first steps, measured with and without the newcomer's loads.)
        if (lane == 0 && !a.trigger_early && n_w_queued < a.trigger_step) grid_launch_dependents();
    } else if (warp == kSWarpMma) {
        // -------------------------------------------------------------- MMA issuer
        // Resolves the grid dependency, then allocates tensor memory (the blocks of the launch before this
        // one have released theirs by then), then issues every MMA of the block: per step eight base MMAs
        // (A = W_base atoms in shared memory) and, per operand set, two delta MMAs for each of its tenants
        // (A = decoded signs in tensor memory, B = that tenant's window of the piece tile).
        grid_dependency_wait();
        ST(2);
        named_bar_arrive(kSBarDep, kSThreads - 32);   // wakes the decode and epilogue warps
        if (lane == 0) mbar_arrive(smem_u32(&ctl->depready));   // ... and the producer
        tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
        tmem_relinquish();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tmemready);
        (void)wait_bar(tmemready, 0, abort_flag, 20);
        tc_fence_after();
        const uint32_t tmem_base = ctl->tmem_base;
        ST(3);
#ifdef BD_TRACE
        int st_step = 0, st_set = 0;
#endif

        const uint32_t idesc_base = io_f16 ? make_idesc_f16(kTileN, (uint32_t)a.Nb) : make_idesc_bf16(kTileN, (uint32_t)a.Nb);
        const uint32_t idesc_delta = make_idesc_e5m2(kTileN, (uint32_t)a.Nd);
        const uint64_t desc0 = make_smem_desc_sw128(0);
        const uint32_t x_atom16 = a.x_atom_bytes >> 4;
        const uint32_t ten_rows16 = (uint32_t)(kPieces * am) * 8u;   // rows per tenant x 128 B >> 4
        Ring wr{0, 0u, a.n_w}, pr{0, 0u, a.n_x8}, sr{0, 0u, a.n_sets};
        uint32_t accphase = 0;
        bool ok = true;
        while (ok && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            ok = warp_all(wait_bar(smem_u32(&ctl->accempty), accphase ^ 1, abort_flag, 3));
            if (!ok) break;
            tc_fence_after();
            for (int p = p0; p < p1 && ok; ++p) {
                const uint32_t first = (p > p0) ? 1u : 0u;   // 0: this step starts the accumulation
                // the step's activation tile and pieces (written by the splitter threads, which fence them)
                ok = warp_all(wait_bar(smem_u32(&ctl->pfull[pr.idx]), pr.par, abort_flag, 13));
                if (!ok) break;
#ifdef BD_TRACE
                if (st_step < 11) ST(9 + 2 * st_step);
#endif
                const uint64_t xdesc = desc0 + ((x_addr + pr.idx * a.x_tile_bytes) >> 4);
                const uint64_t x8desc = desc0 + ((x8_addr + pr.idx * a.x8_atom_bytes) >> 4);
                ok = warp_all(wait_bar(smem_u32(&ctl->wfull[wr.idx]), wr.par, abort_flag, 4));
                if (!ok) break;
#ifdef BD_TRACE
                if (st_step < 11) ST(8 + 2 * st_step);
#endif
                {
                    const uint64_t wdesc = desc0 + ((w_addr + wr.idx * (2 * kSAtomBytes)) >> 4);
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint32_t atom = kk >> 2, k16 = kk & 3;
                            umma_ss(tmem_base, wdesc + (atom * (kSAtomBytes >> 4) + k16 * 2), xdesc + (atom * x_atom16 + k16 * 2),
                                    idesc_base, (kk > 0) ? 1u : first);
                        }
                        tc_commit(smem_u32(&ctl->wempty[wr.idx]));
                    }
                    __syncwarp();
                    wr.step();
                }
                if (!ok) break;
#ifdef BD_TRACE
                ++st_step;
#endif
#pragma unroll
                for (int half = 0; half < 2; ++half, sr.step()) {
                    // The 256 decode threads arrive here once the set is filled (or when they give up
                    // after an abandoned wait, see the end of the decode role).
                    named_bar_sync(kSBarSet0 + sr.idx, kSHandover);
                    if (*abort_flag) { ok = false; break; }
                    tc_fence_after();
#ifdef BD_TRACE
                    if (st_set < 30) ST(30 + st_set);
                    ++st_set;
#endif
                    const uint32_t a_set = tmem_base + a.col_a + (uint32_t)sr.idx * kStreamSetCols;
                    if (elect_one()) {
                        const uint32_t acc = (half > 0) ? 1u : first;
                        for (int j = 0; j < u.nten; ++j) {
                            // tenant j's 16 columns: decode warp half j % kTenStride, its tenant j / kTenStride
                            const uint32_t a_j = a_set + (uint32_t)((j % kTenStride) * kWarpCols + (j / kTenStride) * 16);
                            const uint32_t d_tmem = tmem_base + a.col_delta + (uint32_t)(j * a.Nd);
                            const uint64_t xj = x8desc + (uint32_t)j * ten_rows16 + (uint32_t)(half * 4);
                            umma_ts_f8(d_tmem, a_j, xj, idesc_delta, acc);
                            umma_ts_f8(d_tmem, a_j + 8, xj + 2, idesc_delta, 1u);
                        }
                        tc_commit(smem_u32(&ctl->opfree[sr.idx]));
                    }
                    __syncwarp();
                }
                if (!ok) break;
                if (elect_one()) tc_commit(smem_u32(&ctl->pempty[pr.idx]));
                __syncwarp();
                pr.step();
            }
            if (!ok) break;
            if (elect_one()) tc_commit(smem_u32(&ctl->accfull));
            __syncwarp();
            accphase ^= 1;
        }
    } else if (warp < kSWarpEpi0) {
        // ------------------------------------------- sign decode -> tensor memory
        // Warp (h, quad) owns the 32 weight rows of lane quadrant `quad` and, of every group of four tenants,
        // the tenants 2h and 2h+1.  Per step it takes its tenants' sign words (128 k each) into registers,
        // hands the slot back, and fills its 32 columns of two operand sets per tenant group (64 k each).
        const int h = (warp - kSWarpDecode0) >> 2;
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        // (sleeps on a hardware barrier while the launch before this one is still running: a polling warp would
        // take issue slots from that launch's warps on the same multiprocessor)
        named_bar_sync(kSBarDep, kSThreads - 32);
        bool ok = wait_bar(tmemready, 0, abort_flag, 20);
        tc_fence_after();
        const uint32_t tmem_base = ctl->tmem_base;
        const uint32_t tbuf0 = tmem_base + ((uint32_t)(quad * 32) << 16) + a.col_a + (uint32_t)(h * kWarpCols);
        Ring br{0, 0u, a.n_bits}, sr{0, 0u, a.n_sets};
#ifdef BD_TRACE
        int st_step = 0, st_set = 0;
        long long acc_alu = 0, acc_wst = 0, acc_opf = 0, acc_st = 0, acc_bits = 0, acc_flush = 0, tc0 = clock64();
#endif
        while (ok && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            for (int p = p0; p < p1 && ok; ++p) {
#ifdef BD_TRACE
                if (warp == kSWarpDecode0 && st_step < 10) ST(140 + st_step);
#endif
                ok = wait_bar(smem_u32(&ctl->bfull[br.idx]), br.par, abort_flag, 6);
                if (!ok) break;
#ifdef BD_TRACE
                if (warp == kSWarpDecode0 && st_step < 10) ST(90 + st_step);
                ++st_step;
#endif
                // this warp's tenants j = kTenStride * i + h: their sign words of the step (128 k each), then the
                // slot goes back
                const uint8_t* bsl = smem + bits_off + br.idx * a.bslot_bytes + row * 16;
                uint4 wq[kTenPerWarp];
#pragma unroll
                for (int i = 0; i < kTenPerWarp; ++i) {
                    const int j = kTenStride * i + h;
                    wq[i] = (j < u.nten) ? *reinterpret_cast<const uint4*>(bsl + j * (kTileN * 16)) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int i = 0; i < kTenPerWarp; ++i) asm volatile("" : "+r"(wq[i].x), "+r"(wq[i].w));
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->bempty[br.idx]));
                br.step();
                // tenants of this warp present in the unit (pairs of them share a 32-column store)
                const int nmine = (u.nten > h) ? (u.nten - h + kTenStride - 1) / kTenStride : 0;
#ifdef BD_TRACE
                const long long tstep = clock64();
                acc_bits += tstep - tc0;
                tc0 = tstep;
#endif
                // Two sets per step (64 k each).  The stores of a set are left in flight while the next one is being
                // decoded: their completion is awaited, and the set handed over, just before the next set's first
                // stores (and after the step's last one).
                int pending = -1;
#pragma unroll
                for (int half = 0; half < 2; ++half, sr.step()) {
                    uint32_t r[32];
                    decode_word_e5m2(half ? wq[0].z : wq[0].x, r);
                    decode_word_e5m2(half ? wq[0].w : wq[0].y, r + 8);
                    decode_word_e5m2(half ? wq[1].z : wq[1].x, r + 16);
                    decode_word_e5m2(half ? wq[1].w : wq[1].y, r + 24);
                    // (keeps the decode arithmetic above the wait: the compiler would otherwise sink it to the store)
                    asm volatile("" : "+r"(r[0]), "+r"(r[7]), "+r"(r[8]), "+r"(r[15]), "+r"(r[16]), "+r"(r[23]), "+r"(r[24]), "+r"(r[31]));
                    ST_CLK(tc1);
                    if (pending >= 0) {
                        tc_wait_st();
                        tc_fence_before();
                        named_bar_arrive(kSBarSet0 + pending, kSHandover);
                    }
                    ST_CLK(tc2);
                    ok = wait_bar(smem_u32(&ctl->opfree[sr.idx]), sr.par ^ 1, abort_flag, 7);
                    if (!ok) break;
                    tc_fence_after();
                    ST_CLK(tc3);
#ifdef BD_TRACE
                    if (warp == kSWarpDecode0 && st_set < 30) ST(60 + st_set);
                    ++st_set;
#endif
                    const uint32_t tbuf = tbuf0 + (uint32_t)sr.idx * kStreamSetCols;
                    if (nmine >= 2) tmem_st32(tbuf, r);          // (warp-uniform)
                    else if (nmine == 1) tmem_st16(tbuf, r);
                    if constexpr (kTenPerWarp == 4) {
                        if (nmine >= 3) {
                            decode_word_e5m2(half ? wq[2].z : wq[2].x, r);
                            decode_word_e5m2(half ? wq[2].w : wq[2].y, r + 8);
                            decode_word_e5m2(half ? wq[3].z : wq[3].x, r + 16);
                            decode_word_e5m2(half ? wq[3].w : wq[3].y, r + 24);
                            if (nmine >= 4) tmem_st32(tbuf + 32, r);
                            else tmem_st16(tbuf + 32, r);
                        }
                    }
                    pending = sr.idx;
                    ST_CLK(tc4);
#ifdef BD_TRACE
                    acc_alu += tc1 - tc0; acc_wst += tc2 - tc1; acc_opf += tc3 - tc2; acc_st += tc4 - tc3;
                    tc0 = tc4;
#endif
                }
                if (ok && pending >= 0) {
                    tc_wait_st();
                    tc_fence_before();
                    named_bar_arrive(kSBarSet0 + pending, kSHandover);
                }
#ifdef BD_TRACE
                { const long long te = clock64(); acc_flush += te - tc0; tc0 = te; }
#endif
            }
        }
#ifdef BD_TRACE
        if (warp == kSWarpDecode0) {
            ST_VAL(111, acc_alu); ST_VAL(112, acc_wst); ST_VAL(113, acc_opf); ST_VAL(114, acc_st); ST_VAL(115, acc_bits);
            ST_VAL(116, acc_flush); ST_VAL(117, (unsigned long long)st_set);
        }
#endif
        if (*abort_flag) {
            // A wait was abandoned somewhere in the block.  The issuer may be blocked on one of the named
            // barriers (they have no time-out): arrive on all of them so that it wakes up, sees the flag
            // and leaves.
            __syncwarp();
            for (int s = 0; s < a.n_sets; ++s) named_bar_arrive(kSBarSet0 + s, kSHandover);
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const int etid = threadIdx.x - kSWarpEpi0 * 32;
        const int first_unit = (int)((unsigned)lo / (unsigned)a.P);
        uint16_t* Y = reinterpret_cast<uint16_t*>(a.Y);
        uint32_t accphase = 0;
        bool ok = true;
        // While a tile is being accumulated these four warps split every step's activations into e5m2 pieces
        // (one 8-element task per thread and token row), as soon as the step's activation tile has landed.
        // Each warp walks the steps on its own; pfull[slot] counts all 128 threads.  Steps of the current
        // tile are split with blocking waits (the tile cannot complete without them), later ones whenever
        // there is nothing else to do.
        named_bar_sync(kSBarDep, kSThreads - 32);   // nothing to do before the activations may be read; sleep until then
        grid_dependency_wait();                     // (returns at once: orders this thread's accesses behind the previous kernel's)
        ItemIter si(it);
        bool more_s = si.next();
        Ring pr{0, 0u, a.n_x8};
        int n_split = 0, seg_end = 0;
        Unit us{};
        if (more_s) us = unit_info(a, si.unit);
        auto split_next = [&](bool block) -> bool {
            const uint32_t bar8 = smem_u32(&ctl->pempty[pr.idx]);
            if (block) {
                if (!wait_bar(bar8, pr.par ^ 1, abort_flag, 14)) return false;
            } else if (!warp_all(mbar_test_wait(bar8, pr.par ^ 1))) {
                return false;
            }
            const uint16_t* xg = reinterpret_cast<const uint16_t*>(a.X) + (size_t)us.xrow0 * a.K + (size_t)si.p * kPairK;
            uint8_t* xt = smem + x_off + pr.idx * a.x_tile_bytes;
            uint8_t* x8t = smem + x8_off + pr.idx * a.x8_atom_bytes;
            if (kG == 2 && us.ntok > 8) {
                if (io_f16) split_from_global_wide<true>(a, am, xg, xt, x8t, us.ntok, etid, kSEpiWarps * 32);
                else split_from_global_wide<false>(a, am, xg, xt, x8t, us.ntok, etid, kSEpiWarps * 32);
            } else if (io_f16) split_from_global<true>(a, am, xg, xt, x8t, us.ntok, etid, kSEpiWarps * 32);
            else split_from_global<false>(a, am, xg, xt, x8t, us.ntok, etid, kSEpiWarps * 32);
            fence_proxy_async_smem();   // generic-proxy writes -> visible to the MMAs' async-proxy reads
            mbar_arrive(smem_u32(&ctl->pfull[pr.idx]));
            pr.step();
            ++n_split;
            more_s = si.next();
            if (more_s && si.first) us = unit_info(a, si.unit);
            return true;
        };
        uint32_t tmem_base = 0;
        bool have_tmem = false;
        int pend_unit[2], pend_c0[2], pend_c1[2], npend = 0;   // cut tiles this block has to finish
        while (ok && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            const int n = u.n0 + row;
            const bool whole = (p0 == 0 && p1 == a.P);
            // the tenants' scales, requested now so that their latency is not paid after the accumulators complete
            float alv[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) alv[j] = (j < u.nten) ? __ldg(a.alpha + u.tenant0 + j) : 0.f;
            float al_lane = 0.f, bias_n = 0.f;
            if constexpr (kGen) {
                al_lane = (lane < u.nten) ? __ldg(a.alpha + u.tenant0 + lane) : 0.f;   // lane l: tenant l's scale
                if (a.bias && n < a.N) bias_n = from_io16(__ldg(reinterpret_cast<const uint16_t*>(a.bias) + n), a.f16);
            }
            seg_end += p1 - p0;
            while (ok && n_split < seg_end) ok = split_next(true);
            if (!ok) break;
            // until this tile's accumulators are complete: split ahead whatever has landed
            while (more_s && !warp_all(mbar_test_wait(smem_u32(&ctl->accfull), accphase))) {
                if (!split_next(false)) break;
            }
            float* slotp = nullptr;
            if (!whole && a.cluster <= 1) {
                const int slot = (unit == first_unit) ? 2 * (int)blockIdx.x : 2 * (int)blockIdx.x + 1;
                slotp = a.partials + (size_t)slot * a.slot_floats;
            }
            ok = wait_bar(smem_u32(&ctl->accfull), accphase, abort_flag, 8);
            if (!ok) break;
            tc_fence_after();
            accphase ^= 1;
#ifdef BD_TRACE
            const int st_seg = (unit == first_unit) ? 0 : 1;
            if (warp == kSWarpEpi0) ST(100 + 3 * st_seg);
#endif
            if (!have_tmem) {
                (void)wait_bar(tmemready, 0, abort_flag, 20);   // long since complete: makes the base address visible
                tmem_base = ctl->tmem_base;
                have_tmem = true;
            }
            const uint32_t lane_taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
            if (a.cluster > 1) {
                // Cluster form: this block's partial sums go to its own shared memory (the W_base ring: every load
                // into it has landed and every MMA that read it has completed), token-major, one float per weight
                // row; the cluster's leader adds the blocks' partials up at the end of the kernel.
                const ClusterPartOut out{reinterpret_cast<float*>(smem) + row};
                if constexpr (kMode >= 1 && kMode <= 4) epilogue_decode<kMode, false>(a, u, lane_taddr, out, alv, al_lane);
                else epilogue_decode_any_m<false>(a, u, lane_taddr, out, alv, al_lane, am);
                break;   // (one segment per block)
            }
            auto drain = [&](auto gate) {
                constexpr bool kGate = decltype(gate)::value;
                const EpiOut<kGen, kGate> out{Y, slotp, a.N, n, row, u.xrow0, bias_n, a};
                if constexpr (kMode >= 1 && kMode <= 4) {
                    epilogue_decode<kMode, kGen>(a, u, lane_taddr, out, alv, al_lane);
                } else {
                    epilogue_decode_any_m<kGen>(a, u, lane_taddr, out, alv, al_lane, am);
                }
            };
            if constexpr (kGen) {
                if (a.act == 2) drain(std::true_type{});
                else drain(std::false_type{});
            } else {
                drain(std::false_type{});
            }
            // this warp's arrival on the "accumulators drained" barrier
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->accempty));
#ifdef BD_TRACE
            if (warp == kSWarpEpi0) ST(101 + 3 * st_seg);
#endif
            if (!whole) {
                // This tile is cut across blocks: publish the partial and count arrivals right away (the sooner every
                // block has arrived, the sooner the last one can finish the tile).  If this block is the last to
                // arrive it adds the partials up in block order and writes Y, but only after its other segments
                // have been drained and published: that sum is a chain of round trips to L2 and would hold up
                // the next segment's drain.
                const int first_item = unit * a.P;
                const int c0 = cta_of_item(a, first_item);
                const int c1 = cta_of_item(a, first_item + a.P - 1);
                epi_bar_sync(kSEpiWarps * 32);
                if (*abort_flag) break;
                if (etid == 0) {
                    // release: the partial stores of all epilogue threads (ordered before this by the barrier);
                    // acquire: the other blocks' partials, if this block turns out to be the last
                    unsigned old;
                    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(a.counters + unit) : "memory");
                    ctl->is_last = (old == (unsigned)(c1 - c0)) ? 1u : 0u;
                }
                epi_bar_sync(kSEpiWarps * 32);
                if (*abort_flag) break;
                if (ctl->is_last) {   // (rewritten only after the next segment's first barrier, which every thread passes after this read)
                    pend_unit[npend] = unit;
                    pend_c0[npend] = c0;
                    pend_c1[npend] = c1;
                    ++npend;
                }
            }
#ifdef BD_TRACE
            if (warp == kSWarpEpi0) ST(102 + 3 * st_seg);
#endif
            // the next tile's first steps
            while (more_s && split_next(false)) {
            }
        }
        // Tiles this block was the last to arrive at (at most its first and its last segment).
        for (int k = 0; k < npend && ok && !*abort_flag; ++k) {
            const int un = pend_unit[k], c0 = pend_c0[k], c1 = pend_c1[k];
            const Unit u = unit_info(a, un);
            const int first_item = un * a.P;
            // Block c0 holds the tile's first step; the tile is its first segment only if its range starts
            // exactly there.  Every later block starts inside the tile.
            const int slot0 = (cta_first_item(a, c0) == first_item) ? 2 * c0 : 2 * c0 + 1;
            const float* first = a.partials + (size_t)slot0 * a.slot_floats;
            const float* rest = a.partials + (size_t)(2 * (c0 + 1)) * a.slot_floats;
            if (kGen && a.act == 2) reduce_partials<kGen, kGen>(a, u, etid, kSEpiWarps, first, rest, 2 * (size_t)a.slot_floats, c1 - c0);
            else reduce_partials<kGen, false>(a, u, etid, kSEpiWarps, first, rest, 2 * (size_t)a.slot_floats, c1 - c0);
            if (etid == 0) a.counters[un] = 0u;
#ifdef BD_TRACE
            if (warp == kSWarpEpi0) ST(106 + k);
#endif
        }
        if (!ok) {
            // This warp left on an abandoned wait; a sibling that passed the same wait a moment earlier may be
            // waiting on the epilogue barrier: release it once (it then sees the flag and leaves too).
            __syncwarp();
            named_bar_arrive(1, kSEpiWarps * 32);
        }
    }

    // ------------------------------------------------------------------ teardown
    __syncthreads();
    if (warp == 0) ST(110);
    if (*abort_flag) {
        // A wait was abandoned: give copies and MMAs still in flight a bounded time to land before shared
        // and tensor memory are released.
        if (threadIdx.x == 0) {
            const long long t0 = clock64();
            while (clock64() - t0 < 4000000ll) {
            }
        }
        __syncthreads();
    }
    tc_fence_after();
    // (tensor memory goes back before the cluster barriers below: a block must never hold it while it waits for
    // another block, which might be waiting for tensor memory on the same multiprocessor)
    if (warp == kSWarpMma) tmem_dealloc(ctl->tmem_base, kTmemCols);
    if (a.cluster > 1) {
        // Cluster form: every block's partial sums are in its shared memory.  After a cluster barrier the leader's
        // epilogue threads (one weight row each) add them up in block order, i.e. in k order, read through the
        // distributed shared memory window, apply the fused epilogue and write Y; a second barrier keeps the
        // other blocks' shared memory alive until it has read them.
        if (warp == 0) ST(119);
        cluster_sync_all();
        if (warp == 0) ST(120);
        if (crank == 0 && warp >= kSWarpEpi0 && lo < hi && !*abort_flag) {
            const Unit u = unit_info(a, (int)blockIdx.x / a.cluster);
            const int row = (warp & 3) * 32 + lane;
            const int n = u.n0 + row;
            float bias_n = 0.f;
            if constexpr (kGen) {
                if (a.bias && n < a.N) bias_n = from_io16(__ldg(reinterpret_cast<const uint16_t*>(a.bias) + n), a.f16);
            }
            const uint32_t part = base + (uint32_t)row * 4u;   // this block's part[0][row]; same offset in every block
            uint32_t peer[8];
#pragma unroll
            for (int r = 1; r < 8; ++r) peer[r] = (r < a.cluster) ? mapa_shared(part, (uint32_t)r) : 0u;
            uint16_t* Yp = reinterpret_cast<uint16_t*>(a.Y);
            auto finish = [&](auto gate) {
                constexpr bool kGate = decltype(gate)::value;
                const EpiOut<kGen, kGate> out{Yp, nullptr, a.N, n, row, u.xrow0, bias_n, a};
                for (int tok = 0; tok < u.ntok; tok += 4) {   // (four tokens' remote loads in flight together)
                    float pv[4][8];
#pragma unroll
                    for (int q = 0; q < 4; ++q)
#pragma unroll
                        for (int r = 1; r < 8; ++r)
                            pv[q][r] = (r < a.cluster && tok + q < u.ntok) ? ld_shared_cluster_f32(peer[r] + (uint32_t)(tok + q) * (kTileN * 4u)) : 0.f;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (tok + q < u.ntok) {   // (warp-uniform)
                            float v = reinterpret_cast<const float*>(smem)[(tok + q) * kTileN + row];
#pragma unroll
                            for (int r = 1; r < 8; ++r) v += pv[q][r];
                            out.put(tok + q, v);
                        }
                    }
                }
            };
            if constexpr (kGen) {
                if (a.act == 2) finish(std::true_type{});
                else finish(std::false_type{});
            } else {
                finish(std::false_type{});
            }
        }
        if (warp == kSWarpEpi0) ST(121);
        cluster_sync_relaxed();   // (nothing to publish: the leader's stores to Y need not be waited for here)
    }
    if (warp == 0) ST(118);
}

#ifdef BD_TRACE
extern "C" int bitdelta_debug_set_trace(unsigned long long* buf) {
    return (int)cudaMemcpyToSymbol(g_stream_trace, &buf, sizeof(buf));
}
#endif

cudaError_t launch_gemm_stream(const CUtensorMap& tmW, const CUtensorMap& tmBits, const GemmArgs& args, int grid, uint32_t smem_bytes, bool early_start,
                               cudaStream_t stream) {
    const int gen = (args.f16 || args.act || args.bias != nullptr) ? 5 : 0;
    const int big = (smem_bytes > (uint32_t)kStreamSmemBudget) ? 10 : 0;   // one block per multiprocessor: the instantiation with the larger register budget
    const int mode = big + gen + (args.m <= 4 ? args.m : 5) - 1;
    using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const GemmArgs);
    static const KernelFn kernels[20] = {
        bitdelta_gemm_stream_kernel<1, false, 1>, bitdelta_gemm_stream_kernel<2, false, 1>, bitdelta_gemm_stream_kernel<3, false, 1>,
        bitdelta_gemm_stream_kernel<4, false, 1>, bitdelta_gemm_stream_kernel<5, false, 1>,
        bitdelta_gemm_stream_kernel<1, true, 1>,  bitdelta_gemm_stream_kernel<2, true, 1>,  bitdelta_gemm_stream_kernel<3, true, 1>,
        bitdelta_gemm_stream_kernel<4, true, 1>,  bitdelta_gemm_stream_kernel<5, true, 1>,
        bitdelta_gemm_stream_kernel<1, false, 2>, bitdelta_gemm_stream_kernel<2, false, 2>, bitdelta_gemm_stream_kernel<3, false, 2>,
        bitdelta_gemm_stream_kernel<4, false, 2>, bitdelta_gemm_stream_kernel<5, false, 2>,
        bitdelta_gemm_stream_kernel<1, true, 2>,  bitdelta_gemm_stream_kernel<2, true, 2>,  bitdelta_gemm_stream_kernel<3, true, 2>,
        bitdelta_gemm_stream_kernel<4, true, 2>,  bitdelta_gemm_stream_kernel<5, true, 2>};
    // Per device and instantiation, once: allow the dynamic shared memory and ask for the largest shared-memory
    // carve-out, so that two blocks (of consecutive launches) fit on one multiprocessor.
    static std::atomic<unsigned char> attr_done[64][20];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_done[dev][mode].load()) {
        e = cudaFuncSetAttribute(kernels[mode], cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kernels[mode], cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_done[dev][mode].store(1);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)stream_threads(big ? 2 : 1));
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int nattr = 0;
    if (early_start) {
        attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[nattr].val.programmaticStreamSerializationAllowed = 1;
        ++nattr;
    }
    if (args.cluster > 1) {
        attr[nattr].id = cudaLaunchAttributeClusterDimension;
        attr[nattr].val.clusterDim.x = (unsigned)args.cluster;
        attr[nattr].val.clusterDim.y = 1;
        attr[nattr].val.clusterDim.z = 1;
        ++nattr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = nattr;
    return cudaLaunchKernelEx(&cfg, kernels[mode], tmW, tmBits, args);
}

int stream_max_active_clusters(uint32_t smem_bytes, int cluster) {
    auto kernel = bitdelta_gemm_stream_kernel<1, false, 1>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess) return 0;
    (void)cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(cluster * 64));
    cfg.blockDim = dim3((unsigned)stream_threads(1));
    cfg.dynamicSmemBytes = smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

int stream_blocks_per_sm(uint32_t smem_bytes) {
    auto kernel = bitdelta_gemm_stream_kernel<1, false, 1>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess) return 0;
    (void)cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, stream_threads(1), smem_bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

cudaError_t read_stream_status(unsigned int out[2]) {
    cudaError_t e = cudaMemcpyFromSymbol(out, g_device_status, sizeof(unsigned int) * 2);
    if (e != cudaSuccess) return e;
    if (out[0] != 0) {
        unsigned int zero[2] = {0, 0};
        e = cudaMemcpyToSymbol(g_device_status, zero, sizeof(zero));
    }
    return e;
}

}  // namespace bd
