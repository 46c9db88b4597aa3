// BitDelta fused GEMM on tcgen05 tensor cores (sm_100a).
//
//   Y[b,t,n] = sum_k X[b,t,k] W[n,k] + alpha[b] sum_k X[b,t,k] S[b,n,k]
//
// The product is computed transposed: weight rows sit on the MMA's M side (128
// TMEM lanes), tokens on its N side.  Per 128-wide k step a CTA
//   * TMA-loads a W_base tile and an X tile into 128B-swizzled shared memory,
//   * TMA-loads the tile's sign words (32 bytes per weight row and tenant),
//   * decodes each tenant's signs into packed bf16 +-1 registers with integer
//     ops and stores them into TENSOR MEMORY as the A operand (no shared-memory
//     round trip for the 16x expanded weights),
//   * issues the base MMA (A = W tile from shared memory) into one accumulator
//     and one delta MMA per tenant (A = decoded signs from tensor memory) into a
//     second accumulator,
// and the epilogue forms base + alpha * delta in fp32, rounds once to bf16.
// Work is a flat list of (tile, k step) items cut evenly across a persistent
// grid; tiles cut across CTAs are summed through a workspace by the last CTA
// to arrive, in a fixed order.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include <atomic>
#include <type_traits>

#include "gemm_common.cuh"
#include "gemm_tc.h"
#include "ptx.cuh"

namespace bd {

constexpr int kThreads = 512;
constexpr int kWarpProducer = 0;
constexpr int kWarpMma = 1;
constexpr int kWarpTmem = 2;
constexpr int kWarpDelta0 = 2;     // decode schedule: warps 2..3 issue the delta MMAs of decode group 0 / 1
constexpr int kBarAFull0 = 2;      // named barriers 2..9 : decode group g, buffer b -> id 2 + g*4 + b
constexpr int kWarpDecode0 = 4;    // warps 4..11
constexpr int kWarpEpi0 = 12;      // warps 12..15

struct Ctl {
    uint64_t wfull[kMaxStages];        // W_base tile landed
    uint64_t wempty[kMaxStages];       // ... and was read by the base MMAs (tcgen05.commit)
    uint64_t xfull[kMaxStages];        // bf16 activation tile landed
    uint64_t xempty[kMaxStages];       // ... and was read by the base MMAs (and by the in-kernel split)
    uint64_t x8empty[kMaxStages];      // decode: piece tile free again (both delta issuers' MMAs completed)
    uint64_t bfull[kMaxBitSlots];
    uint64_t bempty[kMaxBitSlots];
    uint64_t afull[kMaxASlots];        // tiled schedule: decoded operand ready (decode warps -> MMA warp)
    uint64_t aempty[2 * kMaxASlots];   // operand buffer free again (tcgen05.commit); decode: [group][buffer]
    uint64_t accfull;
    uint64_t accempty;
    uint64_t x8full[kMaxStages];       // decode: the stage's e5m2 pieces are in place (128 splitter threads, or TMA)
    uint64_t depready;                 // the grid this launch depends on has completed (activations may be read)
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t is_last;
};
static_assert(sizeof(Ctl) <= kSmemCtrlBytes, "control block too large");


// kMode 0: tiled schedule; 1..4 and 8: decode schedule with m = kMode tokens per tenant; 5: decode schedule, any other m;
// 6: tiled schedule with several tenants per unit; 7: tiled schedule on CTA pairs.
// One instantiation per mode keeps each launched kernel's code small (the roles' loops then stay in the
// instruction caches) and turns the schedule switches into compile-time constants.
// kGen: the general form (binary16 I/O, bias, activation); false compiles the plain bf16 product alone, whose
// code is then exactly as short as it can be (the kernel's speed is sensitive to its length).
template <int kMode, bool kGen>
__global__ void __launch_bounds__(kThreads, 1)
bitdelta_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                        const __grid_constant__ CUtensorMap tmX8, const __grid_constant__ CUtensorMap tmBits,
                        const GemmArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t w_addr = base;                                        // ring of W_base tiles
    const uint32_t x_off = a.n_w * a.w_stage_bytes;                      // ring of bf16 activation tiles
    const uint32_t x_addr = base + x_off;
    const uint32_t x8_off = x_off + a.n_x * a.x_tile_bytes;              // ring of e5m2 piece tiles (decode)
    const uint32_t x8_addr = base + x8_off;
    const uint32_t bits_off = x8_off + a.n_x8 * a.x8_atom_bytes;         // sign-word slots
    const uint32_t bits_addr = base + bits_off;
    uint8_t* bits_ptr = smem + bits_off;
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + bits_off + a.n_bits * a.bslot_bytes);
    volatile uint32_t* abort_flag = &ctl->abort_flag;

    constexpr bool kGrouped = kMode == 6;   // tiled schedule with several tenants per unit (16 < m <= 64)
    constexpr bool kPair = kMode == 7;      // tiled schedule on CTA pairs (cluster of two, 256-row MMAs)
    constexpr bool kDec = (kMode >= 1 && kMode <= 5) || kMode == 8;
    // Pair schedule: this CTA's rank in its cluster (0 = leader, issues the MMAs), the leader's view of
    // the barriers both CTAs signal, and the work share of the CLUSTER.
    const uint32_t rank = kPair ? cluster_ctarank() : 0u;
    const int cta_id = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;   // index into the work split
    const int am = ((kMode >= 1 && kMode <= 4) || kMode == 8) ? kMode : a.m;
    const bool convert = kDec && a.convert != 0;
    const bool io_f16 = kGen && a.f16 != 0;
    auto unit_info = [&](const GemmArgs& aa, int un) { return unit_info_t<kDec, kGrouped, kPair>(aa, un, am, (int)rank); };
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // Tiled schedule: signs need few decode threads, the epilogue many -> warps 8..11 drain accumulators
    // instead of decoding.
    constexpr int epi_first_warp = kDec ? kWarpEpi0 : kWarpEpi0 - 4;
    constexpr int n_epi_warps = 16 - epi_first_warp;
    if (threadIdx.x == 32) {
        prefetch_tensormap(&tmW);
        prefetch_tensormap(&tmX);
        prefetch_tensormap(&tmBits);
        if (kDec) prefetch_tensormap(&tmX8);
    }

    // Work: either an even share of the flat item list, or (whole-unit order) units b, b+grid, ...
    const int lo = a.whole_units ? (int)blockIdx.x * a.P : cta_first_item(a, cta_id);
    const int hi = a.whole_units ? (int)a.T : cta_first_item(a, cta_id + 1);
    SegIter it{lo, hi, a.P, a.whole_units ? (int)gridDim.x : 0};
    int unit, p0, p1;

    // Queues the weight loads of one item: its W_base tile into `stage` of the W ring and, if `with_bits`,
    // the sign words of its k-pair into sign-word slot `bslot`.  One thread.
    auto issue_weights_raw = [&](const Unit& u, int p, int stage, int bslot, bool with_bits) {
        // W_base first: the stage's MMAs need it together with the activations, and the first sign-word
        // load of a tile is slow (it pulls whole 128-byte lines, i.e. the signs of 1024 k, out of DRAM).
        const uint32_t bar = smem_u32(&ctl->wfull[stage]);
        const uint32_t dst = w_addr + stage * a.w_stage_bytes;
        const int k0 = p * kPairK;
        if constexpr (kPair) {
            // Both CTAs' tiles of the stage (W_base and half an activation tile each) are counted on the
            // leader's barrier, which only the leader arms.
            if (rank == 0) mbar_arrive_expect_tx(bar, 2u * (a.w_stage_bytes + 2 * a.x_atom_bytes));
            tma_load_3d_pair(dst, &tmW, mapa_shared(bar, 0), 0, u.n0, k0 / kAtomK);
        } else {
            // tiled schedule: the stage's activation tile (same slot index, queued by the activation
            // stream) completes on this barrier too
            mbar_arrive_expect_tx(bar, a.w_stage_bytes + (kDec ? 0u : 2 * a.x_atom_bytes));
            tma_load_3d(dst, &tmW, bar, 0, u.n0, k0 / kAtomK);   // both 64-k atoms of the tile
        }
        if (with_bits) {
            const uint32_t bbar = smem_u32(&ctl->bfull[bslot]);
            mbar_arrive_expect_tx(bbar, a.bslot_bytes);
            tma_load_3d(bits_addr + bslot * a.bslot_bytes, &tmBits, bbar, (p >> 1) * 8, u.n0, u.tenant0);
        }
    };

    // One epilogue thread's share (tasks tid, tid + 128, ...) of the in-kernel activation split: bf16 tile
    // in slot `xs` of its ring -> piece tile in slot `x8s` of its ring.
    auto do_split = [&](int xs, int x8s, int ntok, int tid) {
        // (two instantiations, chosen here: a test of the I/O type inside the split's loops costs the plain
        // product measurable time)
        if (io_f16) split_activations<true>(a, am, smem + x_off + xs * a.x_tile_bytes, smem + x8_off + x8s * a.x8_atom_bytes, ntok, tid, 128);
        else split_activations<false>(a, am, smem + x_off + xs * a.x_tile_bytes, smem + x8_off + x8s * a.x8_atom_bytes, ntok, tid, 128);
        fence_proxy_async_smem();   // generic-proxy writes -> visible to the MMAs' async-proxy reads
        mbar_arrive(smem_u32(&ctl->x8full[x8s]));
        mbar_arrive(smem_u32(&ctl->xempty[xs]));   // this thread is done reading the bf16 tile
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&ctl->wfull[s]), 1);
            mbar_init(smem_u32(&ctl->wempty[s]), 1);
            mbar_init(smem_u32(&ctl->xfull[s]), 1);
            mbar_init(smem_u32(&ctl->xempty[s]), (kDec && convert) ? 129 : 1);   // base issuer (+ the splitter threads)
            mbar_init(smem_u32(&ctl->x8full[s]), (kDec && convert) ? 128 : 1);   // splitter threads, or one TMA load
            mbar_init(smem_u32(&ctl->x8empty[s]), 2);                            // the two delta issuers
        }
        for (int s = 0; s < kMaxBitSlots; ++s) {
            mbar_init(smem_u32(&ctl->bfull[s]), 1);
            mbar_init(smem_u32(&ctl->bempty[s]), kDec ? 8 : 4);
        }
        for (int s = 0; s < kMaxASlots; ++s) mbar_init(smem_u32(&ctl->afull[s]), kPair ? 8 : 4);   // (pair: both CTAs' decode warps)
        for (int s = 0; s < 2 * kMaxASlots; ++s) mbar_init(smem_u32(&ctl->aempty[s]), 1);
        mbar_init(smem_u32(&ctl->accfull), kDec ? 3 : 1);
        mbar_init(smem_u32(&ctl->accempty), kDec ? 4 : (kPair ? 16 : 8));
        mbar_init(smem_u32(&ctl->depready), 1);
        ctl->abort_flag = 0;
        ctl->is_last = 0;
        fence_barrier_init();
        // The first item's weights are requested right here, before the rest of the CTA is set up:
        // every cycle until the first load is queued is added to the launch's latency.
        // (pair schedule: not before the other CTA's barriers exist, i.e. after the cluster barrier below)
        if (!kPair && lo < hi) {
            const int unit0 = (int)((unsigned)lo / (unsigned)a.P);
            issue_weights_raw(unit_info(a, unit0), a.whole_units ? 0 : lo - unit0 * a.P, 0, 0, true);
        }
    }
    if (warp == kWarpTmem) {
        if constexpr (kPair) {
            tmem_alloc_pair(smem_u32(&ctl->tmem_base), kTmemCols);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (kPair) {
        cluster_sync_all();   // both CTAs' barriers are initialised and both hold their tensor memory
        if (threadIdx.x == 0 && lo < hi) {
            const int unit0 = (int)((unsigned)lo / (unsigned)a.P);
            issue_weights_raw(unit_info(a, unit0), lo - unit0 * a.P, 0, 0, true);
        }
    }
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    // A kernel queued behind this one with an early start may begin its own prologue and weight
    // prefetch as soon as SMs free up; it waits for this grid to finish before it touches anything
    // this grid reads or writes.
    if (threadIdx.x == 0) grid_launch_dependents();

    if (warp == kWarpProducer) {
        // ------------------------------------------------------------ TMA producer
        // The whole warp walks the loop (warp-uniform control flow); one elected lane issues.
        // Two independent streams over the same item list:
        //  * weights (W_base tile + sign words) never depend on the kernel queued before this one and
        //    run ahead as far as their rings allow;
        //  * activations wait for the grid dependency (warp 1 completes `depready`) and for a free slot
        //    of their own, shallower ring.
        // Neither stream may block the other, so the warp polls both rings and sleeps on a short
        // suspended wait when neither can advance.
        ItemIter wi(it), xi(it), pi(it);
        int stage = 0, xslot = 0, pslot = 0, bslot = 0;
        uint32_t phase = 0, xphase = 0, pphase = 0, bphase = 0;
        bool ok = true, dep_ok = false;
        bool hold = kDec && a.hold_prefetch != 0;
        Unit uw{}, ux{};
        bool more_w = wi.next();
        // (decode schedule, many token rows per unit: the activation tiles are queued by two of the otherwise
        // idle epilogue warps, so that this warp only serves the weight stream)
        bool more_x = (!kDec || convert) && xi.next();
        if (more_x) ux = unit_info(a, xi.unit);
        // e5m2 piece tiles written by the pre-pass kernel (decode schedule, many token rows per unit)
        bool more_p = false;
        Unit up{};
        if (more_p) up = unit_info(a, pi.unit);
        // Tiled schedule: the sign words are a stream of their own (one small load per k-pair and unit into a
        // deep ring), so that they run far ahead of the W_base tiles: the decode warps work several stages
        // ahead of the MMAs.  In the decode schedules they travel with the W_base stream.
        ItemIter bi(it);
        bool more_b = !kDec && bi.next();
        Unit ub{};
        auto next_pair = [&]() {   // to the next item that starts a k-pair of its segment
            do {
                more_b = bi.next();
            } while (more_b && !bi.first && (bi.p & 1));
            if (more_b && bi.first) ub = unit_info(a, bi.unit);
        };
        if (more_b) {
            ub = unit_info(a, bi.unit);
            next_pair();   // the first pair was queued in the prologue
        }
        if (more_w) {
            // queued by thread 0 in the prologue: W stage 0, sign-word slot 0
            bslot = 1; bphase = 0u;   // (at least two sign-word slots)
            stage = 1 % a.n_w; phase = (a.n_w == 1) ? 1u : 0u;
            uw = unit_info(a, wi.unit);
            more_w = wi.next();
            if (more_w && wi.first) uw = unit_info(a, wi.unit);
        }
        const uint32_t depbar = smem_u32(&ctl->depready);
        long long t_idle = 0;
        int idle = 0;
        while (more_w || more_x || more_p || more_b) {
            bool did = false;
            if (more_x) {
                if (!dep_ok) dep_ok = warp_all(mbar_test_wait(depbar, 0));
                const uint32_t xebar = kDec ? smem_u32(&ctl->xempty[xslot]) : smem_u32(&ctl->wempty[xslot]);
                if (dep_ok && warp_all(mbar_test_wait(xebar, xphase ^ 1))) {
                    if (elect_one()) {
                        const uint32_t bar = kDec ? smem_u32(&ctl->xfull[xslot]) : smem_u32(&ctl->wfull[xslot]);
                        const uint32_t dst = x_addr + xslot * a.x_tile_bytes;
                        const int k0 = xi.p * kPairK;
                        if constexpr (kPair) {
                            // this CTA's half of the token tile, counted on the leader's barrier
                            tma_load_3d_pair(dst, &tmX, mapa_shared(bar, 0), 0, ux.xrow0 + (int)rank * (a.tok_tile / 2), k0 / kAtomK);
                        } else {
                            if (kDec) mbar_arrive_expect_tx(bar, a.x_tile_bytes);
                            tma_load_3d(dst, &tmX, bar, 0, ux.xrow0, k0 / kAtomK);   // both 64-k atoms
                        }
                    }
                    __syncwarp();
                    if (++xslot == a.n_x) { xslot = 0; xphase ^= 1; }
                    more_x = xi.next();
                    if (more_x && xi.first) ux = unit_info(a, xi.unit);
                    did = true;
                }
            }
            if (more_p) {
                if (!dep_ok) dep_ok = warp_all(mbar_test_wait(depbar, 0));
                if (dep_ok && warp_all(mbar_test_wait(smem_u32(&ctl->x8empty[pslot]), pphase ^ 1))) {
                    if (elect_one()) {
                        const uint32_t bar = smem_u32(&ctl->x8full[pslot]);
                        mbar_arrive_expect_tx(bar, a.x8_atom_bytes);
                        tma_load_2d(x8_addr + pslot * a.x8_atom_bytes, &tmX8, bar, pi.p * kPairK, up.tenant0 * kPieces * am);
                    }
                    __syncwarp();
                    if (++pslot == a.n_x8) { pslot = 0; pphase ^= 1; }
                    more_p = pi.next();
                    if (more_p && pi.first) up = unit_info(a, pi.unit);
                    did = true;
                }
            }
            if (!kDec && more_b) {
                if (warp_all(mbar_test_wait(smem_u32(&ctl->bempty[bslot]), bphase ^ 1))) {
                    if (elect_one()) {
                        const uint32_t bbar = smem_u32(&ctl->bfull[bslot]);
                        mbar_arrive_expect_tx(bbar, a.bslot_bytes);
                        tma_load_3d(bits_addr + bslot * a.bslot_bytes, &tmBits, bbar, (bi.p >> 1) * 8, ub.n0, ub.tenant0);
                    }
                    __syncwarp();
                    if (++bslot == a.n_bits) { bslot = 0; bphase ^= 1; }
                    next_pair();
                    did = true;
                }
            }
            if (more_w && hold) {
                // The first sign-word load of a tile pulls whole 128-byte lines (the signs of 1024 k) out of
                // DRAM; until it has landed, further weight requests would only queue in front of it.
                hold = !warp_all(mbar_test_wait(smem_u32(&ctl->bfull[0]), 0));
            }
            if (more_w && !hold) {
                const bool need_slot = kDec && (wi.first || !(wi.p & 1));
                if ((!need_slot || warp_all(mbar_test_wait(smem_u32(&ctl->bempty[bslot]), bphase ^ 1))) &&
                    warp_all(mbar_test_wait(smem_u32(&ctl->wempty[stage]), phase ^ 1))) {
                    if (elect_one()) issue_weights_raw(uw, wi.p, stage, bslot, need_slot);
                    __syncwarp();
                    if (need_slot && ++bslot == a.n_bits) { bslot = 0; bphase ^= 1; }
                    if (++stage == a.n_w) { stage = 0; phase ^= 1; }
                    more_w = wi.next();
                    if (more_w && wi.first) uw = unit_info(a, wi.unit);
                    did = true;
                }
            }
            if (did) {
                idle = 0;
                continue;
            }
            // Nothing can advance: a short suspended wait (tens of ns) on one ring, then look at both again.
            if (more_w && hold) (void)mbar_try_wait_hint(smem_u32(&ctl->bfull[0]), 0u, 64u);
            else if (more_w) (void)mbar_try_wait_hint(smem_u32(&ctl->wempty[stage]), phase ^ 1, 64u);
            else if (more_b) (void)mbar_try_wait_hint(smem_u32(&ctl->bempty[bslot]), bphase ^ 1, 64u);
            else (void)mbar_try_wait_hint(dep_ok ? (kDec ? smem_u32(&ctl->xempty[xslot]) : smem_u32(&ctl->wempty[xslot])) : depbar,
                                          dep_ok ? (xphase ^ 1) : 0u, 64u);
            if (idle == 0) t_idle = clock64();
            if ((++idle & 255) == 0) {
                if (*abort_flag) { ok = false; break; }
                if (clock64() - t_idle > kWaitLimitCycles) {
                    *abort_flag = 1;
                    if (atomicCAS(&g_device_status[0], 0u, 7u) == 0u) g_device_status[1] = 2u;
                    ok = false;
                    break;
                }
            }
        }
        (void)ok;
    } else if (warp == kWarpMma) {
        // -------------------------------------------------------------- MMA issuer
        // Warp-uniform loop, one elected lane issues: descriptors and predicates then live in
        // uniform registers, which keeps the issue cost of a tcgen05.mma at its hardware floor.
        // Operand buffers in tensor memory are handed over as `items`:
        //   tiled schedule : one item = one tenant x 128 k of bf16 signs (64 columns, 8 MMAs of K=16)
        //   decode schedule: one item = all tenants of the unit x 64 k of e5m2 signs (16 columns per
        //                    tenant, 2 MMAs of K=32 per tenant)
        constexpr uint32_t kM = kPair ? 2 * kTileN : kTileN;   // MMA M: both CTAs' weight rows in the pair schedule
        const uint32_t idesc_base = io_f16 ? make_idesc_f16(kM, (uint32_t)a.Nb) : make_idesc_bf16(kM, (uint32_t)a.Nb);
        const uint32_t idesc_delta = kDec ? make_idesc_e5m2(kTileN, (uint32_t)a.Nd)
                                          : (io_f16 ? make_idesc_f16(kM, (uint32_t)a.Nd) : make_idesc_bf16(kM, (uint32_t)a.Nd));
        // Descriptor of a tile = descriptor of address 0 plus (address >> 4): addresses stay below
        // 256 KiB, so the sum never carries out of the 14-bit start-address field.
        const uint64_t desc0 = make_smem_desc_sw128(0);
        const uint32_t w_atom16 = a.w_atom_bytes >> 4, x_atom16 = a.x_atom_bytes >> 4;
        Ring ar{0, 0u, a.a_slots};   // operand buffers in tensor memory (tiled schedule)
        int stage = 0, xslot = 0;
        uint32_t phase = 0, xphase = 0, accphase = 0, item = 0;
        bool ok = true;
        // This warp also tells the producer when the grid this launch depends on has completed.
        grid_dependency_wait();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->depready));
        // (pair schedule: only the leader's warp issues; its MMAs and commits act on both CTAs)
        while (ok && (!kPair || rank == 0) && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            ok = warp_all(wait_bar(smem_u32(&ctl->accempty), accphase ^ 1, abort_flag, 3));
            if (!ok) break;
            tc_fence_after();
            for (int p = p0; p < p1 && ok; ++p) {
                {
                    ok = warp_all(wait_bar(smem_u32(&ctl->wfull[stage]), phase, abort_flag, 4));
                    if (kDec && ok) ok = warp_all(wait_bar(smem_u32(&ctl->xfull[xslot]), xphase, abort_flag, 12));
                    if (!ok) break;
                }
                const uint32_t wbase = w_addr + stage * a.w_stage_bytes;
                const uint32_t xbase = x_addr + xslot * a.x_tile_bytes;
                const uint64_t wdesc = desc0 + (wbase >> 4);
                const uint64_t xdesc = desc0 + (xbase >> 4);
                const uint32_t first = (p > p0) ? 1u : 0u;   // 0: this stage starts the accumulation
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t atom = kk >> 2, k16 = kk & 3;
                        if constexpr (kPair)
                            umma_ss_pair(tmem_base, wdesc + (atom * w_atom16 + k16 * 2), xdesc + (atom * x_atom16 + k16 * 2),
                                         idesc_base, (kk > 0) ? 1u : first);
                        else
                            umma_ss(tmem_base, wdesc + (atom * w_atom16 + k16 * 2), xdesc + (atom * x_atom16 + k16 * 2),
                                    idesc_base, (kk > 0) ? 1u : first);
                    }
                    // decode schedule: nothing else reads the W_base tile, hand it back as soon as these MMAs
                    // have completed
                    if (kDec) {
                        tc_commit(smem_u32(&ctl->wempty[stage]));
                        tc_commit(smem_u32(&ctl->xempty[xslot]));
                    }
                }
                __syncwarp();
                if constexpr (kDec) {
                    // Delta MMAs are issued by the two delta-issuer warps.
                } else {
                    for (int j = 0; j < u.nten && ok; ++j, ++item, ar.step()) {
                        const uint32_t slot = (uint32_t)ar.idx;
                        ok = warp_all(wait_bar(smem_u32(&ctl->afull[slot]), ar.par, abort_flag, 5));
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_base + a.col_delta + (uint32_t)(j * a.Nd);
                        const uint32_t a_tmem = tmem_base + a.col_a + slot * (uint32_t)a.aslot_cols;
                        const uint64_t xwdesc = xdesc + (uint32_t)(j * a.win_rows) * 8u;   // 128 B per row
                        if (elect_one()) {
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {
                                const uint32_t atom = kk >> 2, k16 = kk & 3;
                                if constexpr (kPair)
                                    umma_ts_pair(d_tmem, a_tmem + kk * 8, xwdesc + (atom * x_atom16 + k16 * 2), idesc_delta,
                                                 (kk > 0) ? 1u : first);
                                else
                                    umma_ts(d_tmem, a_tmem + kk * 8, xwdesc + (atom * x_atom16 + k16 * 2), idesc_delta,
                                            (kk > 0) ? 1u : first);
                            }
                            if constexpr (kPair) tc_commit_pair(smem_u32(&ctl->aempty[slot]), 3);
                            else tc_commit(smem_u32(&ctl->aempty[slot]));
                        }
                        __syncwarp();
                    }
                }
                if (!ok) break;
                if (!kDec) {
                    if (elect_one()) {
                        if constexpr (kPair) tc_commit_pair(smem_u32(&ctl->wempty[stage]), 3);
                        else tc_commit(smem_u32(&ctl->wempty[stage]));
                    }
                    __syncwarp();
                }
                if (++stage == a.n_w) { stage = 0; phase ^= 1; }
                if (++xslot == a.n_x) { xslot = 0; xphase ^= 1; }
            }
            if (!ok) break;
            if (elect_one()) {
                if constexpr (kPair) tc_commit_pair(smem_u32(&ctl->accfull), 3);
                else tc_commit(smem_u32(&ctl->accfull));
            }
            __syncwarp();
            accphase ^= 1;
        }
    } else if (warp >= kWarpDelta0 && warp < kWarpDelta0 + 2) {
        // ------------------------------------------------- delta issuers (decode schedule)
        // Warp 2+g serves decode group g (tenants j = g, g+2, ... of the unit).  Per 128-k stage it
        //  * waits for the stage's e5m2 piece tile, and
        //  * per 64-k half waits, on a named barrier, for the group's decode warps to have filled the
        //    operand buffer in tensor memory, issues that half's MMAs and commits the buffer's release.
        // Nothing else writes those tenants' accumulators, so their summation order is fixed.
        if constexpr (kDec) {
            const int g = warp - kWarpDelta0;
            const uint32_t idesc_delta = make_idesc_e5m2(kTileN, (uint32_t)a.Nd);
            const uint64_t desc0 = make_smem_desc_sw128(0);
            const uint32_t ten_rows16 = (uint32_t)(kPieces * am) * 8u;   // rows per tenant x 128 B >> 4
            Ring ar{0, 0u, a.a_slots};   // this group's operand buffers in tensor memory
            int xslot = 0;
            uint32_t xphase = 0, accphase = 0;
            bool ok = true;
            while (ok && it.next(unit, p0, p1)) {
                const Unit u = unit_info(a, unit);
                ok = warp_all(wait_bar(smem_u32(&ctl->accempty), accphase ^ 1, abort_flag, 3));
                if (!ok) break;
                tc_fence_after();
                for (int p = p0; p < p1 && ok; ++p) {
                    // the stage's e5m2 pieces: written by the epilogue warps (few token rows per unit) or loaded
                    // from the pre-pass kernel's output
                    ok = warp_all(wait_bar(smem_u32(&ctl->x8full[xslot]), xphase, abort_flag, 12));
                    if (!ok) break;
                    const uint64_t x8desc = desc0 + ((x8_addr + xslot * a.x8_atom_bytes) >> 4);
                    const uint32_t first = (p > p0) ? 1u : 0u;   // 0: this stage starts the accumulation
                    for (int half = 0; half < a.halves; ++half, ar.step()) {
                        const uint32_t slot = (uint32_t)ar.idx;
                        if (*abort_flag) { ok = false; break; }
                        // The group's 128 decode threads arrive here once the buffer is filled (or when they
                        // give up after an abandoned wait, see the end of the decode role).
                        named_bar_sync(kBarAFull0 + g * 4 + (int)slot, 160);
                        if (*abort_flag) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a_buf = tmem_base + a.col_a + (uint32_t)(g * a.a_slots + (int)slot) * (uint32_t)a.aslot_cols;
                        if (elect_one()) {
                            if (a.halves == 2) {
                                // 64 k per hand-over: two K=32 steps per tenant, 16 operand columns each
                                const uint32_t acc = (half > 0) ? 1u : first;
                                for (int j = g; j < u.nten; j += 2) {
                                    const uint32_t d_tmem = tmem_base + a.col_delta + (uint32_t)(j * a.Nd);
                                    const uint64_t xj = x8desc + (uint32_t)j * ten_rows16 + (uint32_t)(half * 4);
                                    const uint32_t a_j = a_buf + (uint32_t)(j >> 1) * 16;
                                    umma_ts_f8(d_tmem, a_j, xj, idesc_delta, acc);
                                    umma_ts_f8(d_tmem, a_j + 8, xj + 2, idesc_delta, 1u);
                                }
                            } else {
                                // the whole 128-k stage: four K=32 steps per tenant, 32 operand columns each
                                for (int j = g; j < u.nten; j += 2) {
                                    const uint32_t d_tmem = tmem_base + a.col_delta + (uint32_t)(j * a.Nd);
                                    const uint64_t xj = x8desc + (uint32_t)j * ten_rows16;
                                    const uint32_t a_j = a_buf + (uint32_t)(j >> 1) * 32;
                                    umma_ts_f8(d_tmem, a_j, xj, idesc_delta, first);
                                    umma_ts_f8(d_tmem, a_j + 8, xj + 2, idesc_delta, 1u);
                                    umma_ts_f8(d_tmem, a_j + 16, xj + 4, idesc_delta, 1u);
                                    umma_ts_f8(d_tmem, a_j + 24, xj + 6, idesc_delta, 1u);
                                }
                            }
                            tc_commit(smem_u32(&ctl->aempty[g * kMaxASlots + slot]));
                        }
                        __syncwarp();
                    }
                    if (!ok) break;
                    if (elect_one()) tc_commit(smem_u32(&ctl->x8empty[xslot]));
                    __syncwarp();
                    if (++xslot == a.n_x8) { xslot = 0; xphase ^= 1; }
                }
                if (!ok) break;
                if (elect_one()) tc_commit(smem_u32(&ctl->accfull));
                __syncwarp();
                accphase ^= 1;
            }
        }
    } else if (warp >= kWarpDecode0 && warp < epi_first_warp) {
        // ------------------------------------------- sign decode -> tensor memory
        const int dw = warp - kWarpDecode0;    // 0..7
        const int grp = dw >> 2;
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
        Ring ar{0, 0u, a.a_slots};   // this group's (tiled: the CTA's) operand buffers in tensor memory
        int bslot = 0;
        uint32_t bphase = 0, item = 0;
        bool ok = true;
        // shapes with a straight-line decode loop (two operand buffers per group in both)
        const uint32_t minus_one2 = io_f16 ? 0xBC00BC00u : 0xBF80BF80u;   // tiled schedule: packed (-1, -1) in the I/O type
        const bool fast8 = kDec && a.TB == 8 && a.halves == 2 && a.a_slots == 2;
        const bool fast4 = kDec && a.TB == 4 && a.halves == 1 && a.a_slots == 2;
        const uint32_t aempty_g = smem_u32(&ctl->aempty[grp * kMaxASlots]);
        const uint32_t tbuf_g = lane_taddr + a.col_a + (uint32_t)(grp * a.a_slots) * (uint32_t)a.aslot_cols;
        while (ok && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            for (int p = p0; p < p1 && ok; ++p) {
                if (p == p0 || !(p & 1)) {
                    ok = wait_bar(smem_u32(&ctl->bfull[bslot]), bphase, abort_flag, 6);
                    if (!ok) break;
                }
                const uint8_t* bsl = bits_ptr + bslot * a.bslot_bytes + (p & 1) * 16;
                if constexpr (kDec) {
                    // Warp (grp, quad) decodes, for its 32 rows, the tenants j = grp, grp+2, ... (64 k = two
                    // sign words each) into its group's ring of operand buffers, then arrives on the
                    // buffer's named barrier, on which the group's delta issuer waits.
                    //
                    // Full units of the two common shapes run as straight-line code: with two warps per
                    // scheduler nothing hides a warp's own bookkeeping, so every dependent instruction that
                    // is not decode work costs its full latency.
                    if (fast8 && u.nten == 8) {
                        // eight tenants, two 64-k hand-overs per stage into buffers 0 and 1 of the group
                        const uint8_t* src = bsl + (grp * kTileN + row) * 32;
                        uint4 wq[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) wq[i] = *reinterpret_cast<const uint4*>(src + i * (2 * kTileN * 32));
#pragma unroll
                        for (int half = 0; half < 2; ++half, ar.step()) {
                            ok = wait_bar(aempty_g + (uint32_t)ar.idx * 8, ar.par ^ 1, abort_flag, 7);
                            if (!ok) break;
                            tc_fence_after();
                            const uint32_t tbuf = tbuf_g + (uint32_t)ar.idx * (uint32_t)a.aslot_cols;
#pragma unroll
                            for (int i = 0; i < 4; i += 2) {
                                uint32_t r[32];
                                decode_word_e5m2(half ? wq[i].z : wq[i].x, r);
                                decode_word_e5m2(half ? wq[i].w : wq[i].y, r + 8);
                                decode_word_e5m2(half ? wq[i + 1].z : wq[i + 1].x, r + 16);
                                decode_word_e5m2(half ? wq[i + 1].w : wq[i + 1].y, r + 24);
                                tmem_st32(tbuf + (uint32_t)i * 16, r);
                            }
                            tc_wait_st();
                            tc_fence_before();
                            named_bar_arrive(kBarAFull0 + grp * 4 + ar.idx, 160);
                        }
                        item += 2;
                    } else if (fast4 && u.nten == 4) {
                        // four tenants, one 128-k hand-over per stage, buffers alternate
                        const uint8_t* src = bsl + (grp * kTileN + row) * 32;
                        uint4 wq[2];
                        wq[0] = *reinterpret_cast<const uint4*>(src);
                        wq[1] = *reinterpret_cast<const uint4*>(src + 2 * kTileN * 32);
                        const uint32_t slot = (uint32_t)ar.idx;
                        ok = wait_bar(aempty_g + slot * 8, ar.par ^ 1, abort_flag, 7);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t tbuf = tbuf_g + slot * (uint32_t)a.aslot_cols;
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            uint32_t r[32];
                            decode_word_e5m2(wq[i].x, r);
                            decode_word_e5m2(wq[i].y, r + 8);
                            decode_word_e5m2(wq[i].z, r + 16);
                            decode_word_e5m2(wq[i].w, r + 24);
                            tmem_st32(tbuf + (uint32_t)i * 32, r);
                        }
                        tc_wait_st();
                        tc_fence_before();
                        named_bar_arrive(kBarAFull0 + grp * 4 + (int)slot, 160);
                        item += 1;
                        ar.step();
                    } else
                    for (int half = 0; half < a.halves && ok; ++half, ++item, ar.step()) {
                        const uint32_t slot = (uint32_t)ar.idx;
                        ok = wait_bar(smem_u32(&ctl->aempty[grp * kMaxASlots + slot]), ar.par ^ 1, abort_flag, 7);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t tbuf = lane_taddr + a.col_a + (uint32_t)(grp * a.a_slots + (int)slot) * (uint32_t)a.aslot_cols;
                        if (a.halves == 1) {
                            // whole stage: four sign words (128 k) per tenant, 32 operand columns each
                            for (int j = grp; j < u.nten; j += 2) {
                                const uint4 w = *reinterpret_cast<const uint4*>(bsl + (j * kTileN + row) * 32);
                                uint32_t r[32];
                                decode_word_e5m2(w.x, r);
                                decode_word_e5m2(w.y, r + 8);
                                decode_word_e5m2(w.z, r + 16);
                                decode_word_e5m2(w.w, r + 24);
                                tmem_st32(tbuf + (uint32_t)(j >> 1) * 32, r);
                            }
                        } else {
                            // This warp's tenants are j = grp + 2*i, i < 4: fetch all their sign words first, so the
                            // shared-memory latency is paid once, then decode and store.
                            uint2 w[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int j = grp + 2 * i;
                                if (j < u.nten) w[i] = *reinterpret_cast<const uint2*>(bsl + (j * kTileN + row) * 32 + half * 8);
                            }
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int j = grp + 2 * i;
                                if (j < u.nten) {
                                    uint32_t r[16];
                                    decode_word_e5m2(w[i].x, r);
                                    decode_word_e5m2(w[i].y, r + 8);
                                    tmem_st16(tbuf + (uint32_t)i * 16, r);
                                }
                            }
                        }
                        tc_wait_st();
                        tc_fence_before();
                        named_bar_arrive(kBarAFull0 + grp * 4 + (int)slot, 160);
                    }
                } else {
                    for (int j = 0; j < u.nten && ok; ++j, ++item, ar.step()) {
                        const uint4 w = *reinterpret_cast<const uint4*>(bsl + (j * kTileN + row) * 32);
                        const uint32_t slot = (uint32_t)ar.idx;
                        ok = wait_bar(smem_u32(&ctl->aempty[slot]), ar.par ^ 1, abort_flag, 7);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t taddr = lane_taddr + a.col_a + slot * (uint32_t)a.aslot_cols;
                        uint32_t r[32];
                        decode_word(w.x, r, minus_one2);
                        decode_word(w.y, r + 16, minus_one2);
                        tmem_st32(taddr, r);
                        decode_word(w.z, r, minus_one2);
                        decode_word(w.w, r + 16, minus_one2);
                        tmem_st32(taddr + 32, r);
                        tc_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if (kPair && rank != 0) mbar_arrive_cluster(mapa_shared(smem_u32(&ctl->afull[slot]), 0));   // the leader's
                            else mbar_arrive(smem_u32(&ctl->afull[slot]));
                        }
                    }
                }
                if (!ok) break;
                if ((p & 1) || p == p1 - 1) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->bempty[bslot]));
                    if (++bslot == a.n_bits) { bslot = 0; bphase ^= 1; }
                }
            }
        }
        if (kDec && *abort_flag) {
            // A wait was abandoned somewhere in the CTA.  The group's delta issuer may be blocked on one
            // of the named barriers (they have no time-out): arrive on all of them so that it wakes up,
            // sees the abort flag and leaves.
            __syncwarp();
            for (int sl = 0; sl < a.a_slots; ++sl) named_bar_arrive(kBarAFull0 + grp * 4 + sl, 160);
        }
    } else if (warp >= epi_first_warp) {
        // ---------------------------------------------------------------- epilogue
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const int etid = threadIdx.x - epi_first_warp * 32;
        const int ehalf = (warp - epi_first_warp) >> 2;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const int first_unit = (int)((unsigned)lo / (unsigned)a.P);
        uint16_t* Y = reinterpret_cast<uint16_t*>(a.Y);
        uint32_t accphase = 0;
        bool ok = true;
        // Decode schedule with few token rows per unit: these four warps, idle while a tile is being
        // accumulated, also split every stage's activations into e5m2 pieces (one 16-element task per
        // thread), as soon as the stage's activation tile has landed.  Each warp walks the items on its
        // own; x8full[slot] counts all 128 threads.  Items of the current tile are split with blocking
        // waits (the tile cannot complete without them), later ones whenever there is nothing else to do.
        // With many token rows per unit there is nothing to split (a pre-pass kernel has written the
        // pieces), but the same walk lets epilogue warp 0 queue the bf16 activation tiles and warp 1 the
        // piece tiles, each into its own ring, instead of the producer warp.
        const int ew = warp - epi_first_warp;
        const bool splitter = kDec && (convert || ew < 2);
        ItemIter si(it);
        bool more_s = splitter && si.next();
        if (more_s && !convert) grid_dependency_wait();   // activations and pieces come from earlier kernels
        int sslot = 0, s8slot = 0, n_split = 0, seg_end = 0;
        uint32_t sphase = 0, s8phase = 0;
        Unit us{};
        if (more_s) us = unit_info(a, si.unit);
        auto split_next = [&](bool block) -> bool {
            if (!convert) {
                // queue one tile load: bf16 activations (warp 0) or pieces (warp 1), when its slot is free
                const uint32_t ebar = (ew == 0) ? smem_u32(&ctl->xempty[sslot]) : smem_u32(&ctl->x8empty[s8slot]);
                const uint32_t epar = ((ew == 0) ? sphase : s8phase) ^ 1;
                if (block) {
                    if (!warp_all(wait_bar(ebar, epar, abort_flag, 13))) return false;
                } else if (!warp_all(mbar_test_wait(ebar, epar))) {
                    return false;
                }
                if (elect_one()) {
                    if (ew == 0) {
                        const uint32_t bar = smem_u32(&ctl->xfull[sslot]);
                        mbar_arrive_expect_tx(bar, a.x_tile_bytes);
                        tma_load_3d(x_addr + sslot * a.x_tile_bytes, &tmX, bar, 0, us.xrow0, si.p * (kPairK / kAtomK));
                    } else {
                        const uint32_t bar = smem_u32(&ctl->x8full[s8slot]);
                        mbar_arrive_expect_tx(bar, a.x8_atom_bytes);
                        tma_load_2d(x8_addr + s8slot * a.x8_atom_bytes, &tmX8, bar, si.p * kPairK, us.tenant0 * kPieces * am);
                    }
                }
                __syncwarp();
                if (++sslot == a.n_x) { sslot = 0; sphase ^= 1; }
                if (++s8slot == a.n_x8) { s8slot = 0; s8phase ^= 1; }
                ++n_split;
                more_s = si.next();
                if (more_s && si.first) us = unit_info(a, si.unit);
                return true;
            }
            // needs the bf16 tile landed and a free piece tile
            const uint32_t bar = smem_u32(&ctl->xfull[sslot]);
            const uint32_t bar8 = smem_u32(&ctl->x8empty[s8slot]);
            if (block) {
                if (!wait_bar(bar, sphase, abort_flag, 13)) return false;
                if (!wait_bar(bar8, s8phase ^ 1, abort_flag, 14)) return false;
            } else if (!warp_all(mbar_test_wait(bar, sphase) && mbar_test_wait(bar8, s8phase ^ 1))) {
                return false;
            }
            do_split(sslot, s8slot, us.ntok, etid);
            if (++sslot == a.n_x) { sslot = 0; sphase ^= 1; }
            if (++s8slot == a.n_x8) { s8slot = 0; s8phase ^= 1; }
            ++n_split;
            more_s = si.next();
            if (more_s && si.first) us = unit_info(a, si.unit);
            return true;
        };
        while (ok && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            const int n = u.n0 + row;
            const bool whole = (p0 == 0 && p1 == a.P);
            // the tenants' scales, requested now so that their latency is not paid after the accumulators complete
            float alv[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) alv[j] = (j < u.nten) ? __ldg(a.alpha + u.tenant0 + j) : 0.f;
            float al_lane = 0.f, bias_n = 0.f;
            if constexpr (kGen || kGrouped) al_lane = (lane < u.nten) ? __ldg(a.alpha + u.tenant0 + lane) : 0.f;   // lane l: tenant l's scale
            if constexpr (kGen) {
                if (a.bias && n < a.N) bias_n = from_io16(__ldg(reinterpret_cast<const uint16_t*>(a.bias) + n), a.f16);
            }
            if (splitter) {
                seg_end += p1 - p0;
                while (ok && n_split < seg_end) ok = split_next(true);
                if (!ok) break;
                // until this tile's accumulators are complete: split ahead whatever has landed
                while (more_s && !warp_all(mbar_test_wait(smem_u32(&ctl->accfull), accphase))) {
                    if (!split_next(false)) break;
                }
            }
            float* slotp = nullptr;
            if (!whole) {
                const int slot = (unit == first_unit) ? 2 * (int)blockIdx.x : 2 * (int)blockIdx.x + 1;
                slotp = a.partials + (size_t)slot * a.slot_floats;
            }
            ok = wait_bar(smem_u32(&ctl->accfull), accphase, abort_flag, 8);
            if (!ok) break;
            tc_fence_after();
            accphase ^= 1;
            grid_dependency_wait();   // Y and the workspace may still be in use by the previous kernel
            // this warp's arrival on the "accumulators drained" barrier (pair schedule: the leader's)
            auto release_acc = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (kPair && rank != 0) mbar_arrive_cluster(mapa_shared(smem_u32(&ctl->accempty), 0));
                    else mbar_arrive(smem_u32(&ctl->accempty));
                }
            };
            // (the gated form of the general epilogue is separate code, chosen here once per tile)
            auto drain = [&](auto gate) {
                constexpr bool kGate = decltype(gate)::value;
                const EpiOut<kGen, kGate> out{Y, slotp, a.N, n, row, u.xrow0, bias_n, a};
                if constexpr ((kMode >= 1 && kMode <= 4) || kMode == 8) {
                    epilogue_decode<kMode, kGen>(a, u, lane_taddr, out, alv, al_lane);
                } else if constexpr (kMode == 5) {
                    switch (am) {
                        case 5: epilogue_decode<5, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 6: epilogue_decode<6, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 7: epilogue_decode<7, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 8: epilogue_decode<8, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 9: epilogue_decode<9, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 10: epilogue_decode<10, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 11: epilogue_decode<11, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 12: epilogue_decode<12, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 13: epilogue_decode<13, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 14: epilogue_decode<14, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        case 15: epilogue_decode<15, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                        default: epilogue_decode<16, kGen>(a, u, lane_taddr, out, alv, al_lane); break;
                    }
                } else {
                    if constexpr (kGrouped) epilogue_tiled_grouped(a, u, lane_taddr, am, out, ehalf, al_lane);
                    else epilogue_tiled(a, u, lane_taddr, out, ehalf, alv[0], release_acc);
                }
            };
            if constexpr (kGen) {
                if (a.act == 2) drain(std::true_type{});
                else drain(std::false_type{});
            } else {
                drain(std::false_type{});
            }
            if constexpr (kDec || kGrouped) release_acc();
            if (splitter) {
                // the next tile's first stages, before the (slow) fix-up of this one
                while (more_s && split_next(false)) {
                }
            }

            if (!whole) {
                // This tile is cut across CTAs: publish the partial, count arrivals, and let
                // the last CTA to arrive add the partials in CTA order and write Y.
                const int first_item = unit * a.P;
                const int c0 = cta_of_item(a, first_item);
                const int c1 = cta_of_item(a, first_item + a.P - 1);
                // All epilogue threads' partial stores, then one thread's fence (cumulative over what the
                // barrier ordered before it) and the arrival count.
                epi_bar_sync(n_epi_warps * 32);
                if (*abort_flag) break;   // (a sibling left on an abandoned wait and released this barrier once)
                if (etid == 0) {
                    __threadfence();
                    const unsigned old = atomicAdd(&a.counters[kPair ? 2 * unit + (int)rank : unit], 1u);
                    ctl->is_last = (old == (unsigned)(c1 - c0)) ? 1u : 0u;
                }
                epi_bar_sync(n_epi_warps * 32);
                if (*abort_flag) break;   // (a sibling left on an abandoned wait and released this barrier once)
                if (ctl->is_last) {
                    __threadfence();
                    // CTA c0 holds the tile's first item; the tile is its first segment only if its
                    // range starts exactly there.  Every later CTA starts inside the tile.
                    // (pair schedule: c0, c1 count clusters; this CTA adds up the slots of the CTAs of its own rank)
                    const int b0 = kPair ? 2 * c0 + (int)rank : c0;            // first contributing CTA
                    const int bstep = kPair ? 2 : 1;                           // CTAs from one contributor to the next
                    const int slot0 = (cta_first_item(a, c0) == first_item) ? 2 * b0 : 2 * b0 + 1;
                    const float* first = a.partials + (size_t)slot0 * a.slot_floats;
                    const float* rest = a.partials + (size_t)(2 * (b0 + bstep)) * a.slot_floats;
                    if (kGen && a.act == 2) reduce_partials<kGen, kGen>(a, u, etid, n_epi_warps, first, rest, 2 * (size_t)bstep * a.slot_floats, c1 - c0);
                    else reduce_partials<kGen, false>(a, u, etid, n_epi_warps, first, rest, 2 * (size_t)bstep * a.slot_floats, c1 - c0);
                    if (etid == 0) a.counters[kPair ? 2 * unit + (int)rank : unit] = 0u;
                }
                epi_bar_sync(n_epi_warps * 32);   // is_last is rewritten by the next cut tile
                if (*abort_flag) break;   // (a sibling left on an abandoned wait and released this barrier once)
            }
        }
        if (!ok) {
            // This warp left on an abandoned wait; a sibling that passed the same wait a moment earlier may be
            // waiting on the epilogue barrier (which has no time-out): release it once.  It then sees the abort
            // flag and leaves too.
            __syncwarp();
            named_bar_arrive(1, n_epi_warps * 32);
        }
    }

    // ------------------------------------------------------------------ teardown
    __syncthreads();
    if (*abort_flag) {
        // A wait was abandoned: give copies and MMAs still in flight a bounded time to land
        // before shared and tensor memory are released.
        if (threadIdx.x == 0) {
            const long long t0 = clock64();
            while (clock64() - t0 < 4000000ll) {
            }
        }
        __syncthreads();
    }
    tc_fence_after();
    if constexpr (kPair) cluster_sync_all();   // neither CTA's shared or tensor memory goes while the other may still signal it
    if (warp == kWarpTmem) {
        if constexpr (kPair) tmem_dealloc_pair(tmem_base, kTmemCols);
        else tmem_dealloc(tmem_base, kTmemCols);
    }
}


cudaError_t launch_gemm_tc(const CUtensorMap& tmW, const CUtensorMap& tmX, const CUtensorMap& tmX8,
                           const CUtensorMap& tmBits, const GemmArgs& args, int grid, uint32_t smem_bytes,
                           bool early_start, cudaStream_t stream) {
    // the general form only where something beyond the plain bf16 product is asked for
    const int gen = (args.f16 || args.act || args.bias != nullptr) ? 9 : 0;
    // 0 tiled, 1..4 and 8 decode with that many tokens per tenant, 5 decode with any other number up to 16, 6 tiled with
    // several tenants per unit, 7 tiled on CTA pairs
    const int mode = gen + (!args.decode ? (args.pair ? 7 : (args.win_rows > 0 ? 6 : 0)) : (args.m <= 4 ? args.m : (args.m == 8 ? 8 : 5)));
    using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const GemmArgs);
    static const KernelFn kernels[18] = {
        bitdelta_gemm_tc_kernel<0, false>, bitdelta_gemm_tc_kernel<1, false>, bitdelta_gemm_tc_kernel<2, false>,
        bitdelta_gemm_tc_kernel<3, false>, bitdelta_gemm_tc_kernel<4, false>, bitdelta_gemm_tc_kernel<5, false>,
        bitdelta_gemm_tc_kernel<6, false>, bitdelta_gemm_tc_kernel<7, false>, bitdelta_gemm_tc_kernel<8, false>,
        bitdelta_gemm_tc_kernel<0, true>,  bitdelta_gemm_tc_kernel<1, true>,  bitdelta_gemm_tc_kernel<2, true>,
        bitdelta_gemm_tc_kernel<3, true>,  bitdelta_gemm_tc_kernel<4, true>,  bitdelta_gemm_tc_kernel<5, true>,
        bitdelta_gemm_tc_kernel<6, true>,  bitdelta_gemm_tc_kernel<7, true>,  bitdelta_gemm_tc_kernel<8, true>};
    // (per device and instantiation, once; setting it twice from two threads is harmless)
    static std::atomic<unsigned char> attr_done[64][18];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_done[dev][mode].load()) {
        e = cudaFuncSetAttribute(kernels[mode], cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        if (e != cudaSuccess) return e;
        attr_done[dev][mode].store(1);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int nattr = 0;
    if (early_start) {
        attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[nattr].val.programmaticStreamSerializationAllowed = 1;
        ++nattr;
    }
    if (args.pair) {   // clusters of two CTAs
        attr[nattr].id = cudaLaunchAttributeClusterDimension;
        attr[nattr].val.clusterDim.x = 2;
        attr[nattr].val.clusterDim.y = 1;
        attr[nattr].val.clusterDim.z = 1;
        ++nattr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = nattr;
    return cudaLaunchKernelEx(&cfg, kernels[mode], tmW, tmX, tmX8, tmBits, args);
}

int max_active_pairs(uint32_t smem_bytes) {
    auto kernel = bitdelta_gemm_tc_kernel<7, false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * kMaxCtas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
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

// Self-test of the time-out path: one warp waits, with the kernels' own bounded wait, on an mbarrier nobody
// arrives on; the wait gives up after `limit_cycles`, records {time-out, site} in the status word and the
// kernel returns normally.  No tensor memory, no named or cluster barriers, nothing else in flight.
__global__ void __launch_bounds__(32, 1) selftest_timeout_kernel(long long limit_cycles, int site) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncwarp();
    (void)wait_bar_limited(smem_u32(&bar), 0u, &abort_flag, site, limit_cycles);
}

cudaError_t launch_selftest_timeout(long long limit_cycles, int site, cudaStream_t stream) {
    selftest_timeout_kernel<<<1, 32, 0, stream>>>(limit_cycles, site);
    return cudaGetLastError();
}

cudaError_t read_device_status(unsigned int out[2], cudaStream_t stream) {
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return e;
    e = cudaMemcpyFromSymbol(out, g_device_status, sizeof(unsigned int) * 2);
    if (e != cudaSuccess) return e;
    if (out[0] != 0) {
        unsigned int zero[2] = {0, 0};
        e = cudaMemcpyToSymbol(g_device_status, zero, sizeof(zero));
        if (e != cudaSuccess) return e;
    }
    // the other translation units' copies of the status word (all are read, so that all are cleared);
    // a time-out is reported in preference to a range flag
    unsigned int other[2][2] = {{0, 0}, {0, 0}};
    e = read_simple_status(other[0]);
    if (e != cudaSuccess) return e;
    e = read_fp4_status(other[1]);
    if (e != cudaSuccess) return e;
    for (int i = 0; i < 2; ++i) {
        if (other[i][0] != 0 && (out[0] == 0 || (out[0] != kStatusTimeout && other[i][0] == kStatusTimeout))) {
            out[0] = other[i][0];
            out[1] = other[i][1];
        }
    }
    return e;
}

}  // namespace bd
