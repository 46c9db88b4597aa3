// Device-side helpers shared by the tcgen05 BitDelta GEMM kernels (the tiled / grouped schedules in
// gemm_tc.cu and the 4-bit decode kernel in gemm_fp4.cu): bounded mbarrier waits, the walk over a
// thread block's share of the work list, sign decode, the fused epilogues, the split-K fix-up and the
// in-kernel activation split.  Every translation unit that includes this file gets its own copy of the
// device status word; read_device_status() looks at all of them.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "gemm_tc.h"
#include "ptx.cuh"

namespace bd {

constexpr long long kWaitLimitCycles = 4000000000ll;   // every spin gives up after 4e9 SM cycles (~2 s)

static __device__ unsigned int g_device_status[2];   // [0] status code (0 = ok), [1] site of the first failure
constexpr unsigned int kStatusTimeout = 7u;   // BITDELTA_ERR_TIMEOUT: a bounded wait expired ([1] = which one)
constexpr unsigned int kStatusRange = 9u;     // BITDELTA_ERR_RANGE: an activation beyond the decode schedules' range

// Bounded wait on an mbarrier phase.  Returns false if the wait was abandoned
// (limit reached here or in another thread of the CTA).  The slow path is kept out of line: it is
// instantiated at some twenty call sites and would otherwise dominate the kernel's code size.
static __device__ __noinline__ bool wait_bar_limited(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, int site,
                                                     long long limit_cycles) {
    // Poll, and every 64 polls look at the abort flag and the SM cycle counter
    // (cheap to read; the default limit is ~2 s at 2 GHz, longer at lower clocks).
    const long long t0 = clock64();
#pragma unroll 1
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i) {
            if (mbar_try_wait(bar, parity)) return true;
        }
        if (*abort_flag) return false;
        if (clock64() - t0 > limit_cycles) {
            *abort_flag = 1;
            if (atomicCAS(&g_device_status[0], 0u, kStatusTimeout) == 0u) g_device_status[1] = (unsigned)site;
            return false;
        }
    }
}
static __device__ __noinline__ bool wait_bar_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, int site) {
    return wait_bar_limited(bar, parity, abort_flag, site, kWaitLimitCycles);
}
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, int site) {
    if (mbar_try_wait(bar, parity)) return true;
    return wait_bar_slow(bar, parity, abort_flag, site);
}

// Walks the k-pair items [lo, hi) of this CTA as segments (unit, p0, p1).
struct SegIter {
    int cur, hi;
    int P;
    int stride;   // 0: the CTA owns the items [cur, hi); > 0: whole units cur/P, cur/P + stride, ... (see plan.h)
    __device__ __forceinline__ bool next(int& unit, int& p0, int& p1) {
        if (cur >= hi) return false;
        unit = (int)((unsigned)cur / (unsigned)P);
        if (stride > 0) {
            p0 = 0;
            p1 = P;
            cur += stride * P;
            return true;
        }
        p0 = cur - unit * P;
        const int rem = hi - cur;
        const int len = (rem < P - p0) ? rem : (P - p0);
        p1 = p0 + len;
        cur += len;
        return true;
    }
};

// The same walk, one (unit, k-pair) item at a time.
struct ItemIter {
    SegIter seg;
    int unit, p, p1;
    bool first;   // first item of its segment
    __device__ __forceinline__ explicit ItemIter(const SegIter& s) : seg(s), unit(0), p(0), p1(0), first(false) {}
    __device__ __forceinline__ bool next() {
        if (p + 1 < p1) { ++p; first = false; return true; }
        int p0;
        if (!seg.next(unit, p0, p1)) { p = 0; p1 = 0; return false; }
        p = p0;
        first = true;
        return true;
    }
};

// Cursor over a ring of n buffers: index of the current buffer and the parity of its use count.
struct Ring {
    int idx;
    uint32_t par;
    int n;
    __device__ __forceinline__ void step() {
        if (++idx == n) { idx = 0; par ^= 1; }
    }
};

struct Unit {
    int n0;        // first weight row of the tile
    int tenant0;   // first tenant
    int nten;      // tenants in this unit
    int xrow0;     // first row of X (in the [B*m, K] view) staged for this unit
    int ntok;      // output tokens of this unit (rows xrow0 .. xrow0+ntok-1)
};

template <bool kDec, bool kGrouped, bool kPair = false>
__device__ __forceinline__ Unit unit_info_t(const GemmArgs& a, int unit, int am, int rank = 0) {
    Unit u;
    int nt, g;
    if ((kDec || kGrouped) && a.teams > 1) {   // group-major (never in the one-tenant tiled schedule)
        g = (int)((unsigned)unit / (unsigned)a.n_tiles);
        nt = unit - g * a.n_tiles;
    } else {
        nt = unit / a.groups;
        g = unit - nt * a.groups;
    }
    if constexpr (kPair) nt = 2 * nt + rank;   // the pair's two W_base tiles
    u.n0 = nt * kTileN;
    if constexpr (kDec || kGrouped) {   // decode schedules, and the tiled schedule with several tenants per unit
        u.tenant0 = g * a.TB;
        u.nten = min(a.TB, a.B - u.tenant0);
        u.xrow0 = u.tenant0 * am;
        u.ntok = u.nten * am;
    } else {
        const int b = g / a.m_tiles;
        const int mt = g - b * a.m_tiles;
        u.tenant0 = b;
        u.nten = 1;
        u.xrow0 = b * am + mt * a.tok_tile;
        u.ntok = min(a.tok_tile, am - mt * a.tok_tile);
    }
    return u;
}

// 32 packed sign bits (k = 0..31 of the word, LSB first) -> 16 registers of two
// bf16 each, register c = {k = 2c (low half), k = 2c+1 (high half)}, +1 for a
// set bit and -1 for a clear bit.  Only shifts and three-input logic ops: the
// wanted bits are moved onto the two bf16 sign positions and flip the sign of a
// packed (-1, -1) constant (`minus_one2`: 0xBF80BF80 as bf16, 0xBC00BC00 as binary16).
__device__ __forceinline__ void decode_word(uint32_t w, uint32_t* r, uint32_t minus_one2) {
    // even bits of the low half stay at 2c, odd bits move to 2c+16 (junk only on odd positions)
    const uint32_t lo = (w & 0x0000FFFFu) | ((w << 15) & 0xFFFF0000u);
    const uint32_t hi = (w >> 16) | ((w >> 1) & 0xFFFF0000u);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        r[c] = ((lo << (15 - 2 * c)) & 0x80008000u) ^ minus_one2;
        r[8 + c] = ((hi << (15 - 2 * c)) & 0x80008000u) ^ minus_one2;
    }
}

// ------------------------------------------------------------------- epilogue helpers
template <int W>
__device__ __forceinline__ void tmem_ld_w(uint32_t taddr, uint32_t* r) {
    if constexpr (W == 1) tmem_ld1(taddr, r);
    else if constexpr (W == 2) tmem_ld2(taddr, r);
    else if constexpr (W == 4) tmem_ld4(taddr, r);
    else if constexpr (W == 8) tmem_ld8(taddr, r);
    else tmem_ld16(taddr, r);
}

// Fused epilogue on a finished sum: bias, then the activation, then rounding to the I/O type.
__device__ __forceinline__ float epi_finish(float v, float bias, int act) {
    v += bias;
    if (act == 1) v = __fdividef(v, 1.f + __expf(-v));   // SiLU; approximate division (2 ulp) keeps the unrolled epilogues small
    return v;
}
__device__ __forceinline__ uint16_t to_io16(float v, int f16) {
    return f16 ? __half_as_ushort(__float2half_rn(v)) : __bfloat16_as_ushort(__float2bfloat16_rn(v));
}
__device__ __forceinline__ uint16_t finish_io16(float v, float bias, int act, int f16) {
    return to_io16(epi_finish(v, bias, act), f16);
}
__device__ __forceinline__ float from_io16(uint16_t h, int f16) {
    return f16 ? __half2float(__ushort_as_half(h)) : __uint_as_float((uint32_t)h << 16);
}

// kGen = false: bf16 output, no bias, no activation (the plain product).  The two forms are separate code
// on purpose: the epilogue runs once per tile, every instruction of it is fetched cold, and the plain
// product should not pay for the general form's length.
template <bool kGen, bool kGate = false>
struct EpiOut {
    uint16_t* Y;        // output matrix [B*m, N], 16-bit values of the I/O type
    float* slot;        // partial-result slot, or nullptr when this CTA owns the whole tile
    int N, n, row, xrow0;
    float bias;         // of output feature n (0 without a bias)
    const GemmArgs& a;  // kernel parameters (activation code, I/O type)
    // (called by all lanes of a warp together: the gated form exchanges values between neighbouring lanes)
    __device__ __forceinline__ void put(int tok, float v) const {
        if (slot) {
            slot[(size_t)tok * kTileN + row] = v;   // partial sums: finished by the CTA that adds them up
            return;
        }
        if constexpr (kGate) {
            // SiLU gate: weight rows come in pairs (2i: gate, 2i+1: up), i.e. in neighbouring lanes
            const float z = v + bias;
            const float other = __shfl_xor_sync(0xFFFFFFFFu, z, 1);
            if (!(n & 1) && n < N)
                Y[(size_t)(xrow0 + tok) * (N >> 1) + (n >> 1)] = to_io16(__fdividef(z, 1.f + __expf(-z)) * other, a.f16);
            return;
        }
        if (n < N) {
            if constexpr (kGen) Y[(size_t)(xrow0 + tok) * N + n] = finish_io16(v, bias, a.act, a.f16);
            else Y[(size_t)(xrow0 + tok) * N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
        }
    }
};

// Decode schedule, M tokens per tenant: the base accumulator holds tenant j's tokens in columns
// j*M .. j*M+M-1; its delta accumulator starts at column N3*j and holds, for piece q of the
// activation split, token t in column q*M + t.  delta = D0 + D1 + D2 + D3.
// Plain product: the tenant loop is unrolled (the tensor-memory loads of all tenants overlap).  General form
// with more than four tokens per tenant: a real loop, because its body is long, this code runs once per tile
// and every instruction of it is fetched cold, so its length is paid in time.
// `alv[j]`: tenant j's scale (unrolled form); `al_lane`: lane l holds tenant l's scale (loop form).
template <int M, bool kGen, class Out>
__device__ __forceinline__ void epilogue_decode(const GemmArgs& a, const Unit& u, uint32_t lane_taddr,
                                                const Out& out, const float* alv, float al_lane) {
    constexpr int N3 = (kPieces * M + 15) / 16 * 16;
    constexpr int TPB = (N3 == 16) ? 2 : 1;   // tenants drained per wait
    constexpr int kMaxTen = (M <= 4) ? 8 : 4;   // tenants per unit (see the plan)
    constexpr bool kLoop = kGen && M > 4;
    auto drain = [&](int j0) {
        uint32_t rb[16], rd[TPB * N3];
        tmem_ld16(lane_taddr + (uint32_t)(j0 * M), rb);
#pragma unroll
        for (int jj = 0; jj < TPB; ++jj) {
#pragma unroll
            for (int c = 0; c < N3; c += 16)
                tmem_ld16(lane_taddr + a.col_delta + (uint32_t)((j0 + jj) * N3 + c), rd + jj * N3 + c);
        }
        tc_wait_ld();
#pragma unroll
        for (int jj = 0; jj < TPB; ++jj) {
            if (j0 + jj < u.nten) {   // warp-uniform
                float al;
                if constexpr (kLoop) al = __shfl_sync(0xFFFFFFFFu, al_lane, j0 + jj);
                else al = alv[j0 + jj];
#pragma unroll
                for (int t = 0; t < M; ++t) {
                    const float lo = __uint_as_float(rd[jj * N3 + 2 * M + t]) + __uint_as_float(rd[jj * N3 + 3 * M + t]);
                    const float hi = __uint_as_float(rd[jj * N3 + t]) + __uint_as_float(rd[jj * N3 + M + t]);
                    out.put((j0 + jj) * M + t, fmaf(al, hi + lo, __uint_as_float(rb[jj * M + t])));
                }
            }
        }
    };
    if constexpr (kLoop) {
#pragma unroll 1
        for (int j0 = 0; j0 < u.nten; j0 += TPB) drain(j0);
    } else {
#pragma unroll
        for (int j0 = 0; j0 < kMaxTen; j0 += TPB) {
            if (j0 >= u.nten) break;
            drain(j0);
        }
    }
}

// Tiled schedule: one tenant, tokens in columns 0..ntok-1 of both accumulators.
// Two warps share each lane quadrant: warp half h drains the 32-token blocks h, h+2, ...
// `release` hands the accumulators back (this warp's arrival): it is called as soon as the warp's last
// tensor-memory load has completed, before the values of that load are finished and stored.
template <class Out, class Release>
__device__ __forceinline__ void epilogue_tiled(const GemmArgs& a, const Unit& u, uint32_t lane_taddr,
                                               const Out& out, int half, float al, const Release& release) {
    if (32 * half >= u.ntok) release();
    for (int t0 = 32 * half; t0 < u.ntok; t0 += 64) {
        uint32_t rb[32], rd[32];
        tmem_ld32(lane_taddr + (uint32_t)t0, rb);
        tmem_ld32(lane_taddr + a.col_delta + (uint32_t)t0, rd);
        tc_wait_ld();
        if (t0 + 64 >= u.ntok) release();
        const int nvalid = min(32, u.ntok - t0);
#pragma unroll
        for (int t = 0; t < 32; ++t) {
            if (t < nvalid) out.put(t0 + t, fmaf(al, __uint_as_float(rd[t]), __uint_as_float(rb[t])));
        }
    }
}

// Tiled schedule with several tenants per unit (16 < m <= 64): tenant j's base columns start at j*m, its delta
// columns at j*Nd; 16-token chunks, dealt alternately to the two warps of a lane quadrant.
// `al_lane`: lane l holds the scale of the unit's tenant l.
template <class Out>
__device__ __forceinline__ void epilogue_tiled_grouped(const GemmArgs& a, const Unit& u, uint32_t lane_taddr, int m,
                                                       const Out& out, int half, float al_lane) {
    const int chunks = (m + 15) >> 4;
#pragma unroll 1
    for (int c = half; c < u.nten * chunks; c += 2) {
        const int j = c / chunks, t0 = (c - j * chunks) * 16;
        uint32_t rb[16], rd[16];
        tmem_ld16(lane_taddr + (uint32_t)(j * m + t0), rb);
        tmem_ld16(lane_taddr + a.col_delta + (uint32_t)(j * a.Nd + t0), rd);
        tc_wait_ld();
        const float al = __shfl_sync(0xFFFFFFFFu, al_lane, j);
        const int nvalid = min(16, m - t0);
#pragma unroll
        for (int t = 0; t < 16; ++t) {
            if (t < nvalid) out.put(j * m + t0 + t, fmaf(al, __uint_as_float(rd[t]), __uint_as_float(rb[t])));
        }
    }
}

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

// Sums the partial results of a tile cut across CTAs c0..c1 (in that order) and writes Y.
// nwarps*32 threads: thread e owns rows 4*(e%32)..+3 of tokens e/32, e/32+nwarps, ...
template <bool kGen, bool kGate>
__device__ __forceinline__ void reduce_partials(const GemmArgs& a, const Unit& u, int etid, int nwarps,
                                                const float* first, const float* rest, size_t cstride, int nrest) {
    uint16_t* Y = reinterpret_cast<uint16_t*>(a.Y);
    const int r4 = (etid & 31) * 4;
    const int n = u.n0 + r4;
    const bool vec_ok = ((a.N & 3) == 0) && (n + 3 < a.N);
    float bias4[4] = {0.f, 0.f, 0.f, 0.f};
    if (kGen && a.bias) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (n + i < a.N) bias4[i] = from_io16(__ldg(reinterpret_cast<const uint16_t*>(a.bias) + n + i), a.f16);
    }
    for (int tk = etid >> 5; tk < u.ntok; tk += 4 * nwarps) {
        float4 acc[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int t = tk + nwarps * q;
            acc[q] = (t < u.ntok) ? ldcg4(first + (size_t)t * kTileN + r4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        // The other contributions, two at a time: their loads are independent round trips to L2 and are
        // requested together (the sums keep their order).
        for (int c = 0; c < nrest; c += 2) {
            float4 v[2][4];
#pragma unroll
            for (int d = 0; d < 2; ++d) {
                const float* pc = rest + (size_t)(c + d) * cstride;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int t = tk + nwarps * q;
                    v[d][q] = (c + d < nrest && t < u.ntok) ? ldcg4(pc + (size_t)t * kTileN + r4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int d = 0; d < 2; ++d)
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    acc[q].x += v[d][q].x; acc[q].y += v[d][q].y; acc[q].z += v[d][q].z; acc[q].w += v[d][q].w;
                }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int t = tk + nwarps * q;
            if (t < u.ntok) {
                if constexpr (kGate) {
                    {
                        // SiLU gate: rows (n, n+1) and (n+2, n+3) are (gate, up) pairs; N is even and n a multiple of 4
                        const float g0 = acc[q].x + bias4[0], u0 = acc[q].y + bias4[1];
                        const float g1 = acc[q].z + bias4[2], u1 = acc[q].w + bias4[3];
                        uint16_t* dg = Y + (size_t)(u.xrow0 + t) * (a.N >> 1) + (n >> 1);
                        if (n < a.N) dg[0] = to_io16(__fdividef(g0, 1.f + __expf(-g0)) * u0, a.f16);
                        if (n + 2 < a.N) dg[1] = to_io16(__fdividef(g1, 1.f + __expf(-g1)) * u1, a.f16);
                        continue;
                    }
                }
                uint16_t* dst = Y + (size_t)(u.xrow0 + t) * a.N + n;
                uint16_t o0, o1, o2, o3;
                if constexpr (kGen) {
                    o0 = finish_io16(acc[q].x, bias4[0], a.act, a.f16);
                    o1 = finish_io16(acc[q].y, bias4[1], a.act, a.f16);
                    o2 = finish_io16(acc[q].z, bias4[2], a.act, a.f16);
                    o3 = finish_io16(acc[q].w, bias4[3], a.act, a.f16);
                } else {
                    o0 = __bfloat16_as_ushort(__float2bfloat16_rn(acc[q].x));
                    o1 = __bfloat16_as_ushort(__float2bfloat16_rn(acc[q].y));
                    o2 = __bfloat16_as_ushort(__float2bfloat16_rn(acc[q].z));
                    o3 = __bfloat16_as_ushort(__float2bfloat16_rn(acc[q].w));
                }
                if (vec_ok) {
                    *reinterpret_cast<uint2*>(dst) = make_uint2((uint32_t)o0 | ((uint32_t)o1 << 16), (uint32_t)o2 | ((uint32_t)o3 << 16));
                } else {
                    if (n + 0 < a.N) dst[0] = o0;
                    if (n + 1 < a.N) dst[1] = o1;
                    if (n + 2 < a.N) dst[2] = o2;
                    if (n + 3 < a.N) dst[3] = o3;
                }
            }
        }
    }
}

// In-kernel activation split (decode schedule, few token rows per unit).  Task (r, q4, h, pc): token row
// r, 32-k group q4 of the stage, half h of the group's byte slots, pair pc of the half's four k classes.
// Slot 4c+i holds k = c + 8i, so the task's classes c = 4h+2pc, 4h+2pc+1 need, from each of the four
// 16-byte chunks (i = 0..3) of the group, the 4 bytes holding k = 8i+c, 8i+c+1, and produce 8 bytes
// (slots 16h+8pc .. +7) per piece.
// The pieces are taken by TRUNCATION on packed f16 pairs (a bf16 value in the e5m2 range is exact in f16,
// and an e5m2 number is the high byte of an f16 number): p = y with its low byte cleared, y -= p (exact).
// A bf16 value has 8 significant bits and every piece removes the top three of what is left, so the third
// piece leaves nothing and the fourth is zero; no conversion instruction is needed (they are slow enough
// to hold up the decode warps that share a scheduler with the splitting warp).
// `xt` is the stage's X tile (two swizzled 64-k atoms), `x8t` its piece tile.  Thread `tid` of `nthreads`
// takes the tasks tid, tid + nthreads, ...  Small tasks on purpose: 16 per token row spread the work over
// all four epilogue warps, one warp per scheduler.
template <bool kF16>
__device__ __forceinline__ void split_activations(const GemmArgs& a, int am, const uint8_t* xt, uint8_t* x8t, int ntok, int tid,
                                                  int nthreads) {
    const int ntasks = ntok * 16;
    bool out_of_range = false;
    for (int task = tid; task < ntasks; task += nthreads) {
        const int r = task >> 4, q4 = (task >> 2) & 3, h = (task >> 1) & 1, pc = task & 1;
        const int j = r / am, t = r - j * am;
        const uint8_t* src = xt + (q4 >> 1) * a.x_atom_bytes + r * 128 + h * 8 + pc * 4;
        uint32_t y[4];   // y[i]: f16 pair, k = 8i + 4h + 2pc, +1
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int chunk = ((q4 & 1) * 4 + i) ^ (r & 7);
            const uint32_t v = *reinterpret_cast<const uint32_t*>(src + chunk * 16);
            if constexpr (kF16) {
                y[i] = v;   // binary16 already: eleven significant bits, the four pieces take 3 + 3 + 3 + 2
            } else {
                // e5m2 has binary16's exponent range: a bf16 magnitude of 2^16 or more does not fit.  It is
                // clamped to the largest binary16 number (delta term only) and reported through the status word.
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
            // bytes (i = 0..3) of element k, then of element k+1
            const uint32_t t01 = __byte_perm(pq[0], pq[1], 0x7351);   // [p0.b1, p1.b1, p0.b3, p1.b3]
            const uint32_t t23 = __byte_perm(pq[2], pq[3], 0x7351);
            const uint2 w = make_uint2(__byte_perm(t01, t23, 0x5410), __byte_perm(t01, t23, 0x7632));
            const int r8 = j * (kPieces * am) + q * am + t;
            *reinterpret_cast<uint2*>(x8t + r8 * 128 + (((2 * q4 + h) ^ (r8 & 7)) * 16) + pc * 8) = w;
        }
    }
    if (out_of_range) atomicCAS(&g_device_status[0], 0u, kStatusRange);
}

// 32 packed sign bits -> 8 registers of four e5m2 each (+1 = 0x3C, -1 = 0xBC).  Register c takes
// bits c, c+8, c+16, c+24 (its bytes 0..3): one shift lands all four on the byte sign positions, one
// three-input logic op masks them and flips the sign of a packed (-1,-1,-1,-1).  The k order inside
// the group of 32 is therefore permuted (slot 4c+i holds k = c + 8i); the activation pieces are
// stored with the same permutation, so the contraction is unchanged.
__device__ __forceinline__ void decode_word_e5m2(uint32_t w, uint32_t* r) {
#pragma unroll
    for (int c = 0; c < 8; ++c) r[c] = ((w << (7 - c)) & 0x80808080u) ^ 0xBCBCBCBCu;
}

__device__ __forceinline__ void epi_bar_sync(int nthreads) { asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory"); }

}  // namespace bd
