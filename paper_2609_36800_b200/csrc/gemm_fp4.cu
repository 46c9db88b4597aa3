// BitDelta fused GEMM, 4-bit decode schedule (few token rows per unit) on tcgen05 tensor cores.
//
//   Y[b,t,n] = sum_k X[b,t,k] W[n,k] + alpha[b] sum_k X[b,t,k] S[b,n,k]
//
// Same orientation as the other kernels (weight rows on the MMA's M side, tokens on its N side, decoded signs written
// to tensor memory as the A operand), work split and split-K fix-up as in gemm_tc.cu; the delta term runs on the
// block-scaled 4-bit tensor path (tcgen05.mma kind::mxf4, K = 64 per instruction):
//   * Signs are decoded to e2m1 (+1 = 0x2, -1 = 0xA), EIGHT per 32-bit register: per sign word three shifts and four
//     logic operations, four tensor-memory columns.  That is half the integer work and half the tensor-memory store
//     traffic of the 8-bit form, the two things that bound the decode schedules, and half the MMA instructions.
//     Register c of a word holds in nibble i the sign of k = 4i + c.
//   * Activations: every group of 32 consecutive k of a token row (one sign word) is written as 16-bit fixed point
//     relative to the group's largest exponent E (|x| = v * 2^(E-142), v < 2^16: every value within 8 binades of the
//     group's largest is exact, smaller ones are truncated below 2^-16 of it) and v as eight radix-4 digits 0..3; a
//     digit d goes into the operand as the e2m1 value d/2, whose 4-bit code is d itself, with the value's sign in the
//     code's sign bit.  Digit q of all tokens forms row block q of the MMA's B operand, and the B-side SCALE FACTOR
//     of a row and 32-k group (ue8m0, one byte) is E + 2q: the group's exponent and the digit's weight 4^q.  The
//     A-side scale is 1.  A tenant's delta is then the plain sum of its eight accumulator column groups times
//     2^-14, which the epilogue applies together with alpha.  No value of the 16-bit input range saturates or is
//     flagged (exponents above 240, i.e. |x| >= 2^114, are treated as 240).
//   * Units of more than 16 token rows: a pre-pass kernel writes, per tenant group and 128-k step, the
//     shared-memory IMAGE of both activation operands (16-bit tile of the base MMA with its 128-byte swizzle, digit
//     rows with the 64-byte swizzle); the producer fetches an image with one plain bulk copy.  Units of up to 16 token
//     rows: the four epilogue warps write the same image straight into shared memory from X.
// One block per multiprocessor (it needs most of the shared memory), 16 warps: producer, THREE MMA issuers (base; delta
// of the even and of the odd tenants), eight decode warps, four epilogue warps.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <type_traits>

#include "gemm_common.cuh"
#include "gemm_tc.h"
#include "ptx.cuh"

namespace bd {

constexpr int kFWarpProducer = 0;
constexpr int kFWarpMma = 1;                     // base MMAs (A = W_base tile in shared memory)
constexpr int kFWarpDelta0 = 2;                  // warps 2, 3: delta MMAs of the even / odd tenants (A = signs in tensor memory)
constexpr int kFWarpDecode0 = 4;                 // warps 4 .. 11 decode
constexpr int kFDecodeWarps = 8;
constexpr int kFWarpEpi0 = kFWarpDecode0 + kFDecodeWarps;
constexpr int kFEpiWarps = 4;
constexpr int kFThreads = (kFWarpEpi0 + kFEpiWarps) * 32;   // 512
constexpr int kFHandover = kFDecodeWarps / 2 * 32 + 32;      // the four decode warps of a tenant half arrive, its issuer warp syncs
constexpr int kFBarSet0 = 2;                     // named barrier of operand set s, tenant half h: id 2 + 2 s + h
constexpr int kFBarDep = 15;                     // the decode and epilogue warps sleep on it until the grid dependency resolves
constexpr int kFBarImg = 14;                     // resident form: all warps but the producer have written their share of the images

#ifdef BD_TRACE
// Trace build: per block 32 accumulators (cycles) written at the end of each role; see bitdelta_debug_set_trace_fp4.
__device__ long long* g_fp4_trace = nullptr;
#define FT_DECL(n) long long ft_acc[n] = {}; long long ft_t0 = clock64()
#ifdef BD_TRACE_TIMELINE_ONLY   /* (the accumulators' clock reads cost time themselves: leave only the timeline stamps) */
#define FT_ADD(i) do { } while (0)
#else
#define FT_ADD(i) do { const long long ft_t1 = clock64(); ft_acc[i] += ft_t1 - ft_t0; ft_t0 = ft_t1; } while (0)
#endif
#define FT_OUT(base, n) do { if (g_fp4_trace && lane == 0) for (int ft_i = 0; ft_i < (n); ++ft_i) g_fp4_trace[(size_t)blockIdx.x * 32 + (base) + ft_i] = ft_acc[ft_i]; } while (0)
// ... and 16 timestamps (ns, %globaltimer) per block in a second buffer half: [16 .. 31] of the block's second row
#define FT_STAMP(i) do { if (g_fp4_trace && lane == 0) g_fp4_trace[(size_t)(256 + blockIdx.x) * 32 + (i)] = (long long)global_timer_ns(); } while (0)
#ifdef BD_TRACE_STEPS   /* per-step event log behind the 512 x 32 words above: [block][step mod 64][16 events], nanoseconds */
#define FT_EVL(ev, n) do { if (g_fp4_trace) g_fp4_trace[512 * 32 + ((size_t)blockIdx.x * 64 + ((n) & 63)) * 16 + (ev)] = (long long)global_timer_ns(); } while (0)
#else
#define FT_EVL(ev, n) do { } while (0)
#endif
#define FT_EV(ev, n) do { if (lane == 0) FT_EVL(ev, n); } while (0)
#define FT_STAMPL(i) do { if (g_fp4_trace) g_fp4_trace[(size_t)(256 + blockIdx.x) * 32 + (i)] = (long long)global_timer_ns(); } while (0)
#else
#define FT_STAMP(i) do { } while (0)
#define FT_STAMPL(i) do { } while (0)
#define FT_EV(ev, n) do { } while (0)
#define FT_EVL(ev, n) do { } while (0)
#define FT_DECL(n) do { } while (0)
#define FT_ADD(i) do { } while (0)
#define FT_OUT(base, n) do { } while (0)
#endif

struct FCtl {
    uint64_t wfull[kMaxStages];     // W_base tile landed
    uint64_t wempty[kMaxStages];    // ... and was read by its base MMAs
    uint64_t bfull[4];              // sign words of two 128-k steps landed
    uint64_t bempty[4];             // ... and are in the decode warps' registers (8 arrivals)
    uint64_t pfull[4];              // a step's activation image landed
    uint64_t pempty[4];             // ... and was read by the step's MMAs
    uint64_t opfree[2][kFp4MaxSets];   // tenant half h's columns of an operand set in tensor memory free again
    uint64_t accfull;               // all MMAs of a segment have completed
    uint64_t accempty;              // the accumulators were drained (4 epilogue warps)
    uint64_t depready;              // the grid this launch depends on has completed
    uint64_t tmemready;             // tensor memory is allocated (its base address is in tmem_base)
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t is_last;
    uint64_t imgready[4];           // a step's image is in shared memory and its scale factors in tensor memory (4 epilogue warps)
    uint64_t cntready;              // cooperative image pass: this block has counted itself; img_target is set
    uint32_t img_target;            // ... value of the launch-wide counter at which every block's share is written
};
static_assert(sizeof(FCtl) <= kSmemCtrlBytes, "control block too large");

// Eight signs per register: register c, nibble i <- bit 4i + c of the word (1 -> +1.0 = 0x2, 0 -> -1.0 = 0xA).
__device__ __forceinline__ void decode_word_e2m1(uint32_t w, uint32_t* r) {
    r[0] = ((w << 3) & 0x88888888u) ^ 0xAAAAAAAAu;
    r[1] = ((w << 2) & 0x88888888u) ^ 0xAAAAAAAAu;
    r[2] = ((w << 1) & 0x88888888u) ^ 0xAAAAAAAAu;
    r[3] = (w & 0x88888888u) ^ 0xAAAAAAAAu;
}

// Eight 16-bit values hv[i] of one token row (k = k0 + 4i) -> for every digit q the register R[q] whose nibble i is
// the operand code of value i: sign << 3 | digit q of its 16-bit fixed-point magnitude (E: the row's exponent).
__device__ __forceinline__ void fp4_digits8(const uint32_t* hv, int E, uint32_t* R) {
    uint32_t T[8];   // T[i]: nibble q = code of digit q of value i
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int ex = (int)((hv[i] >> 7) & 0xFFu);
        const uint32_t m8 = (hv[i] & 0x7Fu) | (ex ? 0x80u : 0u);
        uint32_t t = (m8 << 8) >> min(E - max(ex, 1), 31);
        t = (t | (t << 8)) & 0x00FF00FFu;    // 8 bits per 16-bit lane
        t = (t | (t << 4)) & 0x0F0F0F0Fu;    // 4 bits per byte
        t = (t | (t << 2)) & 0x33333333u;    // 2 bits per nibble
        T[i] = t | ((hv[i] & 0x8000u) ? 0x88888888u : 0u);
    }
    // 8 x 8 nibble transpose: 16-bit halves between registers i, i+4; bytes between i, i+2; nibbles between i, i+1
    uint32_t A[8], Bv[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        A[i] = __byte_perm(T[i], T[i + 4], 0x5410);
        A[i + 4] = __byte_perm(T[i], T[i + 4], 0x7632);
    }
#pragma unroll
    for (int g = 0; g < 8; g += 4) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            Bv[g + i] = __byte_perm(A[g + i], A[g + i + 2], 0x6240);
            Bv[g + i + 2] = __byte_perm(A[g + i], A[g + i + 2], 0x7351);
        }
    }
#pragma unroll
    for (int g = 0; g < 8; g += 2) {
        R[g] = (Bv[g] & 0x0F0F0F0Fu) | ((Bv[g + 1] & 0x0F0F0F0Fu) << 4);
        R[g + 1] = ((Bv[g] >> 4) & 0x0F0F0F0Fu) | (Bv[g + 1] & 0xF0F0F0F0u);
    }
}

// One task of the activation split: of token row r_local = j*m + t of its unit the 16-byte chunk `tk` of a 128-k
// step (k = 8 tk .. 8 tk + 7) goes to the 16-bit tile, and the eight values k = 32 wd + 4i + c (wd = tk / 4, c = tk % 4)
// to the digit rows j*8m + q*m + t: register c of word wd, the order in which decode_word_e2m1 lays out the signs.
// The four tasks c = 0..3 of a word sit in neighbouring lanes (all active together) and share the group's exponent,
// which task c = 0 writes to the image's scale table (byte 4 r_local + wd).  `xstep`: the row's first value of the
// step; `im`: the step's image (global or shared memory): [16-bit tile | digit rows | scale table].
struct Fp4TaskData {
    uint4 chunk;       // the task's 16-byte chunk of the 16-bit tile
    uint32_t hv[8];    // the eight values k = 32 wd + 4i + c
};
__device__ __forceinline__ void fp4_task_load(const uint16_t* __restrict__ xstep, int tk, Fp4TaskData& d) {
    // (through L1: the four tasks of a word read the same 64 bytes, and X is not written while this kernel may read it)
    d.chunk = __ldg(reinterpret_cast<const uint4*>(xstep) + tk);
    const int wd = tk >> 2, c = tk & 3;
#pragma unroll
    for (int i = 0; i < 8; ++i) d.hv[i] = __ldg(xstep + 32 * wd + 4 * i + c);
}
__device__ __forceinline__ void fp4_task_digits(const Fp4TaskData& d, uint8_t* im, int tk, int r_local, int j, int t, int m,
                                                uint32_t x_tile_bytes, uint32_t sf_off);
__device__ __forceinline__ void fp4_task_finish(const Fp4TaskData& d, uint8_t* im, int tk, int r_local, int j, int t, int m,
                                                uint32_t x_atom_bytes, uint32_t x_tile_bytes, uint32_t sf_off) {
    *reinterpret_cast<uint4*>(im + (tk >> 3) * x_atom_bytes + r_local * 128 + (((tk & 7) ^ (r_local & 7)) * 16)) = d.chunk;
    fp4_task_digits(d, im, tk, r_local, j, t, m, x_tile_bytes, sf_off);
}
// ... its second half: the digit rows and the scale table entry from the eight values d.hv
__device__ __forceinline__ void fp4_task_digits(const Fp4TaskData& d, uint8_t* im, int tk, int r_local, int j, int t, int m,
                                                uint32_t x_tile_bytes, uint32_t sf_off) {
    const int wd = tk >> 2, c = tk & 3;
    uint32_t R[8];
    uint32_t mx = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) mx = max(mx, d.hv[i] & 0x7FFFu);
    const unsigned act = __activemask();
    mx = max(mx, __shfl_xor_sync(act, mx, 1));
    mx = max(mx, __shfl_xor_sync(act, mx, 2));
    const int E = min(max((int)(mx >> 7), 1), 240);
    fp4_digits8(d.hv, E, R);
#pragma unroll
    for (int q = 0; q < kFp4Pieces; ++q) {
        const int n = j * (kFp4Pieces * m) + q * m + t;
        *reinterpret_cast<uint32_t*>(im + x_tile_bytes + n * 64 + ((wd ^ ((n >> 1) & 3)) * 16) + 4 * c) = R[q];
    }
    if (c == 0) im[sf_off + 4 * r_local + wd] = (uint8_t)E;
}
__device__ __forceinline__ void fp4_split_task(const uint16_t* __restrict__ xstep, uint8_t* im, int tk, int r_local, int j, int t,
                                               int m, uint32_t x_atom_bytes, uint32_t x_tile_bytes, uint32_t sf_off) {
    Fp4TaskData d;
    fp4_task_load(xstep, tk, d);
    fp4_task_finish(d, im, tk, r_local, j, t, m, x_atom_bytes, x_tile_bytes, sf_off);
}

// ---------------------------------------------------------------------------------------------- pre-pass
// Block (row, chunk of 2048 k): the row's share of the images of those steps.
__global__ void __launch_bounds__(256) x_split_fp4_kernel(const uint16_t* __restrict__ X, uint8_t* __restrict__ img, int m, int K,
                                                          int TB, int P, uint32_t img_bytes, uint32_t x_atom_bytes,
                                                          uint32_t x_tile_bytes, uint32_t sf_off) {
    // Launched with an early start: the GEMM queued behind this kernel may become resident at once (it prefetches
    // weights and waits for this kernel before it reads an image); this kernel itself reads X and overwrites the
    // images only after the kernel before it (possibly the previous GEMM, still reading them) has completed.
    grid_launch_dependents();
    grid_dependency_wait();
    const int row = blockIdx.x;
    const int b = row / m, t = row - b * m;
    const int g = b / TB, j = b - g * TB;
    const int r_local = j * m + t;
    const uint16_t* x = X + (size_t)row * K;
    uint8_t* img_g = img + (size_t)g * P * img_bytes;
    const int task = blockIdx.y * 256 + threadIdx.x;   // (16 tasks per step: whole groups of four are inside K or outside)
    if (task < K / 8) {
        const int p = task >> 4;
        fp4_split_task(x + (size_t)p * kPairK, img_g + (size_t)p * img_bytes, task & 15, r_local, j, t, m, x_atom_bytes, x_tile_bytes, sf_off);
    }
}

cudaError_t launch_x_split_fp4(const void* X, uint8_t* img, const Plan& p, bool early_start, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.B * p.m), (unsigned)((p.K / 8 + 255) / 256));
    cfg.blockDim = dim3(256u);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early_start ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, x_split_fp4_kernel, reinterpret_cast<const uint16_t*>(X), img, p.m, p.K, p.TB, p.P, p.img_bytes,
                              p.x_atom_bytes, p.x_tile_bytes, p.x_tile_bytes + (uint32_t)p.x8_rows * 64u);
}

// Epilogue of one segment, M tokens per tenant: base accumulator columns j*M + t, tenant j's delta accumulator from
// column 8M*j, digit q of token t in column q*M + t (already weighted by its scale factors).
//   out(j*M + t) = base + (alpha_j * 2^-14) * sum_q D[q*M + t]
template <int M, class Out>
__device__ __forceinline__ void epilogue_fp4(const GemmArgs& a, const Unit& u, uint32_t lane_taddr, const Out& out, float al_lane) {
    constexpr int ND = kFp4Pieces * M;
    constexpr int MB = (M <= 1) ? 1 : (M <= 2) ? 2 : (M <= 4) ? 4 : 8;   // base columns read per tenant (a power of two >= M)
#pragma unroll 1
    for (int j = 0; j < u.nten; ++j) {
        uint32_t rd[ND], rb[MB];
        const uint32_t col = lane_taddr + a.col_delta + (uint32_t)(j * ND);
        if constexpr (MB == 1) tmem_ld1(lane_taddr + (uint32_t)(j * M), rb);
        else if constexpr (MB == 2) tmem_ld2(lane_taddr + (uint32_t)(j * M), rb);
        else if constexpr (MB == 4) tmem_ld4(lane_taddr + (uint32_t)(j * M), rb);
        else tmem_ld8(lane_taddr + (uint32_t)(j * M), rb);
        if constexpr (ND >= 32) {
#pragma unroll
            for (int c = 0; c + 32 <= ND; c += 32) tmem_ld32(col + c, rd + c);
        }
        if constexpr (ND % 32 >= 16) tmem_ld16(col + ND / 32 * 32, rd + ND / 32 * 32);
        if constexpr (ND % 16 >= 8) tmem_ld8(col + ND / 16 * 16, rd + ND / 16 * 16);
        tc_wait_ld();
        const float al = __shfl_sync(0xFFFFFFFFu, al_lane, j) * 6.103515625e-05f;   // tenant j's scale (held by lane j) x 2^-14
#pragma unroll
        for (int t = 0; t < M; ++t) {
            float d = 0.f;
#pragma unroll
            for (int q = 0; q < kFp4Pieces; ++q) d += __uint_as_float(rd[q * M + t]);
            out.put(j * M + t, fmaf(al, d, __uint_as_float(rb[t])));
        }
    }
}

template <class Out>
__device__ __forceinline__ void epilogue_fp4_any_m(const GemmArgs& a, const Unit& u, uint32_t lane_taddr, const Out& out,
                                                   float al_lane, int am) {
    switch (am) {
        case 1: epilogue_fp4<1>(a, u, lane_taddr, out, al_lane); break;
        case 2: epilogue_fp4<2>(a, u, lane_taddr, out, al_lane); break;
        case 3: epilogue_fp4<3>(a, u, lane_taddr, out, al_lane); break;
        case 4: epilogue_fp4<4>(a, u, lane_taddr, out, al_lane); break;
        case 5: epilogue_fp4<5>(a, u, lane_taddr, out, al_lane); break;
        case 6: epilogue_fp4<6>(a, u, lane_taddr, out, al_lane); break;
        case 7: epilogue_fp4<7>(a, u, lane_taddr, out, al_lane); break;
        default: epilogue_fp4<8>(a, u, lane_taddr, out, al_lane); break;
    }
}

// Cluster form: where a block's partial sums go (its own shared memory, [token][128 weight rows] floats).
struct FClusterPartOut {
    float* part_row;   // &part[0][this thread's weight row]
    __device__ __forceinline__ void put(int tok, float v) const { part_row[tok * kTileN] = v; }
};

// The walk over a block's (unit, step) items.  Cluster form (kForm 1): one segment of one unit per block, known without a
// division; the other forms walk the flat list like the 8-bit kernels (gemm_common.cuh).  Every role holds a copy of this
// code and the kernel's speed depends on its length.
// x / d by the multiplier of d (ceil(2^32 / d), 0 for d = 1; exact while x * d < 2^32: the plan sees to that).
__device__ __forceinline__ int fdiv(int x, uint32_t mg) { return mg ? (int)__umulhi((unsigned)x, mg) : x; }

template <int kForm>
struct FSeg {
    int cur, hi;
    int P;
    int stride;   // flat list, whole units: > 0 = units cur/P, cur/P + stride, ...
    int unit1;    // cluster form: the cluster's unit
    uint32_t mg_P;   // flat list: the multiplier of P (fdiv)
    __device__ __forceinline__ bool next(int& unit, int& p0, int& p1) {
        if (cur >= hi) return false;
        if constexpr (kForm == 1) {
            unit = unit1;
            p0 = cur - unit1 * P;
            p1 = hi - unit1 * P;
            cur = hi;
            return true;
        } else {
            unit = fdiv(cur, mg_P);
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
    }
};
template <int kForm>
struct FItem {
    FSeg<kForm> seg;
    int unit, p, p1;
    bool first;   // first item of its segment
    __device__ __forceinline__ explicit FItem(const FSeg<kForm>& s) : seg(s), unit(0), p(0), p1(0), first(false) {}
    __device__ __forceinline__ bool next() {
        if (p + 1 < p1) { ++p; first = false; return true; }
        int p0;
        if (!seg.next(unit, p0, p1)) { p = 0; p1 = 0; return false; }
        p = p0;
        first = true;
        return true;
    }
};

// kTB8: units of up to eight tenants (m <= 4): two operand sets per 128-k step, a set = all tenants x 64 k; else up to
// four tenants (m <= 8): one set per step, a set = all tenants x 128 k.  Either way a decode warp stores 32 columns per
// set: warp (quad, h) owns the weight rows of lane quadrant `quad` and the tenants j = 2i + h.
template <bool kTB8, bool kVariants, int kForm>
__global__ void __launch_bounds__(kFThreads, 1)
bitdelta_gemm_fp4_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmBits, const GemmArgs a) {
    constexpr int kSetsPerStep = kTB8 ? 2 : 1;
    constexpr int kTenPerWarp = kTB8 ? 4 : 2;
    constexpr int kTenCols = kTB8 ? 8 : 16;            // columns of one tenant in a set
    // The opt-in variants (images written in the kernel: by the epilogue warps per step, by all warps up front, or by
    // the launch's blocks together) have an instantiation of their own: the default one carries none of their code
    // (the kernel's code is several times the instruction cache as it is).
    // kForm: 0 = the flat work list only, 1 = the cluster form only, 2 = whichever the launch says (the variants).
    const bool is_cluster = (kForm == 2) ? (a.cluster > 1) : (kForm == 1);
    const int v_resident = kVariants ? a.resident : 0;
    const int v_coop = kVariants ? a.coop : 0;
    const int v_convert = kVariants ? a.convert : 0;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t w_addr = base;                                          // ring of W_base tiles
    const uint32_t bits_off = a.n_w * a.w_stage_bytes;                     // sign-word slots (two steps each)
    const uint32_t bits_addr = base + bits_off;
    const uint32_t img_off = bits_off + a.n_bits * a.bslot_bytes;          // ring of activation images
    const int n_ring = v_resident ? a.n_sf : a.n_img;                      // ... its slots (resident images: the scale-factor slots)
    const uint32_t img_addr = base + img_off;
    FCtl* ctl = reinterpret_cast<FCtl*>(smem + img_off + a.n_img * a.img_bytes);
    volatile uint32_t* abort_flag = &ctl->abort_flag;

    const int am = a.m;
    auto unit_info = [&](const GemmArgs& aa, int un) {
        if constexpr (kForm == 1) {   // (cluster form: one tenant group, no teams)
            Unit u;
            u.n0 = un * kTileN;
            u.tenant0 = 0;
            u.nten = min(aa.TB, aa.B);
            u.xrow0 = 0;
            u.ntok = u.nten * am;
            return u;
        } else {   // (the look-up of gemm_common.cuh for the decode schedules, its divisions by multipliers)
            Unit u;
            int nt, g;
            if (aa.teams > 1) {   // group-major
                g = fdiv(un, aa.mg_tiles);
                nt = un - g * aa.n_tiles;
            } else {
                nt = fdiv(un, aa.mg_groups);
                g = un - nt * aa.groups;
            }
            u.n0 = nt * kTileN;
            u.tenant0 = g * aa.TB;
            u.nten = min(aa.TB, aa.B - u.tenant0);
            u.xrow0 = u.tenant0 * am;
            u.ntok = u.nten * am;
            return u;
        }
    };
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    if (warp == 0) FT_STAMP(0);   // block start
    if (threadIdx.x == 32) {
        prefetch_tensormap(&tmW);
        prefetch_tensormap(&tmBits);
    }

    // Work: an even share of the flat (unit, k-step) list (or whole units round-robin), or, in the cluster form,
    // this block's share of the k-steps of its cluster's unit.
    const int crank = is_cluster ? (int)cluster_ctarank() : 0;
    int lo, hi, cunit = 0;
    if (is_cluster) {
        const int cshift = 31 - __clz(a.cluster);   // (clusters of 2, 4 or 8 blocks)
        cunit = (int)(blockIdx.x >> cshift);
        lo = cunit * a.P + ((crank * a.P) >> cshift);
        hi = cunit * a.P + (((crank + 1) * a.P) >> cshift);
    } else {
        lo = a.whole_units ? (int)blockIdx.x * a.P : cta_first_item(a, (int)blockIdx.x);
        hi = a.whole_units ? (int)a.T : cta_first_item(a, (int)blockIdx.x + 1);
    }
    FSeg<kForm> it{lo, hi, a.P, (a.whole_units && !is_cluster) ? (int)gridDim.x : 0, cunit, a.mg_P};
    int unit, p0, p1;

    // The W_base tile of a step (128 rows x 128 k: both 64-k atoms) in one bulk-tensor copy.  One thread.
    auto issue_w = [&](const Unit& u, int p, int stage) {
        const uint32_t bar = smem_u32(&ctl->wfull[stage]);
        mbar_arrive_expect_tx(bar, a.w_stage_bytes);
        tma_load_3d(w_addr + stage * a.w_stage_bytes, &tmW, bar, 0, u.n0, p * (kPairK / kAtomK));
    };
    // The sign words of the two steps 2*(p/2), 2*(p/2)+1 for all the unit's tenants: one bulk-tensor copy (rows of
    // 32 bytes).  One thread.
    auto issue_bits = [&](const Unit& u, int p, int bslot) {
        const uint32_t bar = smem_u32(&ctl->bfull[bslot]);
        mbar_arrive_expect_tx(bar, a.bslot_bytes);
        tma_load_3d(bits_addr + bslot * a.bslot_bytes, &tmBits, bar, a.bits_row == 32 ? (p >> 1) * 8 : p * 4, u.n0, u.tenant0);
    };
    // The activation image of a step (written by the pre-pass kernel): one plain bulk copy.  One thread.
    auto issue_img = [&](const Unit& u, int p, int slot) {
        const uint32_t bar = smem_u32(&ctl->pfull[slot]);
        mbar_arrive_expect_tx(bar, a.img_bytes);
        const int g = fdiv(u.tenant0, a.mg_TB);
        bulk_load(img_addr + slot * a.img_bytes, a.img + ((size_t)g * a.P + p) * a.img_bytes, a.img_bytes, bar);
    };
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&ctl->wfull[s]), 1);
            mbar_init(smem_u32(&ctl->wempty[s]), 1);
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_u32(&ctl->bfull[s]), 1);
            mbar_init(smem_u32(&ctl->bempty[s]), kFDecodeWarps);
            mbar_init(smem_u32(&ctl->pfull[s]), 1);   // one bulk copy (pre-pass mode)
            mbar_init(smem_u32(&ctl->imgready[s]), kFEpiWarps);
            mbar_init(smem_u32(&ctl->pempty[s]), 3);   // (the three issuers)
        }
        for (int s = 0; s < kFp4MaxSets; ++s) {
            mbar_init(smem_u32(&ctl->opfree[0][s]), 1);
            mbar_init(smem_u32(&ctl->opfree[1][s]), 1);
        }
        mbar_init(smem_u32(&ctl->accfull), 3);   // (the three issuers)
        mbar_init(smem_u32(&ctl->accempty), kFEpiWarps);
        mbar_init(smem_u32(&ctl->depready), 1);
        mbar_init(smem_u32(&ctl->tmemready), 1);
        mbar_init(smem_u32(&ctl->cntready), 1);
        ctl->abort_flag = 0;
        ctl->is_last = 0;
        fence_barrier_init();
    }
    __syncthreads();

    const uint32_t tmemready = smem_u32(&ctl->tmemready);
    // Resident form (cluster form, one segment per block): once the grid dependency has resolved, all warps but the
    // producer write the images of all the block's steps, one task per thread and (token row, 16-byte chunk, step).
    auto write_resident_images = [&]() {
        const Unit u = unit_info(a, cunit);
        const int q0 = lo - cunit * a.P, nsteps = hi - lo;
        const int tid = (int)threadIdx.x - 32;
        const uint32_t sf_off = a.x_tile_bytes + (uint32_t)(a.TB * a.Nd) * 64u;
        const int per_step = u.ntok * 16;
        // Phase A: the 16-bit tiles, one 16-byte chunk per task (three tasks per thread requested together: one round
        // trip to X).  Phase B: the digit rows, from the tiles in shared memory (eight 2-byte shared loads per task instead of
        // eight global ones).
        for (int task0 = tid; task0 < nsteps * per_step; task0 += 3 * (kFThreads - 32)) {
            uint4 ch[3];
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                const int task = task0 + q * (kFThreads - 32);
                if (task < nsteps * per_step) {
                    const int st = (int)((unsigned)task / (unsigned)per_step);
                    const int rem = task - st * per_step;
                    ch[q] = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(a.X) + (size_t)(u.xrow0 + (rem >> 4)) * a.K + (size_t)(q0 + st) * kPairK) + (rem & 15));
                }
            }
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                const int task = task0 + q * (kFThreads - 32);
                if (task < nsteps * per_step) {
                    const int st = (int)((unsigned)task / (unsigned)per_step);
                    const int rem = task - st * per_step;
                    const int r = rem >> 4, tk = rem & 15;
                    *reinterpret_cast<uint4*>(smem + img_off + st * a.img_bytes + (tk >> 3) * a.x_atom_bytes + r * 128 + (((tk & 7) ^ (r & 7)) * 16)) = ch[q];
                }
            }
        }
        named_bar_sync(kFBarImg, kFThreads - 32);
        for (int task = tid; task < nsteps * per_step; task += kFThreads - 32) {
            const int st = (int)((unsigned)task / (unsigned)per_step);
            const int rem = task - st * per_step;
            const int r = rem >> 4, tk = rem & 15;
            const int j = r / am, t = r - j * am;
            uint8_t* im = smem + img_off + st * a.img_bytes;
            const int wd = tk >> 2, c = tk & 3;
            Fp4TaskData d;
            d.chunk = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int kk = 32 * wd + 4 * i + c;   // value k of the step: atom kk / 64, chunk (kk % 64) / 8, element kk % 8
                d.hv[i] = *reinterpret_cast<const uint16_t*>(im + (kk >> 6) * a.x_atom_bytes + r * 128 + ((((kk & 63) >> 3) ^ (r & 7)) * 16) + (kk & 7) * 2);
            }
            fp4_task_digits(d, im, tk, r, j, t, am, a.x_tile_bytes, sf_off);
        }
        fence_proxy_async_smem();   // generic-proxy writes -> visible to the MMAs' async-proxy reads
        named_bar_sync(kFBarImg, kFThreads - 32);
    };

    if (warp == kFWarpProducer) {
        // ------------------------------------------------------------ producer
        // Walks the block's steps three times over, once per stream: W_base tiles and sign words (never written by
        // another kernel: queued before the grid dependency is resolved, as far as their rings allow) and activation
        // images (written by the pre-pass kernel queued before this one: only afterwards).
        FItem<kForm> wi(it), bi(it), xi(it);
        Ring wr{0, 0u, a.n_w}, br{0, 0u, a.n_bits}, xr{0, 0u, n_ring};
        Unit uw{}, ub{}, ux{};
        bool more_w = wi.next(), more_b = bi.next(), more_x = !v_convert && xi.next();   // (convert: the epilogue warps write the images)
        if (more_w) { uw = unit_info(a, wi.unit); ub = uw; ux = uw; }
        long long t_idle = 0;
        int idle = 0;
        bool dep_done = false;
        while (more_w || more_b || more_x) {
            bool did = false;
            if (more_b && warp_all(mbar_test_wait(smem_u32(&ctl->bempty[br.idx]), br.par ^ 1))) {
                if (elect_one()) issue_bits(ub, bi.p, br.idx);
                __syncwarp();
                br.step();
                // the slot also covers the next step if that is the odd step of the same pair and of the same segment
                const bool odd_next = a.bits_row == 32 && ((bi.p & 1) == 0) && (bi.p + 1 < bi.p1);
                more_b = bi.next();
                if (more_b && odd_next) more_b = bi.next();
                if (more_b && bi.first) ub = unit_info(a, bi.unit);
                did = true;
            }
            if (more_w && warp_all(mbar_test_wait(smem_u32(&ctl->wempty[wr.idx]), wr.par ^ 1))) {
                if (elect_one()) issue_w(uw, wi.p, wr.idx);
                __syncwarp();
                wr.step();
                more_w = wi.next();
                if (more_w && wi.first) uw = unit_info(a, wi.unit);
                did = true;
            }
            if (dep_done && more_x && warp_all(mbar_test_wait(smem_u32(&ctl->pempty[xr.idx]), xr.par ^ 1))) {
                if (elect_one()) issue_img(ux, xi.p, xr.idx);
                __syncwarp();
                xr.step();
                more_x = xi.next();
                if (more_x && xi.first) ux = unit_info(a, xi.unit);
                did = true;
            }
            if (did) {
                idle = 0;
                continue;
            }
            if (!dep_done) {
                // The weight rings are full and stay full until the grid dependency resolves: sleep until then.  The first
                // image's source is worked out before, and requested right behind the wait (a few instructions next
                // to the ones this warp has been executing, instead of another trip around the loop).
                const uint8_t* first_src = nullptr;
                if (more_x && !v_coop) first_src = a.img + ((size_t)fdiv(ux.tenant0, a.mg_TB) * a.P + xi.p) * a.img_bytes;
                dep_done = warp_all(mbar_try_wait_hint(smem_u32(&ctl->depready), 0u, 20000u));
                if (dep_done && first_src != nullptr) {
                    if (elect_one()) {   // (the image ring is empty: slot 0, first use)
                        const uint32_t bar = smem_u32(&ctl->pfull[0]);
                        mbar_arrive_expect_tx(bar, a.img_bytes);
                        bulk_load(img_addr, first_src, a.img_bytes, bar);
                    }
                    __syncwarp();
                    xr.step();
                    more_x = xi.next();
                    if (more_x && xi.first) ux = unit_info(a, xi.unit);
                }
                if (dep_done && v_coop) {
                    // Cooperative image pass: every block of the launch writes its share of the activation images to
                    // the workspace and counts itself; the images may be fetched once all have (all blocks of a
                    // cluster-form launch are resident together, one per multiprocessor).  Bounded like every wait.
                    bool ok = warp_all(wait_bar(smem_u32(&ctl->cntready), 0u, abort_flag, 23));
                    const unsigned int target = ctl->img_target;
                    const long long t0 = clock64();
                    while (ok && (int)(ld_acquire_gpu_u32(a.img_counter) - target) < 0) {
                        if (*abort_flag) ok = false;
                        if (clock64() - t0 > kWaitLimitCycles) {
                            *abort_flag = 1;
                            if (atomicCAS(&g_device_status[0], 0u, kStatusTimeout) == 0u) g_device_status[1] = 24u;
                            ok = false;
                        }
                    }
                    FT_STAMP(14);   // every block's share is written
                    fence_proxy_async_all();   // the other blocks' generic-proxy stores -> this warp's bulk copies
                    if (!ok) break;
                }
                continue;
            }
            if (more_x) (void)mbar_try_wait_hint(smem_u32(&ctl->pempty[xr.idx]), xr.par ^ 1, 64u);
            else if (more_b) (void)mbar_try_wait_hint(smem_u32(&ctl->bempty[br.idx]), br.par ^ 1, 64u);
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
        // All of this block's loads are queued: a kernel queued behind this one with an early start may become resident.
        FT_STAMP(2);   // all loads queued
        if (lane == 0) grid_launch_dependents();
    } else if (warp == kFWarpMma) {
        // -------------------------------------------------------------- MMA issuer
        // Tensor memory is taken while the launch before this one may still be running (a block of this kernel fills a
        // multiprocessor: whatever ran here before has left, and only this library's kernels let a dependent start
        // early, after all their blocks hold what they need), so that nothing of it is left to do once the
        // dependency has resolved.
        tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
        tmem_relinquish();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tmemready);
        grid_dependency_wait();
        FT_STAMP(1);   // dependency resolved
        named_bar_arrive(kFBarDep, kFThreads - 32);   // wakes the decode and epilogue warps
        if (lane == 0) mbar_arrive(smem_u32(&ctl->depready));   // ... and the producer
        (void)wait_bar(tmemready, 0, abort_flag, 20);
        tc_fence_after();
        const uint32_t tmem_base = ctl->tmem_base;
        bool ok = true;
        if (v_resident) {
            grid_dependency_wait();   // (returns at once: orders this thread's reads of X behind the previous kernel)
            write_resident_images();
        }

        const uint32_t idesc_base = make_idesc_bf16(kTileN, (uint32_t)a.Nb);
        const uint64_t desc128 = make_smem_desc_sw128(0);
        const uint32_t x_atom16 = a.x_atom_bytes >> 4;
        Ring wr{0, 0u, a.n_w}, pr{0, 0u, n_ring};
        uint32_t accphase = 0;
        [[maybe_unused]] int ev_n = 0;
        FT_DECL(8);
        while (ok && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            FT_ADD(0);
            ok = warp_all(wait_bar(smem_u32(&ctl->accempty), accphase ^ 1, abort_flag, 3));
            FT_ADD(1);
            if (!ok) break;
            tc_fence_after();
            for (int p = p0; p < p1 && ok; ++p) {
                const uint32_t first = (p > p0) ? 1u : 0u;   // 0: this step starts the accumulation
                FT_ADD(0);
                ok = warp_all(wait_bar(smem_u32(&ctl->imgready[pr.idx]), pr.par, abort_flag, 13));
                FT_ADD(2);
                if (p == p0) FT_STAMP(3);   // first image ready (base issuer)
                FT_EV(3, ev_n);
                if (!ok) break;
                const uint32_t img_s = img_addr + (v_resident ? (p - p0) : pr.idx) * a.img_bytes;
                const uint64_t xdesc = desc128 + (img_s >> 4);
                ok = warp_all(wait_bar(smem_u32(&ctl->wfull[wr.idx]), wr.par, abort_flag, 4));
                FT_ADD(3);
                if (p == p0) FT_STAMP(4);   // first W_base tile landed
                FT_EV(4, ev_n);
                if (p == p1 - 1) FT_STAMP(5);   // last W_base tile landed
                if (!ok) break;
                {
                    const uint64_t wdesc = desc128 + ((w_addr + wr.idx * a.w_stage_bytes) >> 4);
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint32_t atom = kk >> 2, k16 = kk & 3;
                            umma_ss(tmem_base, wdesc + (atom * (a.w_atom_bytes >> 4) + k16 * 2), xdesc + (atom * x_atom16 + k16 * 2),
                                    idesc_base, (kk > 0) ? 1u : first);
                        }
                        tc_commit(smem_u32(&ctl->wempty[wr.idx]));
                    }
                    __syncwarp();
                    wr.step();
                }
                if (!ok) break;
                if (elect_one()) tc_commit(smem_u32(&ctl->pempty[pr.idx]));
                __syncwarp();
                pr.step();
                FT_EV(5, ev_n); ++ev_n;
            }
            if (!ok) break;
            if (elect_one()) tc_commit(smem_u32(&ctl->accfull));
            __syncwarp();
            accphase ^= 1;
        }
        FT_ADD(0);
        FT_OUT(0, 8);
    } else if (warp < kFWarpDecode0) {
        // -------------------------------------------------------------- delta MMA issuers
        // Warp 2 + h issues the delta MMAs of the tenants j = 2i + h (A = their decoded signs, filled by the four decode
        // warps of half h).  One thread issues a tcgen05 instruction every ~50 cycles whatever its size, so three
        // issuing threads (this pair and the base issuer) are what keeps the per-step instruction count off the
        // critical path.
        const int h = warp - kFWarpDelta0;
        bool ok = warp_all(wait_bar(tmemready, 0, abort_flag, 20));
        named_bar_sync(kFBarDep, kFThreads - 32);
        tc_fence_after();
        const uint32_t tmem_base = ctl->tmem_base;
        if (v_resident) {
            grid_dependency_wait();
            write_resident_images();
        }
        const uint32_t idesc_delta = make_idesc_mxf4(kTileN, (uint32_t)a.Nd);   // (+ the B-side scale id: which pair of a step's four 32-k groups)
        const uint64_t desc64 = make_smem_desc_sw64(0);
        const uint32_t ten_rows16 = (uint32_t)a.Nd * 4u;      // a tenant's digit rows x 64 B >> 4
        const uint32_t sfa = tmem_base + a.col_sf;
        Ring pr{0, 0u, n_ring}, fr{0, 0u, a.n_sf}, sr{0, 0u, a.n_sets};
        uint32_t accphase = 0;
        [[maybe_unused]] int ev_n = 0;
        FT_DECL(8);
        while (ok && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            FT_ADD(0);
            ok = warp_all(wait_bar(smem_u32(&ctl->accempty), accphase ^ 1, abort_flag, 3));
            FT_ADD(1);
            if (!ok) break;
            tc_fence_after();
            for (int p = p0; p < p1 && ok; ++p) {
                const uint32_t first = (p > p0) ? 1u : 0u;   // 0: this step starts the accumulation
                FT_ADD(0);
                ok = warp_all(wait_bar(smem_u32(&ctl->imgready[pr.idx]), pr.par, abort_flag, 13));
                FT_ADD(2);
                if (h == 0) FT_EV(6, ev_n);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sfb0 = sfa + 4u + (uint32_t)(fr.idx * (kTB8 ? 32 : 16));   // this step's scale factors (four columns per tenant)
                const uint64_t x4desc = desc64 + ((img_addr + (v_resident ? (p - p0) : pr.idx) * a.img_bytes + a.x_tile_bytes) >> 4);
#pragma unroll
                for (int s = 0; s < kSetsPerStep; ++s, sr.step()) {
                    // The 128 decode threads of this half arrive here once their columns of the set are filled (or when
                    // they give up after an abandoned wait, see the end of the decode role).
                    FT_ADD(0);
                    named_bar_sync(kFBarSet0 + 2 * sr.idx + h, kFHandover);
                    FT_ADD(4);
                    if (h == 0) FT_EV(7 + s, ev_n);
                    if (*abort_flag) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_set = tmem_base + a.col_a + (uint32_t)sr.idx * kFp4SetCols + (uint32_t)(h * 32);
                    if (elect_one()) {
                        for (int j = h; j < u.nten; j += 2) {
                            const uint32_t a_j = a_set + (uint32_t)((j >> 1) * kTenCols);
                            const uint32_t d_tmem = tmem_base + a.col_delta + (uint32_t)(j * a.Nd);
                            const uint64_t xj = x4desc + (uint32_t)j * ten_rows16;
                            const uint32_t sfb = sfb0 + (uint32_t)(4 * j);
                            if constexpr (kTB8) {
                                umma_ts_mxf4(d_tmem, a_j, xj + (uint32_t)(s * 2), idesc_delta | ((uint32_t)(2 * s) << 4), sfa, sfb, (s > 0) ? 1u : first);
                            } else {
                                umma_ts_mxf4(d_tmem, a_j, xj, idesc_delta, sfa, sfb, first);
                                umma_ts_mxf4(d_tmem, a_j + 8, xj + 2, idesc_delta | (2u << 4), sfa, sfb, 1u);
                            }
                        }
                        tc_commit(smem_u32(&ctl->opfree[h][sr.idx]));
                    }
                    __syncwarp();
                }
                if (!ok) break;
                if (elect_one()) tc_commit(smem_u32(&ctl->pempty[pr.idx]));
                __syncwarp();
                pr.step();
                fr.step();
                if (h == 0) FT_EV(9, ev_n);
                ++ev_n;
            }
            if (!ok) break;
            if (elect_one()) tc_commit(smem_u32(&ctl->accfull));
            __syncwarp();
            accphase ^= 1;
        }
        FT_ADD(0);
        if (h == 0) FT_OUT(24, 8);
    } else if (warp < kFWarpEpi0) {
        // ------------------------------------------- sign decode -> tensor memory
        const int h = (warp - kFWarpDecode0) >> 2;
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        bool ok = wait_bar(tmemready, 0, abort_flag, 20);
        named_bar_sync(kFBarDep, kFThreads - 32);   // (sleeps while the launch before this one is still running)
        tc_fence_after();
        const uint32_t tmem_base = ctl->tmem_base;
        if (v_resident) {
            grid_dependency_wait();
            write_resident_images();
        }
        const uint32_t tbuf0 = tmem_base + ((uint32_t)(quad * 32) << 16) + a.col_a + (uint32_t)(h * 32);
        Ring br{0, 0u, a.n_bits}, sr{0, 0u, a.n_sets};
        const int bits_row = a.bits_row;
        [[maybe_unused]] int ev_n = 0;
        const bool pair_slots = bits_row == 32;
        int pending = -1;
        FT_DECL(8);
        while (ok && it.next(unit, p0, p1)) {
            for (int p = p0; p < p1 && ok; ++p) {
                // 32-byte rows: a slot holds the steps 2*(p/2) and 2*(p/2)+1 and is waited for at the first step of it that
                // this segment takes; 16-byte rows: a slot per step
                if (!pair_slots || p == p0 || (p & 1) == 0) {
                    FT_ADD(0);
                    ok = wait_bar(smem_u32(&ctl->bfull[br.idx]), br.par, abort_flag, 6);
                    FT_ADD(1);
                    if (!ok) break;
                }
                if (warp == kFWarpDecode0) FT_EV(10, ev_n);
                // this warp's tenants j = 2i + h: their sign words of the step (128 k each)
                const uint8_t* bsl = smem + bits_off + br.idx * a.bslot_bytes + row * bits_row + (pair_slots ? (p & 1) * 16 : 0);
                uint4 wq[kTenPerWarp];
#pragma unroll
                for (int i = 0; i < kTenPerWarp; ++i)   // (tenants past the unit's own have no words in the slot: nothing is read for them)
                    wq[i] = (2 * i + h < a.TB) ? *reinterpret_cast<const uint4*>(bsl + (2 * i + h) * (kTileN * bits_row)) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int i = 0; i < kTenPerWarp; ++i) asm volatile("" : "+r"(wq[i].x), "+r"(wq[i].w));
                if (!pair_slots || (p & 1) == 1 || p + 1 == p1) {   // the slot's last step in this segment: it goes back
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->bempty[br.idx]));
                    br.step();
                }
#pragma unroll
                for (int s = 0; s < kSetsPerStep; ++s, sr.step()) {
                    uint32_t r[32];
                    if constexpr (kTB8) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            decode_word_e2m1(s ? wq[i].z : wq[i].x, r + 8 * i);
                            decode_word_e2m1(s ? wq[i].w : wq[i].y, r + 8 * i + 4);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            decode_word_e2m1(wq[i].x, r + 16 * i);
                            decode_word_e2m1(wq[i].y, r + 16 * i + 4);
                            decode_word_e2m1(wq[i].z, r + 16 * i + 8);
                            decode_word_e2m1(wq[i].w, r + 16 * i + 12);
                        }
                    }
                    // (keeps the decode arithmetic above the waits: the compiler would otherwise sink it to the store)
                    asm volatile("" : "+r"(r[0]), "+r"(r[7]), "+r"(r[8]), "+r"(r[15]), "+r"(r[16]), "+r"(r[23]), "+r"(r[24]), "+r"(r[31]));
                    // the previous set's stores complete, the set is handed over; then this set's buffer must be free
                    FT_ADD(0);
                    if (pending >= 0) {
                        tc_wait_st();
                        tc_fence_before();
                        named_bar_arrive(kFBarSet0 + 2 * pending + h, kFHandover);
                    }
                    FT_ADD(2);
                    ok = wait_bar(smem_u32(&ctl->opfree[h][sr.idx]), sr.par ^ 1, abort_flag, 7);
                    FT_ADD(3);
                    if (warp == kFWarpDecode0) FT_EV(11 + s, ev_n);
                    if (!ok) break;
                    tc_fence_after();
                    tmem_st32(tbuf0 + (uint32_t)sr.idx * kFp4SetCols, r);
                    pending = sr.idx;
                }
                ++ev_n;
            }
        }
        if (ok && pending >= 0) {
            tc_wait_st();
            tc_fence_before();
            named_bar_arrive(kFBarSet0 + 2 * pending + h, kFHandover);
        }
        FT_ADD(0);
        if (warp == kFWarpDecode0) FT_OUT(8, 8);
        if (*abort_flag) {
            // A wait was abandoned somewhere in the block: the issuer may be blocked on one of the named barriers (they
            // have no time-out); arrive on all of them so that it wakes up, sees the flag and leaves.
            __syncwarp();
            for (int s = 0; s < a.n_sets; ++s) named_bar_arrive(kFBarSet0 + 2 * s + h, kFHandover);
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const int etid = threadIdx.x - kFWarpEpi0 * 32;
        const int first_unit = (kForm == 1) ? cunit : fdiv(lo, a.mg_P);
        uint16_t* Y = reinterpret_cast<uint16_t*>(a.Y);
        uint32_t accphase = 0;
        bool ok = wait_bar(tmemready, 0, abort_flag, 20);
        tc_fence_after();
        const uint32_t tmem_base = ctl->tmem_base;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
        {
            // A-side scale factors (four columns: weight rows 32c + lane), once per launch, in this warp's lane quadrant
            // (every quadrant of the tensor core reads its own copy): 2^0.  Ordered before the first MMA by the
            // first image's hand-over below.
            uint32_t sf[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) sf[c] = 0x7F7F7F7Fu;
            tmem_st8(lane_taddr + a.col_sf, sf);
        }
        named_bar_sync(kFBarDep, kFThreads - 32);   // nothing else to do before the grid dependency is resolved; sleep until then
        grid_dependency_wait();                     // (returns at once: orders this thread's accesses behind the previous kernel's)
        if (v_resident) write_resident_images();
        if (warp == kFWarpEpi0) FT_STAMP(11);   // epilogue warps awake, tensor memory ready
        if (v_coop) {
            // This block's share of the launch's activation images (one tenant group): task = (step, token row, chunk).
            const Unit u0 = unit_info(a, 0);
            const uint32_t sf_off0 = a.x_tile_bytes + (uint32_t)(a.TB * a.Nd) * 64u;
            const int per_step = u0.ntok * 16;
            for (int task = (int)blockIdx.x * (kFEpiWarps * 32) + etid; task < a.P * per_step; task += (int)gridDim.x * (kFEpiWarps * 32)) {
                const int p = (int)((unsigned)task / (unsigned)per_step);
                const int rem = task - p * per_step;
                const int r = rem >> 4;
                const int j = r / am, t = r - j * am;
                fp4_split_task(reinterpret_cast<const uint16_t*>(a.X) + (size_t)(u0.xrow0 + r) * a.K + (size_t)p * kPairK,
                               a.img + (size_t)p * a.img_bytes, rem & 15, r, j, t, am, a.x_atom_bytes, a.x_tile_bytes, sf_off0);
            }
            if (warp == kFWarpEpi0) FT_STAMP(12);   // this block's share written
            __threadfence();
            epi_bar_sync(kFEpiWarps * 32);
            if (etid == 0) {
                const unsigned int old = atomicAdd(a.img_counter, 1u);
                ctl->img_target = (old / gridDim.x + 1u) * gridDim.x;   // (the launches of a stream take their turns: whole rounds)
                mbar_arrive(smem_u32(&ctl->cntready));
            }
            if (warp == kFWarpEpi0) FT_STAMP(13);   // counted
        }
        int pend_unit[2], pend_c0[2], pend_c1[2], npend = 0;   // cut tiles this block has to finish
        // While a tile is being accumulated these four warps prepare every step's activation operands.  Units of up to
        // 16 token rows (a.convert): they write the step's image themselves, one task per thread (fp4_split_task);
        // otherwise the producer's bulk copy brings it.  Either way they then move the image's scale table into
        // tensor memory: tenant j's MMAs read the scale factors of their digit rows n = q*m + t from lane n % 32 of
        // column 4 TB slot + 4 j + n / 32, one byte per 32-k group of the step: the group's exponent + 2q.
        // Steps of the current tile are served with blocking waits (the tile cannot complete without them), later
        // ones whenever their image slot is ready.
        FItem<kForm> si(it);
        bool more_s = si.next();
        Ring xr{0, 0u, n_ring}, fr{0, 0u, a.n_sf};
        int n_split = 0, seg_end = 0;
        const int p_first = is_cluster ? lo - cunit * a.P : lo - (int)((unsigned)lo / (unsigned)a.P) * a.P;   // (resident form: the block's first step)
        Unit us{};
        const uint32_t sf_off = a.x_tile_bytes + (uint32_t)(a.TB * a.Nd) * 64u;
        // (digit row n = q*m + t of a tenant: this lane serves n = lane and n = lane + 32)
        const int sf_t0 = lane % am, sf_t1 = (lane + 32) % am;
        const uint32_t sf_q0 = 0x02020202u * (uint32_t)(lane / am), sf_q1 = 0x02020202u * (uint32_t)((lane + 32) / am);
        const bool sf_v0 = lane < a.Nd, sf_v1 = lane + 32 < a.Nd;
        auto split_next = [&](bool block) -> bool {
            // convert: the slot must be free (its step's MMAs complete); else: its image must have landed
            const uint32_t bar = v_convert ? smem_u32(&ctl->pempty[xr.idx]) : smem_u32(&ctl->pfull[xr.idx]);
            const uint32_t par = v_convert ? (xr.par ^ 1) : xr.par;
            if (block) {
                if (!wait_bar(bar, par, abort_flag, 14)) return false;
            } else if (!warp_all(mbar_test_wait(bar, par))) {
                return false;
            }
            if (a.n_sf < n_ring && n_split >= a.n_sf) {
                // Fewer scale-factor slots in tensor memory than images in shared memory: this step's slot is the one of
                // the step n_sf before it, whose MMAs must be complete (the issuers' commits on that step's image slot).
                const int prev = n_split - a.n_sf;
                const uint32_t pbar = smem_u32(&ctl->pempty[prev % n_ring]);
                const uint32_t ppar = (uint32_t)(prev / n_ring) & 1u;
                if (block) {
                    if (!wait_bar(pbar, ppar, abort_flag, 15)) return false;
                } else if (!warp_all(mbar_test_wait(pbar, ppar))) {
                    return false;
                }
                tc_fence_after();
            }
            if (warp == kFWarpEpi0) FT_EV(13, n_split);
            if (si.first) us = unit_info(a, si.unit);
            uint8_t* im = smem + img_off + (v_resident ? (si.p - p_first) : xr.idx) * a.img_bytes;
            if (v_convert == 1) {
                const uint16_t* xstep = reinterpret_cast<const uint16_t*>(a.X) + (size_t)us.xrow0 * a.K + (size_t)si.p * kPairK;
                for (int task = etid; task < us.ntok * 16; task += kFEpiWarps * 32) {
                    const int r = task >> 4;
                    const int j = r / am, t = r - j * am;
                    fp4_split_task(xstep + (size_t)r * a.K, im, task & 15, r, j, t, am, a.x_atom_bytes, a.x_tile_bytes, sf_off);
                }
                fence_proxy_async_smem();   // generic-proxy writes -> visible to the MMAs' async-proxy reads
                epi_bar_sync(kFEpiWarps * 32);
                if (*abort_flag) return false;
            }
            {
                // (a tenant's scale factors start at a multiple of four columns: the MMA wants that alignment; all the
                // tenants' columns of the slot go out in one store, the unused ones with a neutral exponent)
                const uint32_t sf_slot = lane_taddr + a.col_sf + 4u + (uint32_t)(fr.idx * (kTB8 ? 32 : 16));
                const uint8_t* tab = im + sf_off;
                uint32_t r[kTB8 ? 32 : 16];
#pragma unroll
                for (int j = 0; j < (kTB8 ? 8 : 4); ++j) {
                    const bool live = j < us.nten;
                    r[4 * j] = (live && sf_v0) ? *reinterpret_cast<const uint32_t*>(tab + 4 * (j * am + sf_t0)) + sf_q0 : 0x7F7F7F7Fu;
                    r[4 * j + 1] = (live && sf_v1) ? *reinterpret_cast<const uint32_t*>(tab + 4 * (j * am + sf_t1)) + sf_q1 : 0x7F7F7F7Fu;
                    r[4 * j + 2] = 0x7F7F7F7Fu;
                    r[4 * j + 3] = 0x7F7F7F7Fu;
                }
                if constexpr (kTB8) tmem_st32(sf_slot, r);
                else tmem_st16(sf_slot, r);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->imgready[xr.idx]));
                if (warp == kFWarpEpi0) FT_EV(14, n_split);
            }
            xr.step();
            fr.step();
            ++n_split;
            more_s = si.next();
            return true;
        };
        FT_DECL(8);
        while (ok && it.next(unit, p0, p1)) {
            const Unit u = unit_info(a, unit);
            const int n = u.n0 + row;
            const bool whole = (p0 == 0 && p1 == a.P);
            // Lane j holds tenant j's scale.  ONE register, first read in the drain: an array indexed by the drain's tenant
            // loop would live in local memory, and storing it there would make this warp wait for the load (DRAM latency
            // when alpha is cold) right here, before it has handed the first step's scale factors to the issuers.
            const float al_lane = (lane < u.nten) ? __ldg(a.alpha + u.tenant0 + lane) : 0.f;
            seg_end += p1 - p0;
            while (ok && n_split < seg_end) ok = split_next(true);
            if (!ok) break;
            // until this tile's accumulators are complete: serve ahead whatever image slot is ready
            // (cluster form: the block has no other segment, and the kernel is better off without a second copy of that code)
            if constexpr (kForm != 1) {
                while (more_s && !warp_all(mbar_test_wait(smem_u32(&ctl->accfull), accphase))) {
                    if (!split_next(false)) break;
                }
            }
            float* slotp = nullptr;
            if (!whole && !is_cluster) {
                const int slot = (unit == first_unit) ? 2 * (int)blockIdx.x : 2 * (int)blockIdx.x + 1;
                slotp = a.partials + (size_t)slot * a.slot_floats;
            }
            FT_ADD(0);
            ok = wait_bar(smem_u32(&ctl->accfull), accphase, abort_flag, 8);
            FT_ADD(1);
            if (warp == kFWarpEpi0) FT_STAMP(6);   // accumulators complete
            if (!ok) break;
            tc_fence_after();
            accphase ^= 1;
            if (is_cluster) {
                // Cluster form: this block's partial sums go to its own shared memory (the W_base ring: every load
                // into it has landed and every MMA that read it has completed), token-major, one float per weight
                // row; the cluster's leader adds the blocks' partials up at the end of the kernel.
                const FClusterPartOut out{reinterpret_cast<float*>(smem) + row};
                epilogue_fp4_any_m(a, u, lane_taddr, out, al_lane, am);
                break;   // (one segment per block)
            }
            {
                const EpiOut<false, false> out{Y, slotp, a.N, n, row, u.xrow0, 0.f, a};
                epilogue_fp4_any_m(a, u, lane_taddr, out, al_lane, am);
            }
            // this warp's arrival on the "accumulators drained" barrier
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->accempty));
            FT_ADD(2);
            if (!whole) {
                // This tile is cut across blocks: publish the partial and count arrivals right away.  If this block is
                // the last to arrive it adds the partials up in block order and writes Y, after its other segments.
                const int first_item = unit * a.P;
                const int c0 = cta_of_item(a, first_item);
                const int c1 = cta_of_item(a, first_item + a.P - 1);
                epi_bar_sync(kFEpiWarps * 32);
                if (*abort_flag) break;
                if (etid == 0) {
                    unsigned old;
                    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(a.counters + unit) : "memory");
                    ctl->is_last = (old == (unsigned)(c1 - c0)) ? 1u : 0u;
                }
                epi_bar_sync(kFEpiWarps * 32);
                if (*abort_flag) break;
                if (ctl->is_last) {
                    pend_unit[npend] = unit;
                    pend_c0[npend] = c0;
                    pend_c1[npend] = c1;
                    ++npend;
                }
                FT_ADD(3);
            }
        }
        // Tiles this block was the last to arrive at (at most its first and its last segment).
        for (int k = 0; k < npend && ok && !*abort_flag; ++k) {
            const int un = pend_unit[k], c0 = pend_c0[k], c1 = pend_c1[k];
            const Unit u = unit_info(a, un);
            const int first_item = un * a.P;
            const int slot0 = (cta_first_item(a, c0) == first_item) ? 2 * c0 : 2 * c0 + 1;
            const float* first = a.partials + (size_t)slot0 * a.slot_floats;
            const float* rest = a.partials + (size_t)(2 * (c0 + 1)) * a.slot_floats;
            reduce_partials<false, false>(a, u, etid, kFEpiWarps, first, rest, 2 * (size_t)a.slot_floats, c1 - c0);
            if (etid == 0) a.counters[un] = 0u;
        }
        FT_ADD(4);
        if (warp == kFWarpEpi0) FT_OUT(16, 8);
        if (!ok) {
            // This warp left on an abandoned wait; a sibling that passed the same wait a moment earlier may be
            // waiting on the epilogue barrier: release it once (it then sees the flag and leaves too).
            __syncwarp();
            named_bar_arrive(1, kFEpiWarps * 32);
        }
    }

    // ------------------------------------------------------------------ teardown
    __syncthreads();
    if (warp == 0) FT_STAMP(7);   // all roles done
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
    if (warp == kFWarpMma) tmem_dealloc(ctl->tmem_base, kTmemCols);
    if (is_cluster) {
        // Cluster form: after a cluster barrier the leader's epilogue threads (one weight row each) add the blocks'
        // partial sums in block order, i.e. in k order, through the distributed shared memory window and write Y; a
        // second barrier keeps the other blocks' shared memory alive until it has read them.
        cluster_sync_all();
        if (warp == 0) FT_STAMP(8);   // cluster barrier passed
        if (crank == 0 && warp >= kFWarpEpi0 && lo < hi && !*abort_flag) {
            const Unit u = unit_info(a, cunit);
            const int row = (warp & 3) * 32 + lane;
            const int n = u.n0 + row;
            const uint32_t part = base + (uint32_t)row * 4u;   // this block's part[0][row]; same offset in every block
            uint32_t peer[8];
#pragma unroll
            for (int r = 1; r < 8; ++r) peer[r] = (r < a.cluster) ? mapa_shared(part, (uint32_t)r) : 0u;
            const EpiOut<false, false> out{reinterpret_cast<uint16_t*>(a.Y), nullptr, a.N, n, row, u.xrow0, 0.f, a};
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
        }
        if (warp == kFWarpEpi0) FT_STAMP(9);   // leader's sum stored
        cluster_sync_relaxed();
    }
    if (warp == 0) FT_STAMP(10);   // exit
}

#ifdef BD_TRACE
extern "C" int bitdelta_debug_set_trace_fp4(long long* buf) {
    return (int)cudaMemcpyToSymbol(g_fp4_trace, &buf, sizeof(buf));
}
#endif

static void* fp4_kernel(int mode) {   // mode: bit 0 = units of up to eight tenants; + 2 = one of the opt-in variants (either form), + 4 = cluster form
    switch (mode) {
        case 0: return reinterpret_cast<void*>(bitdelta_gemm_fp4_kernel<false, false, 0>);
        case 1: return reinterpret_cast<void*>(bitdelta_gemm_fp4_kernel<true, false, 0>);
        case 2: return reinterpret_cast<void*>(bitdelta_gemm_fp4_kernel<false, true, 2>);
        case 3: return reinterpret_cast<void*>(bitdelta_gemm_fp4_kernel<true, true, 2>);
        case 4: return reinterpret_cast<void*>(bitdelta_gemm_fp4_kernel<false, false, 1>);
        default: return reinterpret_cast<void*>(bitdelta_gemm_fp4_kernel<true, false, 1>);
    }
}

cudaError_t launch_gemm_fp4(const CUtensorMap& tmW, const CUtensorMap& tmBits, const GemmArgs& args, int grid, uint32_t smem_bytes,
                            bool early_start, cudaStream_t stream) {
    const int mode = (args.sets_per_step == 2 ? 1 : 0) + ((args.resident || args.coop || args.convert) ? 2 : (args.cluster > 1 ? 4 : 0));
    static std::atomic<unsigned char> attr_done[64][6];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_done[dev][mode].load()) {
        e = cudaFuncSetAttribute(fp4_kernel(mode), cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        if (e != cudaSuccess) return e;
        attr_done[dev][mode].store(1);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)kFThreads);
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
    switch (mode) {
        case 0: return cudaLaunchKernelEx(&cfg, bitdelta_gemm_fp4_kernel<false, false, 0>, tmW, tmBits, args);
        case 1: return cudaLaunchKernelEx(&cfg, bitdelta_gemm_fp4_kernel<true, false, 0>, tmW, tmBits, args);
        case 2: return cudaLaunchKernelEx(&cfg, bitdelta_gemm_fp4_kernel<false, true, 2>, tmW, tmBits, args);
        case 3: return cudaLaunchKernelEx(&cfg, bitdelta_gemm_fp4_kernel<true, true, 2>, tmW, tmBits, args);
        case 4: return cudaLaunchKernelEx(&cfg, bitdelta_gemm_fp4_kernel<false, false, 1>, tmW, tmBits, args);
        default: return cudaLaunchKernelEx(&cfg, bitdelta_gemm_fp4_kernel<true, false, 1>, tmW, tmBits, args);
    }
}

int fp4_max_active_clusters(uint32_t smem_bytes, int cluster) {
    if (cudaFuncSetAttribute(fp4_kernel(5), cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(cluster * 16));
    cfg.blockDim = dim3((unsigned)kFThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, bitdelta_gemm_fp4_kernel<true, false, 1>, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

cudaError_t read_fp4_status(unsigned int out[2]) {
    cudaError_t e = cudaMemcpyFromSymbol(out, g_device_status, sizeof(unsigned int) * 2);
    if (e != cudaSuccess) return e;
    if (out[0] != 0u) {
        const unsigned int zero[2] = {0u, 0u};
        e = cudaMemcpyToSymbol(g_device_status, zero, sizeof(zero));
    }
    return e;
}

}  // namespace bd
