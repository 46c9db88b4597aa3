// Device-side arguments and launcher of the tcgen05 BitDelta GEMM kernel.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "plan.h"

namespace bd {

struct GemmArgs {
    int B, m, N, K;
    int decode, convert, TB, tok_tile, Nb, Nd, win_rows, chunk_rows, aslot_cols;
    int pair;            // tiled schedule on CTA pairs (see plan.h)
    int f16;             // 0: X, W_base, bias, Y are bf16; 1: IEEE binary16
    int act;             // fused epilogue: 0 none, 1 SiLU (after the bias)
    const void* bias;    // [N] values of the I/O type added to every output row, or nullptr
    int m_tiles, groups, P, whole_units;
    int teams, Tg, cpt, n_tiles;   // work split by teams (see plan.h); q, r then describe one team's cut
    int T;             // work items (< 2^30)
    int q, r;          // T = q * grid + r
    int n_w, n_x, n_x8, n_bits, a_slots, halves;
    int n_sets;          // 4-bit decode kernel: operand sets in tensor memory
    int cluster;         // ... blocks per cluster (one cluster per unit), or 0: flat work list
    int hold_prefetch;   // decode: hold further weight loads until the first sign words have landed
    int fp4;             // 4-bit decode kernel (gemm_fp4.cu) ...
    int n_img;           // ... ring of activation operand images (resident form: one per step of a block)
    int n_sf;            // ... slots of B-side scale factors in tensor memory
    int resident;        // ... the block writes the images of all its steps itself, once, before its main loop
    int coop;            // ... the launch's blocks write the images together into the workspace (no pre-pass kernel)
    unsigned int* img_counter;   // ... and count themselves here when their share is written
    int sets_per_step;   // ... operand sets per 128-k step
    uint32_t mg_P, mg_tiles, mg_groups, mg_TB;   // ... ceil(2^32 / d) for d = P, n_tiles, groups, TB (0 for d = 1): x / d = umulhi(x, mg) while x * d < 2^32
    int bits_row;        // ... bytes per row of a sign-word slot: 32 (a slot per two steps) or 16 (a slot per step)
    uint32_t img_bytes;  // ... bytes of one image (16-bit activation tile, then the e2m1 piece tile)
    uint32_t col_sf;     // ... first scale-factor column in tensor memory
    uint8_t* img;        // ... images written by the pre-pass (or by the launch itself, coop): [group][step][img_bytes]
    uint32_t w_stage_bytes, x_tile_bytes, w_atom_bytes, x_atom_bytes, x8_atom_bytes, bslot_bytes;
    uint32_t col_delta, col_a;
    uint32_t slot_floats;
    const float* alpha;
    const void* X;       // [B*m, K] activations (16-bit values): the 4-bit decode kernel's in-kernel split reads them with
                         // plain loads; the other kernels use their tensor map
    void* Y;
    unsigned int* counters;
    float* partials;
};

// ceil(2^32 / d) (0 for d <= 1): x / d = umulhi(x, magic) as long as x * d < 2^32.
inline uint32_t magic_u32(int d) { return d <= 1 ? 0u : (uint32_t)((0x100000000ull + (unsigned long long)d - 1ull) / (unsigned long long)d); }
inline GemmArgs make_args(const Plan& p, const float* alpha, void* Y, void* workspace) {
    GemmArgs a{};
    a.B = p.B; a.m = p.m; a.N = p.N; a.K = p.K;
    a.decode = p.decode; a.convert = p.convert; a.TB = p.TB; a.tok_tile = p.tok_tile; a.Nb = p.Nb; a.Nd = p.Nd;
    a.win_rows = p.win_rows; a.chunk_rows = p.chunk_rows; a.aslot_cols = p.aslot_cols;
    a.m_tiles = p.m_tiles; a.groups = p.groups; a.P = p.P; a.T = (int)p.T; a.whole_units = p.whole_units;
    a.pair = p.pair;
    a.teams = p.teams; a.Tg = (int)(p.T / p.teams); a.cpt = (p.pair ? p.grid / 2 : p.grid) / p.teams; a.n_tiles = p.n_tiles;
    a.q = a.Tg / a.cpt; a.r = a.Tg % a.cpt;
    a.n_w = p.n_w; a.n_x = p.n_x; a.n_x8 = p.n_x8; a.n_bits = p.n_bits; a.a_slots = p.a_slots; a.hold_prefetch = 1; a.halves = p.halves;
    a.n_sets = p.n_sets; a.cluster = p.cluster;
    a.w_stage_bytes = p.w_stage_bytes; a.x_tile_bytes = p.x_tile_bytes; a.w_atom_bytes = p.w_atom_bytes; a.x_atom_bytes = p.x_atom_bytes;
    a.x8_atom_bytes = p.x8_atom_bytes;
    a.bslot_bytes = p.bslot_bytes;
    a.col_delta = p.col_delta; a.col_a = p.col_a;
    a.slot_floats = (uint32_t)p.slot_floats;
    a.alpha = alpha; a.Y = Y;
    a.counters = reinterpret_cast<unsigned int*>(workspace);
    char* ws = reinterpret_cast<char*>(workspace);
    a.partials = reinterpret_cast<float*>(ws + p.ws_header_bytes);
    a.fp4 = p.fp4; a.n_img = p.n_img; a.n_sf = p.n_sf; a.resident = p.resident; a.coop = p.coop;
    a.img_counter = reinterpret_cast<unsigned int*>(ws + p.ws_header_bytes) - 1; a.sets_per_step = p.sets_per_step; a.bits_row = p.bits_row;
    a.mg_P = magic_u32(p.P); a.mg_tiles = magic_u32(p.n_tiles); a.mg_groups = magic_u32(p.groups); a.mg_TB = magic_u32(p.TB); a.img_bytes = p.img_bytes; a.col_sf = p.col_sf;
    a.img = reinterpret_cast<uint8_t*>(ws + p.ws_header_bytes + p.ws_partials_bytes);
    return a;
}

#ifdef __CUDACC__
#define BD_HD __host__ __device__ __forceinline__
#else
#define BD_HD inline
#endif
// Work split.  The T = q*G + r items (T < 2^30) are cut evenly across the G CTAs: CTA b owns
// [b*q + min(b, r), ...), i.e. the first r CTAs take q+1 items.  32-bit arithmetic only: 64-bit
// divisions cost several hundred cycles each and sit on the kernel's start-up and tail paths.
// With teams (one per tenant group, cpt CTAs each) the same cut is applied to each team's Tg items.
// (Host and device: the kernel uses them, and the plan queries of the C ABI report them.)
BD_HD int cta_first_item(const GemmArgs& a, int b) {
    int base = 0;
    if (a.teams > 1) {
        const int t = (int)((unsigned)b / (unsigned)a.cpt);
        b -= t * a.cpt;
        base = t * a.Tg;
    }
    return base + b * a.q + (b < a.r ? b : a.r);
}
BD_HD int cta_of_item(const GemmArgs& a, int i) {
    int base = 0;
    if (a.teams > 1) {
        const int t = (int)((unsigned)i / (unsigned)a.Tg);
        i -= t * a.Tg;
        base = t * a.cpt;
    }
    const int big = a.r * (a.q + 1);
    return base + ((i < big) ? (int)((unsigned)i / (unsigned)(a.q + 1)) : a.r + (int)((unsigned)(i - big) / (unsigned)a.q));
}

// Workspace regions of the decode schedule.
inline uint8_t* ws_x8(const Plan& p, void* workspace) {
    return reinterpret_cast<uint8_t*>(workspace) + p.ws_header_bytes + p.ws_partials_bytes;
}

// tmX8 is only read in the decode schedule with a pre-pass split; `early_start` launches the kernel so
// that it may begin (prologue, weight prefetch) while the kernel queued just before it is still running.
cudaError_t launch_gemm_tc(const CUtensorMap& tmW, const CUtensorMap& tmX, const CUtensorMap& tmX8,
                           const CUtensorMap& tmBits, const GemmArgs& args, int grid, uint32_t smem_bytes,
                           bool early_start, cudaStream_t stream);

// Status word of the plain kernels' translation unit (read and cleared; the stream must be idle): the pre-pass
// activation split of the 8-bit decode schedule flags out-of-range values there.
cudaError_t read_simple_status(unsigned int out[2]);

// Number of CTA pairs (clusters of two) of the pair schedule's kernel that the current device can hold at once
// with `smem_bytes` of dynamic shared memory each (0 if the query fails).
int max_active_pairs(uint32_t smem_bytes);

// Decode schedule pre-pass: X bf16 [rows, K] -> four e5m2 pieces per element (k permuted inside
// each group of 32) in X8 [B, 4, m, K].
cudaError_t launch_x_split(const void* X, uint8_t* X8, int B, int m, int K, int f16, cudaStream_t stream);

// The 4-bit decode kernel (plan.fp4).  Pre-pass: per tenant group and 128-k step the shared-memory image of the
// activation operands (16-bit tile, eight e2m1 digit rows per token, one exponent per token and 32 k).
cudaError_t launch_x_split_fp4(const void* X, uint8_t* img, const Plan& p, bool early_start, cudaStream_t stream);
cudaError_t launch_gemm_fp4(const CUtensorMap& tmW, const CUtensorMap& tmBits, const GemmArgs& args, int grid, uint32_t smem_bytes,
                            bool early_start, cudaStream_t stream);
int fp4_max_active_clusters(uint32_t smem_bytes, int cluster);
cudaError_t read_fp4_status(unsigned int out[2]);

// One warp that lets a bounded wait expire after `limit_cycles` (see bitdelta_selftest_timeout).
cudaError_t launch_selftest_timeout(long long limit_cycles, int site, cudaStream_t stream);

// Synchronises the stream, reads {status, site} and clears them if set.
cudaError_t read_device_status(unsigned int out[2], cudaStream_t stream);

// Plain kernels (pack / unpack / CUDA-core GEMM).
cudaError_t launch_pack(const int8_t* S, uint32_t* bits, long long words, cudaStream_t stream);
cudaError_t launch_unpack(const uint32_t* bits, int8_t* S, long long words, cudaStream_t stream);
// Compress step: signs and per-tenant scale from fine-tuned weights; `partial` holds B x compress_blocks doubles.
long long compress_blocks(int N, int K);
cudaError_t launch_compress(const void* Wf, const void* Wb, uint32_t* bits, float* alpha, double* partial, int B, int N,
                            int K, cudaStream_t stream);
cudaError_t launch_gemm_simt(const void* X, const void* W, const uint32_t* bits, const float* alpha, const void* bias,
                             void* Y, int B, int m, int N, int K, int f16, int act, cudaStream_t stream);

}  // namespace bd
