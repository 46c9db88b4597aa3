// Host-side schedule of the tcgen05 BitDelta GEMM kernel: tile shapes, shared /
// tensor memory budget, work decomposition and workspace layout.  Pure integer
// arithmetic; shared by the launcher and the workspace-size query.
#pragma once
#include <cstdlib>
#include <cstddef>
#include <cstdint>

namespace bd {

constexpr int kTileN = 128;          // weight rows per tile = MMA M = TMEM lanes
constexpr int kPairK = 128;          // reduction extent of one pipeline stage (two 64-wide swizzle atoms)
constexpr int kAtomK = 64;           // bf16 elements in one 128-byte swizzled row
constexpr int kQuadK = 256;          // reduction extent of one sign-word slot (8 words = 32 bytes per row)
constexpr int kMaxStages = 8;
constexpr int kMaxBitSlots = 8;   // sign-word slots in shared memory: 2 in the decode schedules, up to 8 (small ones) in the tiled one
constexpr int kMaxASlots = 4;
constexpr int kPieces = 4;           // e5m2 pieces an activation is split into for the decode-regime delta MMA
constexpr int kTmemCols = 512;
constexpr int kMaxCtas = 256;        // upper bound on the grid, sizes the workspace
constexpr int kDecodeMaxM = 16;      // m <= 16: tenants are grouped into one tile
constexpr int kSmemBudget = 227 * 1024;
constexpr int kSmemCtrlBytes = 1024; // barriers, TMEM base, flags
constexpr int kFp4MaxSets = 6;      // operand sets of the 4-bit decode kernel in tensor memory, at most
// 4-bit decode schedule (see gemm_fp4.cu): signs and activation pieces as e2m1, block-scaled MMA with constant scales.
constexpr int kFp4Pieces = 8;        // radix-4 digits of a 16-bit fixed-point activation magnitude
constexpr int kFp4MaxM = 8;          // tokens per tenant
constexpr int kFp4SetCols = 64;      // one operand set in tensor memory: 8 tenants x 64 k, or 4 tenants x 128 k

struct Plan {
    int B, m, N, K;
    int decode;        // 1: tenants grouped (m <= 16); 0: token tiles of one tenant
    int TB;            // tenants per unit
    int tok_tile;      // tokens per unit and tenant in the tiled schedule (0 in decode)
    int Nb;            // N of the base MMA  (columns of the base accumulator)
    int Nd;            // N of a delta MMA   (columns of one tenant's delta accumulator)
    int win_rows;      // X-tile row where tenant j's delta window starts = j * win_rows
    int chunk_rows;    // epilogue: rows of the X tile between consecutive 16-token chunks
    int x_rows;        // rows of X staged per stage (TMA box height)
    int N3;            // decode: columns of one tenant's delta accumulator = round16(4 m) (pieces x tokens)
    int x8_rows;       // decode: rows of the e5m2 activation pieces staged per stage (0 in the tiled schedule)
    int convert;       // decode: 1 = the kernel itself splits the activations (few token rows per unit),
                       //         0 = a pre-pass kernel writes the pieces to the workspace
    int aslot_cols;    // TMEM columns of one decoded-operand buffer: decode ceil(TB/2)*16 (one decode group's
                       // tenants x 64 k of e5m2; a_slots buffers per group), tiled 64 (one tenant x 128 k of bf16)
    int n_tiles, m_tiles, groups, units;
    int P;             // k-pairs per unit
    int whole_units;   // 1: CTAs take whole units round-robin (no tile is cut), 0: even shares of the item list
    int teams;         // > 1: one team of grid/teams CTAs per tenant group; units are numbered group-major and each
                       // team cuts its group's items evenly (1: one cut of the whole list, units tile-major)
    long long T;       // total k-pair work items = units * P
    int grid;
    int n_w;           // ring of W_base tiles (128 rows x 128 k of bf16 each)
    int n_x;           // ring of bf16 activation tiles
    int n_x8;          // decode: ring of e5m2 piece tiles
    int n_bits;        // sign-word slots (each holds the signs of one k-pair of one unit)
    int stream;        // 1 = planned for the 4-bit decode kernel (operand sets handed to issuer warps, clusters or the flat list)
    int n_sets;        // 4-bit decode kernel: operand sets in tensor memory
    int cluster;       // 4-bit decode kernel: > 1 = every unit is taken by a cluster of this many blocks, each with an equal
                       // share of the unit's k-steps; their partial results meet in the leader's shared memory
                       // (no workspace traffic, no arrival counters); 0 = the flat work list
    int pair;          // tiled schedule on CTA pairs: a unit is two W_base tiles (256 rows), one per CTA of a cluster of
                       // two; each CTA stages its own weights and half of the activation tile, the pair's leader issues
                       // 256-row MMAs (tcgen05 cta_group::2)
    int fp4;           // 1: the 4-bit decode kernel (gemm_fp4.cu; a pre-pass writes the activation operands)
    int n_img;         // ... ring of activation operand images in shared memory (resident form: one image per step of a block)
    int n_sf;          // ... slots of B-side scale factors in tensor memory (<= n_img unless the images are resident)
    int coop;          // ... 1: cluster form: the launch's blocks write the activation images together, each a share of them, into
                       //     the workspace before their main loops (no pre-pass kernel); 0: a pre-pass kernel writes them
    int resident;      // ... 1: cluster form with few steps per block and few token rows: every block writes the images of all
                       //     its steps into shared memory itself, right after the grid dependency resolves (no pre-pass kernel)
    int bits_row;      // ... bytes per row of a sign-word slot: 32 = one slot per two 128-k steps, 16 = one per step
    int sets_per_step; // ... operand sets per 128-k step (2: eight tenants per unit, 1: four)
    uint32_t img_bytes;   // ... one image: 16-bit activation tile (two atoms) + e2m1 piece tile (64 bytes per row)
    uint32_t col_sf;      // ... first scale-factor column in tensor memory (4 for the A side, then the B side's)
    int a_slots;
    int halves;        // decode: operand hand-overs per 128-k stage (2: 64 k each, 1: the whole stage)
    uint32_t w_stage_bytes, x_tile_bytes, w_atom_bytes, x_atom_bytes, x8_atom_bytes, bslot_bytes, smem_bytes;
    uint32_t col_base, col_delta, col_a;
    size_t slot_floats;   // floats of one partial-result slot: 128 rows x tokens per unit
    size_t ws_header_bytes;   // arrival counters: one u32 per work unit
    size_t ws_partials_bytes; // two partial-result slots per CTA
    size_t ws_x8_bytes;       // decode: e5m2 pieces of X, [B, 4, m, K] bytes
    size_t ws_bytes;
    bool ok;
};

inline int round_up(int a, int b) { return (a + b - 1) / b * b; }

// The pair schedule is taken where it applies unless BITDELTA_PAIR=0 is set (experiments).
inline bool pair_enabled() {
    const char* e = getenv("BITDELTA_PAIR");
    return !(e && e[0] == '0');
}

// The 4-bit decode kernel (gemm_fp4.cu; m <= 8, plain bf16 calls).  By default it is taken where it measures faster than
// the 8-bit decode kernels: where its cluster form applies (one tenant group, clusters of 2-8 blocks per W_base tile),
// and on the flat work list with up to four token rows per tenant (5-20 % faster on fifteen shapes from 8 x 2 x 11008 x
// 4096 to 64 x 1 x 4096 x 4096; with 5-8 rows per tenant its activation images take the room of the W_base stages and the
// 8-bit kernel stays ahead).  BITDELTA_FP4=1: wherever it applies; BITDELTA_FP4=0: never.
inline int fp4_mode() {
    const char* e = getenv("BITDELTA_FP4");
    return (e && e[0] == '1') ? 1 : (e && e[0] == '0') ? 0 : 2;
}

// The cluster form of the 4-bit decode kernel is taken where it applies unless BITDELTA_CLUSTER=0 is set (experiments).
// (experiments) BITDELTA_FP4_BITS16=0: never the one-step sign-word slots of the 4-bit decode kernel.
// Columns of one scale-factor slot of the 4-bit decode kernel: four per tenant, written with one store of 16 or 32 columns.
inline int fp4_sf_slot_cols(int TB) { return TB > 4 ? 32 : 16; }
inline bool fp4_bits16_enabled() {
    const char* e = getenv("BITDELTA_FP4_BITS16");
    return !(e && e[0] == '0');
}
inline bool cluster_enabled() {
    const char* e = getenv("BITDELTA_CLUSTER");
    return !(e && e[0] == '0');
}

// allow_pair = false: the device cannot hold all the pairs (or clusters) at once (see the launcher), plan without them.
// force_tiled: plan the tiled schedule whatever m is (bf16 / binary16 operands for both terms).
// allow_fp4 = false: the call has options the 4-bit decode kernel does not take (binary16, bias, activation).
inline Plan make_plan(int B, int m, int N, int K, int num_sms, int tb_override = 0, int whole_override = 0,
                      bool allow_pair = true, bool force_tiled = false, bool allow_fp4 = true) {
    Plan p{};
    p.B = B; p.m = m; p.N = N; p.K = K;
    p.ok = false;
    if (B <= 0 || m <= 0 || N <= 0 || K <= 0 || (K % 128) != 0) return p;
    p.decode = (m <= kDecodeMaxM && !force_tiled) ? 1 : 0;
    p.n_tiles = (N + kTileN - 1) / kTileN;
    if (p.decode) {
        p.N3 = round_up(kPieces * m, 16);
        const int tb_max = (m <= 4) ? 8 : 4;          // keeps accumulators + two operand buffers within 512 columns
        p.TB = B < tb_max ? B : tb_max;
        if (tb_override > 0 && tb_override <= tb_max && tb_override <= B) p.TB = tb_override;
        p.tok_tile = 0;
        p.groups = (B + p.TB - 1) / p.TB;
        p.m_tiles = 1;
        p.Nb = round_up(p.TB * m, 16);
        p.Nd = p.N3;
        p.win_rows = m;
        p.chunk_rows = m;
        p.x_rows = p.Nb;   // the bf16 tile feeds the base MMA (N = Nb) and the in-kernel split only
        p.x8_rows = round_up((p.TB - 1) * kPieces * m + p.N3, 8);
        p.aslot_cols = ((p.TB + 1) / 2) * 16;
        p.convert = (p.TB * m <= 16) ? 1 : 0;   // 64 converter threads, one 32-k group of one row each
        p.slot_floats = (size_t)kTileN * p.TB * m;
        p.stream = 0;
        p.fp4 = (allow_fp4 && fp4_mode() != 0 && m <= kFp4MaxM) ? 1 : 0;
        if (p.fp4) {
            // 4-bit operands: eight e2m1 pieces per token stacked along N (tenant j's rows start at 8 m j), written by
            // a pre-pass together with the 16-bit tile of the base MMA as one image per (tenant group, 128-k step).
            p.stream = 1;
            // (BITDELTA_FP4_INKERNEL=1, experiments: with few token rows the kernel's epilogue warps write the images themselves;
            // measured slower than the pre-pass: every block of a tile column repeats the split)
            p.convert = (p.TB * m <= 16 && getenv("BITDELTA_FP4_INKERNEL") != nullptr) ? 1 : 0;
            p.Nd = kFp4Pieces * m;
            p.N3 = p.Nd;
            p.x_rows = round_up(p.TB * m, 8);        // (the base MMA's N = Nb may read past the tile's rows: ignored columns)
            p.x8_rows = p.TB * kFp4Pieces * m;
            p.sets_per_step = (p.TB > 4) ? 2 : 1;
        }
    } else if (m <= 64 && B > 1 && tb_override != 1) {
        // Tiled schedule, middle regime (16 < m <= 64): a unit holds several tenants, whose tokens share one
        // W_base tile and one base MMA (N = all their tokens); every tenant keeps its own delta accumulator
        // (N = m rounded up to 16) and its own operand buffer of decoded signs.  Tenant j's delta MMAs read the
        // activation rows from j*m on: a window that runs into the next tenant's rows, whose columns are ignored.
        p.tok_tile = round_up(m, 16);
        p.m_tiles = 1;
        p.Nd = p.tok_tile;
        const int tb_max = 128 / p.Nd;                  // 4 tenants up to m = 32, 2 up to m = 64
        p.TB = B < tb_max ? B : tb_max;
        p.groups = (B + p.TB - 1) / p.TB;
        p.Nb = round_up(p.TB * m, 16);
        p.win_rows = m;
        p.chunk_rows = 16;
        p.x_rows = round_up((p.TB - 1) * m + p.Nd, 8);
        if (p.x_rows < p.Nb) p.x_rows = p.Nb;
        p.N3 = 0;
        p.convert = 0;
        p.x8_rows = 0;
        p.aslot_cols = 64;
        p.slot_floats = (size_t)kTileN * p.TB * m;
    } else {
        p.TB = 1;
        p.tok_tile = m >= 128 ? 128 : round_up(m, 16);
        p.m_tiles = (m + p.tok_tile - 1) / p.tok_tile;
        p.groups = B * p.m_tiles;
        p.Nb = p.tok_tile;
        p.Nd = p.tok_tile;
        p.win_rows = 0;
        p.chunk_rows = 16;
        p.pair = (allow_pair && pair_enabled() && p.tok_tile >= 80 && (p.n_tiles % 2) == 0 && num_sms >= 2) ? 1 : 0;
        p.x_rows = p.pair ? p.tok_tile / 2 : p.tok_tile;   // a pair's CTAs stage half of the token tile each
        p.N3 = 0;
        p.convert = 0;
        p.x8_rows = 0;
        p.aslot_cols = 64;
        p.slot_floats = (size_t)kTileN * p.tok_tile;
    }
    p.units = (p.pair ? p.n_tiles / 2 : p.n_tiles) * p.groups;
    p.P = (K + kPairK - 1) / kPairK;
    p.T = (long long)p.units * p.P;
    if (p.T >= (1ll << 30)) return p;   // the kernel's work-split arithmetic is 32-bit
    int max_grid = num_sms < kMaxCtas ? num_sms : kMaxCtas;
    p.grid = p.T < max_grid ? (int)p.T : max_grid;
    if (p.pair) p.grid = 2 * (int)(p.T < max_grid / 2 ? p.T : max_grid / 2);   // clusters of two
    // Several tenant groups share each W_base tile; cut anywhere, the groups of a tile sit at different k at any
    // moment and W_base is fetched from HBM once per group.  Two work orders keep them in step instead, so
    // that all but the first read of a W_base tile hit L2:
    //  * teams: one team of CTAs per tenant group, units numbered group-major, every team cutting its group's
    //    items (all tiles x all k) the same way: CTA i of every team is at the same (tile, k) at the same
    //    time.  Costs the CTAs left over when the groups do not divide the SM count.
    //  * whole units: every CTA takes whole units in round-robin order, the groups of a tile run on
    //    neighbouring CTAs.  Costs the idle CTAs of the last round.
    // The one that keeps more of the chip busy is taken if that is at least 85 %; else the plain even cut.
    // whole_override (experiments): 1 whole units, 3 teams, 2 not whole units, 4 plain cut.
    p.whole_units = 0;
    p.teams = 1;
    if ((p.decode || p.win_rows > 0) && p.groups > 1) {   // (not the tiled schedule with one tenant per unit)
        double s_whole = 0.0, s_teams = 0.0;
        if (p.units >= max_grid) {
            const int rounds = (p.units + max_grid - 1) / max_grid;
            s_whole = (double)p.units / ((double)rounds * max_grid);
        }
        const long long Tg = (long long)p.n_tiles * p.P;
        int cpt = max_grid / p.groups;
        if (cpt > Tg) cpt = (int)Tg;
        if (cpt >= 1) s_teams = (double)(cpt * p.groups) / max_grid;
        int pick = 0;   // 0 plain cut, 1 whole units, 3 teams
        if (s_teams >= 0.85 && s_teams >= s_whole) pick = 3;
        else if (s_whole >= 0.85) pick = 1;
        if (whole_override == 1 && p.units >= max_grid) pick = 1;
        if (whole_override == 3 && cpt >= 1) pick = 3;
        if (whole_override == 2 && pick == 1) pick = (s_teams >= 0.85) ? 3 : 0;
        if (whole_override == 4) pick = 0;
        if (pick == 1) { p.whole_units = 1; p.grid = max_grid; }
        if (pick == 3) { p.teams = p.groups; p.grid = cpt * p.groups; }
    }

    // Streaming kernel, one tenant group: if clusters of 2, 4 or 8 blocks (one cluster per W_base tile, the k-steps
    // dealt evenly to its blocks) fill at least 80 % of the blocks the flat list would use, take the largest such
    // cluster: no tile is then cut at an arbitrary place, every block has one segment, and the partial sums are
    // added up through distributed shared memory instead of a workspace, arrival counters and L2 round trips.
    p.cluster = 0;
    if (p.stream && p.groups == 1 && allow_pair && cluster_enabled()) {
        for (int c = 8; c >= 2; c >>= 1) {
            if (p.units * c <= max_grid && p.P >= c && 10 * p.units * c >= 8 * p.grid) {
                p.cluster = c;
                p.grid = p.units * c;
                p.whole_units = 0;
                p.teams = 1;
                break;
            }
        }
    }
    // (the 4-bit kernel divides item and unit numbers by multipliers that are exact while the product stays below 2^32)
    if (p.fp4) {
        int dmax = p.P > p.n_tiles ? p.P : p.n_tiles;
        if (p.groups > dmax) dmax = p.groups;
        if ((unsigned long long)p.T * (unsigned long long)dmax >= 0x100000000ull)
            return make_plan(B, m, N, K, num_sms, tb_override, whole_override, allow_pair, force_tiled, false);
    }
    // (default: the flat list of the 4-bit kernel only with up to four token rows per tenant)
    if (p.fp4 && fp4_mode() == 2 && p.cluster <= 1 && m > 4) return make_plan(B, m, N, K, num_sms, tb_override, whole_override, allow_pair, force_tiled, false);

    p.w_atom_bytes = kTileN * 128;
    p.x_atom_bytes = (uint32_t)p.x_rows * 128;
    p.x8_atom_bytes = (uint32_t)p.x8_rows * 128;
    p.w_stage_bytes = 2 * p.w_atom_bytes;
    p.x_tile_bytes = 2 * p.x_atom_bytes;
    p.bslot_bytes = (uint32_t)p.TB * kTileN * 32;
    // Shared memory: rings of W_base tiles, of bf16 activation tiles and (decode) of e5m2 piece tiles, and
    // the sign-word slots.  W_base comes from DRAM (latency ~1.5 us under load); it and the bf16
    // activations are released as soon as the base MMAs have read them.  The piece tiles come from L2 (or
    // are written in place by the in-kernel split), but stay in use until the last delta MMA of their
    // stage has completed, which is the longest hold of all: three of them.  Every remaining byte goes to
    // W_base.  The tiled schedule keeps one ring (activation tile s lives and dies with W_base tile s).
    // Sign words: two slots in the decode schedules (16-64 KB each; they travel with the W_base stream).  In the
    // tiled schedule a slot is 4 KB and the words have a stream of their own that runs well ahead of W_base:
    // the decode warps need them long before the MMAs of their stage (they fill a ring of operand buffers).
    p.n_bits = 2;
    if (!p.decode) {
        p.n_bits = (int)(32768u / p.bslot_bytes);
        if (p.n_bits > kMaxBitSlots) p.n_bits = kMaxBitSlots;
        if (p.n_bits < 2) p.n_bits = 2;
    }
    const int avail = kSmemBudget - 1024 /*alignment slack*/ - kSmemCtrlBytes - p.n_bits * (int)p.bslot_bytes;
    if (p.fp4) {
        // A whole multiprocessor per block: two sign-word slots (256 k each, 32-byte rows: a copy-engine operation costs
        // about a cycle per row whatever its width), three activation images if they fit, the rest for W_base tiles.
        p.img_bytes = (uint32_t)round_up((int)p.x_tile_bytes + p.x8_rows * 64 + 4 * p.TB * p.m, 1024);   // tile, digit rows, scale table
        p.n_bits = 2;
        const int fixed = 1024 + kSmemCtrlBytes + p.n_bits * (int)p.bslot_bytes;
        p.n_img = 3;
        p.n_w = (kSmemBudget - fixed - p.n_img * (int)p.img_bytes) / (int)p.w_stage_bytes;
        p.bits_row = 32;
        if (p.n_w < 3 && fp4_bits16_enabled()) {
            // Three images do not fit next to three W_base stages: three sign-word slots of one step each (16-byte rows,
            // the same depth in steps on average) free a quarter of the sign-word memory for the third image.
            const uint32_t half = p.bslot_bytes / 2;
            const int nw = (kSmemBudget - 1024 - kSmemCtrlBytes - 3 * (int)half - 3 * (int)p.img_bytes) / (int)p.w_stage_bytes;
            if (nw >= 3) {
                p.bits_row = 16;
                p.bslot_bytes = half;
                p.n_bits = 3;
                p.n_w = nw;
            }
        }
        if (p.n_w < 3) {
            p.n_img = 2;
            p.n_w = (kSmemBudget - fixed - p.n_img * (int)p.img_bytes) / (int)p.w_stage_bytes;
        }
        if (p.n_w > 4) p.n_w = 4;
        // (eight tenants of one token row: a fourth W_base stage measured SLOWER than three: 8 x 1 x 4096 x 4096 14.85 vs 14.45
        // us, K = 8192 24.7 vs 23.8, 16 x 1 x 4096 x 4096 25.5 vs 24.7, 8 x 1 x 4096 x 11008 31.1 vs 29.7; with fewer tenants per
        // unit or more token rows per tenant the two are level or the fourth stage is ahead by 0.1-0.2 us)
        if (p.n_w > 3 && p.TB > 4 && m == 1) p.n_w = 3;
        p.n_sf = p.n_img;
        p.resident = 0;
        if (p.cluster > 1 && p.TB * m <= 16 && p.convert == 0 && getenv("BITDELTA_FP4_RESIDENT") != nullptr) {
            // (experiments) Resident images: all the steps of a block ((P + cluster - 1) / cluster of them) if that leaves three
            // W_base stages.  Measured slower than the pre-pass (20.6 vs 17.7 us on 8 x 1 x 4096 x 4096, no faster with the inputs
            // resident in L2): every block repeats the split of its k range, ~250 integer instructions per eight values,
            // before its main loop can start.
            const int steps = (p.P + p.cluster - 1) / p.cluster;
            const int nw = (kSmemBudget - fixed - steps * (int)p.img_bytes) / (int)p.w_stage_bytes;
            if (nw >= 3) {
                p.resident = 1;
                p.convert = 2;
                p.n_img = steps;
                p.n_sf = 3;
                p.n_w = nw > 4 ? 4 : nw;
            }
        }
        // (experiments, BITDELTA_FP4_COOP=1) Cluster form, every block of the launch resident at once: the blocks write the
        // images together, each a share, and count themselves in the workspace; no pre-pass kernel.  Measured slower than
        // the pre-pass (20.5 vs 18.3 us on 8 x 1 x 4096 x 4096): shares written 1.7 us after the grid dependency resolves,
        // but fence + count + the slowest block + the fetch add up to 9.5 us before the first MMA (pre-pass chain: 9.3).
        p.coop = (p.cluster > 1 && !p.resident && p.convert == 0 && getenv("BITDELTA_FP4_COOP") != nullptr) ? 1 : 0;
        p.n_x = p.n_img;
        p.n_x8 = p.n_img;
    } else if (p.decode) {
        p.n_x8 = 3;
        p.n_x = (p.x_tile_bytes <= 4 * 1024) ? 3 : 2;
        p.n_w = (avail - p.n_x * (int)p.x_tile_bytes - p.n_x8 * (int)p.x8_atom_bytes) / (int)p.w_stage_bytes;
        if (p.n_w < 2) {
            p.n_x8 = 2;
            p.n_w = (avail - p.n_x * (int)p.x_tile_bytes - p.n_x8 * (int)p.x8_atom_bytes) / (int)p.w_stage_bytes;
        }
        if (p.n_w > 6) p.n_w = 6;
        if (p.convert && p.n_w >= 3) {
            // Few token rows per unit: the activation and piece tiles are small.  Three W_base stages are
            // enough (deeper rings measured no faster); the rest buys activation slots, so that the epilogue
            // warps can split several stages ahead -- during the start-up of a launch, when nothing else
            // runs, they get through most of a short CTA's stages.
            p.n_w = 3;
            int n = (avail - p.n_w * (int)p.w_stage_bytes) / (int)(p.x_tile_bytes + p.x8_atom_bytes);
            if (n > kMaxStages) n = kMaxStages;
            if (n > p.n_x) { p.n_x = n; p.n_x8 = n; }
        }
    } else {
        p.n_x8 = 0;
        p.n_w = avail / (int)(p.w_stage_bytes + p.x_tile_bytes);
        if (p.n_w > kMaxStages) p.n_w = kMaxStages;
        p.n_x = p.n_w;
    }
    if (p.n_w < 2) return p;
    p.smem_bytes = 1024 + p.n_w * p.w_stage_bytes + p.n_x * p.x_tile_bytes + p.n_x8 * p.x8_atom_bytes +
                   p.n_bits * p.bslot_bytes + kSmemCtrlBytes;
    if (p.fp4) {
        p.smem_bytes = 1024 + p.n_w * p.w_stage_bytes + p.n_img * p.img_bytes + p.n_bits * p.bslot_bytes + kSmemCtrlBytes;
    } else if (p.smem_bytes < 120 * 1024) {
        // One CTA per SM is assumed by this kernel's TMEM allocation: keep the request above half an SM.
        p.smem_bytes = 120 * 1024;
    }

    p.col_base = 0;
    p.col_delta = (uint32_t)p.Nb;
    p.col_a = p.col_delta + (uint32_t)(p.TB * p.Nd);
    int free_cols = kTmemCols - (int)p.col_a;
    p.halves = 2;
    if (p.decode && free_cols >= 2 * 2 * 2 * p.aslot_cols) {
        // Room for two whole-stage buffers per decode group: hand over 128 k at a time, which halves
        // the number of hand-overs (their fixed cost is comparable to the decode work of 64 k).
        p.halves = 1;
        p.aslot_cols *= 2;
    }
    int slots = free_cols / p.aslot_cols;
    if (p.decode) slots /= 2;                          // each of the two decode groups has its own ring
    p.a_slots = slots >= 4 ? 4 : slots >= 2 ? 2 : 0;   // power of two
    if (p.a_slots > kMaxASlots) p.a_slots = kMaxASlots;
    if (p.fp4) {
        // [base | delta accumulators | scale factors: 4 columns for the A side, 4 per tenant and image slot for the B side |
        //  operand sets of 64 columns]
        p.col_sf = p.col_a;
        // (the pre-pass form may keep fewer scale-factor slots than images: two are enough to run, and with wide
        // accumulators the columns are worth more as operand sets)
        for (;;) {
            const int col_a = round_up((int)p.col_sf + 4 + fp4_sf_slot_cols(p.TB) * p.n_sf, 32);
            if (p.n_sf <= 2 || p.convert != 0 || p.resident || (kTmemCols - col_a) / kFp4SetCols >= 4) break;
            --p.n_sf;
        }
        p.col_a = (uint32_t)round_up((int)p.col_sf + 4 + fp4_sf_slot_cols(p.TB) * p.n_sf, 32);
        p.halves = 2;
        p.n_sets = (kTmemCols - (int)p.col_a) / kFp4SetCols;
        if (p.n_sets > kFp4MaxSets) p.n_sets = kFp4MaxSets;
        if (p.n_sets < 2) return p;
        p.a_slots = 2;
    }
    if (p.a_slots < 2) return p;

    // Workspace: arrival counters, two partial-result slots per CTA, then (decode) the e5m2
    // pieces of X written by the activation-split kernel.
    p.ws_header_bytes = (size_t)round_up((p.n_tiles * p.groups + 1) * 4, 1024);   // one arrival counter per W_base tile and group,
                                                                                  // and (last word) the activation-image counter of the 4-bit kernel
    // (sized for the largest grid any device could get, so that the size does not depend on the device;
    // never more CTAs than items)
    const long long items = p.pair ? 2 * p.T : p.T;
    const long long max_ctas = items < kMaxCtas ? items : kMaxCtas;
    p.ws_partials_bytes = (size_t)2 * (size_t)max_ctas * p.slot_floats * sizeof(float);
    p.ws_x8_bytes = p.decode ? (((size_t)B * kPieces * m * K + 1023) / 1024 * 1024) : 0;
    if (p.fp4) p.ws_x8_bytes = (size_t)p.groups * p.P * p.img_bytes;   // one image per (tenant group, 128-k step)
    p.ws_bytes = p.ws_header_bytes + p.ws_partials_bytes + p.ws_x8_bytes;
    p.ok = true;
    return p;
}

}  // namespace bd
