// Device-side data shared by the kernels of the EAD gate step and the host API.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ead {

constexpr int kTileN = 256;        // vocabulary columns per accumulator tile (MMA N)
constexpr int kTileM = 128;        // batch rows per accumulator tile (MMA M = TMEM lanes)
constexpr int kBlockK = 64;        // hidden elements per pipeline stage (128 B of bf16)
constexpr int kUnit = 16;          // granularity of a CTA's vocabulary range (MMA N step)
constexpr int kMaxStages = 8;
constexpr int kMaxCtas = 256;         // upper bound on the LM-head grid (one CTA per SM)
constexpr int kWTileBytes = kTileN * kBlockK * 2;   // 32 KiB
constexpr int kSmemCtrlBytes = 1024;
constexpr int kTransposeBytes = 4 * 32 * 33 * 4;    // four 32 x 33 float tiles (one per epilogue warp)
constexpr int kLmheadThreads = 192;                 // TMA warp, MMA warp, 4 epilogue warps
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegSentinel = -1.0e30f;            // "no logit seen yet"; finite on purpose
constexpr uint32_t kStatusNonFinite = 0x1u;
constexpr uint32_t kStatusWaitExpired = 0x2u;
constexpr uint32_t kStatusBadCount = 0x4u;
constexpr uint32_t kStatusShardMismatch = 0x8u;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // bounded waits give up after 2 s

// Step control block (device resident, one per context).
struct StepCtl {
    int32_t step;       // gate steps taken since the last reset
    int32_t cur_t;      // copy of `step` taken by the compaction kernel for this step
    int32_t n[2];       // rows served by the small / large head in this step
    uint32_t status;    // sticky EAD_STATUS_* bits
    int32_t n_done;     // rows whose sequence has ended (served by neither head)
    int32_t xstep;      // vocabulary-sharded use: steps taken since the exchange buffers were
                        // connected (ead_reset leaves it alone); numbers the exchanged records
    int32_t cur_x;      // copy of `xstep` taken by the compaction kernel for this step
};

// Caller buffers of the current ead_step / ead_run call (device resident so that a
// captured graph does not freeze pointers).  Step `step - run_base` of the run reads
// row block [idx * B, (idx + 1) * B) of the inputs and writes the same of the outputs.
struct RunArgs {
    const uint16_t *h[2];
    int32_t *tok;
    float *H;
    float *Hbar;
    uint8_t *used;
    uint8_t *next;
    float *shard_out;   // vocabulary-sharded use: receives this shard's record per row instead
    int32_t run_base;
    int32_t pad;
};

// Record that one vocabulary shard produces per sequence (caller's row order): the statistics of
// its slice of the active model's logits, with vocabulary indices of the full head.
struct ShardRecord {
    float m, s, t;
    int32_t idx;
    float k;            // sampling: largest perturbed logit of the slice ...
    int32_t ki;         // ... and its index
    int32_t model;      // head the slice belongs to (must agree between the shards)
    int32_t step1;      // 1 + number of the exchange step the record belongs to; written last
};

// Where a shard delivers its records when the exchange runs inside the kernels: all[d] is the
// exchange buffer of shard d ([2][n][B] records: step parity, source shard, row) as addressable
// from this GPU; all[self] is local memory.
constexpr int kMaxShards = 16;
struct ShardLink {
    ShardRecord *all[kMaxShards];
    int32_t n, self;
};
static_assert(sizeof(ShardRecord) == 32, "two 16-byte words per record");

// How the CTAs of the LM-head kernel divide one head.  With n rows on the head there
// are R = ceil(n / 128) row blocks; the first g * R CTAs (g = G / R) form R groups of
// g CTAs; group member `slot` owns the vocabulary units [slot * U / g, (slot + 1) * U / g)
// of 16 columns (U = ceil(V / 16)) for row block rb.  CTAs with the same slot work on
// the same vocabulary range at about the same time, so a weight tile fetched by one is
// an L2 hit for the others.
struct HeadSplit {
    int R, g, rb, slot, active;
    int col_begin, col_end;    // multiples of 16; col_end may exceed V by < 16
};

__host__ __device__ inline HeadSplit split_head(int cta, int G, int n, int V)
{
    HeadSplit s;
    s.R = (n + kTileM - 1) / kTileM;
    if (n <= 0) {
        s.g = 0; s.rb = 0; s.slot = 0; s.active = 0; s.col_begin = s.col_end = 0;
        return s;
    }
    s.g = G / s.R;
    if (s.g < 1) s.g = 1;      // R > G is rejected on the host (B <= 4096 gives R <= 32)
    s.active = cta < s.g * s.R;
    s.rb = cta % s.R;
    s.slot = cta / s.R;
    const long long U = (V + kUnit - 1) / kUnit;
    s.col_begin = static_cast<int>((U * s.slot) / s.g) * kUnit;
    s.col_end = static_cast<int>((U * (s.slot + 1)) / s.g) * kUnit;
    if (!s.active) s.col_begin = s.col_end = 0;
    return s;
}

// How the CTAs of the large-batch kernel (B > 128) divide one head.  With n rows there are
// R = ceil(n / 128) row blocks.  On a head with `two_blocks` set they are taken two at a time
// (units of two blocks); an odd last block is a unit of its own, or, on a head of three blocks
// whose last has at most 64 rows, rides along with the two-block unit as a THIN block: its logits are computed with the
// operands swapped (vocabulary on the MMA's M side, the thin block's rows on N), which takes
// thin16 = rows rounded up to 16 accumulator columns per 128 vocabulary rows instead of a third
// 256-column accumulator; the unit's tiles are then tile_n = 256 - thin16 columns wide, so that
// everything fits the 512 columns of tensor memory.  Without `two_blocks` every block is a unit
// of its own.  Units get CTAs in proportion to their cost and a unit's g CTAs take the head's
// tiles round-robin (member `slot` takes tiles slot, slot + g, ...).  Units of the same kind sweep
// the vocabulary at the same pace, so a weight tile fetched for one is an L2 hit for the others;
// units of different kinds do not, and a head with two kinds reads its weights twice.
struct UnitSplit {
    int active;      // this CTA serves a unit of the head
    int dual;        // 1: row blocks rb and rb + 1; 0: row block rb alone
    int thin16;      // > 0: row block rb + 2 rides along as a thin block of at most thin16 rows
    int tile_n;      // width of a full tile: 256, or 256 - thin16
    int rb;
    int slot, g;     // member index within the unit's group of g CTAs (also the partial slot)
    int rounds;      // whole rounds of tiles: member `slot` takes tile slot + k * g in round k.  The first
    int n_hi;        // n_hi rounds have tiles of w_hi columns, the others of w_lo (both multiples of 16,
    int w_hi, w_lo;  // at most tile_n)
    int tail_col0, tail_cols;   // what is left after the whole rounds is cut evenly (in 16-column
                                // units) among the g members: this member's piece (tail_cols may be 0)
    int n_tiles;     // pieces this member multiplies: rounds + (tail_cols > 0)
};

// A member's share in few pieces (at most this many whole rounds of full tiles) is cut into
// pieces of nearly equal width instead of full tiles and a narrow last one that only some
// members have: on a head of three row blocks and more (measured: step at 25 % large rows
// 843 -> 824 us, at 50 % 1079 -> 1048 us, 300 rows on the small head 144 -> 134 us) and in a
// two-block unit (181 rows on the large head 326 -> 304 us).  Single-block units of a head of one
// or two blocks stream their weights from HBM at the rate their loads in flight allow, and
// narrower tiles in several boxes mean fewer bytes in flight: there the full tiles stay (256 rows
// on the small head 103 us with them, 144 us with even pieces).
constexpr int kEvenRoundsMax = 8;
constexpr int kEvenRoundsMinBlocks = 3;

// Column range [col0, col0 + ncols) of piece k (0 <= k < n_tiles) of a member; vpad = V rounded up to 16.
__host__ __device__ inline void unit_piece(const UnitSplit &s, int k, int vpad, int &col0, int &ncols)
{
    if (k < s.rounds) {
        const int hi = k < s.n_hi ? k : s.n_hi;              // rounds of the wider kind before this one
        const int w = k < s.n_hi ? s.w_hi : s.w_lo;
        col0 = s.g * (hi * s.w_hi + (k - hi) * s.w_lo) + s.slot * w;
        ncols = vpad - col0 < w ? vpad - col0 : w;
    } else {
        col0 = s.tail_col0;
        ncols = s.tail_cols;
    }
}

// Units of a head with n rows (R row blocks): D of two blocks, then T (0 or 1, and only if D = 0)
// of two blocks and a thin one, then S of one block; CTAs per unit gd, gt and gs, in proportion to what the unit
// costs per 256 vocabulary columns and 64 hidden elements: measured 1386 cycles for two blocks
// against 763 for one (18 : 10), a single block of at most 64 rows (an M = 64 tile with half the
// hidden rows) a little less (9).  A unit with a thin block is the only unit of its head.
struct UnitPlan {
    int D, T, S;
    int gd, gt, gs;
    int thin16;
};

__host__ __device__ inline UnitPlan unit_plan(int G, int n, int two_blocks)
{
    UnitPlan u;
    u.D = u.T = u.S = u.gd = u.gt = u.gs = u.thin16 = 0;
    const int R = (n + kTileM - 1) / kTileM;
    if (R <= 0) return u;
    const int last = n - (R - 1) * kTileM;                   // rows of the last block
    if (two_blocks && R == 3 && last <= kTileM / 2) {
        // (with five blocks and more, one two-block unit less and a thin block instead of the
        // single one measured slower: 1076 against 1055 us per step at 50 % large rows)
        u.T = 1;
        u.thin16 = (last + kUnit - 1) / kUnit * kUnit;
    } else {
        // Units of different kinds walk the vocabulary at different rates and cannot share a weight
        // tile in L2, so a head with both kinds reads its weights twice (measured: 3.2 GB per launch
        // against 2.06 GB).  With three row blocks that makes the head HBM-bound, and three single
        // units, which share every tile, are faster (917 against 961 us per step at 25 % large rows).
        u.D = (two_blocks && R != 3) ? R / 2 : 0;
        u.S = R - 2 * u.D;
    }
    if (u.T > 0) {
        u.gt = G;
        return u;
    }
    const int w_single = last <= kTileM / 2 ? 9 : 10;
    if (u.D > 0) {
        u.gd = 18 * G / (18 * u.D + w_single * u.S);
        if (u.gd < 1) u.gd = 1;
    }
    const int left = G - u.gd * u.D;                           // CTAs for the single-block units
    if (u.S > 0) {
        u.gs = left / u.S;
        if (u.gs < 1) {                                        // fewer CTAs than units are rejected on the host
            u.gs = 1;
            if (u.D > 0) u.gd = (G - u.S) / u.D > 0 ? (G - u.S) / u.D : 1;
        }
    }
    return u;
}

__host__ __device__ inline UnitSplit split_units(int cta, int G, int n, int V, int two_blocks)
{
    UnitSplit s;
    s.active = 0; s.dual = 0; s.thin16 = 0; s.tile_n = kTileN; s.rb = 0; s.slot = 0; s.g = 0;
    s.rounds = 0; s.n_hi = 0; s.w_hi = s.w_lo = kTileN; s.tail_col0 = 0; s.tail_cols = 0; s.n_tiles = 0;
    if (n <= 0) return s;
    const UnitPlan u = unit_plan(G, n, two_blocks);
    const int after_d = u.gd * u.D;
    if (cta < after_d) {                           // units interleaved: neighbours in the grid share a slot
        s.active = 1;
        s.dual = 1;
        s.rb = 2 * (cta % u.D);
        s.slot = cta / u.D;
        s.g = u.gd;
    } else if (u.T > 0 && cta - after_d < u.gt) {
        s.active = 1;
        s.dual = 1;
        s.thin16 = u.thin16;
        s.tile_n = kTileN - u.thin16;
        s.rb = 2 * u.D;
        s.slot = cta - after_d;
        s.g = u.gt;
    } else if (u.S > 0 && (cta - after_d) / u.S < u.gs) {
        const int local = cta - after_d;
        s.active = 1;
        s.rb = 2 * u.D + local % u.S;
        s.slot = local / u.S;
        s.g = u.gs;
    }
    if (!s.active) return s;
    // Whole rounds of full tiles, then the rest of the vocabulary in g even pieces, so that the
    // members of a unit finish together (with whole tiles only, a unit of 74 CTAs on 594 tiles
    // would wait a ninth round out for two of its members).
    const int vpad = (V + kUnit - 1) / kUnit * kUnit;
    const int U = vpad / kUnit;                               // 16-column units of the head
    const int tile_u = s.tile_n / kUnit;
    const int tiles = (V + s.tile_n - 1) / s.tile_n;
    s.rounds = tiles / s.g;
    s.w_hi = s.w_lo = s.tile_n;
    if (s.rounds * s.g * s.tile_n > vpad) s.rounds -= 1;     // the last whole round would hold the ragged last tile: deal that round out evenly instead
    s.n_hi = s.rounds;
    if ((n > (kEvenRoundsMinBlocks - 1) * kTileM || s.dual) && s.rounds >= 1 && s.rounds <= kEvenRoundsMax &&
        U > s.rounds * s.g * tile_u) {
        // few pieces: n_p pieces of nearly equal width, the last one again the even rest
        const int u_tot = (U + s.g - 1) / s.g;                // units of the member with the most
        const int n_p = (u_tot + tile_u - 1) / tile_u;
        const int base = u_tot / n_p, extra = u_tot % n_p;    // `extra` pieces of base + 1 units, the others of base
        s.rounds = n_p - 1;
        s.n_hi = extra < s.rounds ? extra : s.rounds;
        s.w_hi = (base + 1) * kUnit;
        s.w_lo = base * kUnit;
    }
    const int rest0 = s.g * (s.n_hi * s.w_hi + (s.rounds - s.n_hi) * s.w_lo);
    const int rest = vpad - rest0;                            // a multiple of 16
    if (rest > 0) {
        const int units16 = rest / kUnit;
        const int per = (units16 + s.g - 1) / s.g * kUnit;    // columns per member, a multiple of 16, <= tile_n
        const int c0 = rest0 + s.slot * per;
        if (c0 < vpad) {
            s.tail_col0 = c0;
            s.tail_cols = vpad - c0 < per ? vpad - c0 : per;
        }
    }
    s.n_tiles = s.rounds + (s.tail_cols > 0 ? 1 : 0);
    return s;
}

// Partial slots that the merge has to fold for compacted row `row` of a head with n rows.
__host__ __device__ inline int unit_slots_of_row(int G, int n, int row, int two_blocks)
{
    const UnitPlan u = unit_plan(G, n, two_blocks);
    const int rb = row / kTileM;
    return rb < 2 * u.D ? u.gd : u.T ? u.gt : u.gs;
}

#ifdef __CUDACC__
struct Partial {
    float m, s, t;
    int idx;
};

// Combines the statistics of two disjoint column sets (m = max z, s = sum exp(z - m),
// t = sum exp(z - m) (z - m) log2 e, idx = lowest column attaining m).  Equal maxima keep the lower column.
__device__ __forceinline__ Partial merge_partial(const Partial &a, const Partial &b)
{
    Partial r;
    r.m = fmaxf(a.m, b.m);
    const float da = (a.m - r.m) * kLog2e, db = (b.m - r.m) * kLog2e;
    const float ea = exp2f(da), eb = exp2f(db);
    r.s = ea * a.s + eb * b.s;
    r.t = ea * fmaf(da, a.s, a.t) + eb * fmaf(db, b.s, b.t);
    if (a.m > b.m) r.idx = a.idx;
    else if (b.m > a.m) r.idx = b.idx;
    else r.idx = min(a.idx, b.idx);
    return r;
}

// A sampled token candidate: largest perturbed logit and its column; equal values keep the
// lower column.
struct Draw {
    float k;
    int ki;
};
__device__ __forceinline__ Draw merge_draw(const Draw &a, const Draw &b)
{
    return (b.k > a.k || (b.k == a.k && b.ki < a.ki)) ? b : a;
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds of two 32x32->64 multiplies
// by 0xD2511F53 / 0xCD9E8D57, key bumped by 0x9E3779B9 / 0xBB67AE85 every round.  Each product
// is one widening multiply (both halves at once).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                               uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = static_cast<uint64_t>(0xD2511F53u) * c0;
        const uint64_t p1 = static_cast<uint64_t>(0xCD9E8D57u) * c2;
        c0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k0;
        c1 = static_cast<uint32_t>(p1);
        c2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k1;
        c3 = static_cast<uint32_t>(p0);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ float lg2_approx(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Standard Gumbel variate from one random word: u = (2k + 1) / 2^24 with k its top 23 bits
// (exact in float32, never 0 or 1), g = -ln(-ln u).  The draw is decided by the largest g, i.e.
// by u next to 1, where -ln u is about 1 - u: there the hardware base-2 logarithm, whose error
// is absolute (2^-22), would be off by percents (seen on a 128 K vocabulary: largest g about
// 11.8, error 0.02, a wrong token).  So -ln u is the series w + w^2/2 + w^3/3 + w^4/4 in
// w = 1 - u (exact in float32) for w < 1/64 and -ln 2 lg2(u) elsewhere, both within 1e-5
// relative; the outer logarithm only needs absolute accuracy.  The perturbed logits then move
// by ~1e-5, two orders of magnitude below the gap under which a different draw counts as a
// near-tie.
__device__ __forceinline__ float gumbel_from_word(uint32_t word)
{
    constexpr float kLn2 = 0.69314718055994531f;
    const float u = static_cast<float>(2u * (word >> 9) + 1u) * 5.9604644775390625e-8f;   // 2^-24
    const float w = 1.0f - u;
    const float series = w * fmaf(w, fmaf(w, fmaf(w, 0.25f, 0.33333334f), 0.5f), 1.0f);
    const float neg_ln_u = w < 0.015625f ? series : -kLn2 * lg2_approx(u);   // in [6e-8, 16.7]
    return -kLn2 * lg2_approx(neg_ln_u);
}
#endif  // __CUDACC__

struct LmheadParams {
    int32_t V[2];          // vocabulary size of the small / large head
    int32_t H[2];
    int32_t a_rows;        // rows of the hidden-state TMA box (multiple of 8, <= 128)
    int32_t n_cols;        // small-batch kernel: batch columns kept per thread (power of two <= 16)
    int32_t stages;
    int32_t slots_stride;  // partial slots per row (>= CTAs x slots per CTA)
    int32_t B;
    const StepCtl *ctl;
    StepCtl *ctl_rw;
    float *part_m;         // [2][B][slots_stride] running max (nats)
    float *part_s;         // sum of exp(z - m)
    float *part_t;         // sum of exp(z - m) * (z - m) * log2(e)
    int32_t *part_i;       // column of the max
    // sampling (temperature > 0): arg max of z / T + Gumbel noise, kept beside the statistics
    int32_t sampling;
    float inv_temperature;
    uint32_t seed_lo, seed_hi;
    float *part_k;         // largest perturbed value
    int32_t *part_ki;      // its column
    const int32_t *perm;   // compacted row -> caller's row (the random stream is per caller row)
    uint32_t ctr_off[2];   // vocabulary-sharded use: first row of this slice in the full head, / 4
    int32_t prefetch_boxes;  // small-batch kernel: 16 KiB weight boxes brought into L2 before the dependency wait
    int32_t half_blocks;     // large-batch kernel: row blocks of at most 64 rows run as M = 64 tiles
    int32_t two_blocks;      // large-batch kernel: bit m set = head m is served in units of two row blocks
    int32_t ring_bytes;      // large-batch kernel: bytes of the stage ring (cut into 48 or 64 KiB stages per head)
};

}  // namespace ead
