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
};

}  // namespace ead
