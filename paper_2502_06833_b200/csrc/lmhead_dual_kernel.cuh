// LM-head projection + online entropy / arg-max statistics for LARGE batches (B > 128), two
// row blocks per weight tile.
//
// Same arithmetic and the same roles as ead_lmhead_kernel (batch rows on the MMA's M side,
// vocabulary on N, logits only ever in tensor memory; warp 0 = TMA producer, warp 1 = MMA
// issuer, warps 2-5 = epilogue).  What differs is what a CTA multiplies per pipeline stage.
// The one-block kernel brings in 16 KiB of hidden rows and 32 KiB of weights per stage and its
// four MMAs read the same 48 KiB back: 96 KiB through a shared-memory port of 128 B/clk = 750
// cycles for 512 cycles of MMA, which is where that kernel stands (744 measured).  Here a CTA
// serves a UNIT: two consecutive 128-row blocks of a head against the same weight tile.  A
// stage holds both blocks' hidden rows and the weight tile once (64 KiB in), its eight MMAs read
// 96 KiB: 160 KiB per 1024 cycles of MMA, a sixth less port time per flop, and the weight tile
// crosses from L2 once for 256 rows.  A head with an odd number of row blocks has one unit of
// a single block (served as in the one-block kernel, as an M = 64 tile if it has at most 64
// rows).
//
// Both accumulators of TMEM are in use at once in a two-block unit, so the epilogue of a tile
// no longer hides behind the MMAs of the next one as a whole: the MMAs of the next tile's first
// block start when the epilogue is done with the first accumulator, those of the second block
// when it is done with the second.  With 80 K blocks per tile (H = 5120) that costs a few
// per cent and the step gains 7 %; with 24 (H = 1536) it costs more than the port gains (measured:
// +6 %), so a head is served in two-block units only if the host says so (p.two_blocks, set for
// hidden sizes of 3072 and more); otherwise every row block is a unit of its own, with the
// one-block kernel's stage (48 KiB, four of them) and double-buffered accumulators; so is the odd
// last block of a head in two-block units.  The ring is re-cut between the heads (64 KiB stages
// for a two-block unit, three of them): the producer first waits until every stage of the previous
// head has been consumed.
//
// A THIN third block.  A head of three row blocks whose last block has at most 64 rows would pay
// a whole single-block unit for them (its own pass of the weights through shared memory, and,
// because units of different kinds cannot share tiles in L2, a second pass through HBM).  Instead
// the two-block unit takes the block along: per stage it also loads the thin block's hidden
// rows (64 x 64, 8 KiB) and issues, after the MMAs of its two blocks, two more with the operands
// swapped: A = 128 rows of the weight tile that is in shared memory anyway (rows 0..127, and
// rows tile_n - 128..tile_n - 1), B = the thin rows, N = thin16 = rows rounded up to 16.  Those
// accumulators (vocabulary in lanes, sequences in columns) take thin16 columns each; the tile
// shrinks to tile_n = 256 - thin16 columns so that block a's accumulator and the first thin one
// share the first 256 columns of tensor memory, block b's and the second thin one the other 256.
// The epilogue transposes 32 x 32 pieces of the thin accumulators with warp shuffles, after which
// lane l holds 32 consecutive logits of thin sequence l and folds them with the routine of the
// other rows; at the end of the head the four warps' statistics (each saw its quarter of every
// tile) are merged through shared memory.  A stage is 72 KiB then, three of them.  The eight thin
// MMAs of a stage cost about 90 cycles each, far more than their 4 cycles of arithmetic (measured:
// 2060 cycles per stage against 1386 without them), so the thin block saves little against a
// single-block unit's 763 per stage; it pays where it also saves the second pass over the weights,
// on a head of three blocks (step at 25 % large rows 880 -> 843 us), and not beside other
// two-block units (five blocks: 1055 -> 1076 us), which is how split_units uses it.
//
// Work split (split_units): the units of a head get CTAs in proportion to their cost (9 : 5 for
// two blocks : one) and a unit's CTAs take its tiles round-robin (member j takes tiles
// j, j + g, ...); what is left after the whole rounds is cut into g even pieces, so the members
// of a unit finish together; a share of few tiles is cut into pieces of nearly equal width where
// that was measured to pay (split_units).  Units of one kind sweep the vocabulary at the same pace whatever
// their number, so a weight tile fetched for one is an L2 hit for the others; units of different
// kinds do not (a head with two kinds reads its weights twice: measured).
#pragma once
#include "lmhead_kernel.cuh"

namespace ead {

constexpr int kDualABytes = kTileM * kBlockK * 2;                          // 16 KiB of hidden rows per block and stage
constexpr int kDualStageBytes = 2 * kDualABytes + kWTileBytes;             // 64 KiB: two blocks' hidden rows + one weight tile
constexpr int kSingleStageBytes = kDualABytes + kWTileBytes;               // 48 KiB: one block's hidden rows + one weight tile
constexpr int kThinABytes = (kTileM / 2) * kBlockK * 2;                    // 8 KiB: the thin block's hidden rows (a 64-row box)
constexpr int kThinStageBytes = 2 * kDualABytes + kThinABytes + kWTileBytes;   // 72 KiB: a full tile is loaded as one 256-row box, of which the last thin16 rows are not used
constexpr int kThinMergeBytes = 4 * (kTileM / 2) * 6 * 4;                  // four warps x 64 sequences x six statistics

// How the stage ring is cut for a unit (of two blocks or of one): stage size, where the weight tile
// sits in a stage, how many stages fit.
struct HeadRing {
    uint32_t stage_bytes, w_off;
    int stages;
};

#ifdef __CUDACC__
__device__ __forceinline__ HeadRing head_ring(const LmheadParams &p, const UnitSplit &sp, bool half_head)
{
    HeadRing r;
    // A head of at most 64 rows brings in 8 KiB of hidden rows per stage: 40 KiB stages, five of
    // them.  (Not so a short block beside other blocks of its head: units that share their weight
    // tiles through L2 must move in step, and with rings of different depth they do not; measured
    // on 181 rows of the small head: 101 us with equal stages, 148 us with 48 and 40 KiB ones.)
    const uint32_t single_a = half_head ? kDualABytes / 2 : kDualABytes;
    r.stage_bytes = sp.thin16 ? kThinStageBytes : sp.dual ? kDualStageBytes : single_a + kWTileBytes;
    r.w_off = sp.thin16 ? 2 * kDualABytes + kThinABytes : sp.dual ? 2 * kDualABytes : single_a;
    r.stages = min(kMaxStages, static_cast<int>(static_cast<uint32_t>(p.ring_bytes) / r.stage_bytes));
    return r;
}

// Transposes a 32 x 32 tile held one row per lane: afterwards v[i] of lane l is what v[l] of lane i was.
__device__ __forceinline__ void warp_transpose32(float (&v)[32], int lane)
{
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const bool up = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (i & s) continue;
            const float send = up ? v[i] : v[i + s];
            const float recv = __shfl_xor_sync(0xffffffffu, send, s);
            if (up) v[i] = recv;
            else v[i + s] = recv;
        }
    }
}

// Folds one thin accumulator into the statistics of the thin sequences.  The accumulator keeps
// vocabulary entry cb + l in the lane l of this warp's quadrant and sequence j in column j
// (thin16 columns from taddr); entries outside [lo, hi) are not the accumulator's to count.
// After the transposition lane l owns sequence 32 * ch + l.
template <bool SAMPLE>
__device__ __forceinline__ void fold_thin(uint32_t taddr, int thin16, int cb, int lo, int hi, int lane, RowStat (&st)[2],
                                          Draw (&dr)[2], const bool (&sampling)[2], uint32_t rng_step,
                                          const uint32_t (&rng_row)[2], const LmheadParams &p, uint32_t ctr_off)
{
    if (max(cb, lo) >= min(cb + 32, hi)) return;              // the same for the whole warp
#pragma unroll
    for (int ch = 0; ch < 2; ++ch) {
        if (ch * 32 >= thin16) break;
        float v[32];
        {
            float h[16];
            tmem_ld_16cols(taddr + ch * 32, h);
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = h[j];
            if (ch * 32 + 16 < thin16) {
                tmem_ld_16cols(taddr + ch * 32 + 16, h);
#pragma unroll
                for (int j = 0; j < 16; ++j) v[16 + j] = h[j];
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[16 + j] = 0.f;
            }
        }
        warp_transpose32(v, lane);
        if (cb < lo || cb + 32 > hi) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = (cb + i >= lo && cb + i < hi) ? v[i] : kNegSentinel;
        }
        rowstat_absorb32(st[ch], v, cb);
        if (SAMPLE && sampling[ch]) draw_absorb32(dr[ch], v, cb, rng_step, rng_row[ch], p, ctr_off);
        __syncwarp();
    }
}

// Folds one accumulator (ncols columns from column col0 of the head) into the statistics of the
// row that this thread owns in it.
template <bool SAMPLE>
__device__ __forceinline__ void fold_accumulator(uint32_t taddr, int ncols, int col0, int col_limit, RowStat &st, Draw &dr,
                                                 bool sampling, uint32_t rng_step, uint32_t rng_row,
                                                 const LmheadParams &p, uint32_t ctr_off)
{
    for (int c = 0; c < ncols; c += 32) {
        float v[32];
        tmem_ld_32cols(taddr + c, v);
        const int cb = col0 + c;
        if (cb + 32 > col_limit) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (cb + j < col_limit) ? v[j] : kNegSentinel;
        }
        rowstat_absorb32(st, v, cb);
        if (SAMPLE && sampling) draw_absorb32(dr, v, cb, rng_step, rng_row, p, ctr_off);
        __syncwarp();
    }
}

// One block of a unit as the epilogue sees it.
struct BlockView {
    int row0;           // first compacted row of the block
    int rows_valid;     // real rows in it (0: the unit has no such block)
    bool half;          // multiplied as an M = 64 tile
};

__device__ __forceinline__ BlockView block_view(const LmheadParams &p, int n, int rb, bool present)
{
    BlockView b;
    b.row0 = rb * kTileM;
    b.rows_valid = present ? max(0, min(kTileM, n - b.row0)) : 0;
    b.half = present && half_block(p, b.rows_valid);
    return b;
}

// tmA*: compacted hidden rows, boxes of 128 x 64; tmH*: the same, boxes of 64 x 64; tmW*: W, boxes
// of 256 x 64; tmQ*, tmT*: W, boxes of 64 x 64 and 16 x 64 (pieces narrower than a tile).
template <bool SAMPLE>
__global__ void __launch_bounds__(kLmheadThreads, 1)
ead_lmhead_dual_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
                       const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
                       const __grid_constant__ CUtensorMap tmT0, const __grid_constant__ CUtensorMap tmT1,
                       const __grid_constant__ CUtensorMap tmH0, const __grid_constant__ CUtensorMap tmH1,
                       const __grid_constant__ CUtensorMap tmQ0, const __grid_constant__ CUtensorMap tmQ1,
                       const LmheadParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                ~static_cast<uintptr_t>(1023));
    SmemCtrl *ctrl = reinterpret_cast<SmemCtrl *>(smem);
    uint8_t *stage0 = smem + kSmemCtrlBytes;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    const int G = gridDim.x;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kMaxStages; ++i) {
            mbar_init(smem_u32(&ctrl->full[i]), 1);
            mbar_init(smem_u32(&ctrl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctrl->tmem_full[i]), 1);
            mbar_init(smem_u32(&ctrl->tmem_empty[i]), 4);   // one arrival per epilogue warp
        }
        mbar_init(smem_u32(&ctrl->drain), 1);
        ctrl->abort = 0;
        fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmA0); tma_prefetch_desc(&tmA1);
        tma_prefetch_desc(&tmW0); tma_prefetch_desc(&tmW1);
        tma_prefetch_desc(&tmT0); tma_prefetch_desc(&tmT1);
        tma_prefetch_desc(&tmH0); tma_prefetch_desc(&tmH1);
        tma_prefetch_desc(&tmQ0); tma_prefetch_desc(&tmQ1);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), 2 * kTileN);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&ctrl->tmem_base);

    // Everything above touched no global memory: it may overlap the kernels before this one.
    griddep_wait();
    griddep_launch_dependents();
    const int n_rows[2] = {p.ctl->n[0], p.ctl->n[1]};
    StepCtl *ctl = p.ctl_rw;

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer
        if (lane == 0) {
            const uint64_t pol_stream = l2_policy_evict_first();
            const uint64_t pol_keep = l2_policy_evict_last();
            uint32_t par = 0;                    // bit s: parity of the number of times slot s has been filled
            bool ok = true;
            for (int m = 0; m < 2 && ok; ++m) {
                const UnitSplit sp = split_units(cta, G, n_rows[m], p.V[m], (p.two_blocks >> m) & 1);
                if (!sp.active) continue;
                const BlockView ba = block_view(p, n_rows[m], sp.rb, true);
                const BlockView bb = block_view(p, n_rows[m], sp.rb + 1, sp.dual != 0);
                const HeadRing ring = head_ring(p, sp, n_rows[m] <= kTileM / 2);
                // The ring may be cut differently for this head: every stage filled so far must have
                // been consumed first (the wait a refill of the slot would do; a slot never filled
                // passes at once).
                for (int s = 0; s < kMaxStages && ok; ++s)
                    ok = wait_bar(smem_u32(&ctrl->empty[s]), ((par >> s) & 1u) ^ 1u, ctrl, ctl);
                if (!ok) break;
                uint32_t s = 0;
                const CUtensorMap *tW = m ? &tmW1 : &tmW0;
                const CUtensorMap *tT = m ? &tmT1 : &tmT0;
                const CUtensorMap *tQ = m ? &tmQ1 : &tmQ0;
                const CUtensorMap *tAa = ba.half ? (m ? &tmH1 : &tmH0) : (m ? &tmA1 : &tmA0);
                const CUtensorMap *tAb = bb.half ? (m ? &tmH1 : &tmH0) : (m ? &tmA1 : &tmA0);
                const CUtensorMap *tAc = m ? &tmH1 : &tmH0;
                const uint32_t a_tx = (ba.half ? kDualABytes / 2 : kDualABytes) +
                                      (sp.dual ? (bb.half ? kDualABytes / 2 : kDualABytes) : 0) +
                                      (sp.thin16 ? kThinABytes : 0);
                // a weight tile needed by several units should stay in L2 for them
                const uint64_t pol_w = (n_rows[m] <= 2 * kTileM) ? pol_stream : pol_keep;
                const int kblocks = (p.H[m] + kBlockK - 1) / kBlockK;
                const int vpad = (p.V[m] + kUnit - 1) / kUnit * kUnit;
                for (int t = 0; t < sp.n_tiles && ok; ++t) {
                    int col0, ncols;
                    unit_piece(sp, t, vpad, col0, ncols);
                    const bool full = ncols == sp.tile_n;     // one box of 256 rows (the narrower tile of a unit with a thin block ignores the last rows)
                    const uint32_t tx = a_tx + (full ? kWTileBytes : static_cast<uint32_t>(ncols) * (kBlockK * 2));
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!wait_bar(smem_u32(&ctrl->empty[s]), ((par >> s) & 1u) ^ 1u, ctrl, ctl)) { ok = false; break; }
                        const uint32_t bar = smem_u32(&ctrl->full[s]);
                        const uint32_t sa = smem_u32(stage0 + static_cast<size_t>(s) * ring.stage_bytes);
                        mbar_arrive_expect_tx(bar, tx);
                        tma_load_2d(sa, tAa, kb * kBlockK, ba.row0, bar, pol_keep);
                        if (sp.dual) tma_load_2d(sa + kDualABytes, tAb, kb * kBlockK, bb.row0, bar, pol_keep);
                        if (sp.thin16) tma_load_2d(sa + 2 * kDualABytes, tAc, kb * kBlockK, bb.row0 + kTileM, bar, pol_keep);
                        const uint32_t sw = sa + ring.w_off;
                        if (full) {
                            tma_load_2d(sw, tW, kb * kBlockK, col0, bar, pol_w);
                        } else {                     // exactly the piece's rows: boxes of 64, then of 16
                            int j = 0;
                            for (; ncols - j >= 64; j += 64)
                                tma_load_2d(sw + j * (kBlockK * 2), tQ, kb * kBlockK, col0 + j, bar, pol_w);
                            for (; j < ncols; j += kUnit)
                                tma_load_2d(sw + j * (kBlockK * 2), tT, kb * kBlockK, col0 + j, bar, pol_w);
                        }
                        par ^= 1u << s;
                        s = (s + 1 == static_cast<uint32_t>(ring.stages)) ? 0 : s + 1;
                    }
                }
            }
            // Before the CTA retires, every copy issued above must have landed: the last fill of
            // slot s completed the phase of parity bit ^ 1 (a slot never filled passes at once).
            for (int s = 0; s < kMaxStages; ++s)
                if (!wait_bar(smem_u32(&ctrl->full[s]), ((par >> s) & 1u) ^ 1u, ctrl, ctl)) break;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t par = 0;                     // as the producer's, for the fills consumed so far
            uint32_t use[2] = {0, 0};             // how often each accumulator has been filled
            uint32_t next_buf = 0;                // single-block units alternate between the accumulators
            bool ok = true;
            for (int m = 0; m < 2 && ok; ++m) {
                const UnitSplit sp = split_units(cta, G, n_rows[m], p.V[m], (p.two_blocks >> m) & 1);
                if (!sp.active) continue;
                const BlockView ba = block_view(p, n_rows[m], sp.rb, true);
                const BlockView bb = block_view(p, n_rows[m], sp.rb + 1, sp.dual != 0);
                const HeadRing ring = head_ring(p, sp, n_rows[m] <= kTileM / 2);
                uint32_t s = 0;
                const int kblocks = (p.H[m] + kBlockK - 1) / kBlockK;
                const int vpad = (p.V[m] + kUnit - 1) / kUnit * kUnit;
                for (int t = 0; t < sp.n_tiles && ok; ++t) {
                    int col0, ncols;
                    unit_piece(sp, t, vpad, col0, ncols);
                    // accumulator of block a (and, in a two-block unit, of block b)
                    const uint32_t buf_a = sp.dual ? 0u : next_buf;
                    const uint32_t buf_b = 1u;
                    if (!sp.dual) next_buf ^= 1u;
                    const uint32_t idesc_a = ba.half ? umma_idesc_bf16_m64(static_cast<uint32_t>(ncols))
                                                     : umma_idesc_bf16_m128(static_cast<uint32_t>(ncols));
                    const uint32_t idesc_b = bb.half ? umma_idesc_bf16_m64(static_cast<uint32_t>(ncols))
                                                     : umma_idesc_bf16_m128(static_cast<uint32_t>(ncols));
                    const uint32_t d_a = tmem_base + buf_a * kTileN, d_b = tmem_base + buf_b * kTileN;
                    // thin accumulators: behind block a's and block b's columns
                    const uint32_t idesc_c = umma_idesc_bf16_m128(static_cast<uint32_t>(sp.thin16 ? sp.thin16 : kUnit));
                    const uint32_t d_c1 = tmem_base + sp.tile_n, d_c2 = tmem_base + kTileN + sp.tile_n;
                    const uint32_t w2_off = ring.w_off + static_cast<uint32_t>(sp.tile_n - kTileM) * (kBlockK * 2);
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!wait_bar(smem_u32(&ctrl->full[s]), (par >> s) & 1u, ctrl, ctl)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint32_t sa = smem_u32(stage0 + static_cast<size_t>(s) * ring.stage_bytes);
                        const uint64_t da = umma_smem_desc(sa);
                        const uint64_t dbk = umma_smem_desc(sa + kDualABytes);
                        const uint64_t dw = umma_smem_desc(sa + ring.w_off);
                        if (kb == 0) {              // the epilogue must be done with the accumulator's last tile
                            if (!wait_bar(smem_u32(&ctrl->tmem_empty[buf_a]), (use[buf_a] & 1u) ^ 1u, ctrl, ctl)) {
                                ok = false;
                                break;
                            }
                            tc_fence_after_sync();
                        }
                        const uint64_t dc = umma_smem_desc(sa + 2 * kDualABytes);     // thin rows (B of the swapped MMAs)
                        const uint64_t dw2 = umma_smem_desc(sa + w2_off);             // weight rows tile_n - 128 ..
#pragma unroll
                        for (int k = 0; k < kBlockK / 16; ++k)   // +32 B (>>4 = 2) per 16 elements of K
                            umma_bf16(d_a, da + 2 * k, dw + 2 * k, idesc_a, (kb | k) != 0);
                        // The thin MMAs stay together: alternating them with the wide ones cost 6 % of
                        // the step (measured).
                        if (sp.thin16) {
#pragma unroll
                            for (int k = 0; k < kBlockK / 16; ++k)
                                umma_bf16(d_c1, dw + 2 * k, dc + 2 * k, idesc_c, (kb | k) != 0);
                        }
                        if (sp.dual) {
                            if (kb == 0) {
                                if (!wait_bar(smem_u32(&ctrl->tmem_empty[buf_b]), (use[buf_b] & 1u) ^ 1u, ctrl, ctl)) {
                                    ok = false;
                                    break;
                                }
                                tc_fence_after_sync();
                            }
#pragma unroll
                            for (int k = 0; k < kBlockK / 16; ++k)
                                umma_bf16(d_b, dbk + 2 * k, dw + 2 * k, idesc_b, (kb | k) != 0);
                            if (sp.thin16) {
#pragma unroll
                                for (int k = 0; k < kBlockK / 16; ++k)
                                    umma_bf16(d_c2, dw2 + 2 * k, dc + 2 * k, idesc_c, (kb | k) != 0);
                            }
                        }
                        umma_commit(smem_u32(&ctrl->empty[s]));   // stage reusable once these MMAs are done
                        par ^= 1u << s;
                        s = (s + 1 == static_cast<uint32_t>(ring.stages)) ? 0 : s + 1;
                    }
                    if (!ok) break;
                    // every MMA issued so far is complete when these arrive: both accumulators are
                    use[buf_a] += 1;
                    umma_commit(smem_u32(&ctrl->tmem_full[buf_a]));
                    if (sp.dual) {
                        use[buf_b] += 1;
                        umma_commit(smem_u32(&ctrl->tmem_full[buf_b]));
                    }
                }
            }
            // All MMAs must have finished before TMEM is released.
            umma_commit(smem_u32(&ctrl->drain));
            wait_bar(smem_u32(&ctrl->drain), 0u, ctrl, ctl);
        }
    } else {
        // ------------------------------------------------------------- epilogue
        const int quad = warp & 3;                   // TMEM lane quadrant this warp may read
        uint32_t use[2] = {0, 0};
        uint32_t next_buf = 0;
        bool ok = true;
        // Once a wait has given up (ok = false) nothing more is folded or stored, but the loop over
        // the heads goes on: every epilogue warp must pass the same named barriers.
        for (int m = 0; m < 2; ++m) {
            const UnitSplit sp = split_units(cta, G, n_rows[m], p.V[m], (p.two_blocks >> m) & 1);
            if (!sp.active) continue;
            const BlockView blk[2] = {block_view(p, n_rows[m], sp.rb, true),
                                      block_view(p, n_rows[m], sp.rb + 1, sp.dual != 0)};
            RowStat st[2];
            Draw dr[2];
            int row[2];
            bool has_rows[2], sampling[2];
            uint32_t rng_row[2];
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                // An M = 128 accumulator keeps row r of the block in TMEM lane r; an M = 64 one keeps
                // its 64 rows in the lower 16 lanes of each 32-lane quadrant.
                const int rib = blk[x].half ? (lane < 16 ? quad * 16 + lane : kTileM) : quad * 32 + lane;
                rowstat_reset(st[x]);
                dr[x] = Draw{-INFINITY, 0x7fffffff};
                row[x] = blk[x].row0 + rib;
                has_rows[x] = (blk[x].half ? quad * 16 : quad * 32) < blk[x].rows_valid;
                const bool live = rib < blk[x].rows_valid;
                sampling[x] = SAMPLE && live;
                rng_row[x] = sampling[x] ? static_cast<uint32_t>(p.perm[m * p.B + row[x]]) : 0u;
                if (!live) row[x] = -1;
            }
            // thin block: after the transposition lane l owns its sequences l and 32 + l
            const BlockView bc = block_view(p, n_rows[m], sp.rb + 2, sp.thin16 != 0);
            RowStat stc[2];
            Draw drc[2];
            int row_c[2];
            bool sampling_c[2];
            uint32_t rng_row_c[2];
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
                rowstat_reset(stc[ch]);
                drc[ch] = Draw{-INFINITY, 0x7fffffff};
                const bool live = ch * 32 + lane < bc.rows_valid;
                row_c[ch] = live ? bc.row0 + ch * 32 + lane : -1;
                sampling_c[ch] = SAMPLE && live;
                rng_row_c[ch] = sampling_c[ch] ? static_cast<uint32_t>(p.perm[m * p.B + row_c[ch]]) : 0u;
            }
            const uint32_t rng_step = static_cast<uint32_t>(p.ctl->cur_t);
            const int vpad = (p.V[m] + kUnit - 1) / kUnit * kUnit;
            for (int t = 0; t < sp.n_tiles && ok; ++t) {
                int col0, ncols;
                unit_piece(sp, t, vpad, col0, ncols);
                const int col_limit = min(p.V[m], col0 + ncols);       // first invalid column
                const uint32_t bufs[2] = {sp.dual ? 0u : next_buf, 1u};
                if (!sp.dual) next_buf ^= 1u;
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    if (x == 1 && !sp.dual) break;
                    const uint32_t buf = bufs[x];
                    if (!wait_bar_warp(smem_u32(&ctrl->tmem_full[buf]), use[buf] & 1u, ctrl, ctl, lane)) {
                        ok = false;
                        break;
                    }
                    use[buf] += 1;
                    tc_fence_after_sync();
                    if (has_rows[x]) {
                        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kTileN;
                        fold_accumulator<SAMPLE>(taddr, ncols, col0, col_limit, st[x], dr[x], sampling[x], rng_step,
                                                 rng_row[x], p, p.ctr_off[m]);
                    }
                    if (sp.thin16) {
                        // first thin accumulator: rows 0..127 of the tile; second: rows tile_n - 128 ..,
                        // of which those below 128 were counted by the first
                        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kTileN + sp.tile_n;
                        const int cb = col0 + (x ? sp.tile_n - kTileM : 0) + quad * 32;
                        fold_thin<SAMPLE>(taddr, sp.thin16, cb, x ? col0 + kTileM : col0, col_limit, lane, stc, drc,
                                          sampling_c, rng_step, rng_row_c, p, p.ctr_off[m]);
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->tmem_empty[buf]));
                }
            }
            if (sp.thin16) {
                // The four warps each saw a quarter of every tile: merge their statistics of the thin
                // sequences through shared memory.  All four come here, whatever `ok`, so that the
                // barrier below is always complete.
                float *mg = reinterpret_cast<float *>(stage0 + p.ring_bytes);
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    float *q = mg + ((quad * 2 + ch) * 32 + lane) * 6;
                    q[0] = stc[ch].m;
                    q[1] = stc[ch].s;
                    q[2] = stc[ch].t;
                    q[3] = __int_as_float(stc[ch].idx);
                    q[4] = drc[ch].k;
                    q[5] = __int_as_float(drc[ch].ki);
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (quad == 0 && ok) {
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        if (row_c[ch] < 0) continue;
                        Partial acc{stc[ch].m, stc[ch].s, stc[ch].t, stc[ch].idx};
                        Draw d = drc[ch];
                        for (int w = 1; w < 4; ++w) {
                            const float *q = mg + ((w * 2 + ch) * 32 + lane) * 6;
                            acc = merge_partial(acc, Partial{q[0], q[1], q[2], __float_as_int(q[3])});
                            d = merge_draw(d, Draw{q[4], __float_as_int(q[5])});
                        }
                        const size_t o = (static_cast<size_t>(m) * p.B + row_c[ch]) * p.slots_stride + sp.slot;
                        p.part_m[o] = acc.m;
                        p.part_s[o] = acc.s;
                        p.part_t[o] = acc.t;
                        p.part_i[o] = acc.idx;
                        if (SAMPLE) {
                            p.part_k[o] = d.k;
                            p.part_ki[o] = d.ki;
                        }
                    }
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");     // the buffer is free for the next head
            }
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (row[x] < 0 || !ok) continue;
                const size_t o = (static_cast<size_t>(m) * p.B + row[x]) * p.slots_stride + sp.slot;
                p.part_m[o] = st[x].m;
                p.part_s[o] = st[x].s;
                p.part_t[o] = st[x].t;
                p.part_i[o] = st[x].idx;
                if (SAMPLE) {
                    p.part_k[o] = dr[x].k;
                    p.part_ki[o] = dr[x].ki;
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem_base, 2 * kTileN);
}
#endif  // __CUDACC__

}  // namespace ead
