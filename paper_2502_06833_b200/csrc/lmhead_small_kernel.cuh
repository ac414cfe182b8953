// LM-head projection + online entropy / arg-max statistics for SMALL batches (B <= 16).
//
// At a handful of sequences the step is bound by streaming the weights from HBM, and an
// MMA with the batch on the M side would spend 128 tensor-core rows on 1-16 real ones.
// This kernel swaps the operands instead: MMA M (TMEM lanes) = 128 vocabulary rows of W,
// MMA N (TMEM columns) = 16 batch columns, K = hidden, so the tensor work is 16x smaller
// and W is the only operand of any size.  One epilogue thread owns one vocabulary row of
// a tile and NB statistics, one per sequence.
//
// The statistics run across all tiles of the CTA's range; at the end of a head every epilogue
// warp reduces its 32 threads and writes one partial per sequence (slot = 4 * CTA + warp),
// in the format of ead_lmhead_kernel, so the merge + gate kernel does not care which of the
// two kernels produced it.
//
// Work distribution: the vocabulary is cut into G contiguous ranges of (almost) equal length,
// in units of 32 rows.  (SMs do not all get the same share of HBM bandwidth - finish times of
// an equal split spread by +-10 % - but which SMs lag changes with the split itself, so
// ranges sized from a measurement do not converge, and the lagging SMs speed up once the
// others are done, so the HBM stays busy; measured cost of the imbalance against dynamic
// scheduling of 256 KB units: 3-4 %.)
//
// Pipeline: per K block of 256 hidden elements (128 for NB = 0) one stage = four (two) 64-wide W boxes
// (<= 128 rows each, 16 KiB) + as many 64-wide boxes of the compacted hidden rows (8 rows if B <= 8, else 16;
// the MMA's N = 16 then reads the following kilobyte as rows 8-15, which only feeds
// accumulator columns nobody reads).  TMEM holds two 16-column accumulators so that the
// epilogue overlaps the next tile's MMAs.
//
// NB = 0 selects the variant for 17..128 sequences: the MMA's N is the number of active rows
// of the head rounded up to 16 (<= 128), the accumulators are 128 columns apart, and the
// epilogue cannot keep one statistic per sequence in registers any more.  Instead each warp
// transposes its 32 vocabulary rows x 32 sequences through a private shared-memory tile, after
// which lane l holds 32 consecutive logits of sequence (chunk * 32 + l) and folds them with the
// same 32-column routine as the large-batch kernel.
#pragma once
#include "lmhead_kernel.cuh"

namespace ead {

constexpr int kSmallTileRows = 128;                    // vocabulary rows per tile (MMA M)
constexpr int kSmallSegRows = 32;                      // granularity of a CTA's vocabulary range
constexpr int kSmallSlotsPerCta = 4;                   // one partial per epilogue warp
constexpr int kSmallN = 16;                            // batch columns (MMA N)
// 64-wide K slabs per stage: four for B <= 16 (measured on the LLaMA B = 1 step: 163.9 us against
// 170.3 with two, the same bytes in flight behind half as many barrier round trips), two for the
// NB = 0 variant, whose hidden-row boxes are up to 16 KiB per slab
__host__ __device__ constexpr int small_slabs(int nb) { return nb == 0 ? 2 : 4; }
constexpr int kSmallWBytes = kSmallTileRows * 64 * 2;  // one 64-wide box of W rows: 16 KiB
constexpr int kMidMaxRows = 128;                       // largest batch of the NB = 0 variant
__host__ __device__ constexpr int small_stage_bytes(int h_rows, int slabs) { return slabs * (h_rows * 128 + kSmallWBytes); }

template <int NB, bool SAMPLE>
__global__ void __launch_bounds__(kLmheadThreads, 1)
ead_lmhead_small_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
                        const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
                        const __grid_constant__ CUtensorMap tmP0, const __grid_constant__ CUtensorMap tmP1,
                        const LmheadParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                ~static_cast<uintptr_t>(1023));
    SmemCtrl *ctrl = reinterpret_cast<SmemCtrl *>(smem);
    uint8_t *stage0 = smem + kSmemCtrlBytes;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int G = gridDim.x;
    const int stages = p.stages;
    const uint32_t h_slab = static_cast<uint32_t>(p.a_rows) * 128;      // hidden rows of one 64-wide K slab
    constexpr int kSlabs = small_slabs(NB);
    constexpr int kSmallBlockK = 64 * kSlabs;                           // hidden elements per stage
    const uint32_t stage_bytes = kSlabs * h_slab + kSlabs * kSmallWBytes;
    constexpr uint32_t kAccCols = NB == 0 ? 128u : static_cast<uint32_t>(kSmallN);   // TMEM columns per accumulator
    float *trans = reinterpret_cast<float *>(stage0 + static_cast<size_t>(stages) * stage_bytes);   // NB = 0 only
    StepCtl *ctl = p.ctl_rw;

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(smem_u32(&ctrl->full[i]), 1);
            mbar_init(smem_u32(&ctrl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctrl->tmem_full[i]), 1);
            mbar_init(smem_u32(&ctrl->tmem_empty[i]), 4);
        }
        mbar_init(smem_u32(&ctrl->drain), 1);
        ctrl->abort = 0;
        fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmA0); tma_prefetch_desc(&tmA1);
        tma_prefetch_desc(&tmW0); tma_prefetch_desc(&tmW1);
        tma_prefetch_desc(&tmP0); tma_prefetch_desc(&tmP1);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), 2 * kAccCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&ctrl->tmem_base);
    const int cta = blockIdx.x;
    int row_begin_m[2], row_end_m[2];            // this CTA's vocabulary range on each head
#pragma unroll
    for (int m = 0; m < 2; ++m) {
        const long long n_seg = (p.V[m] + kSmallSegRows - 1) / kSmallSegRows;
        row_begin_m[m] = static_cast<int>(n_seg * cta / G) * kSmallSegRows;
        row_end_m[m] = static_cast<int>(n_seg * (cta + 1) / G) * kSmallSegRows;
    }
    // Everything above touched no global memory: it may overlap the kernels before this one.
    // So may this: while the previous step's merge and this step's compaction run, HBM is idle.
    // The weights do not depend on them, so the first boxes of this CTA's range are brought
    // into L2 now, for the head that served rows in the previous step (a guess from a counter
    // that the compaction kernel may be rewriting: a wrong guess costs bandwidth, nothing else).
    if (warp == 0 && lane == 0 && p.prefetch_boxes > 0) {
        const int g0 = *reinterpret_cast<const volatile int32_t *>(&p.ctl->n[0]);
        const int g1 = *reinterpret_cast<const volatile int32_t *>(&p.ctl->n[1]);
        const int m = g0 > 0 ? 0 : 1;
        if (g0 > 0 || g1 > 0) {
            const CUtensorMap *tW = m ? &tmW1 : &tmW0;
            const int kcols = (p.H[m] + 63) / 64;
            int left = p.prefetch_boxes;
            for (int row0 = row_begin_m[m]; row0 < row_end_m[m] && left > 0; row0 += kSmallTileRows)
                for (int kc = 0; kc < kcols && left > 0; ++kc, --left) tma_prefetch_l2_2d(tW, kc * 64, row0);
        }
    }
    griddep_wait();
    griddep_launch_dependents();
    const int n_rows[2] = {p.ctl->n[0], p.ctl->n[1]};

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer
        if (lane == 0) {
            const uint64_t pol_keep = l2_policy_evict_last();
            // W is read once per step: streamed lines should leave L2 first, not the hidden rows and
            // not the boxes that the next step's kernel prefetches while this one drains
            // (measured: LLaMA B = 1 step 164.4 -> 161.6 us, small head only 88.5 -> 84.2 us)
            const uint64_t pol_w = l2_policy_evict_first();
            uint32_t it = 0;
            bool ok = true;
            for (int m = 0; m < 2 && ok; ++m) {
                if (n_rows[m] <= 0) continue;
                const int row_begin = row_begin_m[m], row_end = row_end_m[m];
                const CUtensorMap *tA = m ? &tmA1 : &tmA0;
                const CUtensorMap *tW = m ? &tmW1 : &tmW0;
                const CUtensorMap *tP = m ? &tmP1 : &tmP0;
                const int kblocks = (p.H[m] + kSmallBlockK - 1) / kSmallBlockK;
                for (int row0 = row_begin; row0 < row_end && ok; row0 += kSmallTileRows) {
                    const int nrows = min(kSmallTileRows, row_end - row0);        // multiple of 32
                    const uint32_t tx = kSlabs * (h_slab + static_cast<uint32_t>(nrows) * 128);
                    for (int kb = 0; kb < kblocks; ++kb, ++it) {
                        const uint32_t s = it % stages;
                        const uint32_t ph = (it / stages) & 1u;
                        if (!wait_bar(smem_u32(&ctrl->empty[s]), ph ^ 1u, ctrl, ctl)) { ok = false; break; }
                        const uint32_t bar = smem_u32(&ctrl->full[s]);
                        const uint32_t sa = smem_u32(stage0 + static_cast<size_t>(s) * stage_bytes);
                        mbar_arrive_expect_tx(bar, tx);
#pragma unroll
                        for (int h = 0; h < kSlabs; ++h) {
                            const int k0 = kb * kSmallBlockK + h * 64;
                            tma_load_2d(sa + h * h_slab, tA, k0, 0, bar, pol_keep);
                            const uint32_t wdst = sa + kSlabs * h_slab + h * kSmallWBytes;
                            if (nrows == kSmallTileRows) {
                                tma_load_2d(wdst, tW, k0, row0, bar, pol_w);
                            } else {
                                for (int j = 0; j < nrows; j += kSmallSegRows)
                                    tma_load_2d(wdst + j * 128, tP, k0, row0 + j, bar, pol_w);
                            }
                        }
                    }
                }
            }
            // Before the CTA retires, every copy issued above must have landed.
            const uint32_t pending = it < static_cast<uint32_t>(stages) ? it : stages;
            for (uint32_t k = 0; k < pending; ++k) {
                const uint32_t j = it - 1 - k;
                if (!wait_bar(smem_u32(&ctrl->full[j % stages]), (j / stages) & 1u, ctrl, ctl)) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tc = 0;
            bool ok = true;
            for (int m = 0; m < 2 && ok; ++m) {
                if (n_rows[m] <= 0) continue;
                const int row_begin = row_begin_m[m], row_end = row_end_m[m];
                const int kblocks = (p.H[m] + kSmallBlockK - 1) / kSmallBlockK;
                const uint32_t idesc =
                    umma_idesc_bf16_m128(NB == 0 ? static_cast<uint32_t>((n_rows[m] + 15) / 16 * 16) : kSmallN);
                for (int row0 = row_begin; row0 < row_end && ok; row0 += kSmallTileRows, ++tc) {
                    const uint32_t buf = tc & 1u;
                    if (!wait_bar(smem_u32(&ctrl->tmem_empty[buf]), ((tc >> 1) & 1u) ^ 1u, ctrl, ctl)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + buf * kAccCols;
                    for (int kb = 0; kb < kblocks; ++kb, ++it) {
                        const uint32_t s = it % stages;
                        if (!wait_bar(smem_u32(&ctrl->full[s]), (it / stages) & 1u, ctrl, ctl)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint32_t sa = smem_u32(stage0 + static_cast<size_t>(s) * stage_bytes);
#pragma unroll
                        for (int h = 0; h < kSlabs; ++h) {
                            const uint64_t dh = umma_smem_desc(sa + h * h_slab);                         // B: hidden rows
                            const uint64_t dw = umma_smem_desc(sa + kSlabs * h_slab + h * kSmallWBytes);      // A: W rows
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_bf16(d_tmem, dw + 2 * k, dh + 2 * k, idesc, (kb | h | k) != 0);
                        }
                        umma_commit(smem_u32(&ctrl->empty[s]));
                    }
                    if (ok) umma_commit(smem_u32(&ctrl->tmem_full[buf]));
                }
            }
            // All MMAs must have finished before TMEM is released.
            umma_commit(smem_u32(&ctrl->drain));
            wait_bar(smem_u32(&ctrl->drain), 0u, ctrl, ctl);
        }
    } else {
        // ------------------------------------------------------------- epilogue
        const int quad = warp & 3;                     // TMEM lane quadrant this warp may read
        uint32_t tc = 0;
        bool ok = true;
        for (int m = 0; m < 2 && ok; ++m) {
            if (n_rows[m] <= 0) continue;
            const int row_begin = row_begin_m[m], row_end = row_end_m[m];
            if constexpr (NB == 0) {
                float *tbuf = trans + quad * (32 * 33);
                const int n16 = (n_rows[m] + 15) / 16 * 16;
                const int nch = (n16 + 31) / 32;                    // <= 4 chunks of 32 sequences
                const uint32_t rng_step = static_cast<uint32_t>(p.ctl->cur_t);
                RowStat st3[4];
                Draw dr3[4];
                uint32_t rr3[4];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    rowstat_reset(st3[ch]);
                    dr3[ch] = Draw{-INFINITY, 0x7fffffff};
                    const int j = ch * 32 + lane;
                    rr3[ch] = (SAMPLE && j < n_rows[m]) ? static_cast<uint32_t>(p.perm[m * p.B + j]) : 0u;
                }
                for (int row0 = row_begin; row0 < row_end && ok; row0 += kSmallTileRows, ++tc) {
                    const int nrows = min(kSmallTileRows, row_end - row0);
                    const uint32_t buf = tc & 1u;
                    if (!wait_bar_warp(smem_u32(&ctrl->tmem_full[buf]), (tc >> 1) & 1u, ctrl, ctl, lane)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const int cb = row0 + quad * 32;                // vocabulary entries held by this warp's lanes
                    const int limit = min(p.V[m], row0 + nrows);    // first invalid vocabulary entry of the tile
                    if (cb < limit) {
                        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kAccCols;
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            if (ch >= nch) continue;
                            float v[32], w[32];
                            tmem_ld_32cols(taddr + ch * 32, v);
#pragma unroll
                            for (int j = 0; j < 32; ++j) tbuf[j * 33 + lane] = v[j];
                            __syncwarp();
#pragma unroll
                            for (int i = 0; i < 32; ++i) w[i] = tbuf[lane * 33 + i];
                            __syncwarp();
                            if (cb + 32 > limit) {
#pragma unroll
                                for (int i = 0; i < 32; ++i) w[i] = (cb + i < limit) ? w[i] : kNegSentinel;
                            }
                            rowstat_absorb32(st3[ch], w, cb);
                            if (SAMPLE) draw_absorb32(dr3[ch], w, cb, rng_step, rr3[ch], p, p.ctr_off[m]);
                            __syncwarp();
                        }
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->tmem_empty[buf]));
                }
                if (!ok) break;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const int j = ch * 32 + lane;
                    if (ch >= nch || j >= n_rows[m]) continue;
                    const size_t o = (static_cast<size_t>(m) * p.B + j) * p.slots_stride + cta * kSmallSlotsPerCta + quad;
                    p.part_m[o] = st3[ch].m;
                    p.part_s[o] = st3[ch].s;
                    p.part_t[o] = st3[ch].t;
                    p.part_i[o] = st3[ch].idx;
                    if (SAMPLE) {
                        p.part_k[o] = dr3[ch].k;
                        p.part_ki[o] = dr3[ch].ki;
                    }
                }
            } else {
            float sm[NB], ss[NB], stt[NB];
            int sidx[NB];
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                sm[j] = kNegSentinel;
                ss[j] = 0.f;
                stt[j] = 0.f;
                sidx[j] = 0x7fffffff;
            }
            // sampling: largest perturbed value per sequence; the random stream is per caller's row
            float dk[NB];
            int dki[NB];
            uint32_t rng_row[NB];
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                dk[j] = -INFINITY;
                dki[j] = 0x7fffffff;
                rng_row[j] = (SAMPLE && j < n_rows[m]) ? static_cast<uint32_t>(p.perm[m * p.B + j]) : 0u;
            }
            const uint32_t rng_step = static_cast<uint32_t>(p.ctl->cur_t);
            for (int row0 = row_begin; row0 < row_end && ok; row0 += kSmallTileRows, ++tc) {
                const int nrows = min(kSmallTileRows, row_end - row0);
                const uint32_t buf = tc & 1u;
                if (!wait_bar_warp(smem_u32(&ctrl->tmem_full[buf]), (tc >> 1) & 1u, ctrl, ctl, lane)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                float v[16];
                tmem_ld_16cols(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kSmallN, v);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->tmem_empty[buf]));
                const int r_in = quad * 32 + lane;
                const int row = row0 + r_in;                       // vocabulary entry of this thread
                if (r_in < nrows && row < p.V[m]) {
#pragma unroll
                    for (int j = 0; j < NB; ++j) {
                        const float z = v[j];
                        const float mo = sm[j];
                        const float mn = fmaxf(mo, z);
                        const float dm2 = (mo - mn) * kLog2e;       // <= 0
                        const float dz2 = (z - mn) * kLog2e;        // <= 0
                        const float a = ex2_approx(dm2), e = ex2_approx(dz2);
                        stt[j] = fmaf(a, fmaf(dm2, ss[j], stt[j]), e * dz2);
                        ss[j] = fmaf(a, ss[j], e);
                        sidx[j] = (z > mo) ? row : sidx[j];
                        sm[j] = mn;
                    }
                    if (SAMPLE) {
#pragma unroll
                        for (int j = 0; j < NB; ++j) {
                            const uint4 w = philox4x32_10((static_cast<uint32_t>(row) >> 2) + p.ctr_off[m], rng_step, rng_row[j], 0u,
                                                          p.seed_lo, p.seed_hi);
                            const uint32_t word = (row & 3) == 0 ? w.x : (row & 3) == 1 ? w.y : (row & 3) == 2 ? w.z : w.w;
                            const float key = fmaf(v[j], p.inv_temperature, gumbel_from_word(word));
                            if (key > dk[j]) {            // rows ascend within a thread: lowest row wins ties
                                dk[j] = key;
                                dki[j] = row;
                            }
                        }
                    }
                }
                __syncwarp();
            }
            if (!ok) break;
            // ---- end of the head: reduce the 32 threads of this warp, one partial per sequence
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                Partial acc{sm[j], ss[j], stt[j], sidx[j]};
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    Partial q;
                    q.m = __shfl_xor_sync(0xffffffffu, acc.m, o);
                    q.s = __shfl_xor_sync(0xffffffffu, acc.s, o);
                    q.t = __shfl_xor_sync(0xffffffffu, acc.t, o);
                    q.idx = __shfl_xor_sync(0xffffffffu, acc.idx, o);
                    acc = merge_partial(acc, q);
                }
                if (lane == 0 && j < n_rows[m]) {
                    const size_t o = (static_cast<size_t>(m) * p.B + j) * p.slots_stride +
                                     cta * kSmallSlotsPerCta + quad;
                    p.part_m[o] = acc.m;
                    p.part_s[o] = acc.s;
                    p.part_t[o] = acc.t;
                    p.part_i[o] = acc.idx;
                }
                if (SAMPLE) {
                    Draw d{dk[j], dki[j]};
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        Draw q;
                        q.k = __shfl_xor_sync(0xffffffffu, d.k, o);
                        q.ki = __shfl_xor_sync(0xffffffffu, d.ki, o);
                        d = merge_draw(d, q);
                    }
                    if (lane == 0 && j < n_rows[m]) {
                        const size_t o = (static_cast<size_t>(m) * p.B + j) * p.slots_stride +
                                         cta * kSmallSlotsPerCta + quad;
                        p.part_k[o] = d.k;
                        p.part_ki[o] = d.ki;
                    }
                }
            }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem_base, 2 * kAccCols);
}

}  // namespace ead
