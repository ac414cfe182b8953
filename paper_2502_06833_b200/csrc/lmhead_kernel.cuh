// LM-head projection fused with the online softmax-entropy / arg-max reduction.
//
// For each head m (0 = small, 1 = large) with n_m compacted rows, the kernel
// computes z = hc_m * W_m^T (bf16 x bf16 -> fp32 in tensor memory) tile by tile
// and reduces every tile in the epilogue to per-row running statistics
//     m   = max z,   s = sum exp(z - m),   t = sum exp(z - m) * (z - m) * log2(e),
//     idx = lowest column attaining m,
// which is all that Eq. 1-2 of the paper (softmax, Shannon entropy) and the
// greedy token need:  H = ln s - t / (s * log2(e)).  Logits never leave the SM.
//
// Orientation: MMA M (TMEM lanes) = batch rows, MMA N (TMEM columns) = vocabulary,
// K = hidden.  One epilogue thread owns one sequence and walks the columns, so
// the reduction needs no cross-lane traffic.
//
// One persistent CTA per SM, three roles:
//   warp 0      TMA producer: per 64-wide K block, one box of the compacted hidden
//               rows (a_rows x 64) and one box of W (up to 256 x 64) into a ring of
//               shared-memory stages (128-byte swizzle), completion on mbarriers.
//   warp 1      allocates TMEM (2 accumulators x 256 columns) and issues
//               tcgen05.mma (M = 128, N <= 256, K = 16) from one thread.
//   warps 2-5   epilogue: tcgen05.ld 32 columns at a time, online update.
// Accumulators are double buffered so that the epilogue of one tile overlaps the
// MMAs of the next.
//
// A head's rows come in blocks of 128.  Its last block is usually short: with at most 64
// rows it is multiplied as an M = 64 tile (a 64-row hidden box; the accumulator then sits in
// the lower 16 lanes of each 32-lane TMEM quadrant), otherwise as an M = 128 tile whose rows
// beyond the real ones are zeros (the compaction kernel keeps them so).  Neither saves
// cycles - the instruction takes 128 cycles whatever M is - but both save power, which is
// what a run of seconds is bound by.
#pragma once
#include "ead_internal.cuh"
#include "ptx_sm100.cuh"

namespace ead {

struct SmemCtrl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    int32_t tile[2][4];         // small-batch kernel: {first row, end row, range} of this CTA
    uint32_t tmem_base;
    uint32_t abort;
};
static_assert(sizeof(SmemCtrl) <= kSmemCtrlBytes, "control block too large");

// Waits for the phase with the given parity to complete.  Gives up after
// kWaitLimitNs (or as soon as another role has given up), records the event in the
// status word and returns false; the caller then leaves its loop.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, SmemCtrl *c, StepCtl *ctl)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = globaltimer_ns();
    for (;;) {
        // suspended until the phase completes or 4 us have passed: no polling in between
        if (mbar_try_wait_hint(bar, parity, 4000u)) return true;
        if (*reinterpret_cast<volatile uint32_t *>(&c->abort)) return false;
        if (globaltimer_ns() - t0 > kWaitLimitNs) {
            *reinterpret_cast<volatile uint32_t *>(&c->abort) = 1u;
            atomicOr(&ctl->status, kStatusWaitExpired);
            return false;
        }
    }
}

// Warp-collective form: lane 0 waits, the outcome is broadcast.
__device__ __forceinline__ bool wait_bar_warp(uint32_t bar, uint32_t parity, SmemCtrl *c,
                                              StepCtl *ctl, int lane)
{
    uint32_t ok = 0;
    if (lane == 0) ok = wait_bar(bar, parity, c, ctl) ? 1u : 0u;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (ok) {
        while (!mbar_try_wait(bar, parity)) { }   // phase already complete: returns at once
    }
    return ok != 0;
}

struct RowStat {
    float m, ml2, s, t;
    int idx;
};

__device__ __forceinline__ void rowstat_reset(RowStat &st)
{
    st.m = kNegSentinel;
    st.ml2 = kNegSentinel * kLog2e;
    st.s = 0.f;
    st.t = 0.f;
    st.idx = 0x7fffffff;
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Folds 32 consecutive logits (columns col_base ..) into the running statistics.
__device__ __forceinline__ void rowstat_absorb32(RowStat &st, const float (&v)[32], int col_base)
{
    float cm = v[0];
#pragma unroll
    for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
    if (cm > st.m) {
        int j0 = 31;
#pragma unroll
        for (int j = 30; j >= 0; --j) j0 = (v[j] == cm) ? j : j0;
        const float dm2 = (st.m - cm) * kLog2e;          // <= 0: rescale to the new maximum
        const float a = ex2_approx(dm2);
        st.t = a * fmaf(dm2, st.s, st.t);
        st.s *= a;
        st.m = cm;
        st.ml2 = cm * kLog2e;
        st.idx = col_base + j0;
    }
    float s = st.s, t = st.t;
    const float nml2 = -st.ml2;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const float d2 = fmaf(v[j], kLog2e, nml2);        // (z - m) * log2(e)
        const float e = ex2_approx(d2);
        s += e;
        t = fmaf(e, d2, t);
    }
    st.s = s;
    st.t = t;
}

// Temperature sampling: folds 32 consecutive logits (columns cb .., cb a multiple of 16) of the
// sequence with random-stream coordinates (step, row) into its running draw.
__device__ __forceinline__ void draw_absorb32(Draw &dr, const float (&v)[32], int cb, uint32_t rng_step,
                                              uint32_t rng_row, const LmheadParams &p, uint32_t ctr_off)
{
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
        const uint4 w = philox4x32_10((static_cast<uint32_t>(cb + j) >> 2) + ctr_off, rng_step, rng_row, 0u, p.seed_lo,
                                       p.seed_hi);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            // masked columns hold the sentinel: their value can never win
            const float key = fmaf(v[j + q], p.inv_temperature, gumbel_from_word(ww[q]));
            if (key > dr.k) {
                dr.k = key;
                dr.ki = cb + j + q;
            }
        }
    }
}

// Whether a row block with `rows` real rows is multiplied as an M = 64 tile.  The instruction
// takes as long as the M = 128 one, but it reads half the hidden rows (so only 64 are brought in)
// and switches half the multipliers, which under the power cap is what a padded block costs.
__device__ __forceinline__ bool half_block(const LmheadParams &p, int rows)
{
    return p.half_blocks && rows <= kTileM / 2;
}

// SAMPLE: also track the arg max of z / T + Gumbel noise (temperature sampling).
template <bool SAMPLE>
__global__ void __launch_bounds__(kLmheadThreads, 1)
ead_lmhead_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
                  const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
                  const __grid_constant__ CUtensorMap tmT0, const __grid_constant__ CUtensorMap tmT1,
                  const __grid_constant__ CUtensorMap tmH0, const __grid_constant__ CUtensorMap tmH1,
                  const LmheadParams p)
{
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: required by the 128-byte swizzle of the operand tiles
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                ~static_cast<uintptr_t>(1023));
    SmemCtrl *ctrl = reinterpret_cast<SmemCtrl *>(smem);
    uint8_t *stage0 = smem + kSmemCtrlBytes;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    const int G = gridDim.x;
    const int stages = p.stages;
    const uint32_t a_bytes = static_cast<uint32_t>(p.a_rows) * (kBlockK * 2);
    const uint32_t stage_bytes = a_bytes + kWTileBytes;

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
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
            uint32_t it = 0;
            bool ok = true;
            for (int m = 0; m < 2 && ok; ++m) {
                const HeadSplit sp = split_head(cta, G, n_rows[m], p.V[m]);
                if (!sp.active) continue;
                const CUtensorMap *tA = m ? &tmA1 : &tmA0;
                const CUtensorMap *tW = m ? &tmW1 : &tmW0;
                const CUtensorMap *tT = m ? &tmT1 : &tmT0;
                // a row block of at most 64 rows is multiplied as an M = 64 tile: half the hidden box
                const bool half = half_block(p, n_rows[m] - sp.rb * kTileM);
                if (half) tA = m ? &tmH1 : &tmH0;
                const uint32_t a_tx = half ? a_bytes / 2 : a_bytes;
                // a weight tile shared by several row blocks should stay in L2 for them
                const uint64_t pol_w = (sp.R == 1) ? pol_stream : pol_keep;
                const int kblocks = (p.H[m] + kBlockK - 1) / kBlockK;
                for (int col0 = sp.col_begin; col0 < sp.col_end && ok; col0 += kTileN) {
                    const int ncols = min(kTileN, sp.col_end - col0);
                    const uint32_t tx = a_tx + static_cast<uint32_t>(ncols) * (kBlockK * 2);
                    for (int kb = 0; kb < kblocks; ++kb, ++it) {
                        const uint32_t s = it % stages;
                        const uint32_t ph = (it / stages) & 1u;
                        if (!wait_bar(smem_u32(&ctrl->empty[s]), ph ^ 1u, ctrl, ctl)) { ok = false; break; }
                        const uint32_t bar = smem_u32(&ctrl->full[s]);
                        const uint32_t sa = smem_u32(stage0 + static_cast<size_t>(s) * stage_bytes);
                        mbar_arrive_expect_tx(bar, tx);
                        tma_load_2d(sa, tA, kb * kBlockK, sp.rb * kTileM, bar, pol_keep);
                        if (ncols == kTileN) {
                            tma_load_2d(sa + a_bytes, tW, kb * kBlockK, col0, bar, pol_w);
                        } else {
                            for (int j = 0; j < ncols; j += kUnit)
                                tma_load_2d(sa + a_bytes + j * (kBlockK * 2), tT, kb * kBlockK, col0 + j,
                                            bar, pol_w);
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
                const HeadSplit sp = split_head(cta, G, n_rows[m], p.V[m]);
                if (!sp.active) continue;
                const int kblocks = (p.H[m] + kBlockK - 1) / kBlockK;
                for (int col0 = sp.col_begin; col0 < sp.col_end && ok; col0 += kTileN, ++tc) {
                    const int ncols = min(kTileN, sp.col_end - col0);
                    const uint32_t buf = tc & 1u;
                    if (!wait_bar(smem_u32(&ctrl->tmem_empty[buf]), ((tc >> 1) & 1u) ^ 1u, ctrl, ctl)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t idesc = half_block(p, n_rows[m] - sp.rb * kTileM)
                                               ? umma_idesc_bf16_m64(static_cast<uint32_t>(ncols))
                                               : umma_idesc_bf16_m128(static_cast<uint32_t>(ncols));
                    const uint32_t d_tmem = tmem_base + buf * kTileN;
                    for (int kb = 0; kb < kblocks; ++kb, ++it) {
                        const uint32_t s = it % stages;
                        if (!wait_bar(smem_u32(&ctrl->full[s]), (it / stages) & 1u, ctrl, ctl)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint32_t sa = smem_u32(stage0 + static_cast<size_t>(s) * stage_bytes);
                        const uint64_t da = umma_smem_desc(sa);
                        const uint64_t db = umma_smem_desc(sa + a_bytes);
#pragma unroll
                        for (int k = 0; k < kBlockK / 16; ++k)   // +32 B (>>4 = 2) per 16 elements of K
                            umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                        umma_commit(smem_u32(&ctrl->empty[s]));   // stage reusable once these MMAs are done
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
        const int quad = warp & 3;                   // TMEM lane quadrant this warp may read
        uint32_t tc = 0;
        bool ok = true;
        for (int m = 0; m < 2 && ok; ++m) {
            const HeadSplit sp = split_head(cta, G, n_rows[m], p.V[m]);
            if (!sp.active) continue;
            const int rows_valid = min(kTileM, n_rows[m] - sp.rb * kTileM);
            // An M = 128 accumulator keeps row r of the block in TMEM lane r; an M = 64 one keeps
            // its 64 rows in the lower 16 lanes of each 32-lane quadrant (row r in lane
            // (r / 16) * 32 + r % 16), the upper 16 lanes hold nothing.
            const bool half = half_block(p, rows_valid);
            const int row_in_block = half ? (lane < 16 ? quad * 16 + lane : kTileM) : quad * 32 + lane;
            const bool warp_has_rows = (half ? quad * 16 : quad * 32) < rows_valid;
            RowStat st;
            rowstat_reset(st);
            // sampling: this thread's sequence draws from its own stream (caller's row, step)
            Draw dr{-INFINITY, 0x7fffffff};
            const bool row_live = sp.rb * kTileM + row_in_block < n_rows[m];
            const bool sampling = SAMPLE && row_live;
            const uint32_t rng_row = sampling ? static_cast<uint32_t>(p.perm[m * p.B + sp.rb * kTileM + row_in_block]) : 0u;
            const uint32_t rng_step = static_cast<uint32_t>(p.ctl->cur_t);
            for (int col0 = sp.col_begin; col0 < sp.col_end && ok; col0 += kTileN, ++tc) {
                const int ncols = min(kTileN, sp.col_end - col0);
                const uint32_t buf = tc & 1u;
                if (!wait_bar_warp(smem_u32(&ctrl->tmem_full[buf]), (tc >> 1) & 1u, ctrl, ctl, lane)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                if (warp_has_rows) {
                    const int col_limit = min(p.V[m], col0 + ncols);       // first invalid column
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kTileN;
                    for (int c = 0; c < ncols; c += 32) {
                        float v[32];
                        tmem_ld_32cols(taddr + c, v);
                        const int cb = col0 + c;
                        if (cb + 32 > col_limit) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = (cb + j < col_limit) ? v[j] : kNegSentinel;
                        }
                        rowstat_absorb32(st, v, cb);
                        if (SAMPLE && sampling) draw_absorb32(dr, v, cb, rng_step, rng_row, p, p.ctr_off[m]);
                        __syncwarp();
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->tmem_empty[buf]));
            }
            const int row = sp.rb * kTileM + row_in_block;
            if (ok && row < n_rows[m]) {
                const size_t o = (static_cast<size_t>(m) * p.B + row) * p.slots_stride + sp.slot;
                p.part_m[o] = st.m;
                p.part_s[o] = st.s;
                p.part_t[o] = st.t;
                p.part_i[o] = st.idx;
                if (SAMPLE) {
                    p.part_k[o] = dr.k;
                    p.part_ki[o] = dr.ki;
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem_base, 2 * kTileN);
}

}  // namespace ead
