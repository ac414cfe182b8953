// The integer / per-row kernels around the LM-head contraction:
//   ead_compact_kernel     splits the batch by active model and gathers the active
//                          model's hidden row of every sequence into a dense operand
//   ead_merge_gate_kernel  merges the per-CTA partial statistics into the entropy of
//                          Eq. 2 and the greedy token, then runs the window / dwell /
//                          threshold part of Algorithm 1 (Eq. 3-4) and updates the state
//   ead_set_args_kernel, ead_reset_kernel   bookkeeping
#pragma once
#include "ead_internal.cuh"
#include "ptx_sm100.cuh"

namespace ead {

constexpr int kCompactThreads = 256;
constexpr int kGateThreads = 256;

__global__ void ead_set_args_kernel(RunArgs *dst, RunArgs a, const StepCtl *ctl)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        a.run_base = ctl->step;
        *dst = a;
    }
}

__global__ void ead_reset_kernel(StepCtl *ctl, uint8_t *flag, int32_t *c, int32_t *nfill, float *ring,
                                 uint32_t *usage, uint8_t *done, int B, int w, int start_model)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        ctl->step = 0;
        ctl->cur_t = 0;
        ctl->n[0] = ctl->n[1] = 0;
        ctl->n_done = 0;
        ctl->status = 0;
    }
    if (i < B) {
        flag[i] = static_cast<uint8_t>(start_model);
        c[i] = 0;
        nfill[i] = 0;
        done[i] = 0;
        usage[i] = usage[B + i] = usage[2 * B + i] = 0u;
    }
    for (int k = i; k < B * w; k += gridDim.x * blockDim.x) ring[k] = 0.f;
}

// Stable partition of the rows by model flag; rows whose sequence has ended ("done") go to
// neither head and get their outputs here (token -1, NaN entropies, model unchanged).  Every
// CTA recomputes the (tiny) scan over the B flags and then copies the rows b = blockIdx.x,
// blockIdx.x + gridDim.x, ...   perm[m * B + r] = original row of compacted row r of head m.
__global__ void __launch_bounds__(kCompactThreads)
ead_compact_kernel(StepCtl *ctl, const RunArgs *args, const uint8_t *flag, const uint8_t *done, int B, int Hs,
                   int Hl, uint16_t *hc_s, uint16_t *hc_l, int32_t *perm, int zero_pad)
{
    extern __shared__ uint32_t pos_sh[];         // [B]: position | class << 30 (0 small, 1 large, 2 done)
    __shared__ int32_t warp_tot[kCompactThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    griddep_launch_dependents();                 // the LM-head kernel may set itself up meanwhile
    griddep_wait();                              // flags and step counter come from the previous step
    const int step = ctl->step;
    const int idx = step - args->run_base;

    const int per = (B + kCompactThreads - 1) / kCompactThreads;
    const int b0 = min(B, tid * per), b1 = min(B, b0 + per);
    int cnt = 0;                                  // large rows in the low half, done rows in the high half
    for (int b = b0; b < b1; ++b) cnt += done[b] ? 0x10000 : (flag[b] ? 1 : 0);
    int incl = cnt;                               // inclusive scan of both counts at once (B <= 4096)
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int before = 0, total = 0;
#pragma unroll
    for (int k = 0; k < kCompactThreads / 32; ++k) {
        const int v = warp_tot[k];
        if (k < warp) before += v;
        total += v;
    }
    const int excl = before + incl - cnt;
    int pos_l = excl & 0xffff;                    // large rows before b0
    int pos_s = b0 - pos_l - (excl >> 16);        // small rows before b0
    for (int b = b0; b < b1; ++b) {
        if (done[b]) {
            pos_sh[b] = 2u << 30;
            continue;
        }
        const int f = flag[b] ? 1 : 0;
        const int pos = f ? pos_l++ : pos_s++;
        pos_sh[b] = static_cast<uint32_t>(pos) | (static_cast<uint32_t>(f) << 30);
        if (blockIdx.x == 0) perm[f * B + pos] = b;
    }
    if (blockIdx.x == 0 && tid == 0) {
        const int total_large = total & 0xffff, total_done = total >> 16;
        ctl->n[0] = B - total_large - total_done;
        ctl->n[1] = total_large;
        ctl->n_done = total_done;
        ctl->cur_t = step;
        ctl->cur_x = ctl->xstep;
    }
    __syncthreads();

    for (int b = blockIdx.x; b < B; b += gridDim.x) {
        const uint32_t e = pos_sh[b];
        const int f = static_cast<int>(e >> 30), pos = static_cast<int>(e & 0x3fffffffu);
        if (f == 2) {                             // ended sequence: nothing is computed for it
            if (tid == 0) {
                const size_t o = static_cast<size_t>(idx) * B + b;
                const float nan = __int_as_float(0x7fc00000);
                if (args->tok) args->tok[o] = -1;
                if (args->H) args->H[o] = nan;
                if (args->Hbar) args->Hbar[o] = nan;
                if (args->used) args->used[o] = flag[b];
                if (args->next) args->next[o] = flag[b];
            }
            continue;
        }
        const int H = f ? Hl : Hs;
        const uint4 *src = reinterpret_cast<const uint4 *>(args->h[f] + (static_cast<size_t>(idx) * B + b) * H);
        uint4 *dst = reinterpret_cast<uint4 *>((f ? hc_l : hc_s) + static_cast<size_t>(pos) * H);
        for (int k = tid; k < H / 8; k += kCompactThreads) dst[k] = __ldg(src + k);
    }

    // Large-batch LM-head kernel: a head's last row block is multiplied as a whole 128-row tile.
    // The rows between the head's last real row and the end of that block would otherwise hold
    // hidden states of earlier steps; they never reach an output either way, but the tensor
    // cores draw power by the bits that toggle, and under the power cap a block padded with
    // zeros runs at a higher clock than one padded with old data.
    if (zero_pad) {
        const int total_large = total & 0xffff, total_done = total >> 16;
        const int n_m[2] = {B - total_large - total_done, total_large};
        const int pad_s = (kTileM - n_m[0] % kTileM) % kTileM;
        const int pad_l = (kTileM - n_m[1] % kTileM) % kTileM;
        for (int q = blockIdx.x; q < pad_s + pad_l; q += gridDim.x) {
            const int f = q < pad_s ? 0 : 1;
            const int row = n_m[f] + (f ? q - pad_s : q);
            const int H = f ? Hl : Hs;
            uint4 *dst = reinterpret_cast<uint4 *>((f ? hc_l : hc_s) + static_cast<size_t>(row) * H);
            for (int k = tid; k < H / 8; k += kCompactThreads) dst[k] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
}

struct GateParams {
    int32_t B, V, w, d_min, unit, G, slots_stride;
    int32_t n_slots;           // > 0: partial slots per row as written by the small-batch kernel
    int32_t units;             // != 0: partials come from the large-batch kernel (units of row blocks);
                               // bit m of two_blocks set = head m is served in units of two row blocks
    int32_t two_blocks;
    float tau;
    StepCtl *ctl;
    const RunArgs *args;
    const float *part_m, *part_s, *part_t;
    const int32_t *part_i;
    int32_t sampling;          // != 0: the token is the sampled candidate, not the arg max
    const float *part_k;
    const int32_t *part_ki;
    const int32_t *perm;
    uint8_t *flag;
    int32_t *c;
    int32_t *nfill;
    float *ring;
    uint32_t *usage;           // [3][B]: tokens by the small model, by the large model, switches
    uint8_t *done;             // [B]: the sequence has produced the end-of-sequence token
    int32_t eos_token;         // < 0: none
    // vocabulary-sharded use: after the cross-CTA merge the kernels hand on one ShardRecord per
    // row (indices shifted by v_off of the row's head): reduce_only = 1 writes it to
    // args->shard_out and stops (the caller exchanges), 2 stores it into the exchange buffer of
    // every shard named in `link` (peer memory) and stops, 3 stores it likewise, then waits for
    // the row's records of all shards and finishes the step
    int32_t reduce_only;
    int32_t v_off[2];
    const ShardLink *link;
};

__device__ __forceinline__ uint32_t ld_acquire_sys(const int32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys(int32_t *p, int32_t v)
{
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Vocabulary-sharded use: folds the records that the n shards delivered for sequence b and
// exchange step `step1` (shard order) into acc / draw.  With `patient` the thread first waits
// for each record's step word (bounded: one deadline for all its waits; an expiry sets
// EAD_STATUS_WAIT_EXPIRED and ends the patience).  Returns whether every record belongs to
// this step and to the head `model`.
__device__ __forceinline__ bool gather_shard_records(const GateParams &p, const ShardRecord *all, int n_shards, int b,
                                                     int model, int step1, bool patient, Partial &acc, Draw &draw)
{
    bool agree = true;
    const unsigned long long t0 = patient ? globaltimer_ns() : 0ull;
    for (int s = 0; s < n_shards; ++s) {
        const ShardRecord *rec = all + static_cast<size_t>(s) * p.B + b;
        int got = static_cast<int>(ld_acquire_sys(&rec->step1));
        while (got != step1 && patient) {
            __nanosleep(64);
            got = static_cast<int>(ld_acquire_sys(&rec->step1));
            if (got != step1 && globaltimer_ns() - t0 > kWaitLimitNs) {
                atomicOr(&p.ctl->status, kStatusWaitExpired);
                patient = false;
            }
        }
        // ordinary loads: the acquire above orders them after the writer's release of the step word
        const float4 lo = *reinterpret_cast<const float4 *>(rec);
        const float2 hi = *reinterpret_cast<const float2 *>(&rec->k);
        const int rmodel = rec->model;
        agree = agree && got == step1 && rmodel == model;
        acc = merge_partial(acc, Partial{lo.x, lo.y, lo.z, __float_as_int(lo.w)});
        draw = merge_draw(draw, Draw{hi.x, __float_as_int(hi.y)});
    }
    return agree;
}

// Everything after the merge for one compacted row (executed by one thread): Eq. 2 in the
// fused form, then the tail of Algorithm 1's loop body (window, counter, Eq. 4), state update
// and outputs scattered back to the caller's row.
// State of one sequence as finish_row needs it; `ring` points at the w window slots (global or a
// shared-memory copy, in which case the new entropy is also written through to `ring_global`).
struct RowState {
    int b, model, nf, c, run_base;
    const float *ring;
    float *ring_global;
};

__device__ __forceinline__ RowState load_row_state(const GateParams &p, int m, int r)
{
    RowState st;
    st.b = p.perm[m * p.B + r];
    st.model = p.flag[st.b];
    st.nf = p.nfill[st.b];
    st.c = p.c[st.b];
    st.run_base = p.args->run_base;
    st.ring_global = p.ring + static_cast<size_t>(st.b) * p.w;
    st.ring = st.ring_global;
    return st;
}

__device__ __forceinline__ void finish_row(const GateParams &p, const RowState &st, const Partial &acc_in, int t_step,
                                           const Draw &draw_in, const RunArgs &out)
{
    Partial acc = acc_in;
    Draw draw = draw_in;
    if (p.reduce_only) {                          // one vocabulary shard: hand the slice's statistics on
        const int off = p.v_off[st.model];
        const int step1 = p.ctl->cur_x + 1;
        const float4 lo = make_float4(acc.m, acc.s, acc.t,
                                      __int_as_float(acc.idx == 0x7fffffff ? acc.idx : acc.idx + off));
        const float2 hi = make_float2(draw.k, __int_as_float(draw.ki == 0x7fffffff ? draw.ki : draw.ki + off));
        if (p.reduce_only == 1) {
            ShardRecord *dst = reinterpret_cast<ShardRecord *>(out.shard_out) + st.b;
            *reinterpret_cast<float4 *>(dst) = lo;
            *reinterpret_cast<float2 *>(&dst->k) = hi;
            dst->model = st.model;
            dst->step1 = step1;
            return;
        }
        // Exchange inside the kernel: the record goes straight into every shard's buffer (plain
        // stores, over NVLink for the peers); the step word follows with release semantics, so a
        // reader that sees it sees the record.  Buffers alternate with the step's parity: a shard
        // can be at most one step ahead of another (its next gate needs that shard's next record).
        const ShardLink &lk = *p.link;
        const size_t slot = (static_cast<size_t>((step1 - 1) & 1) * lk.n + lk.self) * p.B + st.b;
        for (int d = 0; d < lk.n; ++d) {
            ShardRecord *dst = lk.all[d] + slot;
            *reinterpret_cast<float4 *>(dst) = lo;
            *reinterpret_cast<float2 *>(&dst->k) = hi;
            dst->model = st.model;
        }
        for (int d = 0; d < lk.n; ++d) st_release_sys(&(lk.all[d] + slot)->step1, step1);
        if (p.reduce_only == 2) return;           // the caller runs the step's second half apart
        // Whole step in this kernel: wait for the row's records of all shards in the local
        // buffer, fold them in shard order (every shard folds the same values in the same
        // order) and carry on as on one GPU.
        acc = Partial{kNegSentinel, 0.f, 0.f, 0x7fffffff};
        draw = Draw{-INFINITY, 0x7fffffff};
        const ShardRecord *all = lk.all[lk.self] + static_cast<size_t>((step1 - 1) & 1) * lk.n * p.B;
        const bool patient = !(p.ctl->status & kStatusWaitExpired);   // none at all once a wait has expired
        if (!gather_shard_records(p, all, lk.n, st.b, st.model, step1, patient, acc, draw)) {
            atomicOr(&p.ctl->status, kStatusShardMismatch);          // a shard is on another step or saw other flags
            acc.s = 0.f;                                              // reported like a non-finite row: state untouched
        }
    }
    // ---- Eq. 2 in the fused form  H = ln Z - E_p[z] = ln s - t / (s log2 e)   (nats)
    float H = logf(acc.s) - acc.t / (acc.s * kLog2e);
    const bool finite = isfinite(H) && acc.s > 0.f;
    if (H < 0.f) H = 0.f;                         // rounding can leave -1e-7 for a one-hot row
    if (p.unit == 1) H *= kLog2e;                 // bits, as Eq. 2 is printed

    const int b = st.b;
    const size_t o = static_cast<size_t>(t_step - st.run_base) * p.B + b;
    int model = st.model;
    if (!finite) {
        // non-finite logits: report, leave window, counter and model untouched
        atomicOr(&p.ctl->status, kStatusNonFinite);
        if (out.tok) out.tok[o] = -1;
        if (out.H) out.H[o] = __int_as_float(0x7fc00000);
        if (out.Hbar) out.Hbar[o] = __int_as_float(0x7fc00000);
        if (out.used) out.used[o] = static_cast<uint8_t>(model);
        if (out.next) out.next[o] = static_cast<uint8_t>(model);
        return;
    }
    // ---- Algorithm 1: append H_t to W; mean of the last w entries (those present)
    int nf = st.nf;
    const int slot = nf % p.w;
    st.ring_global[slot] = H;
    nf += 1;
    const int cnt = nf < p.w ? nf : p.w;
    if (nf >= 2 * p.w) nf -= p.w;                  // same slot sequence, and the counter stays bounded
    float sum = 0.f;
    for (int k = 0; k < cnt; ++k) sum += (k == slot) ? H : st.ring[k];     // slot order, as stored
    const float Hbar = sum / static_cast<float>(cnt);
    // ---- c <- c + 1; Eq. 4
    int c = st.c < (1 << 30) ? st.c + 1 : st.c;   // saturates far above any d_min instead of wrapping
    const int used = model;
    if (c >= p.d_min) {
        if (model == 0 && Hbar > p.tau) { model = 1; c = 0; }
        else if (model == 1 && Hbar <= p.tau) { model = 0; c = 0; }
    }
    p.nfill[b] = nf;
    p.c[b] = c;
    p.flag[b] = static_cast<uint8_t>(model);
    p.usage[used * p.B + b] += 1u;                     // this row is owned by this thread: no atomics
    if (model != used) p.usage[2 * p.B + b] += 1u;
    const int token = p.sampling ? draw.ki : acc.idx;
    if (p.eos_token >= 0 && token == p.eos_token) p.done[b] = 1;    // "while not done" ends for this row
    if (out.tok) out.tok[o] = token;
    if (out.H) out.H[o] = H;
    if (out.Hbar) out.Hbar[o] = Hbar;
    if (out.used) out.used[o] = static_cast<uint8_t>(used);
    if (out.next) out.next[o] = static_cast<uint8_t>(model);
}

__device__ __forceinline__ Draw warp_merge_draw(Draw d)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Draw q;
        q.k = __shfl_xor_sync(0xffffffffu, d.k, o);
        q.ki = __shfl_xor_sync(0xffffffffu, d.ki, o);
        d = merge_draw(d, q);
    }
    return d;
}

__device__ __forceinline__ Partial warp_merge(Partial acc)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Partial q;
        q.m = __shfl_xor_sync(0xffffffffu, acc.m, o);
        q.s = __shfl_xor_sync(0xffffffffu, acc.s, o);
        q.t = __shfl_xor_sync(0xffffffffu, acc.t, o);
        q.idx = __shfl_xor_sync(0xffffffffu, acc.idx, o);
        acc = merge_partial(acc, q);
    }
    return acc;
}

// One warp per compacted row: partials of the large-batch LM-head kernels (one slot per CTA of the
// row's group, or per member of the unit that serves the row).
__global__ void __launch_bounds__(kGateThreads) ead_merge_gate_kernel(const GateParams p)
{
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * (kGateThreads / 32) + (threadIdx.x >> 5);
    griddep_launch_dependents();
    griddep_wait();                              // partials of the LM-head kernel
    const int n0 = p.ctl->n[0], n1 = p.ctl->n[1];
    const int t_step = p.ctl->cur_t;
    const int nd = p.ctl->n_done;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (n0 + n1 + nd != p.B) atomicOr(&p.ctl->status, kStatusBadCount);
        if (!p.reduce_only || p.reduce_only == 3) p.ctl->step = t_step + 1;   // nobody in this kernel reads `step`
        if (p.reduce_only == 3) p.ctl->xstep = p.ctl->cur_x + 1;
    }
    if (i >= n0 + n1 || n0 + n1 + nd != p.B) return;
    const int m = i < n0 ? 0 : 1;
    const int r = m ? i - n0 : i;
    const int n_m = m ? n1 : n0;
    // partial slots of the row: one per member of the group that served its row block
    int g;
    if (p.units) {
        g = unit_slots_of_row(p.G, n_m, r, (p.two_blocks >> m) & 1);
    } else {
        const int R = (n_m + kTileM - 1) / kTileM;
        g = p.G / R;
        if (g < 1) g = 1;
    }

    // ---- cross-CTA merge, fixed order: each lane folds its slots in ascending
    //      order, then a butterfly over the lanes (no float atomics: deterministic)
    const size_t base = (static_cast<size_t>(m) * p.B + r) * p.slots_stride;
    Partial acc{kNegSentinel, 0.f, 0.f, 0x7fffffff};
    Draw draw{-INFINITY, 0x7fffffff};
    for (int s = lane; s < g; s += 32) {
        const Partial q{p.part_m[base + s], p.part_s[base + s], p.part_t[base + s], p.part_i[base + s]};
        acc = merge_partial(acc, q);
        if (p.sampling) draw = merge_draw(draw, Draw{p.part_k[base + s], p.part_ki[base + s]});
    }
    acc = warp_merge(acc);
    if (p.sampling) draw = warp_merge_draw(draw);
    if (lane == 0) finish_row(p, load_row_state(p, m, r), acc, t_step, draw, *p.args);
}

// One block per compacted row: the 4 G partials of the small-batch kernel.  Thread t folds slots t, t + 256, ... in ascending order, then lanes, then warps:
// a fixed order again.
__global__ void __launch_bounds__(kGateThreads) ead_merge_gate_wide_kernel(const GateParams p)
{
    __shared__ Partial wsum[kGateThreads / 32];
    __shared__ Draw dsum[kGateThreads / 32];
    __shared__ float ring_sh[64];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int i = blockIdx.x;
    griddep_launch_dependents();
    // This kernel is released as soon as the LM-head kernel is past its own dependency wait,
    // i.e. after the compaction kernel has finished: row counts, permutation and the state of
    // the previous step are final, and loading them here hides their latency behind the
    // LM-head kernel.  Only the partials need the wait below.
    const int n0 = p.ctl->n[0], n1 = p.ctl->n[1];
    const int t_step = p.ctl->cur_t;
    const int nd = p.ctl->n_done;
    const bool live = i < n0 + n1 && n0 + n1 + nd == p.B;
    const int m = i < n0 ? 0 : 1;
    const int r = m ? i - n0 : i;
    RowState st{};
    if (live) {
        if (threadIdx.x == 0) st = load_row_state(p, m, r);
        const int b = p.perm[m * p.B + r];
        if (threadIdx.x < p.w) ring_sh[threadIdx.x] = p.ring[static_cast<size_t>(b) * p.w + threadIdx.x];
    }
    st.ring = ring_sh;
    __syncthreads();
    griddep_wait();                              // partials of the LM-head kernel
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (n0 + n1 + nd != p.B) atomicOr(&p.ctl->status, kStatusBadCount);
        if (!p.reduce_only || p.reduce_only == 3) p.ctl->step = t_step + 1;
        if (p.reduce_only == 3) p.ctl->xstep = p.ctl->cur_x + 1;
    }
    if (!live) return;
    const size_t base = (static_cast<size_t>(m) * p.B + r) * p.slots_stride;
    Partial acc{kNegSentinel, 0.f, 0.f, 0x7fffffff};
    Draw draw{-INFINITY, 0x7fffffff};
    for (int s = threadIdx.x; s < p.n_slots; s += kGateThreads) {
        const Partial q{p.part_m[base + s], p.part_s[base + s], p.part_t[base + s], p.part_i[base + s]};
        acc = merge_partial(acc, q);
        if (p.sampling) draw = merge_draw(draw, Draw{p.part_k[base + s], p.part_ki[base + s]});
    }
    acc = warp_merge(acc);
    if (p.sampling) draw = warp_merge_draw(draw);
    if (lane == 0) {
        wsum[warp] = acc;
        dsum[warp] = draw;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        acc = wsum[0];
        draw = dsum[0];
#pragma unroll
        for (int k = 1; k < kGateThreads / 32; ++k) {
            acc = merge_partial(acc, wsum[k]);
            draw = merge_draw(draw, dsum[k]);
        }
        finish_row(p, st, acc, t_step, draw, *p.args);
    }
}

// Vocabulary-sharded use, the step's second half.  One thread per sequence folds the records of
// all n shards for this step in shard order and finishes the step exactly as the single-GPU
// merge does.  Every shard runs this on the same records in the same order, so the per-sequence
// state stays identical on all of them without further communication.
// (Whole steps of a connected context do not come here: there the merge kernels finish the rows
// themselves.)  Outputs `out` are [B].
//   from_exchange = 0: `all` = [n][B] records gathered by the caller
//   from_exchange = 1: records arrive in this shard's exchange buffer (link->all[self]), stored
//           there by the merge kernels of all shards; the thread waits for each record's step
//           word (bounded: a shard that never delivers sets EAD_STATUS_WAIT_EXPIRED)
__global__ void __launch_bounds__(128)
ead_shard_gate_kernel(const GateParams p, const ShardRecord *all, int n_shards, RunArgs out, int from_exchange)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    griddep_launch_dependents();
    griddep_wait();                               // this shard's own records, state of the last step
    const int t_step = p.ctl->cur_t;
    const int step1 = p.ctl->cur_x + 1;
    if (from_exchange) {
        const ShardLink &lk = *p.link;
        n_shards = lk.n;
        all = lk.all[lk.self] + static_cast<size_t>((step1 - 1) & 1) * lk.n * p.B;
    }
    out.run_base = t_step;
    if (b == 0) {                                 // nobody in this kernel reads step or xstep
        p.ctl->step = t_step + 1;
        p.ctl->xstep = step1;
    }
    if (b >= p.B) return;
    const int model = p.flag[b];
    const size_t o = static_cast<size_t>(t_step - out.run_base) * p.B + b;
    if (p.done[b]) {                              // ended sequence: as the compaction kernel reports it
        const float nan = __int_as_float(0x7fc00000);
        if (out.tok) out.tok[o] = -1;
        if (out.H) out.H[o] = nan;
        if (out.Hbar) out.Hbar[o] = nan;
        if (out.used) out.used[o] = static_cast<uint8_t>(model);
        if (out.next) out.next[o] = static_cast<uint8_t>(model);
        return;
    }
    Partial acc{kNegSentinel, 0.f, 0.f, 0x7fffffff};
    Draw draw{-INFINITY, 0x7fffffff};
    // one deadline for all of this thread's waits; none at all once a wait has expired before
    const bool patient = from_exchange && !(p.ctl->status & kStatusWaitExpired);
    const bool agree = gather_shard_records(p, all, n_shards, b, model, step1, patient, acc, draw);
    if (!agree) {                                 // a shard is on another step or saw other flags
        atomicOr(&p.ctl->status, kStatusShardMismatch);
        acc.s = 0.f;                              // reported like a non-finite row: state untouched
    }
    RowState st;
    st.b = b;
    st.model = model;
    st.nf = p.nfill[b];
    st.c = p.c[b];
    st.run_base = out.run_base;
    st.ring_global = p.ring + static_cast<size_t>(b) * p.w;
    st.ring = st.ring_global;
    finish_row(p, st, acc, t_step, draw, out);
}

}  // namespace ead
