// Host side of the C ABI declared in include/ead.h: context set-up (state, scratch,
// TMA descriptors), step orchestration and CUDA-graph replay of the T-step loop.
#include "../../include/ead.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "ead_internal.cuh"
#include "gate_kernels.cuh"
#include "lmhead_kernel.cuh"
#include "lmhead_dual_kernel.cuh"
#include "lmhead_small_kernel.cuh"

using namespace ead;

namespace {

constexpr int kMidCols = 32;              // value of ead_ctx::small_cols that selects ead_lmhead_small_kernel<0>
// 16 KiB weight boxes per CTA fetched into L2 ahead of the dependency wait.  Measured optimum on the
// LLaMA-shaped heads: 64 for B <= 16 (one head per step at B = 1: 160.7 us per step against 162.5 with 32
// and 161.8 with 128), 32 for 17..128 sequences (both heads live in most steps and only one is guessed:
// 256 us against 259 with 64).
constexpr int kPrefetchBoxesSmall = 64;
constexpr int kPrefetchBoxesMid = 32;
constexpr int kGraphChunk = 32;           // gate steps unrolled in the replayed graph
constexpr uint32_t kStateMagic = 0x45414433u;   // "EAD3"
constexpr size_t kHostStageBytes = 64u << 20;   // per staging buffer of ead_run_host

struct StateHeader {
    uint32_t magic;
    int32_t B, w, step;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 matrix [rows, cols] row major -> tiles of box_rows x 64 elements, 128-byte swizzle,
// out-of-range elements read as zero.
bool encode_bf16_2d(CUtensorMap *tm, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(kBlockK), box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct ead_ctx {
    ead_config cfg{};
    cudaStream_t stream = nullptr;
    cudaStream_t cap_stream = nullptr;     // capture happens on a private stream
    int G = 0, a_rows = 0, stages = 0, slots_stride = 0;
    int two_blocks = 0;                    // large-batch kernel: bit m = head m is served in units of two row blocks
    size_t ring_bytes = 0;                 // ... and the bytes of its stage ring
    int V_large = 0;                       // vocabulary of the large head (cfg.V_large, or cfg.V if that is 0)
    int small_cols = 0;                    // > 0: swapped-operand kernel: batch columns per thread (1..16), or
                                           // kMidCols for its 17..128-sequence variant
    int small_slots = 0;                   // partial slots per row it writes (one per CTA and epilogue warp)
    size_t smem_bytes = 0;
    const void *W[2] = {nullptr, nullptr};
    // device state and scratch (owned)
    StepCtl *ctl = nullptr;
    RunArgs *args = nullptr;
    uint8_t *flag = nullptr, *done = nullptr;
    int32_t *c = nullptr, *nfill = nullptr, *perm = nullptr, *part_i = nullptr, *part_ki = nullptr;
    float *part_k = nullptr;
    uint32_t *usage = nullptr;
    float *ring = nullptr, *part_m = nullptr, *part_s = nullptr, *part_t = nullptr;
    uint16_t *hc[2] = {nullptr, nullptr};
    ShardLink *link = nullptr;             // vocabulary-sharded contexts: where the records go (device)
    bool connected = false;                // ead_shard_connect has filled `link`
    CUtensorMap tmA[2], tmH[2], tmW[2], tmT[2], tmP[2], tmQ[2];   // hidden rows (boxes of a_rows and of 64 rows); W boxes of 256|128, 16, 32 and 64 rows
    cudaGraphExec_t g_one = nullptr, g_chunk = nullptr;
    int64_t launches = 0;
    // staging of ead_run_host (allocated on first use)
    cudaStream_t in_stream = nullptr, out_stream = nullptr;
    uint16_t *st_h[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};
    void *st_out[2] = {nullptr, nullptr};
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_comp[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    int st_steps = 0;
};

namespace {

#define EAD_CUDA(x)                          \
    do {                                     \
        if ((x) != cudaSuccess) {            \
            cudaGetLastError();              \
            return EAD_ECUDA;                \
        }                                    \
    } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Launches `kernel`; with `pdl` the launch carries the programmatic-stream-serialization
// attribute: the kernel may start while its predecessor in the stream is still running and
// synchronises with it through griddepcontrol.wait.
template <typename... KArgs, typename... Args>
cudaError_t launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl,
                   Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

GateParams gate_params(const ead_ctx *x, int reduce_only)
{
    const ead_config &c = x->cfg;
    GateParams gp{};
    gp.B = c.B;
    gp.V = c.V;
    gp.w = c.w;
    gp.d_min = c.d_min;
    gp.unit = c.unit;
    gp.G = x->G;
    gp.slots_stride = x->slots_stride;
    gp.n_slots = x->small_slots;
    gp.units = x->small_cols ? 0 : 1;
    gp.two_blocks = x->two_blocks;
    gp.tau = c.tau;
    gp.ctl = x->ctl;
    gp.args = x->args;
    gp.part_m = x->part_m;
    gp.part_s = x->part_s;
    gp.part_t = x->part_t;
    gp.part_i = x->part_i;
    gp.sampling = c.temperature > 0.f ? 1 : 0;
    gp.part_k = x->part_k;
    gp.part_ki = x->part_ki;
    gp.perm = x->perm;
    gp.flag = x->flag;
    gp.c = x->c;
    gp.nfill = x->nfill;
    gp.ring = x->ring;
    gp.usage = x->usage;
    gp.done = x->done;
    gp.eos_token = c.eos_token;
    gp.reduce_only = reduce_only;
    gp.link = x->link;
    gp.v_off[0] = c.vocab_offset_small;
    gp.v_off[1] = c.vocab_offset_large;
    return gp;
}

// The three kernels of one gate step, in stream order.  With `ev` (4 events) the
// boundaries between the kernels are recorded for timing and the kernels do not overlap;
// otherwise each kernel's set-up overlaps the tail of the one before it.
// shard_mode (vocabulary-sharded contexts): 1 = stop after the merge, records to the caller's
// buffer; 2 = records into every shard's exchange buffer, then the same thread waits for the
// row's records of all shards and finishes the step; 3 = as 2 without the second half.
int enqueue_step(ead_ctx *x, cudaStream_t s, cudaEvent_t *ev = nullptr, int shard_mode = 0)
{
    const ead_config &c = x->cfg;
    const bool pdl = ev == nullptr;
    const int cgrid = std::min(c.B, 4 * x->G);
    cudaError_t e = cudaSuccess;
    if (ev) cudaEventRecord(ev[0], s);
    e = launch(ead_compact_kernel, dim3(cgrid), dim3(kCompactThreads), static_cast<size_t>(c.B) * sizeof(int32_t), s, pdl,
               x->ctl, x->args, x->flag, x->done, c.B, c.H_small, c.H_large, x->hc[0], x->hc[1], x->perm,
               x->small_cols ? 0 : 1);
    if (e != cudaSuccess) return EAD_ECUDA;
    if (ev) cudaEventRecord(ev[1], s);

    LmheadParams lp{};
    lp.V[0] = c.V;
    lp.V[1] = x->V_large;
    lp.H[0] = c.H_small;
    lp.H[1] = c.H_large;
    lp.a_rows = x->a_rows;
    lp.n_cols = x->small_cols;
    lp.stages = x->stages;
    lp.slots_stride = x->slots_stride;
    lp.B = c.B;
    lp.ctl = x->ctl;
    lp.ctl_rw = x->ctl;
    lp.part_m = x->part_m;
    lp.part_s = x->part_s;
    lp.part_t = x->part_t;
    lp.part_i = x->part_i;
    lp.sampling = c.temperature > 0.f ? 1 : 0;
    lp.inv_temperature = c.temperature > 0.f ? 1.f / c.temperature : 0.f;
    lp.seed_lo = static_cast<uint32_t>(c.seed);
    lp.seed_hi = static_cast<uint32_t>(c.seed >> 32);
    lp.part_k = x->part_k;
    lp.part_ki = x->part_ki;
    lp.perm = x->perm;
    lp.prefetch_boxes = !pdl ? 0 : x->small_cols == kMidCols ? kPrefetchBoxesMid : kPrefetchBoxesSmall;     // nothing to overlap with when the kernels are timed apart
    lp.ctr_off[0] = static_cast<uint32_t>(c.vocab_offset_small) >> 2;
    lp.ctr_off[1] = static_cast<uint32_t>(c.vocab_offset_large) >> 2;
    const dim3 lgrid(x->G), lblock(kLmheadThreads);
#define EAD_LAUNCH_SMALL(NB)                                                                                   \
    e = lp.sampling ? launch(ead_lmhead_small_kernel<NB, true>, lgrid, lblock, x->smem_bytes, s, pdl, x->tmA[0],  \
                             x->tmA[1], x->tmW[0], x->tmW[1], x->tmP[0], x->tmP[1], lp)                        \
                    : launch(ead_lmhead_small_kernel<NB, false>, lgrid, lblock, x->smem_bytes, s, pdl, x->tmA[0], \
                             x->tmA[1], x->tmW[0], x->tmW[1], x->tmP[0], x->tmP[1], lp)
    switch (x->small_cols) {
        case 0:
            lp.half_blocks = 1;
            lp.two_blocks = x->two_blocks;
            lp.ring_bytes = static_cast<int32_t>(x->ring_bytes);
            e = lp.sampling ? launch(ead_lmhead_dual_kernel<true>, lgrid, lblock, x->smem_bytes, s, pdl, x->tmA[0],
                                     x->tmA[1], x->tmW[0], x->tmW[1], x->tmT[0], x->tmT[1], x->tmH[0], x->tmH[1], x->tmQ[0], x->tmQ[1], lp)
                            : launch(ead_lmhead_dual_kernel<false>, lgrid, lblock, x->smem_bytes, s, pdl, x->tmA[0],
                                     x->tmA[1], x->tmW[0], x->tmW[1], x->tmT[0], x->tmT[1], x->tmH[0], x->tmH[1], x->tmQ[0], x->tmQ[1], lp);
            break;
        case 1: EAD_LAUNCH_SMALL(1); break;
        case 2: EAD_LAUNCH_SMALL(2); break;
        case 4: EAD_LAUNCH_SMALL(4); break;
        case 8: EAD_LAUNCH_SMALL(8); break;
        case 16: EAD_LAUNCH_SMALL(16); break;
        default: EAD_LAUNCH_SMALL(0); break;     // kMidCols
    }
#undef EAD_LAUNCH_SMALL
    if (e != cudaSuccess) return EAD_ECUDA;
    if (ev) cudaEventRecord(ev[2], s);

    const GateParams gp = gate_params(x, shard_mode == 3 ? 2 : shard_mode == 2 ? 3 : shard_mode);
    const int rows_per_block = kGateThreads / 32;
    if (x->small_cols)
        e = launch(ead_merge_gate_wide_kernel, dim3(c.B), dim3(kGateThreads), 0, s, pdl, gp);
    else
        e = launch(ead_merge_gate_kernel, dim3((c.B + rows_per_block - 1) / rows_per_block), dim3(kGateThreads), 0, s,
                   pdl, gp);
    if (e != cudaSuccess) return EAD_ECUDA;
    if (ev) cudaEventRecord(ev[3], s);
    return cudaGetLastError() == cudaSuccess ? EAD_OK : EAD_ECUDA;
}

int step_mode(const ead_ctx *x) { return x->cfg.shard_count > 0 ? 2 : 0; }
int kernels_per_step(const ead_ctx *) { return 3; }
// Sharded contexts take whole steps only once their exchange buffers are known.
bool can_step(const ead_ctx *x) { return x->cfg.shard_count == 0 || x->connected; }

int build_graph(ead_ctx *x, int steps, cudaGraphExec_t *out)
{
    cudaGraph_t graph = nullptr;
    EAD_CUDA(cudaStreamBeginCapture(x->cap_stream, cudaStreamCaptureModeThreadLocal));
    int rc = EAD_OK;
    for (int i = 0; i < steps && rc == EAD_OK; ++i) rc = enqueue_step(x, x->cap_stream, nullptr, step_mode(x));
    cudaError_t e = cudaStreamEndCapture(x->cap_stream, &graph);
    if (rc != EAD_OK || e != cudaSuccess || !graph) {
        if (graph) cudaGraphDestroy(graph);
        cudaGetLastError();
        return EAD_ECUDA;
    }
    e = cudaGraphInstantiate(out, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return EAD_ECUDA;
    }
    return EAD_OK;
}

int set_args(ead_ctx *x, const void *hs, const void *hl, int32_t *tok, float *H, float *Hbar, uint8_t *used,
             uint8_t *next, cudaStream_t s, float *shard_out = nullptr)
{
    RunArgs a{};
    a.shard_out = shard_out;
    a.h[0] = static_cast<const uint16_t *>(hs);
    a.h[1] = static_cast<const uint16_t *>(hl);
    a.tok = tok;
    a.H = H;
    a.Hbar = Hbar;
    a.used = used;
    a.next = next;
    ead_set_args_kernel<<<1, 32, 0, s>>>(x->args, a, x->ctl);
    x->launches += 1;
    return cudaGetLastError() == cudaSuccess ? EAD_OK : EAD_ECUDA;
}

int run_device(ead_ctx *x, int T, const void *hs, const void *hl, int32_t *tok, float *H, float *Hbar,
               uint8_t *used, uint8_t *next)
{
    int rc = set_args(x, hs, hl, tok, H, Hbar, used, next, x->stream);
    if (rc != EAD_OK) return rc;
    int left = T;
    while (left >= kGraphChunk) {
        EAD_CUDA(cudaGraphLaunch(x->g_chunk, x->stream));
        left -= kGraphChunk;
    }
    while (left > 0) {
        EAD_CUDA(cudaGraphLaunch(x->g_one, x->stream));
        left -= 1;
    }
    x->launches += static_cast<int64_t>(kernels_per_step(x)) * T;
    return EAD_OK;
}

void free_staging(ead_ctx *x)
{
    for (int i = 0; i < 2; ++i) {
        for (int m = 0; m < 2; ++m) {
            if (x->st_h[i][m]) cudaFree(x->st_h[i][m]);
            x->st_h[i][m] = nullptr;
        }
        if (x->st_out[i]) cudaFree(x->st_out[i]);
        x->st_out[i] = nullptr;
        if (x->ev_in[i]) cudaEventDestroy(x->ev_in[i]);
        if (x->ev_comp[i]) cudaEventDestroy(x->ev_comp[i]);
        if (x->ev_out[i]) cudaEventDestroy(x->ev_out[i]);
        x->ev_in[i] = x->ev_comp[i] = x->ev_out[i] = nullptr;
    }
    if (x->in_stream) cudaStreamDestroy(x->in_stream);
    if (x->out_stream) cudaStreamDestroy(x->out_stream);
    x->in_stream = x->out_stream = nullptr;
    x->st_steps = 0;
}

// Bytes of one step of outputs in the staging layout: tok | H | Hbar | used | next,
// each [steps, B], sections 16-byte aligned for a given number of steps.
struct OutLayout {
    size_t off_tok, off_H, off_Hbar, off_used, off_next, total;
};
OutLayout out_layout(int steps, int B)
{
    auto up = [](size_t v) { return (v + 255) & ~static_cast<size_t>(255); };
    OutLayout l;
    const size_t n = static_cast<size_t>(steps) * B;
    l.off_tok = 0;
    l.off_H = up(l.off_tok + 4 * n);
    l.off_Hbar = up(l.off_H + 4 * n);
    l.off_used = up(l.off_Hbar + 4 * n);
    l.off_next = up(l.off_used + n);
    l.total = up(l.off_next + n);
    return l;
}

int ensure_staging(ead_ctx *x)
{
    if (x->st_steps) return EAD_OK;
    const ead_config &c = x->cfg;
    const size_t per_step = static_cast<size_t>(c.B) * (c.H_small + c.H_large) * 2;
    // about 64 MB per buffer, but room for one 32-step graph if that takes no more than 512 MB
    // (large batches: a chunk of single-step replays loses the overlap between the steps)
    const size_t lo = std::max<size_t>(1, std::min<size_t>(kGraphChunk, (512u << 20) / per_step));
    int steps = static_cast<int>(std::max<size_t>(lo, kHostStageBytes / per_step));
    steps = std::min(steps, 256);
    if (steps > kGraphChunk) steps -= steps % kGraphChunk;
    EAD_CUDA(cudaStreamCreateWithFlags(&x->in_stream, cudaStreamNonBlocking));
    EAD_CUDA(cudaStreamCreateWithFlags(&x->out_stream, cudaStreamNonBlocking));
    const OutLayout l = out_layout(steps, c.B);
    for (int i = 0; i < 2; ++i) {
        EAD_CUDA(cudaMalloc(&x->st_h[i][0], static_cast<size_t>(steps) * c.B * c.H_small * 2));
        EAD_CUDA(cudaMalloc(&x->st_h[i][1], static_cast<size_t>(steps) * c.B * c.H_large * 2));
        EAD_CUDA(cudaMalloc(&x->st_out[i], l.total));
        EAD_CUDA(cudaEventCreateWithFlags(&x->ev_in[i], cudaEventDisableTiming));
        EAD_CUDA(cudaEventCreateWithFlags(&x->ev_comp[i], cudaEventDisableTiming));
        EAD_CUDA(cudaEventCreateWithFlags(&x->ev_out[i], cudaEventDisableTiming));
    }
    x->st_steps = steps;
    return EAD_OK;
}

}  // namespace

extern "C" {

const char *ead_strerror(int code)
{
    switch (code) {
        case EAD_OK: return "ok";
        case EAD_EINVALID_ARG: return "invalid argument";
        case EAD_EALIGNMENT: return "pointer not 16-byte aligned or hidden size not a multiple of 8";
        case EAD_ECUDA: return "CUDA call failed";
        case EAD_EUNSUPPORTED_ARCH: return "device is not sm_100";
        case EAD_EDEVICE_FAULT: return "device status word reports a kernel-side error";
        case EAD_ESTATE: return "state blob does not match this context";
        case EAD_ELIMIT: return "size exceeds a built-in limit (EAD_STATIC_MAX_B / EAD_STATIC_MAX_H)";
        default: return "unknown error";
    }
}

int ead_create(const ead_config *cfg, const void *W_small, const void *W_large, ead_ctx **out)
{
    if (!cfg || !W_small || !W_large || !out) return EAD_EINVALID_ARG;
    *out = nullptr;
    if (cfg->B < 1 || cfg->B > 4096 || cfg->V < 1 || cfg->H_small < 8 || cfg->H_large < 8 || cfg->w < 1 ||
        cfg->w > 64 || (cfg->unit != 0 && cfg->unit != 1) || (cfg->start_model != 0 && cfg->start_model != 1) ||
        !(cfg->temperature >= 0.f) || !(cfg->temperature < 3.0e38f) || cfg->V_large < 0 || cfg->shard_count < 0 ||
        cfg->shard_count > kMaxShards ||
        cfg->vocab_offset_small < 0 || cfg->vocab_offset_large < 0 ||
        (cfg->shard_count == 0 && (cfg->vocab_offset_small || cfg->vocab_offset_large)) ||
        // a sharded context sees one slice: the end-of-sequence token indexes the full vocabulary
        (cfg->shard_count == 0 && cfg->eos_token >= std::min(cfg->V, cfg->V_large > 0 ? cfg->V_large : cfg->V)))
        return EAD_EINVALID_ARG;
    if (cfg->vocab_offset_small % kUnit || cfg->vocab_offset_large % kUnit) return EAD_EALIGNMENT;
    if (cfg->H_small % 8 || cfg->H_large % 8 || !aligned16(W_small) || !aligned16(W_large)) return EAD_EALIGNMENT;

    int ndev = 0;
    EAD_CUDA(cudaGetDeviceCount(&ndev));
    if (cfg->device < 0 || cfg->device >= ndev) return EAD_EINVALID_ARG;
    EAD_CUDA(cudaSetDevice(cfg->device));
    cudaDeviceProp prop;
    EAD_CUDA(cudaGetDeviceProperties(&prop, cfg->device));
    if (prop.major != 10) return EAD_EUNSUPPORTED_ARCH;

    ead_ctx *x = new (std::nothrow) ead_ctx();
    if (!x) return EAD_ECUDA;
    x->cfg = *cfg;
    x->stream = static_cast<cudaStream_t>(cfg->stream);
    x->V_large = cfg->V_large > 0 ? cfg->V_large : cfg->V;
    x->W[0] = W_small;
    x->W[1] = W_large;
    x->G = std::min(prop.multiProcessorCount, kMaxCtas);
    if ((cfg->B + kTileM - 1) / kTileM > x->G) {   // the work split needs one CTA per row block at least
        delete x;
        return EAD_EINVALID_ARG;
    }
    x->slots_stride = (x->G + 31) & ~31;
    const size_t smem_max = prop.sharedMemPerBlockOptin;
    size_t stage_bytes;
    if (cfg->B <= kSmallN) {
        // latency regime: swapped-operand kernel, batch columns rounded up to a power of two
        x->small_cols = 1;
        while (x->small_cols < cfg->B) x->small_cols *= 2;
        x->a_rows = cfg->B <= 8 ? 8 : kSmallN;
        stage_bytes = small_stage_bytes(x->a_rows, small_slabs(1));
        x->small_slots = x->G * kSmallSlotsPerCta;
        x->slots_stride = (x->small_slots + 31) & ~31;
    } else if (cfg->B <= kMidMaxRows) {
        // still bound by streaming the weights: same kernel, sequences in chunks of 32
        x->small_cols = kMidCols;
        x->a_rows = (cfg->B + 15) / 16 * 16;
        stage_bytes = small_stage_bytes(x->a_rows, small_slabs(0));
        x->small_slots = x->G * kSmallSlotsPerCta;
        x->slots_stride = (x->small_slots + 31) & ~31;
    } else {
        // tensor-bound regime.  A head with a long K loop (48 K blocks and more) is served in units of
        // two row blocks: the epilogue that no longer hides then costs less than the shared-memory
        // traffic saved (measured: H = 5120 all-large step -7 %, H = 1536 all-small step +6 %).
        x->a_rows = kTileM;
        stage_bytes = kSingleStageBytes;           // what launch_info reports: stages of a one-block head
        x->two_blocks = (cfg->H_small >= 48 * kBlockK ? 1 : 0) | (cfg->H_large >= 48 * kBlockK ? 2 : 0);
    }
    const size_t extra = x->small_cols == kMidCols ? kTransposeBytes : 0;   // transpose tiles of its epilogue
    x->stages = static_cast<int>(
        std::min<size_t>(kMaxStages, (smem_max - kSmemCtrlBytes - 1024 - 1024 - extra) / stage_bytes));
    x->smem_bytes = kSmemCtrlBytes + 1024 + x->stages * stage_bytes + extra;
    if (!x->small_cols) {                          // the kernel cuts the whole ring into 48 or 64 KiB stages per head
        x->ring_bytes = (smem_max - kSmemCtrlBytes - 2048 - kThinMergeBytes) & ~static_cast<size_t>(1023);
        x->smem_bytes = kSmemCtrlBytes + 1024 + x->ring_bytes + kThinMergeBytes;   // merge buffer of the thin block behind the ring
    }

    const int B = cfg->B;
    // compacted operands are padded to whole row blocks (zeros) so that no TMA box of
    // hidden rows reaches past the tensor
    const size_t Bpad = (static_cast<size_t>(B) + kTileM - 1) / kTileM * kTileM;
    const size_t np = 2ull * B * x->slots_stride;
    int rc = EAD_OK;
    auto fail = [&](int code) {
        ead_destroy(x);
        return code;
    };
    if (x->stages < 2) return fail(EAD_ECUDA);
    if (cudaStreamCreateWithFlags(&x->cap_stream, cudaStreamNonBlocking) != cudaSuccess) return fail(EAD_ECUDA);
    if (cudaMalloc(&x->ctl, sizeof(StepCtl)) != cudaSuccess || cudaMalloc(&x->args, sizeof(RunArgs)) != cudaSuccess ||
        cudaMalloc(&x->flag, B) != cudaSuccess || cudaMalloc(&x->done, B) != cudaSuccess || cudaMalloc(&x->c, 4ull * B) != cudaSuccess ||
        cudaMalloc(&x->nfill, 4ull * B) != cudaSuccess || cudaMalloc(&x->perm, 8ull * B) != cudaSuccess ||
        cudaMalloc(&x->ring, 4ull * B * cfg->w) != cudaSuccess ||
        cudaMalloc(&x->usage, 12ull * B) != cudaSuccess ||
        cudaMalloc(&x->hc[0], 2ull * Bpad * cfg->H_small) != cudaSuccess ||
        cudaMalloc(&x->hc[1], 2ull * Bpad * cfg->H_large) != cudaSuccess ||
        cudaMalloc(&x->part_m, 4 * np) != cudaSuccess || cudaMalloc(&x->part_s, 4 * np) != cudaSuccess ||
        cudaMalloc(&x->part_t, 4 * np) != cudaSuccess || cudaMalloc(&x->part_i, 4 * np) != cudaSuccess ||
        cudaMalloc(&x->part_k, 4 * np) != cudaSuccess || cudaMalloc(&x->part_ki, 4 * np) != cudaSuccess)
        return fail(EAD_ECUDA);
    if (cfg->shard_count > 0) {
        if (cudaMalloc(&x->link, sizeof(ShardLink)) != cudaSuccess) return fail(EAD_ECUDA);
        cudaMemsetAsync(x->link, 0, sizeof(ShardLink), x->stream);
    }
    cudaMemsetAsync(x->ctl, 0, sizeof(StepCtl), x->stream);
    cudaMemsetAsync(x->args, 0, sizeof(RunArgs), x->stream);
    cudaMemsetAsync(x->perm, 0, 8ull * B, x->stream);
    cudaMemsetAsync(x->hc[0], 0, 2ull * Bpad * cfg->H_small, x->stream);
    cudaMemsetAsync(x->hc[1], 0, 2ull * Bpad * cfg->H_large, x->stream);
    cudaMemsetAsync(x->part_m, 0, 4 * np, x->stream);
    cudaMemsetAsync(x->part_s, 0, 4 * np, x->stream);
    cudaMemsetAsync(x->part_t, 0, 4 * np, x->stream);
    cudaMemsetAsync(x->part_i, 0, 4 * np, x->stream);
    cudaMemsetAsync(x->part_k, 0, 4 * np, x->stream);
    cudaMemsetAsync(x->part_ki, 0, 4 * np, x->stream);

    const int Hm[2] = {cfg->H_small, cfg->H_large};
    const int Vm[2] = {cfg->V, x->V_large};
    for (int m = 0; m < 2; ++m) {
        const uint32_t wbox = static_cast<uint32_t>(
            std::min(x->small_cols ? kSmallTileRows : kTileN, (Vm[m] + kUnit - 1) / kUnit * kUnit));
        if (!encode_bf16_2d(&x->tmA[m], x->hc[m], Bpad, Hm[m], x->a_rows) ||
            !encode_bf16_2d(&x->tmH[m], x->hc[m], Bpad, Hm[m], std::min(x->a_rows, kTileM / 2)) ||
            !encode_bf16_2d(&x->tmW[m], x->W[m], Vm[m], Hm[m], wbox) ||
            !encode_bf16_2d(&x->tmT[m], x->W[m], Vm[m], Hm[m], kUnit) ||
            !encode_bf16_2d(&x->tmP[m], x->W[m], Vm[m], Hm[m], kSmallSegRows) ||
            !encode_bf16_2d(&x->tmQ[m], x->W[m], Vm[m], Hm[m],
                            static_cast<uint32_t>(std::min(64, (Vm[m] + kUnit - 1) / kUnit * kUnit))))
            return fail(EAD_ECUDA);
    }
    // the attribute belongs to the kernel on this device, not to the context: ask for the
    // device maximum so that contexts with different stage counts can coexist
    const void *lmhead_kernels[] = {
        reinterpret_cast<const void *>(ead_lmhead_dual_kernel<false>),
        reinterpret_cast<const void *>(ead_lmhead_dual_kernel<true>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<1, false>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<2, false>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<4, false>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<8, false>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<16, false>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<1, true>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<2, true>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<4, true>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<8, true>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<16, true>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<0, false>),
        reinterpret_cast<const void *>(ead_lmhead_small_kernel<0, true>)};
    for (const void *k : lmhead_kernels) {
        cudaFuncAttributes fa;
        if (cudaFuncGetAttributes(&fa, k) != cudaSuccess) return fail(EAD_ECUDA);
        const size_t dyn_max = smem_max - fa.sharedSizeBytes;      // static shared memory counts too
        if (x->smem_bytes > dyn_max) return fail(EAD_ECUDA);
        if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(dyn_max)) !=
            cudaSuccess)
            return fail(EAD_ECUDA);
    }
    if (cudaFuncSetAttribute(ead_compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 * 4096) !=
        cudaSuccess)
        return fail(EAD_ECUDA);

    rc = ead_reset(x);
    if (rc != EAD_OK) return fail(rc);
    rc = build_graph(x, 1, &x->g_one);
    if (rc == EAD_OK) rc = build_graph(x, kGraphChunk, &x->g_chunk);
    if (rc != EAD_OK) return fail(rc);
    if (cudaStreamSynchronize(x->stream) != cudaSuccess) return fail(EAD_ECUDA);
    *out = x;
    return EAD_OK;
}

int ead_reset(ead_ctx *x)
{
    if (!x) return EAD_EINVALID_ARG;
    const ead_config &c = x->cfg;
    const int threads = 256;
    ead_reset_kernel<<<(c.B + threads - 1) / threads, threads, 0, x->stream>>>(x->ctl, x->flag, x->c, x->nfill,
                                                                              x->ring, x->usage, x->done, c.B, c.w,
                                                                              c.start_model);
    x->launches += 1;
    return cudaGetLastError() == cudaSuccess ? EAD_OK : EAD_ECUDA;
}

int ead_step(ead_ctx *x, const void *h_small, const void *h_large, int32_t *tok, float *H, float *Hbar,
             uint8_t *model_used, uint8_t *next_model)
{
    if (!x || !h_small || !h_large || !can_step(x)) return EAD_EINVALID_ARG;
    if (!aligned16(h_small) || !aligned16(h_large)) return EAD_EALIGNMENT;
    int rc = set_args(x, h_small, h_large, tok, H, Hbar, model_used, next_model, x->stream);
    if (rc != EAD_OK) return rc;
    rc = enqueue_step(x, x->stream, nullptr, step_mode(x));
    x->launches += kernels_per_step(x);
    return rc;
}

int ead_run(ead_ctx *x, int32_t T, const void *h_small_seq, const void *h_large_seq, int32_t *tok, float *H,
            float *Hbar, uint8_t *model_used, uint8_t *next_model)
{
    if (!x || T < 0 || !h_small_seq || !h_large_seq || !can_step(x)) return EAD_EINVALID_ARG;
    if (!aligned16(h_small_seq) || !aligned16(h_large_seq)) return EAD_EALIGNMENT;
    if (T == 0) return EAD_OK;
    return run_device(x, T, h_small_seq, h_large_seq, tok, H, Hbar, model_used, next_model);
}

int ead_run_timed(ead_ctx *x, int32_t T, const void *h_small_seq, const void *h_large_seq, int32_t *tok, float *H,
                  float *Hbar, uint8_t *model_used, uint8_t *next_model, float *kernel_ms)
{
    if (!x || T < 0 || !h_small_seq || !h_large_seq || !kernel_ms || x->cfg.shard_count > 0) return EAD_EINVALID_ARG;
    if (!aligned16(h_small_seq) || !aligned16(h_large_seq)) return EAD_EALIGNMENT;
    kernel_ms[0] = kernel_ms[1] = kernel_ms[2] = 0.f;
    if (T == 0) return EAD_OK;
    constexpr int kBatch = 64;                 // steps between synchronisations
    std::vector<cudaEvent_t> ev(4 * kBatch, nullptr);
    int rc = EAD_OK;
    for (auto &e : ev)
        if (cudaEventCreate(&e) != cudaSuccess) rc = EAD_ECUDA;
    if (rc == EAD_OK) rc = set_args(x, h_small_seq, h_large_seq, tok, H, Hbar, model_used, next_model, x->stream);
    double acc[3] = {0, 0, 0};
    for (int t0 = 0; t0 < T && rc == EAD_OK; t0 += kBatch) {
        const int n = std::min(kBatch, T - t0);
        for (int i = 0; i < n && rc == EAD_OK; ++i) rc = enqueue_step(x, x->stream, &ev[4 * i]);
        x->launches += 3ll * n;
        if (rc == EAD_OK && cudaStreamSynchronize(x->stream) != cudaSuccess) rc = EAD_ECUDA;
        for (int i = 0; i < n && rc == EAD_OK; ++i)
            for (int k = 0; k < 3; ++k) {
                float ms = 0.f;
                if (cudaEventElapsedTime(&ms, ev[4 * i + k], ev[4 * i + k + 1]) != cudaSuccess) rc = EAD_ECUDA;
                acc[k] += ms;
            }
    }
    for (auto &e : ev)
        if (e) cudaEventDestroy(e);
    for (int k = 0; k < 3; ++k) kernel_ms[k] = static_cast<float>(acc[k]);
    if (rc != EAD_OK) cudaGetLastError();
    return rc;
}

int ead_run_host(ead_ctx *x, int32_t T, const void *h_small_seq, const void *h_large_seq, int32_t *tok, float *H,
                 float *Hbar, uint8_t *model_used, uint8_t *next_model)
{
    if (!x || T < 0 || !h_small_seq || !h_large_seq || !can_step(x)) return EAD_EINVALID_ARG;
    if (T == 0) return EAD_OK;
    int rc = ensure_staging(x);
    if (rc != EAD_OK) return rc;
    const ead_config &c = x->cfg;
    const int S = x->st_steps;
    const OutLayout l = out_layout(S, c.B);
    const size_t row_s = static_cast<size_t>(c.B) * c.H_small * 2, row_l = static_cast<size_t>(c.B) * c.H_large * 2;
    const uint8_t *hs = static_cast<const uint8_t *>(h_small_seq), *hl = static_cast<const uint8_t *>(h_large_seq);
    // Chunks grow from 4 steps to the staging size: the first chunk's copy is the one nothing
    // can hide, so it is kept short; from then on copies run under the computation.
    int t0 = 0, ramp = 4;
    // A failed call inside the loop must not leave copies to or from the caller's buffers in
    // flight: every error path falls through to the synchronisation below.
#define EAD_TRY(x)                     \
    if (rc == EAD_OK && (x) != cudaSuccess) rc = EAD_ECUDA
    for (int k = 0; t0 < T && rc == EAD_OK; ++k) {
        const int i = k & 1;
        const int n = std::min(std::min(S, ramp), T - t0);
        ramp = std::min(S, 2 * ramp);
        const size_t cells = static_cast<size_t>(n) * c.B;
        // inputs of chunk k -> staging buffer i, once the compute that read it (chunk k-2) is done
        if (k >= 2) EAD_TRY(cudaStreamWaitEvent(x->in_stream, x->ev_comp[i], 0));
        EAD_TRY(cudaMemcpyAsync(x->st_h[i][0], hs + t0 * row_s, n * row_s, cudaMemcpyHostToDevice, x->in_stream));
        EAD_TRY(cudaMemcpyAsync(x->st_h[i][1], hl + t0 * row_l, n * row_l, cudaMemcpyHostToDevice, x->in_stream));
        EAD_TRY(cudaEventRecord(x->ev_in[i], x->in_stream));
        // compute, once the inputs are in and the previous results of buffer i have been read back
        EAD_TRY(cudaStreamWaitEvent(x->stream, x->ev_in[i], 0));
        if (k >= 2) EAD_TRY(cudaStreamWaitEvent(x->stream, x->ev_out[i], 0));
        uint8_t *o = static_cast<uint8_t *>(x->st_out[i]);
        if (rc == EAD_OK)
            rc = run_device(x, n, x->st_h[i][0], x->st_h[i][1], reinterpret_cast<int32_t *>(o + l.off_tok),
                            reinterpret_cast<float *>(o + l.off_H), reinterpret_cast<float *>(o + l.off_Hbar),
                            o + l.off_used, o + l.off_next);
        EAD_TRY(cudaEventRecord(x->ev_comp[i], x->stream));
        // results of chunk k -> host
        EAD_TRY(cudaStreamWaitEvent(x->out_stream, x->ev_comp[i], 0));
        const size_t o0 = static_cast<size_t>(t0) * c.B;
        if (tok) EAD_TRY(cudaMemcpyAsync(tok + o0, o + l.off_tok, 4 * cells, cudaMemcpyDeviceToHost, x->out_stream));
        if (H) EAD_TRY(cudaMemcpyAsync(H + o0, o + l.off_H, 4 * cells, cudaMemcpyDeviceToHost, x->out_stream));
        if (Hbar) EAD_TRY(cudaMemcpyAsync(Hbar + o0, o + l.off_Hbar, 4 * cells, cudaMemcpyDeviceToHost, x->out_stream));
        if (model_used)
            EAD_TRY(cudaMemcpyAsync(model_used + o0, o + l.off_used, cells, cudaMemcpyDeviceToHost, x->out_stream));
        if (next_model)
            EAD_TRY(cudaMemcpyAsync(next_model + o0, o + l.off_next, cells, cudaMemcpyDeviceToHost, x->out_stream));
        EAD_TRY(cudaEventRecord(x->ev_out[i], x->out_stream));
        t0 += n;
    }
#undef EAD_TRY
    // the call is synchronous, also when it fails
    const cudaError_t s_in = cudaStreamSynchronize(x->in_stream);
    const cudaError_t s_comp = cudaStreamSynchronize(x->stream);
    const cudaError_t s_out = cudaStreamSynchronize(x->out_stream);
    if (rc == EAD_OK && (s_in != cudaSuccess || s_comp != cudaSuccess || s_out != cudaSuccess)) rc = EAD_ECUDA;
    if (rc != EAD_OK) cudaGetLastError();
    return rc;
}

int ead_shard_range(int32_t V, int32_t n_shards, int32_t shard, int32_t *begin, int32_t *end)
{
    if (V < 1 || n_shards < 1 || shard < 0 || shard >= n_shards || !begin || !end) return EAD_EINVALID_ARG;
    const int64_t U = (static_cast<int64_t>(V) + kTileM - 1) / kTileM;      // whole 128-row tiles, last one ragged
    if (n_shards > U) return EAD_EINVALID_ARG;                               // some shard would be empty
    *begin = static_cast<int32_t>(U * shard / n_shards * kTileM);
    *end = static_cast<int32_t>(std::min<int64_t>(V, U * (shard + 1) / n_shards * kTileM));
    return EAD_OK;
}

size_t ead_shard_exchange_bytes(int32_t B, int32_t n_shards)
{
    if (B < 1 || n_shards < 1) return 0;
    return 2ull * n_shards * B * sizeof(ShardRecord);
}

int ead_shard_connect(ead_ctx *x, int32_t shard, void *const *exchange)
{
    if (!x || !exchange || x->cfg.shard_count < 1 || shard < 0 || shard >= x->cfg.shard_count) return EAD_EINVALID_ARG;
    ShardLink lk{};
    lk.n = x->cfg.shard_count;
    lk.self = shard;
    for (int d = 0; d < lk.n; ++d) {
        if (!exchange[d]) return EAD_EINVALID_ARG;
        if (!aligned16(exchange[d])) return EAD_EALIGNMENT;
        lk.all[d] = static_cast<ShardRecord *>(exchange[d]);
    }
    EAD_CUDA(cudaStreamSynchronize(x->stream));
    EAD_CUDA(cudaMemcpy(x->link, &lk, sizeof lk, cudaMemcpyHostToDevice));
    const int32_t zero[2] = {0, 0};                  // record numbering restarts with the fresh buffers
    EAD_CUDA(cudaMemcpy(&x->ctl->xstep, zero, sizeof zero, cudaMemcpyHostToDevice));
    x->connected = true;
    return EAD_OK;
}

int ead_shard_partials(ead_ctx *x, const void *h_small, const void *h_large, void *records)
{
    if (!x || !h_small || !h_large || x->cfg.shard_count < 1 || (!records && !x->connected)) return EAD_EINVALID_ARG;
    if (!aligned16(h_small) || !aligned16(h_large) || !aligned16(records)) return EAD_EALIGNMENT;
    int rc = set_args(x, h_small, h_large, nullptr, nullptr, nullptr, nullptr, nullptr, x->stream,
                      static_cast<float *>(records));
    if (rc != EAD_OK) return rc;
    rc = enqueue_step(x, x->stream, nullptr, records ? 1 : 3);
    x->launches += 3;
    return rc;
}

int ead_shard_gate(ead_ctx *x, const void *all_records, int32_t n_shards, int32_t *tok, float *H, float *Hbar,
                   uint8_t *model_used, uint8_t *next_model)
{
    if (!x || x->cfg.shard_count < 1 || n_shards != x->cfg.shard_count || (!all_records && !x->connected))
        return EAD_EINVALID_ARG;
    if (!aligned16(all_records)) return EAD_EALIGNMENT;
    RunArgs out{};
    out.tok = tok;
    out.H = H;
    out.Hbar = Hbar;
    out.used = model_used;
    out.next = next_model;
    const GateParams gp = gate_params(x, 0);
    ead_shard_gate_kernel<<<(x->cfg.B + 127) / 128, 128, 0, x->stream>>>(
        gp, static_cast<const ShardRecord *>(all_records), n_shards, out, all_records ? 0 : 1);
    x->launches += 1;
    return cudaGetLastError() == cudaSuccess ? EAD_OK : EAD_ECUDA;
}

int ead_status(ead_ctx *x, uint32_t *status_word)
{
    if (!x) return EAD_EINVALID_ARG;
    EAD_CUDA(cudaStreamSynchronize(x->stream));
    StepCtl h{};
    EAD_CUDA(cudaMemcpy(&h, x->ctl, sizeof h, cudaMemcpyDeviceToHost));
    if (status_word) *status_word = h.status;
    if (h.status & (kStatusWaitExpired | kStatusBadCount)) return EAD_EDEVICE_FAULT;
    return (h.status & kStatusShardMismatch) ? EAD_ESTATE : EAD_OK;
}

size_t ead_state_size(const ead_ctx *x)
{
    if (!x) return 0;
    const size_t B = x->cfg.B;
    return sizeof(StateHeader) + 2 * (B + ((4 - B % 4) % 4)) /*flag, done*/ + 4 * B /*c*/ + 4 * B /*nfill*/ + 12 * B /*usage*/ +
           4 * B * x->cfg.w;
}

int ead_get_state(ead_ctx *x, void *blob, size_t size)
{
    if (!x || !blob) return EAD_EINVALID_ARG;
    if (size != ead_state_size(x)) return EAD_ESTATE;
    EAD_CUDA(cudaStreamSynchronize(x->stream));
    const size_t B = x->cfg.B, pad = (4 - B % 4) % 4;
    uint8_t *p = static_cast<uint8_t *>(blob);
    StepCtl h{};
    EAD_CUDA(cudaMemcpy(&h, x->ctl, sizeof h, cudaMemcpyDeviceToHost));
    StateHeader hd{kStateMagic, x->cfg.B, x->cfg.w, h.step};
    memcpy(p, &hd, sizeof hd);
    p += sizeof hd;
    EAD_CUDA(cudaMemcpy(p, x->flag, B, cudaMemcpyDeviceToHost));
    memset(p + B, 0, pad);
    p += B + pad;
    EAD_CUDA(cudaMemcpy(p, x->done, B, cudaMemcpyDeviceToHost));
    memset(p + B, 0, pad);
    p += B + pad;
    EAD_CUDA(cudaMemcpy(p, x->c, 4 * B, cudaMemcpyDeviceToHost));
    p += 4 * B;
    EAD_CUDA(cudaMemcpy(p, x->nfill, 4 * B, cudaMemcpyDeviceToHost));
    p += 4 * B;
    EAD_CUDA(cudaMemcpy(p, x->usage, 12 * B, cudaMemcpyDeviceToHost));
    p += 12 * B;
    EAD_CUDA(cudaMemcpy(p, x->ring, 4 * B * x->cfg.w, cudaMemcpyDeviceToHost));
    return EAD_OK;
}

int ead_set_state(ead_ctx *x, const void *blob, size_t size)
{
    if (!x || !blob) return EAD_EINVALID_ARG;
    if (size != ead_state_size(x)) return EAD_ESTATE;
    const uint8_t *p = static_cast<const uint8_t *>(blob);
    StateHeader hd;
    memcpy(&hd, p, sizeof hd);
    if (hd.magic != kStateMagic || hd.B != x->cfg.B || hd.w != x->cfg.w || hd.step < 0) return EAD_ESTATE;
    EAD_CUDA(cudaStreamSynchronize(x->stream));
    const size_t B = x->cfg.B, pad = (4 - B % 4) % 4;
    p += sizeof hd;
    for (size_t i = 0; i < B; ++i)
        if (p[i] > 1 || p[B + pad + i] > 1) return EAD_ESTATE;
    {
        // dwell counters and window fill counts index device arrays: a negative one is not a state
        const uint8_t *q = p + 2 * (B + pad);
        for (size_t i = 0; i < 2 * B; ++i) {
            int32_t v;
            memcpy(&v, q + 4 * i, 4);
            if (v < 0) return EAD_ESTATE;
        }
    }
    EAD_CUDA(cudaMemcpy(&x->ctl->step, &hd.step, 4, cudaMemcpyHostToDevice));
    EAD_CUDA(cudaMemcpy(x->flag, p, B, cudaMemcpyHostToDevice));
    p += B + pad;
    EAD_CUDA(cudaMemcpy(x->done, p, B, cudaMemcpyHostToDevice));
    p += B + pad;
    EAD_CUDA(cudaMemcpy(x->c, p, 4 * B, cudaMemcpyHostToDevice));
    p += 4 * B;
    EAD_CUDA(cudaMemcpy(x->nfill, p, 4 * B, cudaMemcpyHostToDevice));
    p += 4 * B;
    EAD_CUDA(cudaMemcpy(x->usage, p, 12 * B, cudaMemcpyHostToDevice));
    p += 12 * B;
    EAD_CUDA(cudaMemcpy(x->ring, p, 4 * B * x->cfg.w, cudaMemcpyHostToDevice));
    return EAD_OK;
}

int ead_usage(ead_ctx *x, uint64_t *counts, uint32_t *per_row)
{
    if (!x || !counts) return EAD_EINVALID_ARG;
    EAD_CUDA(cudaStreamSynchronize(x->stream));
    const size_t B = x->cfg.B;
    std::vector<uint32_t> h(3 * B);
    EAD_CUDA(cudaMemcpy(h.data(), x->usage, 12 * B, cudaMemcpyDeviceToHost));
    for (int k = 0; k < 3; ++k) {
        uint64_t s = 0;
        for (size_t b = 0; b < B; ++b) s += h[k * B + b];
        counts[k] = s;
    }
    if (per_row) memcpy(per_row, h.data(), 12 * B);
    return EAD_OK;
}

double ead_parameter_ratio(uint64_t tokens_small, uint64_t tokens_large, double P_small, double P_large)
{
    const double total = static_cast<double>(tokens_small) + static_cast<double>(tokens_large);
    const double alpha = static_cast<double>(tokens_small) / total, beta = static_cast<double>(tokens_large) / total;
    return (alpha * P_small + beta * P_large) / P_large;
}

int ead_set_done(ead_ctx *x, const uint8_t *done)
{
    if (!x || !done) return EAD_EINVALID_ARG;
    for (int b = 0; b < x->cfg.B; ++b)
        if (done[b] > 1) return EAD_EINVALID_ARG;
    EAD_CUDA(cudaStreamSynchronize(x->stream));
    EAD_CUDA(cudaMemcpy(x->done, done, x->cfg.B, cudaMemcpyHostToDevice));
    return EAD_OK;
}

int ead_get_done(ead_ctx *x, uint8_t *done)
{
    if (!x || !done) return EAD_EINVALID_ARG;
    EAD_CUDA(cudaStreamSynchronize(x->stream));
    EAD_CUDA(cudaMemcpy(done, x->done, x->cfg.B, cudaMemcpyDeviceToHost));
    return EAD_OK;
}

int64_t ead_kernel_launches(const ead_ctx *x) { return x ? x->launches : 0; }

int ead_launch_info(const ead_ctx *x, int32_t *info, int32_t n)
{
    if (!x || !info || n < 0) return EAD_EINVALID_ARG;
    const int32_t v[4] = {x->G, x->stages, x->a_rows, static_cast<int32_t>(x->smem_bytes)};
    for (int i = 0; i < n && i < 4; ++i) info[i] = v[i];
    return EAD_OK;
}

int ead_plan_split(int32_t cta, int32_t G, int32_t n_rows, int32_t V, int32_t *out)
{
    if (!out || cta < 0 || G < 1 || cta >= G || n_rows < 0 || V < 1) return EAD_EINVALID_ARG;
    if ((n_rows + kTileM - 1) / kTileM > G) return EAD_EINVALID_ARG;   // more row blocks than CTAs
    const HeadSplit s = split_head(cta, G, n_rows, V);
    out[0] = s.active;
    out[1] = s.rb;
    out[2] = s.slot;
    out[3] = s.col_begin;
    out[4] = s.col_end;
    out[5] = s.g;
    return EAD_OK;
}

int ead_plan_units(int32_t cta, int32_t G, int32_t n_rows, int32_t V, int32_t two_blocks, int32_t *out)
{
    if (!out || cta < 0 || G < 1 || cta >= G || n_rows < 0 || V < 1) return EAD_EINVALID_ARG;
    if ((n_rows + kTileM - 1) / kTileM > G) return EAD_EINVALID_ARG;   // more row blocks than CTAs
    const UnitSplit s = split_units(cta, G, n_rows, V, two_blocks ? 1 : 0);
    out[0] = s.active;
    out[1] = s.dual;
    out[2] = s.rb;
    out[3] = s.slot;
    out[4] = s.g;
    out[5] = s.rounds;
    out[6] = s.tail_col0;
    out[7] = s.tail_cols;
    out[8] = s.thin16;
    out[9] = s.tile_n;
    out[10] = s.n_hi;
    out[11] = s.w_hi;
    out[12] = s.w_lo;
    return EAD_OK;
}

void ead_destroy(ead_ctx *x)
{
    if (!x) return;
    cudaSetDevice(x->cfg.device);
    cudaStreamSynchronize(x->stream);
    if (x->in_stream) cudaStreamSynchronize(x->in_stream);
    if (x->out_stream) cudaStreamSynchronize(x->out_stream);
    free_staging(x);
    if (x->g_one) cudaGraphExecDestroy(x->g_one);
    if (x->g_chunk) cudaGraphExecDestroy(x->g_chunk);
    if (x->cap_stream) cudaStreamDestroy(x->cap_stream);
    void *bufs[] = {x->ctl, x->args, x->flag, x->c, x->nfill, x->perm, x->ring, x->hc[0], x->hc[1],
                    x->part_m, x->part_s, x->part_t, x->part_i, x->usage, x->part_k, x->part_ki, x->done, x->link};
    for (void *b : bufs)
        if (b) cudaFree(b);
    cudaGetLastError();
    delete x;
}

}  // extern "C"

// =====================================================================================
// Allocation-free entry point.  Everything below is independent of ead_ctx: its scratch
// is the file-scope device array g_static_scratch, shared by all calls on a device.
// =====================================================================================
namespace {

constexpr int kStaticSlots = 160;          // partial slots per row (>= CTAs launched)
constexpr int kStaticMaxDevices = 64;

// Layout of the built-in scratch array.
struct StaticScratch {
    StepCtl ctl;
    unsigned char pad[256 - sizeof(StepCtl)];
    float part_m[EAD_STATIC_MAX_B * kStaticSlots];
    float part_s[EAD_STATIC_MAX_B * kStaticSlots];
    float part_t[EAD_STATIC_MAX_B * kStaticSlots];
    int32_t part_i[EAD_STATIC_MAX_B * kStaticSlots];
    uint16_t hidden[EAD_STATIC_MAX_B * EAD_STATIC_MAX_H];   // padded copy of the hidden rows
};

// In host code this name is only a handle for cudaGetSymbolAddress, not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

struct StaticDevice {
    bool ready = false;
    StaticScratch *scratch = nullptr;      // device address of g_static_scratch on this device
    int sms = 0;
    int smem_optin = 0;
};
StaticDevice g_static_dev[kStaticMaxDevices];
std::mutex g_static_mu;

// Copies the caller's rows into the padded operand (rows B .. a_rows-1 are cleared, so the
// TMA box never reads what an earlier call left there) and writes the control block.
__global__ void ead_static_stage_kernel(StaticScratch *sc, const uint16_t *h, int B, int H, int a_rows)
{
    const int row = blockIdx.x;
    if (row == 0 && threadIdx.x == 0) {
        sc->ctl.step = 0;
        sc->ctl.cur_t = 0;
        sc->ctl.n[0] = B;
        sc->ctl.n[1] = 0;
        sc->ctl.status = 0;
    }
    if (row >= a_rows) return;
    uint4 *dst = reinterpret_cast<uint4 *>(sc->hidden + static_cast<size_t>(row) * H);
    if (row < B) {
        const uint4 *src = reinterpret_cast<const uint4 *>(h + static_cast<size_t>(row) * H);
        for (int k = threadIdx.x; k < H / 8; k += blockDim.x) dst[k] = __ldg(src + k);
    } else {
        for (int k = threadIdx.x; k < H / 8; k += blockDim.x) dst[k] = make_uint4(0, 0, 0, 0);
    }
}

// One warp per row: merge the G per-CTA partials in fixed order, then Eq. 2 in the fused
// form and the arg max.
__global__ void __launch_bounds__(kGateThreads)
ead_static_merge_kernel(const StaticScratch *sc, int B, int G, int32_t *tok, float *H_out, uint32_t *status)
{
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (kGateThreads / 32) + (threadIdx.x >> 5);
    if (r >= B) return;
    const size_t base = static_cast<size_t>(r) * kStaticSlots;
    Partial acc{kNegSentinel, 0.f, 0.f, 0x7fffffff};
    for (int s = lane; s < G; s += 32) {
        const Partial q{sc->part_m[base + s], sc->part_s[base + s], sc->part_t[base + s], sc->part_i[base + s]};
        acc = merge_partial(acc, q);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Partial q;
        q.m = __shfl_xor_sync(0xffffffffu, acc.m, o);
        q.s = __shfl_xor_sync(0xffffffffu, acc.s, o);
        q.t = __shfl_xor_sync(0xffffffffu, acc.t, o);
        q.idx = __shfl_xor_sync(0xffffffffu, acc.idx, o);
        acc = merge_partial(acc, q);
    }
    if (lane != 0) return;
    float H = logf(acc.s) - acc.t / (acc.s * kLog2e);
    const bool finite = isfinite(H) && acc.s > 0.f;
    if (H < 0.f) H = 0.f;
    uint32_t st = sc->ctl.status;
    if (!finite) st |= kStatusNonFinite;
    if (tok) tok[r] = finite ? acc.idx : -1;
    if (H_out) H_out[r] = finite ? H : __int_as_float(0x7fc00000);
    if (status && st) atomicOr(status, st);
}

__global__ void ead_static_clear_status_kernel(uint32_t *status)
{
    if (status) *status = 0;
}

// Once per device, with that device current: device address of the array, device limits.
int static_device_setup(int device, StaticDevice **out)
{
    if (device < 0 || device >= kStaticMaxDevices) return EAD_EINVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mu);
    StaticDevice &d = g_static_dev[device];
    if (!d.ready) {
        int major = 0;
        EAD_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
        if (major != 10) return EAD_EUNSUPPORTED_ARCH;
        void *ptr = nullptr;
        EAD_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr) return EAD_ECUDA;
        EAD_CUDA(cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, device));
        EAD_CUDA(cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device));
        EAD_CUDA(cudaFuncSetAttribute(ead_lmhead_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, d.smem_optin));
        d.scratch = static_cast<StaticScratch *>(ptr);
        d.ready = true;
    }
    *out = &d;
    return EAD_OK;
}

}  // namespace

extern "C" int ead_head_entropy_static(const void *W, const void *h, int32_t B, int32_t V, int32_t H, int32_t *tok,
                                       float *H_out, uint32_t *status, int32_t device, void *stream)
{
    if (!W || !h || B < 1 || V < 1 || H < 8) return EAD_EINVALID_ARG;
    if (B > EAD_STATIC_MAX_B || H > EAD_STATIC_MAX_H) return EAD_ELIMIT;
    if (H % 8 || !aligned16(W) || !aligned16(h)) return EAD_EALIGNMENT;
    int ndev = 0;
    EAD_CUDA(cudaGetDeviceCount(&ndev));
    if (device < 0 || device >= ndev) return EAD_EINVALID_ARG;
    EAD_CUDA(cudaSetDevice(device));
    StaticDevice *d = nullptr;
    int rc = static_device_setup(device, &d);
    if (rc != EAD_OK) return rc;
    StaticScratch *sc = d->scratch;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    const int G = std::min(d->sms, kStaticSlots);
    const int a_rows = std::min(kTileM, (B + 7) & ~7);
    const size_t stage_bytes = static_cast<size_t>(a_rows) * kBlockK * 2 + kWTileBytes;
    const int stages = static_cast<int>(
        std::min<size_t>(kMaxStages, (static_cast<size_t>(d->smem_optin) - kSmemCtrlBytes - 1024) / stage_bytes));
    if (stages < 2) return EAD_ECUDA;
    const size_t smem_bytes = kSmemCtrlBytes + 1024 + stages * stage_bytes;

    // TMA descriptors are built on the host and travel as kernel arguments: no device memory.
    CUtensorMap tmA, tmW, tmT;
    const uint32_t wbox = static_cast<uint32_t>(std::min(kTileN, (V + kUnit - 1) / kUnit * kUnit));
    if (!encode_bf16_2d(&tmA, sc->hidden, kTileM, H, a_rows) || !encode_bf16_2d(&tmW, W, V, H, wbox) ||
        !encode_bf16_2d(&tmT, W, V, H, kUnit))
        return EAD_ECUDA;

    ead_static_clear_status_kernel<<<1, 1, 0, s>>>(status);
    ead_static_stage_kernel<<<a_rows, 128, 0, s>>>(sc, static_cast<const uint16_t *>(h), B, H, a_rows);
    LmheadParams lp{};
    lp.V[0] = V;
    lp.V[1] = V;
    lp.H[0] = H;
    lp.H[1] = H;
    lp.a_rows = a_rows;
    lp.stages = stages;
    lp.slots_stride = kStaticSlots;
    lp.B = EAD_STATIC_MAX_B;
    lp.ctl = &sc->ctl;
    lp.ctl_rw = &sc->ctl;
    lp.part_m = sc->part_m;
    lp.part_s = sc->part_s;
    lp.part_t = sc->part_t;
    lp.part_i = sc->part_i;
    ead_lmhead_kernel<false><<<G, kLmheadThreads, smem_bytes, s>>>(tmA, tmA, tmW, tmW, tmT, tmT, tmA, tmA, lp);
    const int rows_per_block = kGateThreads / 32;
    ead_static_merge_kernel<<<(B + rows_per_block - 1) / rows_per_block, kGateThreads, 0, s>>>(sc, B, G, tok, H_out,
                                                                                             status);
    return cudaGetLastError() == cudaSuccess ? EAD_OK : EAD_ECUDA;
}
