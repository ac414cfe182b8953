/*
 * ead.h - C ABI of the B200 (sm_100a) library for the gate step of Entropy
 * Adaptive Decoding (EAD).
 *
 * One "gate step" is one pass through the loop body of the paper's
 * Algorithm 1 for a batch of B independent sequences: project the active
 * model's final hidden state through that model's LM head (the last stage of
 * "l <- M_t(x + y)"), take the softmax of the raw logits (Eq. 1) and its
 * Shannon entropy (Eq. 2), pick the greedy token (the temperature -> 0 limit
 * of the sampling lines), append the entropy to the sequence's window and
 * average the last w entries (Eq. 3 / "mean(W[-w:])"), count the token
 * (c <- c + 1) and apply the dwell + threshold rule (Eq. 4) that selects the
 * model for the next token.
 *
 * Conventions
 *   - Every function returns 0 (EAD_OK) or a negative EAD_E* code; nothing
 *     throws or aborts across this boundary.  ead_strerror names a code.
 *   - Pointers marked "dev" are device pointers on cfg.device, "host" are
 *     host pointers.  Weights, hidden states and outputs are BORROWED: the
 *     library never copies or frees them; they must stay valid until the work
 *     enqueued with them has finished.  All per-sequence state (window,
 *     dwell counter, model flag) is OWNED by the context.
 *   - bf16 matrices are row major; their base must be 16-byte aligned and
 *     H_small, H_large must be multiples of 8 (16-byte rows).
 *   - Work is enqueued on cfg.stream and is asynchronous with respect to the
 *     host unless stated otherwise.  Calls on one context must not overlap on
 *     the device (one stream); the context is not thread safe.
 *   - The library needs an sm_100 device and has no other code path:
 *     ead_create fails with EAD_EUNSUPPORTED_ARCH elsewhere.
 *   - Models are numbered 0 = small (M_S), 1 = large (M_L).
 */
#ifndef EAD_H_
#define EAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define EAD_OK                  0
#define EAD_EINVALID_ARG      (-1)  /* NULL where not allowed, size out of range            */
#define EAD_EALIGNMENT        (-2)  /* pointer not 16-byte aligned or H not a multiple of 8 */
#define EAD_ECUDA             (-3)  /* a CUDA runtime / driver call failed                  */
#define EAD_EUNSUPPORTED_ARCH (-4)  /* device is not sm_100                                 */
#define EAD_EDEVICE_FAULT     (-5)  /* the device status word reports a kernel-side error   */
#define EAD_ESTATE            (-6)  /* state blob of the wrong size or version              */
#define EAD_ELIMIT            (-7)  /* size beyond a fixed built-in limit (see EAD_STATIC_*)  */

/* Bits of the device status word (ead_status). */
#define EAD_STATUS_NONFINITE   0x1u /* some row saw a NaN / infinite logit (row gets H = NaN) */
#define EAD_STATUS_WAIT_EXPIRED 0x2u /* a bounded wait inside a kernel ran out                 */
#define EAD_STATUS_BAD_COUNT   0x4u /* internal row counts inconsistent                       */
#define EAD_STATUS_SHARD_MISMATCH 0x8u /* vocabulary shards disagree on the step or on a row's model */

typedef struct ead_ctx ead_ctx; /* opaque */

/* Hyper-parameters follow the "Require" line of Algorithm 1 (tau, w, d_min);
 * the paper's experiments use w = 5 and d_min = 10. */
typedef struct ead_config {
    int32_t B;           /* sequences in the batch, 1 .. 4096                                 */
    int32_t V;           /* vocabulary size shared by both heads, >= 1                        */
    int32_t H_small;     /* hidden size of M_S, multiple of 8, >= 8                           */
    int32_t H_large;     /* hidden size of M_L, multiple of 8, >= 8                           */
    int32_t w;           /* window length of Eq. 3, 1 .. 64                                   */
    int32_t d_min;       /* minimum tokens on a model before a switch (Eq. 4); <= 1 = none    */
    float   tau;         /* threshold of Eq. 4, compared with the rolling mean in `unit`      */
    int32_t unit;        /* 0: entropy in nats; 1: in bits (Eq. 2 as printed, log base 2)     */
    int32_t start_model; /* model of the first token; Algorithm 1 starts on 0 (small)         */
    int32_t device;      /* CUDA device ordinal                                               */
    void   *stream;      /* cudaStream_t to enqueue on (borrowed); NULL = legacy default      */
    float   temperature; /* T of Algorithm 1's sampling lines; 0 = greedy (arg max)           */
    uint64_t seed;       /* seed of the sampling random stream (used when temperature > 0)    */
    int32_t eos_token;   /* token that ends a sequence ("while not done"); < 0 = none         */
    int32_t V_large;     /* vocabulary of M_L if it differs from V (the paper allows models of
                            different architectures); 0 = same as V.  Tokens of a step are
                            indices into the vocabulary of the model that produced them      */
    int32_t shard_count; /* 0: this context holds the whole heads.  n >= 1: it holds one of n
                            vocabulary slices (see ead_shard_connect); V and V_large are then the
                            rows of its slices                                                   */
    int32_t vocab_offset_small; /* sharded: row of the full small head at which this slice starts,
                                   a multiple of 16; tokens are reported in full-head indices   */
    int32_t vocab_offset_large; /* the same for the large head                                  */
} ead_config;

/*
 * Creates a context: allocates the per-sequence state of Algorithm 1's
 * initialisation (empty window, c = 0, M_t = start_model) plus scratch, and
 * encodes the TMA descriptors of the two heads.
 *   W_small  dev, bf16 [V, H_small], one row per vocabulary entry (borrowed, read only)
 *   W_large  dev, bf16 [V_large or V, H_large]
 *   out      host, receives the context
 * Synchronises the device once.  Errors: EAD_EINVALID_ARG, EAD_EALIGNMENT,
 * EAD_EUNSUPPORTED_ARCH, EAD_ECUDA.
 */
int ead_create(const ead_config *cfg, const void *W_small, const void *W_large, ead_ctx **out);

/*
 * One gate step (one iteration of Algorithm 1's loop) for all B sequences.
 *   h_small     dev, bf16 [B, H_small]: final hidden state of M_S per sequence
 *   h_large     dev, bf16 [B, H_large]: the same for M_L
 *               Only the row of the model that is active for a sequence is read.
 *   tok         dev, int32 [B]: next token: with cfg.temperature = 0 the arg max (lowest index
 *               among equal maxima); with cfg.temperature = T > 0 a draw from softmax(l / T),
 *               realised as arg max of l_i / T + g_i with standard Gumbel g_i = -ln(-ln u_i),
 *               u_i = (2k + 1) / 2^24, k = top 23 bits of word (i mod 4) of
 *               Philox4x32-10(counter = {i / 4, step, row, 0}, key = seed), step = number of
 *               gate steps of the context since the last reset.  -1 for a row with
 *               non-finite logits
 *   H           dev, float [B]: entropy of Eq. 2 in cfg.unit
 *   Hbar        dev, float [B]: rolling mean of Eq. 3 after this token
 *   model_used  dev, uint8 [B]: model that produced this token
 *   next_model  dev, uint8 [B]: model selected for the next token (Eq. 4)
 * Any output pointer may be NULL to skip it.  Row b of every output belongs to
 * row b of the inputs.  Asynchronous.  Errors: EAD_EINVALID_ARG,
 * EAD_EALIGNMENT, EAD_ECUDA.
 */
int ead_step(ead_ctx *ctx, const void *h_small, const void *h_large, int32_t *tok, float *H,
             float *Hbar, uint8_t *model_used, uint8_t *next_model);

/*
 * T consecutive gate steps with the hidden states of all steps resident on
 * the device; step t reads h_*_seq[t] and writes row t of each output.  The
 * T-step loop is replayed from CUDA graphs; the result is bit-identical to T
 * calls of ead_step.  Continues from the context's current state.
 *   h_small_seq  dev, bf16 [T, B, H_small];  h_large_seq  dev, bf16 [T, B, H_large]
 *   outputs      dev, [T, B] each, as in ead_step; any may be NULL
 * Asynchronous.  Errors as ead_step.
 */
int ead_run(ead_ctx *ctx, int32_t T, const void *h_small_seq, const void *h_large_seq,
            int32_t *tok, float *H, float *Hbar, uint8_t *model_used, uint8_t *next_model);

/*
 * The same T steps as ead_run, but every buffer is a HOST pointer: hidden
 * states are copied to the device and results back through internal staging
 * buffers, in chunks that overlap with the computation.  Synchronous: returns
 * when the outputs are complete, and also when it fails: before an error is
 * returned every copy already enqueued to or from the caller's buffers has ended.
 * Any output may be NULL.  Pinned host memory makes the copies faster but is not required.
 */
int ead_run_host(ead_ctx *ctx, int32_t T, const void *h_small_seq, const void *h_large_seq,
                 int32_t *tok, float *H, float *Hbar, uint8_t *model_used, uint8_t *next_model);

/*
 * DIAGNOSTIC (measurement aid, not part of the gate step's interface; so are
 * ead_kernel_launches, ead_launch_info, ead_plan_split and ead_plan_units below).
 * The same T steps as ead_run, launched kernel by kernel (no graph replay) with
 * CUDA events around every kernel on cfg.stream, to attribute device time.
 *   kernel_ms  host, float [3]: summed device time in milliseconds of the
 *              compaction, LM-head and merge+gate kernels over the T steps
 * Synchronous (waits for the stream).  Results are identical to ead_run; the
 * event records make it slower, so it is a measurement aid, not the fast path.
 */
int ead_run_timed(ead_ctx *ctx, int32_t T, const void *h_small_seq, const void *h_large_seq,
                  int32_t *tok, float *H, float *Hbar, uint8_t *model_used, uint8_t *next_model,
                  float *kernel_ms);

/* Back to Algorithm 1's initial state (empty window, c = 0, start model) and a
 * cleared status word.  Asynchronous. */
int ead_reset(ead_ctx *ctx);

/* Waits for the context's stream, then reports the device status word
 * (EAD_STATUS_* bits, sticky until ead_reset).  Returns EAD_EDEVICE_FAULT if
 * EAD_STATUS_WAIT_EXPIRED or EAD_STATUS_BAD_COUNT is set, EAD_ESTATE if
 * EAD_STATUS_SHARD_MISMATCH is set, else EAD_OK. */
int ead_status(ead_ctx *ctx, uint32_t *status_word);

/*
 * Checkpoint of the per-sequence state (window contents, dwell counters, model
 * flags, number of steps taken).  ead_state_size gives the blob size for this
 * context; ead_get_state copies device -> host, ead_set_state host -> device.
 * Both wait for the stream.  A blob is only valid for a context with the same
 * B and w; ead_set_state also rejects (EAD_ESTATE, nothing copied) a blob whose flags are
 * not 0 / 1 or whose dwell counters or window fill counts are negative.
 * Errors: EAD_EINVALID_ARG, EAD_ESTATE, EAD_ECUDA.
 */
size_t ead_state_size(const ead_ctx *ctx);
int ead_get_state(ead_ctx *ctx, void *host_blob, size_t size);
int ead_set_state(ead_ctx *ctx, const void *host_blob, size_t size);

/*
 * Done mask ("while not done" of Algorithm 1).  A sequence becomes done when it produces
 * cfg.eos_token, or when the caller marks it here.  From the next step on a done row takes no
 * part: no logits are computed for it, its outputs are token -1, NaN entropies and its
 * unchanged model in model_used / next_model, and its window, counters and model stay frozen.
 * ead_reset clears the mask.  Both calls wait for the stream.
 *   done  host, uint8 [B], each 0 or 1
 * Errors: EAD_EINVALID_ARG, EAD_ECUDA.
 */
int ead_set_done(ead_ctx *ctx, const uint8_t *done);
int ead_get_done(ead_ctx *ctx, uint8_t *done);

/*
 * Usage accounting since the last ead_reset (the paper's "large model usage" column and the
 * count of model switches), summed over the B sequences.  Rows with non-finite logits in a
 * step are not counted for that step.  Waits for the stream.
 *   counts  host, uint64 [3]: {tokens produced by M_S, tokens produced by M_L, switches}
 *   per_row host, uint32 [3 * B] or NULL: the same three counters per sequence, row major [3][B]
 * Errors: EAD_EINVALID_ARG, EAD_ECUDA.
 */
int ead_usage(ead_ctx *ctx, uint64_t *counts, uint32_t *per_row);

/*
 * The footnote of the paper's Table 1: average parameters per forward pass relative to the
 * large model, (alpha P_S + beta P_L) / P_L, with alpha = tokens_small / total and
 * beta = tokens_large / total.  Pure host arithmetic; returns NaN if both counts are 0.
 */
double ead_parameter_ratio(uint64_t tokens_small, uint64_t tokens_large, double P_small, double P_large);

/* DIAGNOSTIC.  Number of kernels the library has launched through this context so far
 * (graph replays count their kernel nodes). */
int64_t ead_kernel_launches(const ead_ctx *ctx);

/* DIAGNOSTIC.  Launch geometry chosen at creation, for reporting: fills up to n ints with
 * {CTAs of the LM-head kernel, pipeline stages, rows of the hidden-state TMA
 * box, dynamic shared memory bytes}.  For B > 128 the stage count is that of a single-block unit
 * (48 KiB stages); the kernel cuts the same ring into 64 or 72 KiB stages for units of two blocks
 * and into 40 KiB ones for a head of at most 64 rows. */
int ead_launch_info(const ead_ctx *ctx, int32_t *info, int32_t n);

/*
 * Vocabulary-sharded gate step (several GPUs, one sequence batch).  The softmax of Eq. 1 and
 * the entropy of Eq. 2 are sums over the vocabulary and the greedy / sampled token is a maximum
 * over it, so the vocabulary rows of both heads can be split over n GPUs: each computes the
 * statistics of its slice, the slices' statistics are exchanged (n x B records of 32 bytes:
 * the only traffic between the GPUs), and every GPU merges all of them in shard order and runs
 * the window / dwell / threshold part of Algorithm 1 itself.  All GPUs then hold identical
 * per-sequence state and identical outputs, bit for bit, without further communication.  The
 * paper describes one device; this split is the build's own.
 *
 * Each GPU creates a context with cfg.shard_count = n (<= 16), cfg.V / cfg.V_large = rows of its
 * slices, cfg.vocab_offset_* = where they start, and the slice pointers as W_small / W_large;
 * all other fields equal on all GPUs.  Every GPU gets the full hidden rows at every step.
 *
 * ead_shard_range: the slice [*begin, *end) of a head of V rows that shard `shard` of n_shards
 * takes when the rows are dealt out in whole tiles of 128 (host arithmetic, needs no GPU).
 * Errors: EAD_EINVALID_ARG (also when n_shards exceeds the number of tiles).
 *
 * The exchange can run in two ways.
 *
 * (1) Inside the kernels, over peer memory.  Every shard owns an exchange buffer of
 * ead_shard_exchange_bytes(B, n) bytes, zero-filled, 16-byte aligned, mapped into the address
 * space of every other shard's GPU (peer access, an IPC handle, symmetric memory).
 *     ead_shard_connect(ctx, shard, exchange)   exchange: host array [n]; entry d = shard d's
 *                                               buffer as addressable from this GPU (entry
 *                                               `shard` is this context's own, local buffer)
 * From then on ead_step / ead_run / ead_run_host work as on one GPU, called on every shard with
 * the same hidden states: after its cross-CTA merge each shard stores its B records straight
 * into all n exchange buffers (plain stores; the record's step word last, with release
 * semantics at system scope), and the thread that stored a row's record then waits until that
 * row's records of all n shards for this step have arrived in the local buffer and finishes
 * the row: a sharded step is the same three kernels as an unsharded one.  Buffers alternate with
 * the parity of the step, which suffices because a shard cannot run more than one step ahead
 * of another.  The wait is bounded (2 s): a shard that never delivers sets
 * EAD_STATUS_WAIT_EXPIRED, the rows are reported like non-finite rows, and later steps do not
 * wait again.  Waits for the stream; restarts the numbering of exchanged records, so all shards
 * connect (to zero-filled buffers) at the same point of their runs.  ead_reset, ead_set_state
 * and ead_set_done must be applied on all shards alike.
 * Errors: EAD_EINVALID_ARG, EAD_EALIGNMENT, EAD_ECUDA.  Before ead_shard_connect the stepping
 * calls return EAD_EINVALID_ARG on a sharded context; ead_run_timed always does.
 *
 * (2) By the caller, between two library calls (NCCL or any other all-gather that is ordered
 * on the context's stream); no peer mapping needed:
 *     ead_shard_partials(ctx, h_small, h_large, records);      // this GPU's [B] records
 *     <all-gather the n record arrays, in shard order, into all_records on every GPU>
 *     ead_shard_gate(ctx, all_records, n, tok, H, Hbar, model_used, next_model);
 *   records      dev, [B] x EAD_SHARD_RECORD_BYTES, 16-byte aligned: per sequence (caller's row
 *                order) {float m, s, t; int32 idx; float k; int32 ki; int32 model; int32 step1}:
 *                max, sum exp(z - m), sum exp(z - m)(z - m) log2 e and arg max of the slice's
 *                logits, the sampling candidate, the head they belong to, and 1 + the number
 *                of sharded steps this context has taken.  Rows of ended sequences are not
 *                written.
 *   all_records  dev, [n_shards][B] records, shard s at index s
 *   outputs      as in ead_step
 * Both calls are asynchronous on the context's stream.  On a connected context `records` and
 * `all_records` may be NULL: the two halves of a step of way (1), called apart.
 *
 * In both ways a record whose model or step number differs from this context's sets
 * EAD_STATUS_SHARD_MISMATCH and leaves the row's state untouched (outputs as for a non-finite
 * row).  Errors of (2): EAD_EINVALID_ARG (also: context not created with shard_count >= 1, or
 * n_shards not equal to it), EAD_EALIGNMENT, EAD_ECUDA.
 */
#define EAD_SHARD_RECORD_BYTES 32
#define EAD_SHARD_MAX 16
int ead_shard_range(int32_t V, int32_t n_shards, int32_t shard, int32_t *begin, int32_t *end);
size_t ead_shard_exchange_bytes(int32_t B, int32_t n_shards);
int ead_shard_connect(ead_ctx *ctx, int32_t shard, void *const *exchange);
int ead_shard_partials(ead_ctx *ctx, const void *h_small, const void *h_large, void *records);
int ead_shard_gate(ead_ctx *ctx, const void *all_records, int32_t n_shards, int32_t *tok, float *H,
                   float *Hbar, uint8_t *model_used, uint8_t *next_model);

/*
 * DIAGNOSTIC.  How the one-block LM-head kernel (the one behind ead_head_entropy_static) divides
 * one head among its CTAs (host-side replica of the rule
 * the kernel applies on the device; pure arithmetic, needs no GPU).  With n rows on a head
 * there are R = ceil(n / 128) row blocks; CTA `cta` of `G` serves row block out[1] and
 * vocabulary columns [out[3], out[4]) (multiples of 16; the end may exceed V by < 16).
 *   out  host, int32 [6]: {active, row_block, slot, col_begin, col_end, group_size}
 * Errors: EAD_EINVALID_ARG.
 */
int ead_plan_split(int32_t cta, int32_t G, int32_t n_rows, int32_t V, int32_t *out);

/*
 * DIAGNOSTIC.  The same for the kernel that serves B > 128, whose CTAs work in UNITS of row blocks
 * (host-side replica of the device rule; needs no GPU).  With two_blocks != 0 (heads with a hidden
 * size of 3072 and more) a unit is two consecutive 128-row blocks against one weight tile.  An odd
 * last block is a unit of its own.  A head of exactly three row blocks is different: if its last
 * block has at most 64 rows, the two-block unit takes it along as a thin third block (thin16 =
 * its rows rounded up to 16) and works on tiles of tile_n = 256 - thin16 columns; otherwise it is
 * served one block per unit, as is every head with two_blocks == 0.  Units get CTAs in
 * proportion to their cost (two blocks : one = 9 : 5); member `slot` of a unit's `group` CTAs takes
 * tile slot of every whole round k < rounds, then its piece [tail_col0, tail_col0 + tail_cols) of
 * what the whole rounds leave over (cut evenly in 16-column units; tail_cols may be 0).  The
 * tiles of the first n_hi rounds are w_hi columns wide, those of the other rounds w_lo (round k
 * begins where round k - 1 ends: at group * (min(k, n_hi) * w_hi + max(0, k - n_hi) * w_lo)).  With
 * more than eight whole rounds of full tiles, no rest, or single-block units on a head of at most
 * two row blocks, all are tile_n wide; otherwise a member's share is cut into pieces of nearly
 * equal width.
 *   out  host, int32 [13]: {active, two_blocks, first_row_block, slot, group, rounds, tail_col0,
 *                           tail_cols, thin16, tile_n, n_hi, w_hi, w_lo}
 * Errors: EAD_EINVALID_ARG (also: more row blocks than CTAs).
 */
int ead_plan_units(int32_t cta, int32_t G, int32_t n_rows, int32_t V, int32_t two_blocks, int32_t *out);

/* Waits for outstanding work and frees everything the context owns.  NULL is allowed. */
void ead_destroy(ead_ctx *ctx);

/*
 * Entropy and greedy token of one LM head for a dense batch, WITHOUT any allocation.
 * (The paper has no counterpart: this is a service entry point of the library; what it
 * computes per row is Eq. 1-2 and the arg max, exactly as one ead_step does for rows
 * that are on that head.)
 *
 * For callers that are not allowed to allocate device memory: code that runs while the
 * framework's allocator is frozen (inside a memory-planned inference engine, under a
 * fixed memory budget that has already been handed out, or in a latency-critical section
 * where cudaMalloc's implicit device synchronisation is unacceptable).  ead_create and
 * ead_run_host call cudaMalloc; this function calls neither cudaMalloc nor cudaFree nor
 * any allocating library routine.  Its scratch memory (per-CTA partial statistics, a
 * padded copy of the hidden rows, a control block) lives in one array compiled into the
 * library, about 2.4 MB, which every GPU that loads the library holds until the process
 * exits.  That fixes the limits:
 *     B <= EAD_STATIC_MAX_B (128),  H <= EAD_STATIC_MAX_H (8192),  H a multiple of 8.
 * Larger sizes are rejected with EAD_ELIMIT before anything is launched.
 *
 *   W        dev, bf16 [V, H] row major, 16-byte aligned (borrowed, read only)
 *   h        dev, bf16 [B, H] row major, 16-byte aligned: one hidden row per sequence
 *   tok      dev, int32 [B]: greedy token, lowest index among equal maxima (-1 for a row
 *            with non-finite logits); may be NULL
 *   H_out    dev, float [B]: entropy in nats (NaN for a row with non-finite logits); may be NULL
 *   status   dev, uint32 [1]: receives EAD_STATUS_* bits of this call; may be NULL
 *   device   CUDA device ordinal; made current by the call
 *   stream   cudaStream_t to enqueue on; NULL = legacy default stream
 *
 * Asynchronous: four kernels are enqueued on `stream` (status clear, staging of the hidden
 * rows, the LM-head contraction, the merge).  The first call on a device also
 * looks up the device address of the built-in array and the device's limits; make that
 * first call outside any stream capture.
 * Every call on a device uses the SAME array.  The call rewrites all of it that it later
 * reads (nothing of an earlier call leaks into the result), but two calls whose kernels
 * overlap on the GPU (different streams, no dependency) race on it: keep calls on one
 * device ordered.  Not thread safe with respect to other calls on the same device.
 * Errors: EAD_EINVALID_ARG, EAD_EALIGNMENT, EAD_ELIMIT, EAD_EUNSUPPORTED_ARCH, EAD_ECUDA.
 */
#define EAD_STATIC_MAX_B 128
#define EAD_STATIC_MAX_H 8192
int ead_head_entropy_static(const void *W, const void *h, int32_t B, int32_t V, int32_t H,
                            int32_t *tok, float *H_out, uint32_t *status, int32_t device,
                            void *stream);

/* Static, NUL-terminated description of an EAD_E* code. */
const char *ead_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* EAD_H_ */
