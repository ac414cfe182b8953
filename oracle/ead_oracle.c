/*
 * CPU oracle for the gate step of Entropy Adaptive Decoding (EAD).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of
 * what the method computes, used by the tests, the smoke check and the CPU
 * baseline leg of the benchmark.  The CUDA library never calls it, and it
 * shares no code with the CUDA library.
 *
 * What follows the paper:
 *   - oracle_logits      "l <- M_t(x + y)" of Algorithm 1, restricted to the
 *                        last layer of M_t: the LM-head projection z = W h.
 *   - oracle_entropy     Eq. 1 (softmax of the raw logits, no temperature)
 *                        and Eq. 2 (Shannon entropy).  Eq. 2 uses log2 (bits);
 *                        unit 0 returns nats, unit 1 bits.
 *   - oracle_greedy      replaces the temperature-sampling lines of
 *                        Algorithm 1 by their T -> 0 limit: the arg max,
 *                        lowest index among equal maxima.
 *   - oracle_gate_step   Algorithm 1 from "Append H_t to W" to the end of the
 *                        loop body: mean of the last w entries of W (only the
 *                        entries that exist while fewer than w were appended),
 *                        c <- c + 1, and, once c >= d_min, the two-sided
 *                        threshold test of Eq. 4 with c <- 0 at a switch.
 *   - oracle_run         Algorithm 1 for B independent sequences and a fixed
 *                        number T of tokens, hidden states given as inputs.
 *   - oracle_sample      the sampling lines of Algorithm 1: l' = l / T, p' =
 *                        softmax(l'), token ~ p'.  The draw is realised as the
 *                        arg max of l'_i + g_i with independent standard Gumbel
 *                        g_i = -ln(-ln u_i) (an exact sampler of p'), the
 *                        uniforms u_i coming from Philox4x32-10 (Salmon, Moraes,
 *                        Dror, Shaw, SC'11) keyed by (seed) and counted by
 *                        (vocabulary index / 4, step, row): the same stream the
 *                        CUDA path implements from the same published definition.
 *   - oracle_parameter_ratio   the footnote of Table 1: average parameters per
 *                        forward pass relative to the large model,
 *                        (alpha P_S + beta P_L) / P_L with alpha, beta the usage
 *                        shares of the small and the large model.
 *
 * Readings where the paper is silent: a row whose logits contain a NaN or an
 * infinity produces H = NaN, token -1, and leaves W, c and the model flag as
 * they were.  0 * log 0 counts as 0.
 *
 * Pins (tests/test_oracle_pins.py): uniform logits give ln V, one-hot logits
 * give 0, shift invariance, a two-level closed form, brute force on tiny V,
 * bits = nats / ln 2, hand-worked window/threshold traces, and the
 * "small for d_min tokens, then large" trace for a threshold below every
 * entropy; the parameter-ratio column of Table 1 recomputed from its usage
 * column.  The end-to-end run on the benchmark configurations has no value
 * printed by the paper to compare with: parity unpinned for oracle_run beyond
 * the composition of its pinned parts.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE float32: widening is exact. */
static double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

void oracle_widen_bf16(const uint16_t *src, int64_t n, double *dst)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = bf16_to_f64(src[i]);
}

/* z_i = sum_j W[i, j] * h[j], j ascending.  W is [V, H] row major, bf16 bits. */
void oracle_logits(const uint16_t *W, int64_t V, int64_t H, const uint16_t *h, double *z)
{
    double *hd = (double *)malloc((size_t)H * sizeof(double));
    oracle_widen_bf16(h, H, hd);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < V; ++i) {
        const uint16_t *w = W + i * H;
        double acc = 0.0;
        for (int64_t j = 0; j < H; ++j) acc += bf16_to_f64(w[j]) * hd[j];
        z[i] = acc;
    }
    free(hd);
}

static int all_finite(const double *z, int64_t V)
{
    for (int64_t i = 0; i < V; ++i)
        if (!isfinite(z[i])) return 0;
    return 1;
}

/* Eq. 1 then Eq. 2.  p may be NULL; otherwise it receives the softmax. */
double oracle_entropy(const double *z, int64_t V, int unit, double *p_out)
{
    if (V <= 0 || !all_finite(z, V)) return NAN;
    double m = z[0];
    for (int64_t i = 1; i < V; ++i)
        if (z[i] > m) m = z[i];
    /* exp(l_i) / sum_j exp(l_j), with the common factor exp(-m) taken out so
       that the exponentials stay in range; the quotient is unchanged. */
    double Z = 0.0;
    for (int64_t i = 0; i < V; ++i) Z += exp(z[i] - m);
    double H = 0.0;
    for (int64_t i = 0; i < V; ++i) {
        double p = exp(z[i] - m) / Z;
        if (p_out) p_out[i] = p;
        if (p > 0.0) H -= p * log(p);
    }
    if (unit == 1) H /= log(2.0);
    return H;
}

/* Lowest index attaining the maximum; also the gap between the two largest
   logits (0 when the maximum is attained twice), for near-tie bookkeeping. */
int64_t oracle_greedy(const double *z, int64_t V, double *gap_out)
{
    if (V <= 0 || !all_finite(z, V)) {
        if (gap_out) *gap_out = NAN;
        return -1;
    }
    int64_t best = 0;
    for (int64_t i = 1; i < V; ++i)
        if (z[i] > z[best]) best = i;
    if (gap_out) {
        double second = -INFINITY;
        for (int64_t i = 0; i < V; ++i)
            if (i != best && z[i] > second) second = z[i];
        *gap_out = (V > 1) ? z[best] - second : INFINITY;
    }
    return best;
}

/* ---- Philox4x32-10 as published: 10 rounds of two 32x32 -> 64 multiplies with the
 *      constants 0xD2511F53, 0xCD9E8D57 and the key bumped by 0x9E3779B9, 0xBB67AE85. */
void oracle_philox4x32(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Uniform in (0, 1) for vocabulary entry i of sequence `row` at its `step`-th token:
 * the top 23 bits k of word (i mod 4) of block (i / 4), as (2k + 1) / 2^24 (an odd
 * multiple of 2^-24: exact in float32 and float64, never 0 or 1). */
double oracle_uniform(uint64_t seed, int64_t row, int64_t step, int64_t i)
{
    uint32_t ctr[4] = {(uint32_t)(i >> 2), (uint32_t)step, (uint32_t)row, 0u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    oracle_philox4x32(ctr, key, out);
    uint32_t k = out[i & 3] >> 9;
    return (double)(2u * k + 1u) / 16777216.0;
}

/* Sampling lines of Algorithm 1 at temperature T > 0 (see the header).  Returns the
 * token; gap_out receives the difference of the two largest perturbed values. */
int64_t oracle_sample(const double *z, int64_t V, double T, uint64_t seed, int64_t row,
                      int64_t step, double *gap_out)
{
    if (V <= 0 || !all_finite(z, V)) {
        if (gap_out) *gap_out = NAN;
        return -1;
    }
    int64_t best = -1;
    double best_v = -INFINITY, second = -INFINITY;
    for (int64_t i = 0; i < V; ++i) {
        double lp = z[i] / T;                                /* l' = l / T          */
        double g = -log(-log(oracle_uniform(seed, row, step, i)));
        double v = lp + g;                                   /* arg max = draw from softmax(l') */
        if (v > best_v) {
            second = best_v;
            best_v = v;
            best = i;
        } else if (v > second) {
            second = v;
        }
    }
    if (gap_out) *gap_out = (V > 1) ? best_v - second : INFINITY;
    return best;
}

/*
 * One pass through the tail of Algorithm 1's loop body for one sequence.
 *   hist     entropy window W as the paper keeps it: an append-only list
 *   n        number of entries in hist (updated)
 *   c        tokens since the last switch (updated)
 *   model    0 = small, 1 = large (updated)
 * Returns the rolling mean.  H = NaN leaves everything untouched.
 */
double oracle_gate_step(double *hist, int64_t *n, int32_t *c, int32_t *model,
                        double H, int32_t w, int32_t d_min, double tau)
{
    if (isnan(H)) return NAN;
    hist[*n] = H;                       /* Append H_t to W            */
    *n += 1;
    int64_t cnt = (*n < (int64_t)w) ? *n : (int64_t)w;
    double sum = 0.0;                   /* mean(W[-w:])               */
    for (int64_t i = *n - cnt; i < *n; ++i) sum += hist[i];
    double Hbar = sum / (double)cnt;
    *c += 1;                            /* c <- c + 1                 */
    if (*c >= d_min) {
        if (*model == 0 && Hbar > tau) {
            *model = 1;
            *c = 0;
        } else if (*model == 1 && Hbar <= tau) {
            *model = 0;
            *c = 0;
        }
    }
    return Hbar;
}

/* Runs oracle_gate_step over a given entropy sequence (for the hand traces). */
void oracle_gate_trace(const double *H, int64_t T, int32_t w, int32_t d_min, double tau,
                       int32_t start_model, double *Hbar, uint8_t *used, uint8_t *next,
                       int32_t *c_after)
{
    double *hist = (double *)malloc((size_t)(T > 0 ? T : 1) * sizeof(double));
    int64_t n = 0;
    int32_t c = 0, model = start_model;
    for (int64_t t = 0; t < T; ++t) {
        used[t] = (uint8_t)model;
        Hbar[t] = oracle_gate_step(hist, &n, &c, &model, H[t], w, d_min, tau);
        next[t] = (uint8_t)model;
        if (c_after) c_after[t] = c;
    }
    free(hist);
}

/*
 * A sequence whose token equals eos_token (>= 0) is done: that step is complete, later
 * steps of the row report token -1, NaN entropies and the unchanged model.
 * Algorithm 1 (greedy for temperature 0, sampled otherwise) for the rows listed in `rows` (n_rows of
 * them, indices into [0, B)) and T tokens.  Inputs are bf16 bit patterns:
 * W_small [V, H_small], W_large [V, H_large], h_small [T, B, H_small],
 * h_large [T, B, H_large].  Outputs are [T, n_rows], row k of an output
 * belonging to sequence rows[k]:
 *   tok, H (in `unit`), Hbar, used (model that produced token t), next (model
 *   after the switch test), gap (difference of the two largest logits),
 *   c_after (dwell counter after the step).  Any output pointer may be NULL.
 */
void oracle_run(int64_t B, int64_t T, int64_t V, int64_t V_large, int64_t H_small, int64_t H_large,
                int32_t w, int32_t d_min, double tau, int32_t unit, int32_t start_model,
                const uint16_t *W_small, const uint16_t *W_large,
                const uint16_t *h_small, const uint16_t *h_large,
                const int64_t *rows, int64_t n_rows,
                int32_t *tok, double *H, double *Hbar, uint8_t *used, uint8_t *next,
                double *gap, int32_t *c_after, double temperature, uint64_t seed, int32_t eos_token)
{
    double *z = (double *)malloc((size_t)(V > V_large ? V : V_large) * sizeof(double));
    double *hist = (double *)malloc((size_t)(T > 0 ? T : 1) * sizeof(double));
    for (int64_t k = 0; k < n_rows; ++k) {
        int64_t b = rows[k];
        int64_t n = 0;                  /* W <- []      */
        int32_t c = 0;                  /* c <- 0       */
        int32_t model = start_model;    /* M_t <- M_S   */
        int done = 0;                   /* "while not done": set by the end-of-sequence token */
        for (int64_t t = 0; t < T; ++t) {
            int64_t o = t * n_rows + k;
            if (used) used[o] = (uint8_t)model;
            if (done) {                 /* the loop has ended for this sequence: nothing is computed */
                if (tok) tok[o] = -1;
                if (H) H[o] = NAN;
                if (Hbar) Hbar[o] = NAN;
                if (next) next[o] = (uint8_t)model;
                if (gap) gap[o] = NAN;
                if (c_after) c_after[o] = c;
                continue;
            }
            /* the two models may have different vocabularies (V for M_S, V_large for M_L) */
            int64_t Vm = model == 0 ? V : V_large;
            if (model == 0)
                oracle_logits(W_small, Vm, H_small, h_small + (t * B + b) * H_small, z);
            else
                oracle_logits(W_large, Vm, H_large, h_large + (t * B + b) * H_large, z);
            double Ht = oracle_entropy(z, Vm, unit, NULL);
            double g;
            /* the entropy above is taken before any temperature scaling; the token is the
               arg max (temperature 0) or a draw from softmax(l / T) */
            int64_t tk = temperature > 0.0 ? oracle_sample(z, Vm, temperature, seed, b, t, &g)
                                           : oracle_greedy(z, Vm, &g);
            double Hb = oracle_gate_step(hist, &n, &c, &model, Ht, w, d_min, tau);
            if (tok) tok[o] = (int32_t)tk;
            if (H) H[o] = Ht;
            if (Hbar) Hbar[o] = Hb;
            if (next) next[o] = (uint8_t)model;
            if (gap) gap[o] = g;
            if (c_after) c_after[o] = c;
            if (eos_token >= 0 && tk == eos_token) done = 1;
        }
    }
    free(hist);
    free(z);
}

/* Footnote of Table 1.  usage_large = beta in [0, 1]; alpha = 1 - beta. */
double oracle_parameter_ratio(double usage_large, double P_small, double P_large)
{
    double alpha = 1.0 - usage_large, beta = usage_large;
    return (alpha * P_small + beta * P_large) / P_large;
}

/*
 * Tokens produced by each model and number of switches in a [T] trace of one sequence
 * (Table 1's usage column counts generated tokens).  `tok` may be NULL; if given, a step
 * whose token is -1 produced nothing (Algorithm 1's "while not done" had ended for the
 * sequence, or its logits were not finite) and counts neither as a token nor as a switch.
 */
void oracle_usage(const uint8_t *used, const uint8_t *next, const int32_t *tok, int64_t T,
                  int64_t *tokens_small, int64_t *tokens_large, int64_t *switches)
{
    int64_t s = 0, l = 0, sw = 0;
    for (int64_t t = 0; t < T; ++t) {
        if (tok && tok[t] < 0) continue;
        if (used[t]) l += 1; else s += 1;
        if (next[t] != used[t]) sw += 1;
    }
    *tokens_small = s;
    *tokens_large = l;
    *switches = sw;
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
