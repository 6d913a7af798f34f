/*
 * CPU oracle for the speculative-decoding step: counter-based uniforms, vocabulary softmax,
 * lossless rejection sampling and paged-KV bookkeeping.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the method computes; it is
 * compiled by gcc into liboracle.so and used by the tests, by the smoke check and by the benchmark's
 * CPU-baseline leg.  The product (the CUDA library) neither links nor imports it, and it shares no code,
 * table or constant generator with the CUDA path.
 *
 * What it follows.  The paper states the method in one sentence (Introduction, third paragraph): a draft
 * proposes several tokens, the target verifies them with a rejection procedure that keeps the target's
 * output distribution; Section 2.1 repeats that rollouts follow the verifier policy by construction, and
 * Section 2.2 defines the acceptance length as the number of tokens produced per speculation step
 * (so between 1 and k+1, Section 4.2).  The concrete rule used here is the standard one those
 * citations define: accept draft token d_i when u_i < min(1, p_i(d_i)/q_i(d_i)); at the first rejected
 * position resample from norm(max(0, p - q)); when all k are accepted draw a bonus token from p_{k+1}.
 *
 * Everything is scalar loops, fp32 storage and fp64 arithmetic, one sequence after another, in index order.
 *
 * Pins (tests/test_oracle_*.py): Philox known-answer vectors from the Random123 distribution; softmax
 * against scipy; exact enumeration and a chi-square test of the emitted-token distribution at V=8;
 * draft == target accepts everything; the i.i.d. mean-length closed form; residual invariants; one-hot
 * drafts; block conservation for the KV bookkeeping.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------------------
 * Uniforms.  Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
 * SC'11): ten rounds of two 32x32->64 multiplies, a key schedule that adds the golden-ratio / sqrt(3)
 * constants each round.  Reading chosen where the paper is silent on the generator:
 *   key     = (low 32 bits of seed, high 32 bits of seed)
 *   counter = (step, sequence index, slot, stream tag)
 *   uniform = (first output word >> 8) * 2^-24, which lies in [0,1) and is exact in fp32.
 * ---------------------------------------------------------------------------------------------------- */
void spec_oracle_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        uint64_t prod0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t prod1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
        uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

float spec_oracle_uniform(uint64_t seed, uint32_t step, uint32_t seq, uint32_t slot, uint32_t stream)
{
    uint32_t ctr[4] = { step, seq, slot, stream };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t out[4];
    spec_oracle_philox4x32_10(ctr, key, out);
    return (float)(out[0] >> 8) * (1.0f / 16777216.0f);
}

/* Fills u[n_seq][n_slots] with the uniforms of one step and one stream. */
void spec_oracle_uniforms(uint64_t seed, uint32_t step, uint32_t stream, int n_seq, int n_slots, float* u)
{
    for (int b = 0; b < n_seq; ++b)
        for (int s = 0; s < n_slots; ++s)
            u[(size_t)b * n_slots + s] = spec_oracle_uniform(seed, step, (uint32_t)b, (uint32_t)s, stream);
}

/* ------------------------------------------------------------------------------------------------------
 * Vocabulary softmax at temperature T (T scales the logits of both models before the softmax).
 *   m = max_v l_v;  Z = sum_v exp((l_v - m)/T);  p_v = exp((l_v - m)/T) / Z     (fp64, rounded to fp32)
 * Optionally reports m and Z.
 * ---------------------------------------------------------------------------------------------------- */
void spec_oracle_softmax_row(const float* logits, int V, double temperature, float* probs,
                             double* row_max, double* row_sumexp)
{
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) if ((double)logits[v] > m) m = (double)logits[v];
    double Z = 0.0;
    for (int v = 0; v < V; ++v) Z += exp(((double)logits[v] - m) / temperature);
    if (probs)
        for (int v = 0; v < V; ++v) probs[v] = (float)(exp(((double)logits[v] - m) / temperature) / Z);
    if (row_max) *row_max = m;
    if (row_sumexp) *row_sumexp = Z;
}

/* log p(token) of one logit row at temperature T: (l_t - m)/T - log sum_v exp((l_v - m)/T), in fp64.  This is the
 * verifier-side log-probability that an RL loss uses (Section 2.3: it must come from the target, not the draft). */
double spec_oracle_logprob(const float* logits, int V, double temperature, int token)
{
    double m, Z;
    spec_oracle_softmax_row(logits, V, temperature, NULL, &m, &Z);
    return ((double)logits[token] - m) / temperature - log(Z);
}

void spec_oracle_softmax(const float* logits, int rows, int V, double temperature, float* probs)
{
    for (int r = 0; r < rows; ++r)
        spec_oracle_softmax_row(logits + (size_t)r * V, V, temperature, probs + (size_t)r * V, NULL, NULL);
}

/* ------------------------------------------------------------------------------------------------------
 * Inverse CDF over non-negative weights w[0..V-1] (not normalised).
 *   S = sum_v w_v (index order);  answer = smallest v with  sum_{j<=v} w_j  >  u*S.
 * The comparison is strict, so a zero-weight bin is never chosen and u = 0 picks the first positive bin.
 * If rounding leaves the running sum at or below u*S after the last bin, the last positive bin is taken.
 * margin (optional) = distance, in units of S, from u to the nearer edge of the chosen bin; the tests use
 * it to recognise draws that sit on a bin edge.  Returns -1 when no weight is positive.
 * ---------------------------------------------------------------------------------------------------- */
static int invcdf(const double* w, int V, double u, double* margin)
{
    double S = 0.0;
    for (int v = 0; v < V; ++v) S += w[v];
    if (!(S > 0.0) || !isfinite(S)) return -1;
    double target = u * S, run = 0.0;
    int chosen = -1, last_pos = -1;
    double lo = 0.0, hi = 0.0;
    for (int v = 0; v < V; ++v) {
        double before = run;
        run += w[v];
        if (w[v] > 0.0) last_pos = v;
        if (run > target) { chosen = v; lo = before; hi = run; break; }
    }
    if (chosen < 0) { chosen = last_pos; lo = hi = S; }
    if (margin) {
        double a = fabs(u - lo / S), b = fabs(u - hi / S);
        *margin = a < b ? a : b;
    }
    return chosen;
}

int spec_oracle_invcdf_f32(const float* w, int V, float u, double* margin)
{
    double* wd = (double*)malloc(sizeof(double) * (size_t)V);
    for (int v = 0; v < V; ++v) wd[v] = (double)w[v];
    int r = invcdf(wd, V, (double)u, margin);
    free(wd);
    return r;
}

/* ------------------------------------------------------------------------------------------------------
 * One rejection-sampling step for ONE sequence.
 *   p      [k+1][V] target probabilities p_1..p_{k+1}   (fp32)
 *   q      [k][V]   draft  probabilities q_1..q_k       (fp32)
 *   draft  [k]      draft tokens d_1..d_k, d_i drawn from q_i
 *   u      [k+1]    uniforms: u[i-1] decides position i (i=1..k); u[k] drives the resample / bonus draw.
 *                   Every slot is positional: u[i-1] belongs to position i whether or not earlier
 *                   positions were accepted.
 * Steps: accept_i = u_i < min(1, p_i(d_i)/q_i(d_i)) in fp64 on the fp32 values (q_i(d_i) = 0 is read as
 * "accept iff p_i(d_i) > 0", the limit of u*q < p); n = length of the all-accepted prefix; if n < k the
 * next token is drawn from max(0, p_{n+1} - q_{n+1}) (fp64 difference, normalised by the inverse CDF),
 * else from p_{k+1}.  Output: out_tokens = d_1..d_n, token, then -1; n_emitted = n + 1.
 * flags bit 0: the residual had no positive mass (possible only with garbage input); the draw then falls
 * back to p_{n+1}.  margins (optional, [k+1]): |u_i - min(1, ratio_i)| for i<k and the bin-edge distance of
 * the final draw at [k].
 * ---------------------------------------------------------------------------------------------------- */
void spec_oracle_reject_sample_seq(int k, int V, const float* p, const float* q, const int32_t* draft,
                                   const float* u, int32_t* out_tokens, int32_t* n_emitted,
                                   uint32_t* flags, double* margins)
{
    uint32_t fl = 0;
    int n = 0, still = 1;
    for (int i = 0; i < k; ++i) {
        int d = draft[i];
        double pd = (double)p[(size_t)i * V + d];
        double qd = (double)q[(size_t)i * V + d];
        double thr;
        if (qd > 0.0) { thr = pd / qd; if (thr > 1.0) thr = 1.0; }
        else          { thr = pd > 0.0 ? 1.0 : 0.0; }
        int acc = (double)u[i] < thr;
        if (margins) margins[i] = fabs((double)u[i] - thr);
        if (still && acc) n += 1; else still = 0;
    }
    double* w = (double*)malloc(sizeof(double) * (size_t)V);
    int token;
    double mg = 0.0;
    if (n < k) {
        const float* pr = p + (size_t)n * V;
        const float* qr = q + (size_t)n * V;
        for (int v = 0; v < V; ++v) {
            double r = (double)pr[v] - (double)qr[v];
            w[v] = r > 0.0 ? r : 0.0;
        }
        token = invcdf(w, V, (double)u[k], &mg);
        if (token < 0) {
            fl |= 1u;
            for (int v = 0; v < V; ++v) w[v] = (double)pr[v];
            token = invcdf(w, V, (double)u[k], &mg);
        }
    } else {
        const float* pr = p + (size_t)k * V;
        for (int v = 0; v < V; ++v) w[v] = (double)pr[v];
        token = invcdf(w, V, (double)u[k], &mg);
    }
    free(w);
    if (token < 0) { fl |= 2u; token = 0; }
    for (int i = 0; i < n; ++i) out_tokens[i] = draft[i];
    out_tokens[n] = token;
    for (int i = n + 1; i <= k; ++i) out_tokens[i] = -1;
    *n_emitted = n + 1;
    if (margins) margins[k] = mg;
    if (flags) *flags = fl;
}

/* The batch form: sequence b uses the uniforms Philox(seed; step, b, slot 0..k, stream 0). */
void spec_oracle_reject_sample(int B, int k, int V, const float* p, const float* q, const int32_t* draft,
                               uint64_t seed, uint32_t step, int32_t* out_tokens, int32_t* n_emitted,
                               uint32_t* flags, double* margins)
{
    float u[64];
    for (int b = 0; b < B; ++b) {
        for (int s = 0; s <= k; ++s) u[s] = spec_oracle_uniform(seed, step, (uint32_t)b, (uint32_t)s, 0u);
        spec_oracle_reject_sample_seq(k, V, p + (size_t)b * (k + 1) * V, q + (size_t)b * k * V,
                                      draft + (size_t)b * k, u, out_tokens + (size_t)b * (k + 1),
                                      n_emitted + b, flags ? flags + b : NULL,
                                      margins ? margins + (size_t)b * (k + 1) : NULL);
    }
}

/* Draft sampling: d = invcdf(q, u) with the stream-1 uniform of (step, b, slot). */
void spec_oracle_sample_rows(int B, int V, const float* probs, const float* u, int32_t* tokens,
                             double* margins)
{
    for (int b = 0; b < B; ++b)
        tokens[b] = spec_oracle_invcdf_f32(probs + (size_t)b * V, V, u[b], margins ? margins + b : NULL);
}

/* ------------------------------------------------------------------------------------------------------
 * Paged-KV bookkeeping.  The paper is silent here; this is the reading used throughout:
 *   seq_len[b]     number of valid KV entries of sequence b (positions 0..seq_len-1)
 *   block_table    [B][max_blocks], physical block id of each 16-token (block_tokens) logical block, -1 = none
 *   free_stack     [num_blocks] ids of free blocks, the top of the stack is free_stack[free_top-1]
 * reserve: every sequence, in index order, pops blocks (logical index increasing) until it owns
 *          ceil((seq_len + k + 1)/block_tokens) of them, i.e. room for the k+1 positions of a verify.
 *          If the stack cannot serve the whole batch nothing is changed and -1 is returned.
 * commit : seq_len += n_emitted (the position of the last committed token plus the n accepted drafts are
 *          kept); logical blocks whose first slot is >= the new seq_len are pushed back (sequence order,
 *          logical index increasing) and their table entries reset to -1.
 * ---------------------------------------------------------------------------------------------------- */
int spec_oracle_kv_reserve(int B, int k, int block_tokens, int max_blocks, const int32_t* seq_len,
                           int32_t* block_table, int32_t* free_stack, int32_t* free_top)
{
    long need_total = 0;
    for (int b = 0; b < B; ++b) {
        if (seq_len[b] < 0) continue;                      /* retired slot */
        int need = (seq_len[b] + k + 1 + block_tokens - 1) / block_tokens;
        if (need > max_blocks) return -2;
        for (int j = 0; j < need; ++j) if (block_table[(size_t)b * max_blocks + j] < 0) need_total += 1;
    }
    if (need_total > *free_top) return -1;
    for (int b = 0; b < B; ++b) {
        if (seq_len[b] < 0) continue;
        int need = (seq_len[b] + k + 1 + block_tokens - 1) / block_tokens;
        for (int j = 0; j < need; ++j) {
            int32_t* e = &block_table[(size_t)b * max_blocks + j];
            if (*e < 0) { *free_top -= 1; *e = free_stack[*free_top]; }
        }
    }
    return 0;
}

void spec_oracle_kv_commit(int B, int block_tokens, int max_blocks, const int32_t* n_emitted,
                           int32_t* seq_len, int32_t* block_table, int32_t* free_stack, int32_t* free_top)
{
    for (int b = 0; b < B; ++b) {
        if (seq_len[b] < 0) continue;                      /* retired slot: holds nothing, commits nothing */
        seq_len[b] += n_emitted[b];
        int keep = (seq_len[b] + block_tokens - 1) / block_tokens;
        for (int j = keep; j < max_blocks; ++j) {
            int32_t* e = &block_table[(size_t)b * max_blocks + j];
            if (*e >= 0) { free_stack[*free_top] = *e; *free_top += 1; *e = -1; }
        }
    }
}

/* replace: sequences finish at different lengths (the long tail of response lengths, Section 5.1) and their slots are
 * refilled.  For every listed slot, in list order: all its blocks go back to the free stack (logical order), then blocks
 * for new_len[i] cached positions are popped.  new_len[i] < 0 retires the slot: it keeps no block, its length stays -1
 * and reserve / commit pass it over until it is replaced again.  Returns -1 (nothing changed) if the stack cannot
 * serve the list. */
int spec_oracle_kv_replace(int n, const int32_t* slots, const int32_t* new_len, int block_tokens, int max_blocks,
                           int32_t* seq_len, int32_t* block_table, int32_t* free_stack, int32_t* free_top)
{
    long avail = *free_top, need = 0;
    for (int i = 0; i < n; ++i) {
        for (int j = 0; j < max_blocks; ++j) if (block_table[(size_t)slots[i] * max_blocks + j] >= 0) avail += 1;
        need += new_len[i] < 0 ? 0 : (new_len[i] + block_tokens - 1) / block_tokens;
    }
    if (need > avail) return -1;
    for (int i = 0; i < n; ++i) {
        int32_t* row = block_table + (size_t)slots[i] * max_blocks;
        for (int j = 0; j < max_blocks; ++j)
            if (row[j] >= 0) { free_stack[*free_top] = row[j]; *free_top += 1; row[j] = -1; }
        int blocks = new_len[i] < 0 ? 0 : (new_len[i] + block_tokens - 1) / block_tokens;
        for (int j = 0; j < blocks; ++j) { *free_top -= 1; row[j] = free_stack[*free_top]; }
        seq_len[slots[i]] = new_len[i] < 0 ? -1 : new_len[i];
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------------------
 * 8-bit KV cache (the precision the paper's deployment simulator assumes, Section 5.1): a cached value x is stored
 * as e4m3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities, largest finite value 448,
 * smallest subnormal 2^-9) of x / scale, rounded to nearest with ties to even and saturating at +-448; the
 * attention reads it back as code * scale.  NaN maps to the NaN code 0x7f.
 * ---------------------------------------------------------------------------------------------------- */
static uint8_t e4m3_from_float(float x)
{
    if (x != x) return 0x7f;
    const uint8_t sign = signbit(x) ? 0x80 : 0x00;
    const double a = fabs((double)x);
    if (a >= 448.0) return (uint8_t)(sign | 0x7e);                 /* saturate: 0x7e is 448 */
    if (a < 0.015625) {                                             /* below 2^-6: subnormal grid, spacing 2^-9 */
        const double r = nearbyint(a * 512.0);                      /* default rounding mode: ties to even */
        return (uint8_t)(sign | (uint8_t)r);                        /* r = 8 is the code of the first normal, 2^-6 */
    }
    int e;
    (void)frexp(a, &e);                                             /* a = m * 2^e with m in [0.5, 1): a = 1.f * 2^(e-1) */
    int exp_field = e - 1 + 7;
    double r = nearbyint(ldexp(a, -(e - 1)) * 8.0);                 /* 8 + mantissa, in [8, 16] */
    if (r >= 16.0) { r = 8.0; exp_field += 1; }
    if (exp_field > 15 || (exp_field == 15 && r > 14.0)) return (uint8_t)(sign | 0x7e);
    return (uint8_t)(sign | (uint8_t)(exp_field << 3) | (uint8_t)((int)r - 8));
}

static float e4m3_to_float(uint8_t c)
{
    int sign = c & 0x80, ef = (c >> 3) & 0xf, mf = c & 7;
    double v;
    if (ef == 15 && mf == 7) return NAN;
    if (ef == 0) v = mf / 512.0;
    else v = ldexp(1.0 + mf / 8.0, ef - 7);
    return (float)(sign ? -v : v);
}

void spec_oracle_e4m3_quantize(size_t n, const float* x, float scale, uint8_t* codes)
{
    for (size_t i = 0; i < n; ++i) codes[i] = e4m3_from_float(x[i] / scale);
}

/* 8-bit operands of a projection (the precision the paper's simulator assumes, Section 5.1): every row of a matrix gets
 * its own scale, the largest magnitude of the row mapped to the largest e4m3 value, scale = amax / 448 in fp32 (1 for an
 * all-zero row); code = round_e4m3(x / scale). */
void spec_oracle_e4m3_quantize_rows(size_t rows, size_t k, const float* x, float* scales, uint8_t* codes)
{
    for (size_t r = 0; r < rows; ++r) {
        float amax = 0.0f;
        for (size_t i = 0; i < k; ++i) { const float a = fabsf(x[r * k + i]); if (a > amax) amax = a; }
        const float sc = amax > 0.0f ? amax / 448.0f : 1.0f;
        scales[r] = sc;
        for (size_t i = 0; i < k; ++i) codes[r * k + i] = e4m3_from_float(x[r * k + i] / sc);
    }
}

void spec_oracle_e4m3_dequantize(size_t n, const uint8_t* codes, float scale, float* x)
{
    for (size_t i = 0; i < n; ++i) x[i] = e4m3_to_float(codes[i]) * scale;
}
