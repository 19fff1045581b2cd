/*
 * polyspec_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, double-precision CPU statement of the verification rule of
 * polybasic speculative decoding (chained speculative sampling).  It exists so
 * that the CUDA library can be checked against something written directly from
 * the paper.  It shares no code with the CUDA path, is never called by it, and
 * only the tests, the smoke check and the benchmark's CPU-baseline leg may load
 * it.  There is no blocking, fusion or reordering here: every step is the
 * definition written out, one vocabulary entry at a time, in index order.
 *
 * What follows the paper, and where:
 *   - the model chain M_1 (target) ... M_n and the per-position distributions
 *     p_i(x | x_<=t) over the vocabulary: Section 3.1 (Problem Formulation);
 *   - the block of K tokens drafted by M_n is checked bottom-up, by M_{n-1}
 *     first and M_1 last: Section 3.1; this is pso_verify_chain_seq's loop;
 *   - Verify(x_i, p_i) with a break at the first failure: Algorithm 1, the inner
 *     for-loop; the verification rule is speculative sampling (Sections 2, 3.1,
 *     3.2), i.e. accept with probability min(1, p/q);
 *   - VerifyBlock / SampleOne: Algorithm 1's M_1 branch, read as prefix
 *     acceptance with a replacement token drawn from the normalised residual
 *     max(0, p - q) at the first rejected position, or from the next row of p
 *     when the whole block is accepted -- the only reading under which the
 *     output keeps the target distribution, as the abstract and Section 5 claim;
 *   - the acceptance length of Eq. 1 is `accepted_len`.
 *
 * Parity pins (tests/test_oracle_*.py): library softmax, exact enumeration of
 * the emitted-stream law on tiny vocabularies (single level and chains), p == q,
 * disjoint supports, residual mass 1 - sum min(p,q), numpy searchsorted for the
 * inverse CDF, the capped-geometric mean of Theorem 3.3's proof.  No function
 * here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { PSO_F32 = 0, PSO_BF16 = 1, PSO_F64 = 2 };   /* storage type of a logits buffer */

enum {
    PSO_OK = 0,
    PSO_BAD_ROW_NAN = 1,       /* a NaN or +inf logit */
    PSO_BAD_ROW_EMPTY = 2,     /* no finite logit in the row */
    PSO_BAD_TOKEN = 3,         /* token id outside [0, V) */
    PSO_BAD_ARG = 4
};

/* One stored logit as a double.  bf16 is the upper half of an IEEE float. */
static double pso_load(const void* base, int dtype, int64_t i)
{
    if (dtype == PSO_F32) return (double)((const float*)base)[i];
    if (dtype == PSO_F64) return ((const double*)base)[i];
    uint32_t bits = (uint32_t)((const uint16_t*)base)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static const void* pso_row(const void* base, int dtype, int64_t V, int64_t r)
{
    size_t elem = (dtype == PSO_F32) ? 4u : (dtype == PSO_F64) ? 8u : 2u;
    return (const char*)base + (size_t)r * (size_t)V * elem;
}

/*
 * Temperature softmax of one logits row: P(v) = exp((z_v - mx)/T) / Z with
 * mx the largest logit and Z summed in index order (Section 3.1: the
 * distribution p_i(x | x_<=t) over the vocabulary; the temperature is the
 * benchmark's, applied to every model alike).  -inf logits get probability 0.
 */
int pso_softmax_row(const void* row, int dtype, int64_t V, double T, double* P)
{
    if (!row || !P || V <= 0 || !(T > 0.0) || isinf(T)) return PSO_BAD_ARG;
    double mx = -INFINITY;
    for (int64_t v = 0; v < V; ++v) {
        double z = pso_load(row, dtype, v);
        if (isnan(z) || (isinf(z) && z > 0)) return PSO_BAD_ROW_NAN;
        if (z > mx) mx = z;
    }
    if (isinf(mx)) return PSO_BAD_ROW_EMPTY;
    double Z = 0.0;
    for (int64_t v = 0; v < V; ++v) {
        double z = pso_load(row, dtype, v);
        double e = isinf(z) ? 0.0 : exp((z - mx) / T);
        P[v] = e;
        Z += e;
    }
    for (int64_t v = 0; v < V; ++v) P[v] /= Z;
    return PSO_OK;
}

/*
 * Inverse CDF in ascending vocabulary order: the first v whose running sum of
 * w exceeds `target` (strictly, so a zero-mass entry is never returned).  If
 * rounding leaves no such v, the last entry with positive mass is returned.
 * info[0] = distance from target to the nearer edge of the chosen entry's CDF
 * interval divided by `total`; info[1] = total; info[2], info[3] = the nearest
 * positive-mass entries before and after the chosen one (-1 if none).
 */
static int32_t pso_inverse_cdf(const double* w, int64_t V, double target, double total, double* info)
{
    double c = 0.0, lo = 0.0, hi = 0.0;
    int64_t chosen = -1, last_pos = -1, prev = -1;
    for (int64_t v = 0; v < V; ++v) {
        double before = c;
        c += w[v];
        if (c > target) { chosen = v; lo = before; hi = c; break; }
        if (w[v] > 0.0) last_pos = v;
    }
    if (chosen < 0) {              /* rounding: fall back to the last positive-mass entry */
        if (last_pos < 0) {        /* no mass at all: nothing to sample */
            if (info) { info[0] = 0.0; info[1] = total; info[2] = -1.0; info[3] = -1.0; }
            return -1;
        }
        chosen = last_pos;
        hi = c;
        lo = c - w[chosen];
        target = c;
    }
    for (int64_t v = chosen - 1; v >= 0; --v) if (w[v] > 0.0) { prev = v; break; }
    int64_t succ = -1;
    for (int64_t v = chosen + 1; v < V; ++v) if (w[v] > 0.0) { succ = v; break; }
    if (info) {
        double dl = target - lo, dh = hi - target;
        info[0] = (dl < dh ? dl : dh) / total;
        info[1] = total;
        info[2] = (double)prev;
        info[3] = (double)succ;
    }
    return (int32_t)chosen;
}

/*
 * One verification of one sequence by one adjacent pair (verifier p, drafter-side q).
 *
 *   p_rows  [>= m+1 rows, V]  verifier logits; row j is position j+1, row m the bonus row
 *   q_rows  [>= m rows,   V]  logits of the distribution the block tokens were drawn from
 *   tokens  [m], u_accept [m], u_s: block tokens, accept uniforms, the one sampling uniform
 *
 * Algorithm 1's inner loop: positions are tested in order with
 *     accept  iff  u_j * Q_j(x_j) <= P_j(x_j)        (u_j <= min(1, P/Q), division-free)
 * and the loop breaks at the first failure; a = number accepted (Eq. 1 is its mean).
 * If a < m the replacement token is the inverse CDF, at u_s, of the residual
 * r(v) = max(0, P_{a+1}(v) - Q_{a+1}(v)) (if the residual sums to 0 in floating
 * point, of P_{a+1}, flagged); if a == m it is the inverse CDF of P_{m+1} (bonus).
 *
 * Outputs: accepted_len, next_token; P_at/Q_at [m] (NaN for positions never reached);
 * accept_margin [m] = |u_j - min(1, P/Q)| (NaN if not reached); sample_info [4] as in
 * pso_inverse_cdf; *used_fallback = 1 when the residual was empty.
 * scratch: 2*V doubles.  Returns PSO_OK or the reason the input is unusable, in
 * which case accepted_len = next_token = -1.
 */
int pso_verify_level_seq(const void* p_rows, const void* q_rows, int dtype, int64_t V, int m,
                         const int32_t* tokens, const float* u_accept, float u_s, double T,
                         int32_t* accepted_len, int32_t* next_token,
                         double* P_at, double* Q_at, double* accept_margin,
                         double* sample_info, int32_t* used_fallback, double* scratch)
{
    *accepted_len = -1;
    *next_token = -1;
    if (used_fallback) *used_fallback = 0;
    for (int j = 0; j < m; ++j) {
        if (P_at) P_at[j] = NAN;
        if (Q_at) Q_at[j] = NAN;
        if (accept_margin) accept_margin[j] = NAN;
    }
    if (!p_rows || V <= 0 || m < 0 || !scratch || (m > 0 && (!q_rows || !tokens || !u_accept)))
        return PSO_BAD_ARG;
    double* P = scratch;
    double* Q = scratch + V;

    int a = 0;
    int rejected = 0;
    for (int j = 0; j < m; ++j) {
        int32_t x = tokens[j];
        if (x < 0 || (int64_t)x >= V) return PSO_BAD_TOKEN;
        int st = pso_softmax_row(pso_row(p_rows, dtype, V, j), dtype, V, T, P);
        if (st) return st;
        st = pso_softmax_row(pso_row(q_rows, dtype, V, j), dtype, V, T, Q);
        if (st) return st;
        double u = (double)u_accept[j];
        double px = P[x], qx = Q[x];
        if (P_at) P_at[j] = px;
        if (Q_at) Q_at[j] = qx;
        if (accept_margin) {
            double ratio = (qx > 0.0) ? px / qx : INFINITY;
            accept_margin[j] = fabs(u - (ratio < 1.0 ? ratio : 1.0));
        }
        if (u * qx <= px) {
            a += 1;
        } else {
            rejected = 1;           /* P and Q now hold the rows of the rejected position */
            break;
        }
    }

    int32_t next;
    if (rejected) {
        double S = 0.0;
        for (int64_t v = 0; v < V; ++v) {
            double r = P[v] - Q[v];
            Q[v] = r > 0.0 ? r : 0.0;
            S += Q[v];
        }
        if (S > 0.0) {
            next = pso_inverse_cdf(Q, V, (double)u_s * S, S, sample_info);
        } else {
            if (used_fallback) *used_fallback = 1;
            next = pso_inverse_cdf(P, V, (double)u_s, 1.0, sample_info);
        }
    } else {
        int st = pso_softmax_row(pso_row(p_rows, dtype, V, m), dtype, V, T, P);
        if (st) return st;
        next = pso_inverse_cdf(P, V, (double)u_s, 1.0, sample_info);
    }
    *accepted_len = a;
    *next_token = next;
    return PSO_OK;
}

/*
 * The chain for one sequence (Section 3.1: the block drafted by M_n is checked
 * bottom-up, by M_{n-1} first and M_1 last).  Array index l = 0 .. n-2 is the level whose
 * verifier is model l (model 0 = M_1, the target); the bottom level l = n-2 runs first.
 *
 *   model_rows[i]  first logits row of model i for this sequence, model_nrows[i] rows
 *   k[l]           largest block level l verifies
 *   stream in      the bottom level's block is draft_tokens[0 .. bottom_len)
 *   uniforms       level l's uniforms start at uniforms + l*u_level_stride:
 *                  [j < k[l]] accept uniforms, [kmax] the sampling uniform
 *
 * Level l checks the first m_l = min(k[l], length of the stream handed up) tokens of
 * that stream with p = model l's rows and q = model l+1's rows: the stream a level
 * emits (accepted prefix plus its replacement or bonus token) is distributed as
 * sequential samples of that level's verifier, so the verifier's own rows are the
 * right q one level up.  The stream of level 0 is the committed output.
 *
 * Outputs per level l: accepted_len[l], block_len[l] (= m_l), out_len[l],
 * out_tokens[l*(kmax+1) ...] (entries past out_len are -1), accept_margin[l*kmax ...],
 * sample_info[l*4 ...], used_fallback[l].  On a bad input at some level, that level
 * and every level above it report -1 and the status is returned.
 */
int pso_verify_chain_seq(const void* const* model_rows, const int32_t* model_nrows, int n,
                         const int32_t* k, const int32_t* draft_tokens, int bottom_len,
                         const float* uniforms, int64_t u_level_stride, int kmax,
                         int64_t V, int dtype, double T,
                         int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens,
                         int32_t* out_len, double* accept_margin, double* sample_info,
                         int32_t* used_fallback, double* scratch)
{
    if (n < 2 || !model_rows || !model_nrows || !k || kmax < 1 || !scratch) return PSO_BAD_ARG;
    int L = n - 1;
    for (int l = 0; l < L; ++l) {
        accepted_len[l] = -1; block_len[l] = -1; out_len[l] = -1;
        if (used_fallback) used_fallback[l] = 0;
        for (int j = 0; j <= kmax; ++j) out_tokens[(size_t)l * (kmax + 1) + j] = -1;
        if (k[l] < 0 || k[l] > kmax) return PSO_BAD_ARG;
        if (model_nrows[l] < k[l] + 1) return PSO_BAD_ARG;
    }
    if (model_nrows[n - 1] < k[L - 1] || bottom_len < 0 || bottom_len > k[L - 1]) return PSO_BAD_ARG;

    int32_t* stream = (int32_t*)malloc(sizeof(int32_t) * (size_t)(kmax + 2));
    if (!stream) return PSO_BAD_ARG;
    int stream_len = bottom_len;
    for (int j = 0; j < bottom_len; ++j) stream[j] = draft_tokens[j];

    int status = PSO_OK;
    for (int l = L - 1; l >= 0; --l) {
        int m = stream_len < k[l] ? stream_len : k[l];
        const float* u = uniforms + (size_t)l * (size_t)u_level_stride;
        int32_t a, next;
        status = pso_verify_level_seq(model_rows[l], model_rows[l + 1], dtype, V, m, stream, u, u[kmax], T,
                                      &a, &next, NULL, NULL,
                                      accept_margin ? accept_margin + (size_t)l * kmax : NULL,
                                      sample_info ? sample_info + (size_t)l * 4 : NULL,
                                      used_fallback ? used_fallback + l : NULL, scratch);
        if (status) break;
        accepted_len[l] = a;
        block_len[l] = m;
        out_len[l] = a + 1;
        int32_t* out = out_tokens + (size_t)l * (kmax + 1);
        for (int j = 0; j < a; ++j) out[j] = stream[j];
        out[a] = next;
        stream[a] = next;            /* the emitted stream becomes the block one level up */
        stream_len = a + 1;
    }
    free(stream);
    return status;
}

/*
 * Greedy matching, the other verification rule Section 3.1 names beside speculative
 * sampling, and the one Section 4.5 compares
 * acceptance-length variance against: a block token is accepted iff it is the verifier's
 * most likely token at its position, the loop breaks at the first mismatch, and the
 * token emitted after the accepted prefix is the verifier's most likely token there (at
 * the first mismatch, or in the bonus row after a fully accepted block).  No uniforms, no
 * temperature (the arg max does not depend on it) and no drafter distribution: only the
 * verifier's rows and the block tokens matter.
 *
 * Arg max of one row: the first index holding the largest logit.  A row holding NaN or
 * +inf, or no finite logit, is unusable, as in the sampling rule.
 */
int pso_argmax_row(const void* row, int dtype, int64_t V, int32_t* arg)
{
    if (!row || !arg || V <= 0) return PSO_BAD_ARG;
    double best = -INFINITY;
    int64_t at = -1;
    for (int64_t v = 0; v < V; ++v) {
        double z = pso_load(row, dtype, v);
        if (isnan(z) || (isinf(z) && z > 0)) return PSO_BAD_ROW_NAN;
        if (z > best) { best = z; at = v; }
    }
    if (at < 0) return PSO_BAD_ROW_EMPTY;
    *arg = (int32_t)at;
    return PSO_OK;
}

/*
 * The chain under greedy matching, one sequence; arguments as in pso_verify_chain_seq
 * without uniforms and temperature.  model_rows[n-1] (the bottom drafter's logits) is
 * never read and may be NULL.
 */
int pso_verify_chain_greedy_seq(const void* const* model_rows, const int32_t* model_nrows, int n,
                                const int32_t* k, const int32_t* draft_tokens, int bottom_len, int kmax,
                                int64_t V, int dtype,
                                int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens, int32_t* out_len)
{
    if (n < 2 || !model_rows || !model_nrows || !k || kmax < 1) return PSO_BAD_ARG;
    int L = n - 1;
    for (int l = 0; l < L; ++l) {
        accepted_len[l] = -1; block_len[l] = -1; out_len[l] = -1;
        for (int j = 0; j <= kmax; ++j) out_tokens[(size_t)l * (kmax + 1) + j] = -1;
        if (k[l] < 0 || k[l] > kmax || model_nrows[l] < k[l] + 1 || !model_rows[l]) return PSO_BAD_ARG;
    }
    if (bottom_len < 0 || bottom_len > k[L - 1]) return PSO_BAD_ARG;
    int32_t* stream = (int32_t*)malloc(sizeof(int32_t) * (size_t)(kmax + 2));
    if (!stream) return PSO_BAD_ARG;
    int stream_len = bottom_len;
    for (int j = 0; j < bottom_len; ++j) stream[j] = draft_tokens[j];
    int status = PSO_OK;
    for (int l = L - 1; l >= 0 && status == PSO_OK; --l) {
        int m = stream_len < k[l] ? stream_len : k[l];
        int a = 0;
        int32_t next = -1;
        for (int j = 0; j <= m; ++j) {          /* row j scores position j; row m is the bonus row */
            if (j < m && (stream[j] < 0 || (int64_t)stream[j] >= V)) { status = PSO_BAD_TOKEN; break; }
            int32_t top;
            status = pso_argmax_row(pso_row(model_rows[l], dtype, V, j), dtype, V, &top);
            if (status) break;
            if (j < m && stream[j] == top) { a += 1; continue; }
            next = top;                          /* first mismatch, or the bonus row */
            break;
        }
        if (status) break;
        accepted_len[l] = a;
        block_len[l] = m;
        out_len[l] = a + 1;
        int32_t* out = out_tokens + (size_t)l * (kmax + 1);
        for (int j = 0; j < a; ++j) out[j] = stream[j];
        out[a] = next;
        stream[a] = next;
        stream_len = a + 1;
    }
    free(stream);
    return status;
}
