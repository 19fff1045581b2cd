/*
 * polyspec.h -- C ABI of libpolyspec: the chained speculative-sampling verification
 * step of polybasic speculative decoding, as CUDA kernels for sm_100a.
 *
 * Vocabulary of the paper (Section 3.1, Problem Formulation): a chain of models
 * M_1 (the target) ... M_n (the smallest drafter); p_i(x | x_<=t) is model i's
 * distribution over the vocabulary at a position; M_n drafts a block of tokens that is
 * checked bottom-up, by M_{n-1} first and M_1 last; the acceptance length of a
 * verifier (Eq. 1) is the number of consecutive block tokens it accepts.  A *level* is
 * one adjacent pair: verifier M_l checking the token stream handed up by M_{l+1}.
 *
 * The rule at a level (Algorithm 1: Verify in the inner loop with a break at the first
 * failure, then VerifyBlock / SampleOne for the level above; the rule itself is
 * speculative sampling, Sections 2 and 3.1):
 *   P_j = softmax(logits_p[j] / T), Q_j = softmax(logits_q[j] / T);
 *   position j is accepted iff  u_j * Q_j(x_j) <= P_j(x_j)   (u_j <= min(1, P/Q));
 *   accepted_len = a = number of accepted positions before the first rejection;
 *   next_token   = inverse CDF at the sampling uniform of
 *                    normalised max(0, P_{a+1} - Q_{a+1})   if a < block_len (residual)
 *                    P_{block_len+1}                         if a = block_len (bonus row),
 *                  in ascending vocabulary order, first v whose running sum exceeds u * total.
 * The emitted stream (x_1..x_a, next_token) is what the next level up verifies, with
 * that level's q = this level's verifier rows.
 *
 * Conventions for every call
 *   - All pointers are DEVICE pointers owned by the caller unless a parameter says
 *     "host".  Logits buffers must be 16-byte aligned and V must be a multiple of 8 (the
 *     kernels read logits eight at a time; other V return POLYSPEC_ERR_UNSUPPORTED).
 *     Row-major, innermost dimension = vocabulary.
 *   - Calls only enqueue work on `cuda_stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and return; outputs are valid once the stream has synchronised.
 *   - The library allocates no device memory: the caller passes a workspace of at least
 *     the size the matching *_workspace call reports, 256-byte aligned.  Concurrent calls
 *     need distinct workspaces.
 *   - Uniforms are caller-supplied floats in the open interval (0, 1); the library draws
 *     no random numbers.  Outputs are a pure function of the inputs.
 *   - Problems visible on the host (NULL pointers, sizes out of range, misalignment,
 *     temperature <= 0 or not finite, workspace too small) return an error status and
 *     launch nothing.  Problems only visible on the device (a token outside [0, V), a row
 *     holding NaN / +inf or no finite logit) never trap: the affected sequence gets
 *     accepted_len = next_token = -1 (and -1 in every later level of a chain) and
 *     *device_status is set to POLYSPEC_ERR_BAD_INPUT_ON_DEVICE.
 *   - No kernel polls memory without a limit.  The kernels of the logits path wait on nothing but
 *     hardware barriers (block, cluster, grid dependency) that every participant reaches
 *     unconditionally.  The LM-head projection waits on its TMA copies and on the tensor core with
 *     bounded polls: should one ever run out, *device_status becomes POLYSPEC_ERR_TIMEOUT, the
 *     outputs of that call are undefined, and the kernel still returns.
 */
#ifndef POLYSPEC_H
#define POLYSPEC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define POLYSPEC_MAX_K       32   /* largest block a level may verify */
#define POLYSPEC_MAX_MODELS   8   /* largest chain */

typedef enum {
    POLYSPEC_OK = 0,
    POLYSPEC_ERR_INVALID_ARG = 1,
    POLYSPEC_ERR_UNSUPPORTED = 2,
    POLYSPEC_ERR_WORKSPACE = 3,
    POLYSPEC_ERR_CUDA = 4,
    POLYSPEC_ERR_TIMEOUT = 5,
    POLYSPEC_ERR_BAD_INPUT_ON_DEVICE = 6,
    POLYSPEC_ERR_SCRATCH_LIMIT = 7      /* problem too large for the built-in scratch of a *_static call */
} polyspec_status;

typedef enum { POLYSPEC_F32 = 0, POLYSPEC_BF16 = 1 } polyspec_dtype;

/* Static strings; never NULL. */
const char* polyspec_status_string(polyspec_status s);
/* major * 10000 + minor * 100 + patch */
int polyspec_version(void);
/* The CUDA runtime's message for the most recent call that returned POLYSPEC_ERR_CUDA ("no error" if none did).
 * Static string; not synchronised between host threads. */
const char* polyspec_last_cuda_error(void);

/*
 * polyspec_verify_level -- one adjacent pair (verifier p, drafter-side q) over a batch of
 * independent sequences: Algorithm 1's Verify loop plus the replacement / bonus token.
 *
 *   logits_p      [B, k+1, V]  verifier logits; row j scores block position j, row k is the bonus row
 *   logits_q      [B, k,   V]  logits of the distribution the block tokens were drawn from
 *   draft_tokens  [B, k]       block tokens, each in [0, V)
 *   uniforms      [B, k+1]     [b, j<k] accept uniform of position j; [b, k] the sampling uniform
 *   block_len     [B] or NULL  tokens actually presented per sequence (0..k); NULL means k
 *   accepted_len  out [B]      0..block_len[b]
 *   next_token    out [B]      residual sample if accepted_len < block_len, else bonus sample
 *   p_at_draft, q_at_draft  out [B, k] or NULL: P_j(x_j), Q_j(x_j) for j < block_len, 0 elsewhere
 *   device_status out [1] or NULL: left untouched when all is well (zero it before the call)
 */
polyspec_status polyspec_verify_level_workspace(int B, int k, int V, polyspec_dtype dt, size_t* bytes /* host out */);
polyspec_status polyspec_verify_level(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms,
    const int32_t* block_len, int B, int k, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * polyspec_verify_chain -- n models, n-1 levels, verified bottom-up in one call
 * (Section 3.1; Algorithm 1 is the n = 3 case).  Level index l = 0 .. n-2: verifier is
 * models[l]; models[0] = M_1 (target), models[n-1] = M_n (bottom drafter).
 *
 *   models        host array [n_models]: device pointer to [B, rows, V] logits and its row
 *                 count; rows >= k[l] + 1 for l < n-1, rows >= k[n-2] for the drafter
 *   k             host [n_models-1]; k[l] = largest block level l verifies; k[n-2] = draft length
 *   draft_tokens  [B, k[n-2]]
 *   uniforms      [n_models-1, B, kmax+1], kmax = max k[l]; level l uses [l, b, j < k[l]] for
 *                 its accept tests and [l, b, kmax] as its sampling uniform
 *   Level l verifies the first min(k[l], out_len[l+1]) tokens of the stream emitted by
 *   level l+1 against q = models[l+1]'s rows.
 *   accepted_len, block_len, out_len   out [n_models-1, B]; out_len = accepted_len + 1
 *   out_tokens    out [n_models-1, B, kmax+1]: stream emitted by each level, -1 past out_len;
 *                 level 0's stream is the committed output
 */
typedef struct {
    const void* logits;   /* device pointer, [B, rows, V] */
    int rows;
} polyspec_model_logits;

polyspec_status polyspec_verify_chain_workspace(int n_models, const int* k /* host */, const int* rows /* host [n_models] */,
                                                int B, int V, polyspec_dtype dt, size_t* bytes /* host out */);
polyspec_status polyspec_verify_chain(
    const polyspec_model_logits* models /* host */, int n_models, const int* k /* host */,
    const int32_t* draft_tokens, const float* uniforms, int B, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens, int32_t* out_len,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The two halves of polyspec_verify_chain, for callers that want to time or overlap them:
 *   polyspec_chain_row_stats  the temperature-softmax normaliser of every row of every model
 *                             (the single pass over all logits; Section 3.1's p_i over the
 *                             vocabulary) written to the workspace;
 *   polyspec_chain_walk       everything after it (Algorithm 1's accept loop, first rejection,
 *                             replacement / bonus token, hand-off between levels), reading the
 *                             workspace the first half filled on the same stream.
 * Calling one after the other with the same arguments is exactly polyspec_verify_chain.
 */
polyspec_status polyspec_chain_row_stats(
    const polyspec_model_logits* models /* host */, int n_models, const int* k /* host */, int B, int V,
    polyspec_dtype dt, float temperature, int32_t* device_status, void* workspace, size_t workspace_bytes,
    void* cuda_stream);
polyspec_status polyspec_chain_walk(
    const polyspec_model_logits* models /* host */, int n_models, const int* k /* host */,
    const int32_t* draft_tokens, const float* uniforms, int B, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens, int32_t* out_len,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * polyspec_verify_chain_host -- the same call for a caller whose buffers live in HOST
 * memory (pinned memory makes the copies asynchronous): logits, draft tokens and
 * uniforms are copied to a device staging area inside the caller's workspace, the chain
 * runs, and the four outputs are copied back, all on `cuda_stream`.  Every data pointer
 * here is a host pointer with the layouts above; `host_status` (host, [1], may be NULL)
 * receives the device status word.  Outputs are valid after the stream synchronises.
 */
polyspec_status polyspec_verify_chain_host_workspace(int n_models, const int* k, const int* rows, int B, int V,
                                                     polyspec_dtype dt, size_t* bytes /* host out */);
polyspec_status polyspec_verify_chain_host(
    const polyspec_model_logits* models_host /* host array of HOST logits pointers */, int n_models, const int* k,
    const int32_t* draft_tokens_host, const float* uniforms_host, int B, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len_host, int32_t* block_len_host, int32_t* out_tokens_host, int32_t* out_len_host,
    int32_t* host_status, void* workspace /* device */, size_t workspace_bytes, void* cuda_stream);

/*
 * polyspec_verify_from_hidden -- polyspec_verify_level with the LM-head projection fused
 * in front (the last op of the model forwards in Algorithm 1, "p_{1:K} <- M_2(...)" and
 * "v <- M_1(...)"): logits[b, j, v] = sum_d hidden[b, j, d] * W[v, d], bf16 inputs,
 * fp32 accumulation on the tensor cores; logits are never passed in.
 *
 *   hidden_p [B, k+1, d_p] bf16, W_p [V, d_p] bf16 (row-major, d contiguous)
 *   hidden_q [B, rows_q, d_q] bf16 with rows_q = k or k + 1 (a row k is projected but not used), W_q [V, d_q] bf16
 *   d_p, d_q multiples of 64; V a multiple of 8; all four buffers 16-byte aligned
 *   the remaining arguments are those of polyspec_verify_level
 */
polyspec_status polyspec_verify_from_hidden_workspace(int B, int k, int V, int d_p, int d_q, size_t* bytes /* host out */);
polyspec_status polyspec_verify_from_hidden(
    const void* hidden_p, const void* W_p, const void* hidden_q, const void* W_q, int rows_q,
    const int32_t* draft_tokens, const float* uniforms, const int32_t* block_len,
    int B, int k, int V, int d_p, int d_q, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * polyspec_verify_chain_greedy -- the chain under greedy matching, the other verification rule
 * Section 3.1 names and Section 4.5 compares with speculative sampling: a block token is accepted
 * iff it is the verifier's most likely token at its position (first index on ties), the loop breaks
 * at the first mismatch, and the token emitted after the accepted prefix is the verifier's most
 * likely token there (at the first mismatch, or in the bonus row after a fully accepted block).
 * No uniforms, no temperature; the emitted stream of a level is that verifier's own greedy text.
 *
 *   models, k, draft_tokens and the four outputs are those of polyspec_verify_chain; only the
 *   verifiers models[0 .. n_models-2] are read (rows >= k[l] + 1); models[n_models-1].logits may be
 *   NULL.  One pass over the verifiers' logits, no second pass.
 */
polyspec_status polyspec_verify_chain_greedy_workspace(int n_models, const int* k /* host */, const int* rows /* host [n_models] */,
                                                       int B, int V, polyspec_dtype dt, size_t* bytes /* host out */);
polyspec_status polyspec_verify_chain_greedy(
    const polyspec_model_logits* models /* host */, int n_models, const int* k /* host */, const int32_t* draft_tokens,
    int B, int V, polyspec_dtype dt,
    int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens, int32_t* out_len,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The two halves of polyspec_verify_from_hidden, for callers that want to time or overlap them:
 *   polyspec_from_hidden_project  both LM-head projections (one launch): logits and, from the same
 *                                 accumulators, every row's softmax-normaliser partials into the workspace;
 *   polyspec_from_hidden_verify   everything after it, reading the workspace the first half filled
 *                                 on the same stream.
 * Calling one after the other with the same sizes and workspace is exactly polyspec_verify_from_hidden.
 */
polyspec_status polyspec_from_hidden_project(
    const void* hidden_p, const void* W_p, const void* hidden_q, const void* W_q, int rows_q,
    int B, int k, int V, int d_p, int d_q, float temperature, int32_t* device_status, void* workspace, size_t workspace_bytes,
    void* cuda_stream);
polyspec_status polyspec_from_hidden_verify(
    int rows_q, const int32_t* draft_tokens, const float* uniforms, const int32_t* block_len,
    int B, int k, int V, int d_p, int d_q, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * polyspec_lm_head -- the projection of polyspec_verify_from_hidden on its own (the last op
 * of a model forward in Algorithm 1): logits[r, v] = sum_d hidden[r, d] * W[v, d].
 *
 *   hidden  [rows, d] bf16, W [V, d] bf16, both row-major and 16-byte aligned; d a multiple of 64,
 *           V a multiple of 4
 *   logits  out [rows, V] fp32, 16-byte aligned
 *   No workspace.  device_status as above (only POLYSPEC_ERR_TIMEOUT can be reported here).
 */
polyspec_status polyspec_lm_head(const void* hidden, const void* W, int rows, int V, int d, float* logits,
                                 int32_t* device_status, void* cuda_stream);

/*
 * polyspec_verify_level with the vocabulary sharded over n_ranks ranks (the layout a tensor-parallel
 * LM head leaves the logits in): rank r holds entries [r * V_local, (r + 1) * V_local) of every row,
 * as logits_p [B, k+1, V_local] and logits_q [B, k, V_local]; the rule is Algorithm 1's Verify loop
 * and replacement / bonus token over the whole vocabulary V = n_ranks * V_local, unchanged.
 * The normaliser, the accept tests and the inverse-CDF search need sums over all slices, so a level
 * is three calls per rank with two small exchanges and one reduction between them, which the caller
 * performs (all-gather, all-gather, max); the library itself never talks to another rank:
 *
 *   polyspec_sharded_level_stats   writes this rank's stats record (stats_record_bytes)
 *        -- all-gather the records into [n_ranks][stats_record_bytes], rank order --
 *   polyspec_sharded_level_decide  accept tests on every rank (identical results): accepted_len [B];
 *                                  writes this rank's mass record (mass_record_bytes)
 *        -- all-gather the mass records into [n_ranks][mass_record_bytes] --
 *   polyspec_sharded_level_pick    next_token [B]: the token (index in the whole vocabulary) on the one
 *                                  rank whose slice contains it, -1 on the others
 *        -- max over ranks of next_token --
 *
 *   draft_tokens [B, k] hold indices in the whole vocabulary; uniforms, block_len, accepted_len,
 *   p_at_draft, q_at_draft, temperature and device_status are those of polyspec_verify_level and must be
 *   the same on every rank.  The three calls of a level share one workspace, whose contents carry from
 *   call to call; records are opaque, 16-byte aligned device buffers.  V_local a multiple of 8,
 *   n_ranks <= 64.  An unusable input gives accepted_len = next_token = -1 on every rank.
 *   With n_ranks = 1 the result is bit-identical to polyspec_verify_level.
 */
polyspec_status polyspec_sharded_level_sizes(int B, int k, int V_local, polyspec_dtype dt, int n_ranks,
                                             size_t* workspace_bytes, size_t* stats_record_bytes,
                                             size_t* mass_record_bytes /* host out, all three */);
polyspec_status polyspec_sharded_level_stats(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, int B, int k, int V_local, int rank, int n_ranks,
    polyspec_dtype dt, float temperature, void* stats_record /* out */, int32_t* device_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream);
polyspec_status polyspec_sharded_level_decide(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms, const int32_t* block_len,
    int B, int k, int V_local, int rank, int n_ranks, polyspec_dtype dt, float temperature,
    const void* stats_records /* all ranks' */, int32_t* accepted_len, float* p_at_draft, float* q_at_draft,
    void* mass_record /* out */, int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);
polyspec_status polyspec_sharded_level_pick(
    const void* logits_p, const void* logits_q, const float* uniforms, int B, int k, int V_local, int rank, int n_ranks,
    polyspec_dtype dt, float temperature, const void* mass_records /* all ranks' */, int32_t* next_token,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * polyspec_verify_chain with the vocabulary sharded over n_ranks ranks: every model's logits as
 * [B, rows, V_local] slices (models[i].logits, models[i].rows as in polyspec_verify_chain), levels verified
 * bottom-up (Section 3.1).  One stats call covers every row of every model; each level then takes a
 * gather call (the logits at its block tokens, which only exist once the level below is done), decide
 * and pick as in the single-level calls, and a hand-off that turns (accepted length, token) into the
 * block of the level above.  Per chain: all-gather of the stats records; per level, for
 * level = n_models-2 down to 0: all-gather of the gather records, all-gather of the mass records, max of
 * next_token, then polyspec_sharded_chain_handoff on every rank.
 *
 *   block_tokens [B, kmax+1], block_len [B]: the block the current level verifies, the same on every
 *       rank; the caller fills them with the draft tokens and k[n_models-2] (or fewer) before the
 *       bottom level, the hand-off rewrites them for the level above (block_len -1: unusable input below)
 *   uniforms [n_models-1, B, kmax+1], accepted_len, block_len_out, out_tokens, out_len: those of
 *       polyspec_verify_chain (block_len_out is its block_len output); each call touches its level's part
 *   With n_ranks = 1 the four outputs are bit-identical to polyspec_verify_chain's.
 */
polyspec_status polyspec_sharded_chain_sizes(int n_models, const int* k /* host */, const int* rows /* host [n_models] */, int B,
                                             int V_local, polyspec_dtype dt, int n_ranks, size_t* workspace_bytes,
                                             size_t* stats_record_bytes, size_t* gather_record_bytes,
                                             size_t* mass_record_bytes /* host out, all four */);
polyspec_status polyspec_sharded_chain_stats(
    const polyspec_model_logits* models /* host */, int n_models, const int* k /* host */, int B, int V_local, int rank, int n_ranks,
    polyspec_dtype dt, float temperature, void* stats_record /* out */, int32_t* device_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream);
polyspec_status polyspec_sharded_chain_gather(
    const polyspec_model_logits* models, int n_models, const int* k, int level, const int32_t* block_tokens, const int32_t* block_len,
    int B, int V_local, int rank, int n_ranks, polyspec_dtype dt, void* gather_record /* out */,
    void* workspace, size_t workspace_bytes, void* cuda_stream);
polyspec_status polyspec_sharded_chain_decide(
    const polyspec_model_logits* models, int n_models, const int* k, int level, const int32_t* block_tokens, const int32_t* block_len,
    const float* uniforms, int B, int V_local, int rank, int n_ranks, polyspec_dtype dt, float temperature,
    const void* stats_records /* all ranks' */, const void* gather_records /* all ranks' */, int32_t* accepted_len,
    int32_t* block_len_out, void* mass_record /* out */, int32_t* device_status, void* workspace, size_t workspace_bytes,
    void* cuda_stream);
polyspec_status polyspec_sharded_chain_pick(
    const polyspec_model_logits* models, int n_models, const int* k, int level, const float* uniforms, int B, int V_local, int rank,
    int n_ranks, polyspec_dtype dt, float temperature, const void* mass_records /* all ranks' */, int32_t* next_token /* [B] */,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);
polyspec_status polyspec_sharded_chain_handoff(
    int n_models, const int* k, int level, int B, const int32_t* accepted_len, const int32_t* next_token /* after the max */,
    int32_t* block_tokens /* in/out */, int32_t* block_len /* in/out */, int32_t* out_tokens, int32_t* out_len, void* cuda_stream);

/*
 * Cost model of Section 3.2 (host arithmetic only; nothing is launched).
 *
 * polyspec_cost_total_time -- Lemma 3.1 (Eq. 3): the time to generate N tokens with n models,
 *     T = sum_{i=1}^{n-1} (N / L_i) T_i + beta (N / L_{n-1}) T_n,
 *   T[0..n-1] the forward-pass costs T_1..T_n, L[0..n-2] the acceptance lengths L_1..L_{n-1} (Eq. 1:
 *   what polyspec_verify_chain reports as accepted_len, averaged), beta the drafter's scaling factor.
 *   Returns NaN for n < 2, a NULL array or a non-positive L.
 * polyspec_cost_insertion -- Theorem 3.2, first condition, with the quantities of Table 1: inserting
 *   M_new between M_i and M_{i+1} pays off iff
 *     T_new / T_i  <  L_new (1 / L_i - 1 / L_{i-new}),
 *   L_i the acceptance length of the pair (M_i, M_{i+1}) before the insertion, L_{i-new} that of
 *   (M_i, M_new) and L_new that of (M_new, M_{i+1}) after it.  Writes both sides (either pointer may be
 *   NULL) and returns 1 if the condition holds, 0 if not, -1 on non-positive inputs.
 * polyspec_cost_insertion_drafter -- Theorem 3.2, second condition, as its proof derives it (the three-model
 *   case, M_new between M_i and the drafter M_{i+1}): the insertion also pays off if
 *     T_new / T_{i+1}  <  beta (L_new / L_i - 1),
 *   the sign of the last two terms of the difference of the two Lemma 3.1 totals; L_new and L_i as above,
 *   T_{i+1} the drafter's forward-pass cost, beta its scaling factor (Lemma 3.1).  The theorem's statement
 *   prints other subscripts for this condition; the proof's are used.  Same outputs and return values.
 */
double polyspec_cost_total_time(int n, const double* T /* host [n] */, const double* L /* host [n-1] */, double beta, double N);
int polyspec_cost_insertion(double T_new, double T_i, double L_new, double L_i, double L_i_new,
                            double* lhs /* host out */, double* rhs /* host out */);
int polyspec_cost_insertion_drafter(double T_new, double T_next, double L_new, double L_i, double beta,
                                    double* lhs /* host out */, double* rhs /* host out */);

/*
 * Staged verification with a threshold (Section 3.3, "Staged Verification"; Algorithm 1, three models)
 * for a batch of independent sequences.  Algorithm 1's loop: M_3 drafts K tokens, M_2 verifies them, what
 * M_2 hands on joins `accepted` (count `cnt`); once cnt >= mu, M_1 verifies the accumulated block in one
 * pass, the verified part is committed, t advances, `accepted` and cnt are reset.  Each M_2 round hands on
 * its whole emitted stream (accepted prefix plus the replacement or bonus token), which is distributed as
 * M_2's own samples, so the pass of M_1 verifies it against q = M_2's rows and the committed text keeps
 * M_1's distribution; a round therefore always adds a token.  Accumulation also stops when one more round
 * might not fit the largest block a level verifies (cnt + K + 1 > POLYSPEC_MAX_K).
 *
 * The two verifications of an iteration are ordinary polyspec_verify_level calls (per-sequence block_len);
 * these calls keep the loop's bookkeeping on the device, so that the loop needs no host read-back per step:
 *
 *   polyspec_staged_init          zeroes the state, remaining = B
 *   per iteration of Algorithm 1's loop, for all sequences at once:
 *     polyspec_staged_round_begin   -> pos2 [B] (= t + cnt), tokens2 [B, K] (M_3's drafts there), uniforms2 [B, K+1],
 *                                      block_len2 [B] (K, or 0 for a sequence that is finished)
 *       -- caller: logits of M_2 at positions pos2 .. pos2+K and of M_3 at pos2 .. pos2+K-1 (the model forwards),
 *          then polyspec_verify_level(M_2 rows, M_3 rows, tokens2, uniforms2, block_len2) -> accepted_len2, next_token2 --
 *     polyspec_staged_accumulate    appends each round's stream; where cnt >= mu (or the block is full): pos1 [B] (= t),
 *                                      tokens1 [B, kcap] (= accepted), uniforms1 [B, kcap+1], block_len1 [B] (= cnt);
 *                                      block_len1 = 0 elsewhere
 *       -- caller: logits of M_1 at pos1 .. pos1+kcap and of M_2 at pos1 .. pos1+kcap-1, then
 *          polyspec_verify_level(M_1 rows, M_2 rows, tokens1, uniforms1, block_len1) -> accepted_len1, next_token1 --
 *     polyspec_staged_commit        where block_len1 > 0: commits accepted[0 .. a1) and M_1's token, t += a1 + 1,
 *                                      cnt = 0; a sequence with n_tokens committed is finished
 *   *remaining (device) counts the sequences still running; a sequence needs at most mu iterations per pass of M_1,
 *   so reading it back once every mu iterations is at most one read-back per pass.
 *
 *   drafts [B, N] int32: M_3's proposal per position (synthetic stand-in: position-indexed);
 *   u2 [B, R, K+1]: row r serves a sequence's r-th round; u1 [B, C, POLYSPEC_MAX_K+1]: row c serves its c-th pass of
 *   M_1, slots 0..m-1 the accept tests, slot POLYSPEC_MAX_K the sampling uniform.
 *   State arrays (device, caller-owned): t, cnt, rounds, cycles, n_committed, done [B]; accepted [B, POLYSPEC_MAX_K];
 *   committed [B, cap] (-1 where nothing was committed); presented, per_cycle [B, C] (block length and tokens
 *   committed of each pass); remaining [1].  kcap >= min(POLYSPEC_MAX_K, mu + K).  done: 0 running, else a
 *   POLYSPEC_STAGED_* code (EXHAUSTED: out of positions N, of uniform rows R / C; BAD_INPUT: a level call reported -1).
 */
#define POLYSPEC_STAGED_FINISHED  1
#define POLYSPEC_STAGED_EXHAUSTED 2
#define POLYSPEC_STAGED_BAD_INPUT 3
typedef struct {
    int B, K, mu, kcap, N, R, C, cap, n_tokens;
    int32_t *t, *cnt, *rounds, *cycles, *n_committed, *done;
    int32_t *accepted, *committed, *presented, *per_cycle, *remaining;
} polyspec_staged_state;
polyspec_status polyspec_staged_init(const polyspec_staged_state* s /* host */, void* cuda_stream);
polyspec_status polyspec_staged_round_begin(const polyspec_staged_state* s /* host */, const int32_t* drafts, const float* u2,
                                            int32_t* pos2, int32_t* tokens2, float* uniforms2, int32_t* block_len2, void* cuda_stream);
polyspec_status polyspec_staged_accumulate(const polyspec_staged_state* s /* host */, const int32_t* tokens2, const int32_t* block_len2,
                                           const int32_t* accepted_len2, const int32_t* next_token2, const float* u1,
                                           int32_t* pos1, int32_t* tokens1, float* uniforms1, int32_t* block_len1, void* cuda_stream);
polyspec_status polyspec_staged_commit(const polyspec_staged_state* s /* host */, const int32_t* block_len1, const int32_t* accepted_len1,
                                       const int32_t* next_token1, void* cuda_stream);

/*
 * polyspec_verify_level_static -- polyspec_verify_level without a workspace argument.
 * (The paper has no counterpart to this call; it exists for integration reasons only.)
 *
 * Some callers cannot give the library a workspace because they cannot allocate device
 * memory at the point where they verify: a plugin invoked from inside a serving engine
 * that owns every byte of the device, code running under a fixed post-start-up memory
 * budget, a callback in which cudaMalloc is forbidden.  For them the row-statistics
 * partials live in a fixed array of POLYSPEC_STATIC_SCRATCH_BYTES inside the library image
 * (each GPU that loads the library holds that much until the process exits).  The call
 * allocates nothing, neither through CUDA nor through any library.
 *
 *   - Inputs and outputs are the caller's, exactly as in polyspec_verify_level.
 *   - Limit: the call needs polyspec_verify_level_workspace(B, k, V, dt) bytes; if that
 *     exceeds POLYSPEC_STATIC_SCRATCH_BYTES it returns POLYSPEC_ERR_SCRATCH_LIMIT and launches
 *     nothing.  (1 MiB covers e.g. B = 256, k = 8, V = 152064 in bf16.)
 *   - The device that owns `cuda_stream` must be current.  The first call on each device
 *     looks up the device address of the array (a one-time set-up step); make that first
 *     call before starting any stream capture.
 *   - All calls on a device share the one array.  A call overwrites every entry it later
 *     reads, so leftovers from earlier calls do not matter, but two calls whose kernels
 *     overlap on the GPU (different streams) race: serialise them.
 */
#define POLYSPEC_STATIC_SCRATCH_BYTES (1u << 20)
size_t polyspec_static_scratch_bytes(void);
polyspec_status polyspec_verify_level_static(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms,
    const int32_t* block_len, int B, int k, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* POLYSPEC_H */
