// Staged verification with a threshold (Section 3.3, "Staged Verification"; Algorithm 1) for a batch of
// independent sequences: the bookkeeping of Algorithm 1's loop -- the accumulated block `accepted`, its count
// `cnt`, the committed length t, which uniforms come next -- kept on the device, one thread per sequence, so
// that the loop around the two level calls of an iteration needs no host read-back.  The verification rule
// itself is not here: each iteration's two polyspec_verify_level calls do that.
#include "polyspec_kernels.cuh"

namespace polyspec {
namespace {

constexpr int kMaxBlock = POLYSPEC_MAX_K;

// Inputs of the M_2 level call of this iteration: the K tokens M_3 drafted from position t + cnt on, the next
// row of M_2-round uniforms, block_len = K (0 for a sequence that sits this iteration out).
__global__ void staged_round_begin_kernel(polyspec_staged_state s, const int32_t* drafts, const float* u2,
                                          int32_t* pos2, int32_t* tokens2, float* uniforms2, int32_t* block_len2)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= s.B) return;
    const int K = s.K;
    int st = s.done[b];
    int pos = 0;
    if (st == 0) {
        pos = s.t[b] + s.cnt[b];
        if (pos + K + 1 > s.N || s.rounds[b] >= s.R) {        // out of positions or of uniforms
            st = POLYSPEC_STAGED_EXHAUSTED;
            s.done[b] = st;
            atomicSub(s.remaining, 1);
            pos = 0;
        }
    }
    const bool active = st == 0;
    pos2[b] = active ? pos : 0;
    block_len2[b] = active ? K : 0;
    for (int j = 0; j < K; ++j) tokens2[static_cast<size_t>(b) * K + j] = active ? drafts[static_cast<size_t>(b) * s.N + pos + j] : 0;
    const float* u = u2 + (static_cast<size_t>(b) * s.R + (active ? s.rounds[b] : 0)) * (K + 1);
    for (int j = 0; j <= K; ++j) uniforms2[static_cast<size_t>(b) * (K + 1) + j] = u[j];
}

// After the M_2 level call: the round's whole emitted stream (accepted prefix and the replacement / bonus token) joins
// `accepted`; where cnt has reached the threshold -- or one more round might not fit a block -- the inputs of the M_1
// level call are laid out (block = accepted, q = M_2's rows from position t on), block_len = cnt; elsewhere block_len = 0.
__global__ void staged_accumulate_kernel(polyspec_staged_state s, const int32_t* tokens2, const int32_t* block_len2,
                                         const int32_t* accepted_len2, const int32_t* next_token2, const float* u1,
                                         int32_t* pos1, int32_t* tokens1, float* uniforms1, int32_t* block_len1)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= s.B) return;
    const int K = s.K, kcap = s.kcap;
    int32_t* acc = s.accepted + static_cast<size_t>(b) * kMaxBlock;
    int st = s.done[b];
    int cnt = s.cnt[b];
    if (st == 0 && block_len2[b] == K) {
        const int a2 = accepted_len2[b];
        if (a2 < 0 || a2 > K) {                                // the level call met unusable input
            st = POLYSPEC_STAGED_BAD_INPUT;
        } else {
            for (int j = 0; j < a2; ++j) acc[cnt + j] = tokens2[static_cast<size_t>(b) * K + j];
            acc[cnt + a2] = next_token2[b];
            cnt += a2 + 1;
            s.cnt[b] = cnt;
            s.rounds[b] += 1;
        }
    }
    bool verify = st == 0 && (cnt >= s.mu || cnt + K + 1 > kMaxBlock);
    if (verify && (s.cycles[b] >= s.C || s.t[b] + cnt + 1 > s.N || cnt > kcap)) {
        st = POLYSPEC_STAGED_EXHAUSTED;
        verify = false;
    }
    if (st != 0 && s.done[b] == 0) {
        s.done[b] = st;
        atomicSub(s.remaining, 1);
    }
    pos1[b] = st == 0 ? s.t[b] : 0;
    block_len1[b] = verify ? cnt : 0;
    const float* u = u1 + (static_cast<size_t>(b) * s.C + (verify ? s.cycles[b] : 0)) * (kMaxBlock + 1);
    for (int j = 0; j < kcap; ++j) {
        tokens1[static_cast<size_t>(b) * kcap + j] = (verify && j < cnt) ? acc[j] : 0;
        uniforms1[static_cast<size_t>(b) * (kcap + 1) + j] = u[j];
    }
    uniforms1[static_cast<size_t>(b) * (kcap + 1) + kcap] = u[kMaxBlock];       // the pass's sampling uniform
}

// After the M_1 level call: the verified prefix and M_1's token are committed, t advances, `accepted` and cnt are reset.
__global__ void staged_commit_kernel(polyspec_staged_state s, const int32_t* block_len1, const int32_t* accepted_len1,
                                     const int32_t* next_token1)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= s.B) return;
    const int m = block_len1[b];
    if (s.done[b] != 0 || m <= 0) return;
    const int a1 = accepted_len1[b];
    if (a1 < 0 || a1 > m) {
        s.done[b] = POLYSPEC_STAGED_BAD_INPUT;
        atomicSub(s.remaining, 1);
        return;
    }
    const int32_t* acc = s.accepted + static_cast<size_t>(b) * kMaxBlock;
    int32_t* text = s.committed + static_cast<size_t>(b) * s.cap;
    int n = s.n_committed[b];
    for (int j = 0; j <= a1; ++j)
        if (n + j < s.cap) text[n + j] = j < a1 ? acc[j] : next_token1[b];
    n += a1 + 1;
    const int c = s.cycles[b];
    s.presented[static_cast<size_t>(b) * s.C + c] = m;
    s.per_cycle[static_cast<size_t>(b) * s.C + c] = a1 + 1;
    s.cycles[b] = c + 1;
    s.n_committed[b] = n;
    s.t[b] += a1 + 1;
    s.cnt[b] = 0;
    if (n >= s.n_tokens) {
        s.done[b] = POLYSPEC_STAGED_FINISHED;
        atomicSub(s.remaining, 1);
    }
}

polyspec_status check_state(const polyspec_staged_state* s)
{
    if (!s) return POLYSPEC_ERR_INVALID_ARG;
    if (s->B <= 0 || s->K < 1 || s->K > kMaxBlock - 1 || s->mu < 1 || s->mu > kMaxBlock || s->N <= 0 || s->R <= 0 || s->C <= 0 ||
        s->cap <= 0 || s->n_tokens <= 0)
        return POLYSPEC_ERR_INVALID_ARG;
    const int need = s->mu + s->K < kMaxBlock ? s->mu + s->K : kMaxBlock;       // the longest block a pass can be handed
    if (s->kcap < need || s->kcap > kMaxBlock) return POLYSPEC_ERR_INVALID_ARG;
    if (!s->t || !s->cnt || !s->rounds || !s->cycles || !s->n_committed || !s->done || !s->accepted || !s->committed ||
        !s->presented || !s->per_cycle || !s->remaining)
        return POLYSPEC_ERR_INVALID_ARG;
    return POLYSPEC_OK;
}

}  // namespace
}  // namespace polyspec

using namespace polyspec;

extern "C" {

polyspec_status polyspec_staged_init(const polyspec_staged_state* s, void* cuda_stream)
{
    polyspec_status st = check_state(s);
    if (st != POLYSPEC_OK) return st;
    cudaStream_t q = static_cast<cudaStream_t>(cuda_stream);
    const size_t nb = static_cast<size_t>(s->B) * sizeof(int32_t);
    int32_t* zeroed[6] = {s->t, s->cnt, s->rounds, s->cycles, s->n_committed, s->done};
    for (int32_t* p : zeroed)
        if (cuda_failed(cudaMemsetAsync(p, 0, nb, q))) return POLYSPEC_ERR_CUDA;
    if (cuda_failed(cudaMemsetAsync(s->accepted, 0, nb * kMaxBlock, q))) return POLYSPEC_ERR_CUDA;
    if (cuda_failed(cudaMemsetAsync(s->committed, 0xff, nb * s->cap, q))) return POLYSPEC_ERR_CUDA;      // -1
    if (cuda_failed(cudaMemsetAsync(s->presented, 0, nb * s->C, q))) return POLYSPEC_ERR_CUDA;
    if (cuda_failed(cudaMemsetAsync(s->per_cycle, 0, nb * s->C, q))) return POLYSPEC_ERR_CUDA;
    const int32_t B = s->B;
    if (cuda_failed(cudaMemcpyAsync(s->remaining, &B, sizeof B, cudaMemcpyHostToDevice, q))) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

polyspec_status polyspec_staged_round_begin(const polyspec_staged_state* s, const int32_t* drafts, const float* u2,
                                            int32_t* pos2, int32_t* tokens2, float* uniforms2, int32_t* block_len2, void* cuda_stream)
{
    polyspec_status st = check_state(s);
    if (st != POLYSPEC_OK) return st;
    if (!drafts || !u2 || !pos2 || !tokens2 || !uniforms2 || !block_len2) return POLYSPEC_ERR_INVALID_ARG;
    staged_round_begin_kernel<<<(s->B + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(*s, drafts, u2, pos2, tokens2,
                                                                                                     uniforms2, block_len2);
    return cuda_failed(cudaGetLastError()) ? POLYSPEC_ERR_CUDA : POLYSPEC_OK;
}

polyspec_status polyspec_staged_accumulate(const polyspec_staged_state* s, const int32_t* tokens2, const int32_t* block_len2,
                                           const int32_t* accepted_len2, const int32_t* next_token2, const float* u1,
                                           int32_t* pos1, int32_t* tokens1, float* uniforms1, int32_t* block_len1, void* cuda_stream)
{
    polyspec_status st = check_state(s);
    if (st != POLYSPEC_OK) return st;
    if (!tokens2 || !block_len2 || !accepted_len2 || !next_token2 || !u1 || !pos1 || !tokens1 || !uniforms1 || !block_len1)
        return POLYSPEC_ERR_INVALID_ARG;
    staged_accumulate_kernel<<<(s->B + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        *s, tokens2, block_len2, accepted_len2, next_token2, u1, pos1, tokens1, uniforms1, block_len1);
    return cuda_failed(cudaGetLastError()) ? POLYSPEC_ERR_CUDA : POLYSPEC_OK;
}

polyspec_status polyspec_staged_commit(const polyspec_staged_state* s, const int32_t* block_len1, const int32_t* accepted_len1,
                                       const int32_t* next_token1, void* cuda_stream)
{
    polyspec_status st = check_state(s);
    if (st != POLYSPEC_OK) return st;
    if (!block_len1 || !accepted_len1 || !next_token1) return POLYSPEC_ERR_INVALID_ARG;
    staged_commit_kernel<<<(s->B + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(*s, block_len1, accepted_len1, next_token1);
    return cuda_failed(cudaGetLastError()) ? POLYSPEC_ERR_CUDA : POLYSPEC_OK;
}

}  // extern "C"
