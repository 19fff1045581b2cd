// Greedy matching (the other verification rule Section 3.1 names, compared with speculative
// sampling in Section 4.5): a block token is accepted iff it is the verifier's most likely token
// at its position, the loop breaks at the first mismatch (Algorithm 1's Verify loop), and the token
// emitted after the accepted prefix is the verifier's most likely token there -- at the first
// mismatch, or in the bonus row after a fully accepted block.
//
// The pass over the logits (arg max of every verifier row) is the row-statistics kernel in its
// arg-max mode; this kernel is the rest: one CTA of four warps per sequence merges the arg-max
// partials of the rows a level needs, compares them with the block, writes the level's outputs
// and hands the emitted stream to the level above.  No logits are read here, nothing waits.
#include "polyspec_kernels.cuh"

namespace polyspec {
namespace {

constexpr int kGreedyThreads = 128;
constexpr int kGreedyWarps = kGreedyThreads / 32;

// Arg max of one row from its partials (value, first index as int bits; -1 marks a segment with NaN
// or +inf): larger value wins, equal values go to the lower index.  Returns -1 for an unusable row
// (a marked segment, or no finite logit at all).  Every lane returns the same result.
__device__ __forceinline__ int merge_argmax(const float2* part, int parts, int lane)
{
    float best = -INFINITY;
    int at = 0x7fffffff;
    bool marked = false;
    for (int i = lane; i < parts; i += 32) {
        const float2 ps = part[i];
        const int a = __float_as_int(ps.y);
        marked |= a < 0;
        if (ps.x > best || (ps.x == best && a < at)) { best = ps.x; at = a; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oa = __shfl_xor_sync(0xffffffffu, at, o);
        if (ov > best || (ov == best && oa < at)) { best = ov; at = oa; }
    }
    marked = __any_sync(0xffffffffu, marked);
    return (marked || best == -INFINITY) ? -1 : at;
}

__global__ void __launch_bounds__(kGreedyThreads) greedy_walk_kernel(const WalkParams p)
{
    __shared__ int tok[kMaxK + 2];
    __shared__ int top[kMaxK + 1];      // arg max of the verifier's rows 0..m, -1 if unusable
    __shared__ int sh_a, sh_next, sh_bad;

    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = p.n_levels;

    int stream_len = p.k[L - 1];
    if (p.bottom_len) stream_len = max(0, min(stream_len, p.bottom_len[b]));
    if (tid < p.k[L - 1]) tok[tid] = p.draft_tokens[static_cast<size_t>(b) * p.k[L - 1] + tid];
    __syncthreads();

    bool dead = false;
    for (int l = L - 1; l >= 0; --l) {
        const size_t lb = static_cast<size_t>(l) * p.B + b;
        if (dead) {               // an unusable input below: this level reports -1 as well
            if (tid == 0) {
                p.accepted_len[lb] = -1;
                if (p.block_len) p.block_len[lb] = -1;
                if (p.out_len) p.out_len[lb] = -1;
            }
            if (p.out_tokens && tid <= p.kmax) p.out_tokens[lb * (p.kmax + 1) + tid] = -1;
            continue;
        }
        const int m = min(p.k[l], stream_len);
        const int grow = p.t.row_begin[l] + b * p.t.rows[l];
        for (int r = warp; r <= m; r += kGreedyWarps) {
            const int a = merge_argmax(p.partials + static_cast<size_t>(grow + r) * p.parts, p.parts, lane);
            if (lane == 0) top[r] = a;
        }
        __syncthreads();
        if (warp == 0) {
            // positions in order: an out-of-range token or an unusable row met before the loop stops
            // spoils the sequence; the loop stops at the first mismatch, else at the bonus row m
            const bool in_block = lane < m;
            const int x = in_block ? tok[lane] : 0;
            const bool tok_bad = in_block && (x < 0 || x >= p.V);
            const bool row_bad = in_block && top[lane] < 0;
            const bool match = in_block && !tok_bad && !row_bad && x == top[lane];
            const unsigned stop_mask = __ballot_sync(0xffffffffu, in_block && !match);
            const unsigned bad_mask = __ballot_sync(0xffffffffu, tok_bad || row_bad);
            const int a = stop_mask ? (__ffs(stop_mask) - 1) : m;          // accepted length
            bool bad = (bad_mask & ((a < 32 ? (2u << a) : 0u) - 1u)) != 0;  // spoiled at a position <= a
            if (a == m && top[m] < 0) bad = true;                          // unusable bonus row
            if (lane == 0) {
                sh_a = a;
                sh_next = bad ? -1 : top[a];
                sh_bad = bad ? 1 : 0;
            }
        }
        __syncthreads();
        const int a = sh_a, next = sh_next;
        if (sh_bad) {
            dead = true;
            if (tid == 0) {
                p.accepted_len[lb] = -1;
                if (p.block_len) p.block_len[lb] = -1;
                if (p.out_len) p.out_len[lb] = -1;
                if (p.device_status) atomicCAS(p.device_status, 0, static_cast<int>(POLYSPEC_ERR_BAD_INPUT_ON_DEVICE));
            }
            if (p.out_tokens && tid <= p.kmax) p.out_tokens[lb * (p.kmax + 1) + tid] = -1;
            __syncthreads();
            continue;
        }
        if (tid == 0) {
            p.accepted_len[lb] = a;
            if (p.block_len) p.block_len[lb] = m;
            if (p.out_len) p.out_len[lb] = a + 1;
        }
        if (p.out_tokens && tid <= p.kmax)
            p.out_tokens[lb * (p.kmax + 1) + tid] = (tid < a) ? tok[tid] : (tid == a ? next : -1);
        __syncthreads();
        if (tid == 0) tok[a] = next;
        stream_len = a + 1;
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_greedy_walk(const WalkParams& p, cudaStream_t stream)
{
    if (p.B <= 0) return cudaSuccess;
    greedy_walk_kernel<<<p.B, kGreedyThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace polyspec
