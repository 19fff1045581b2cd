// Internal declarations shared by the kernels and the C-ABI layer of libpolyspec.
// Product code: nothing here is shared with, or derived from, the CPU oracle.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "polyspec.h"

namespace polyspec {

constexpr int kMaxModels = POLYSPEC_MAX_MODELS;
constexpr int kMaxLevels = POLYSPEC_MAX_MODELS - 1;
constexpr int kMaxK = POLYSPEC_MAX_K;

// Records the runtime's code for polyspec_last_cuda_error; true if `e` is an error.
bool cuda_failed(cudaError_t e);

// Reference exponent of a stretch of a row that holds no finite logit (its sum is 0).
constexpr float kEmptyRef = -1.0e30f;

// Elements one warp covers per tile in the sampling pass (32 lanes x 8 elements).
constexpr int kTile = 256;
// Largest vocabulary the sampling pass keeps tile sums for in shared memory.
constexpr int kMaxTiles = 8192;
constexpr int kMaxV = kMaxTiles * kTile;

// Which logits rows exist: model i has rows[i] rows per sequence, B sequences, stored
// [B, rows[i], V]; global row index = row_begin[i] + b * rows[i] + j.
struct RowTable {
    const void* logits[kMaxModels];
    int rows[kMaxModels];
    int row_begin[kMaxModels + 1];
    int n_models;
};

// Row statistics (softmax normaliser) pass.  A row is cut into `parts` segments of `seg`
// elements; one work item is one segment and yields one partial (E, s) meaning
// sum_v 2^(z_v * c - E) = s with E an integer-valued float, c = log2(e) / T.
struct StatsParams {
    RowTable t;
    int V;
    int seg;
    int parts;
    int n_items;
    float c;
    float2* partials;   // [total rows, parts]
};

// Decision + sampling pass: one CTA walks one sequence up the chain.
struct WalkParams {
    RowTable t;
    int V;
    int parts;
    float c;
    const float2* partials;
    int n_levels;
    int k[kMaxLevels];
    int kmax;
    int B;
    const int32_t* draft_tokens;   // [B, k[n_levels-1]]
    const int32_t* bottom_len;     // [B] or nullptr
    const float* uniforms;         // [n_levels, B, kmax+1]
    int32_t* accepted_len;         // [n_levels, B]
    int32_t* block_len;            // [n_levels, B] or nullptr
    int32_t* out_tokens;           // [n_levels, B, kmax+1] or nullptr
    int32_t* out_len;              // [n_levels, B] or nullptr
    int32_t* next_token;           // [B] or nullptr (single-level call)
    float* p_at;                   // [B, k[0]] or nullptr (single-level call)
    float* q_at;                   // [B, k[0]] or nullptr
    int32_t* device_status;        // [1] or nullptr
    int cluster;                   // CTAs per sequence (set by launch_walk)
};

// How the row-statistics pass is cut up for a problem size (same answer for the
// workspace query and the launch).
struct StatsPlan {
    int seg;
    int parts;
    long long total_rows;
    long long n_items;
    size_t partial_bytes;
};
StatsPlan plan_stats(long long total_rows, int V, polyspec_dtype dt);

// argmax = true: the same pass produces arg-max partials (largest logit, index as int bits or -1)
// for greedy matching instead of the softmax normaliser.
cudaError_t launch_stats(polyspec_dtype dt, const StatsParams& p, cudaStream_t stream, bool argmax = false);
cudaError_t launch_walk(polyspec_dtype dt, const WalkParams& p, cudaStream_t stream);
// Greedy matching: reads arg-max partials (launch_stats with argmax = true) of the verifiers' rows only.
cudaError_t launch_greedy_walk(const WalkParams& p, cudaStream_t stream);

// The level call as two launches on a workspace that holds the partials only (api.cu); polyspec_verify_level_static
// runs it on the library's built-in scratch.
polyspec_status verify_level_two_launch_workspace(int B, int k, int V, polyspec_dtype dt, size_t* bytes);
polyspec_status verify_level_two_launch(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms,
    const int32_t* block_len, int B, int k, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream);

// LM-head projection on the tensor cores: out[r, v] = sum_d hidden[r, d] * W[v, d], bf16 inputs
// (hidden [rows, d], W [V, d], both row-major and 16-byte aligned, d a multiple of 64), fp32
// output [rows, V].  Up to two projections (the verifier's and the drafter's) share one launch.
struct LmHeadProblem {
    const void* hidden;
    const void* W;
    int rows;
    int d;
    float* out;
    float2* partials;   // nullptr, or [rows, lmhead_parts(V)]: row-statistics partials written by the epilogue
};
// Number of row-statistics partials per row the projection writes: one per 128 vocabulary entries
// (one per CTA of the pair that owns a 256-entry tile).
inline int lmhead_parts(int V) { return 2 * ((V + 255) / 256); }
// c = log2(e) / T, used only when partials are requested.
cudaError_t launch_lmhead(const LmHeadProblem* probs, int n, int V, float c, int32_t* device_status, cudaStream_t stream);

}  // namespace polyspec
