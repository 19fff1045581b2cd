// The C-ABI entry points of libpolyspec: argument checks, workspace layout, kernel launches.
// Every step of the verification itself runs in the kernels; nothing is computed on the host.
#include <cmath>
#include <cstring>

#include "polyspec_kernels.cuh"

using namespace polyspec;

namespace {

constexpr double kLog2e = 1.4426950408889634074;

// The runtime's code for the most recent POLYSPEC_ERR_CUDA (see polyspec_last_cuda_error).
cudaError_t g_last_cuda_error = cudaSuccess;

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t elem_size(polyspec_dtype dt) { return dt == POLYSPEC_BF16 ? 2 : 4; }

// Fills the row table; returns the total number of rows or -1 on overflow.
long long fill_rows(RowTable& t, const void* const* logits, const int* rows, int n, int B)
{
    long long acc = 0;
    t.n_models = n;
    for (int i = 0; i < kMaxModels; ++i) { t.logits[i] = nullptr; t.rows[i] = 0; t.row_begin[i] = 0; }
    for (int i = 0; i < n; ++i) {
        t.logits[i] = logits[i];
        t.rows[i] = rows[i];
        t.row_begin[i] = static_cast<int>(acc);
        acc += static_cast<long long>(B) * rows[i];
        if (acc > 0x3fffffffLL) return -1;
    }
    for (int i = n; i <= kMaxModels; ++i) t.row_begin[i] = static_cast<int>(acc);
    return acc;
}

struct ChainArgs {
    const void* logits[kMaxModels];
    int rows[kMaxModels];
    int n_models;
    int k[kMaxLevels];
    const int32_t* draft_tokens;
    const int32_t* bottom_len;
    const float* uniforms;
    int B, V;
    polyspec_dtype dt;
    float temperature;
    int32_t *accepted_len, *block_len, *out_tokens, *out_len, *next_token;
    float *p_at, *q_at;
    int32_t* device_status;
    void* workspace;
    size_t workspace_bytes;
    cudaStream_t stream;
    int parts_override;     // > 0: the partials were written by the LM-head projection, this many per row
    uint32_t spin_limit;    // 0: default; otherwise the try_wait attempts a copy wait may take (test hook)
};

polyspec_status check_chain_shape(int n_models, const int* k, const int* rows, int B, int V, polyspec_dtype dt,
                                  long long* total_rows)
{
    if (n_models < 2 || n_models > kMaxModels || !k || !rows) return POLYSPEC_ERR_INVALID_ARG;
    if (B <= 0 || V <= 0) return POLYSPEC_ERR_INVALID_ARG;
    if (dt != POLYSPEC_F32 && dt != POLYSPEC_BF16) return POLYSPEC_ERR_INVALID_ARG;
    if (V % 8 != 0 || V > kMaxV) return POLYSPEC_ERR_UNSUPPORTED;
    const int L = n_models - 1;
    long long acc = 0;
    for (int l = 0; l < L; ++l) {
        if (k[l] < 1 || k[l] > kMaxK) return POLYSPEC_ERR_INVALID_ARG;
        if (rows[l] < k[l] + 1) return POLYSPEC_ERR_INVALID_ARG;
    }
    if (rows[n_models - 1] < k[L - 1]) return POLYSPEC_ERR_INVALID_ARG;
    for (int i = 0; i < n_models; ++i) {
        acc += static_cast<long long>(B) * rows[i];
        if (acc > 0x3fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    }
    const StatsPlan pl = plan_stats(acc, V, dt);
    if (pl.n_items > 0x7fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    *total_rows = acc;
    return POLYSPEC_OK;
}

// Bytes a chain call needs: the partials.
size_t chain_workspace_bytes(long long total_rows, int /*n_models*/, int /*B*/, int V, polyspec_dtype dt)
{
    return plan_stats(total_rows, V, dt).partial_bytes;
}

// Checks shared by both halves; fills the plan and the row table.
polyspec_status prepare_chain(const ChainArgs& a, StatsPlan* pl, StatsParams* sp)
{
    long long total_rows = 0;
    polyspec_status st = check_chain_shape(a.n_models, a.k, a.rows, a.B, a.V, a.dt, &total_rows);
    if (st != POLYSPEC_OK) return st;
    if (!(a.temperature > 0.0f) || !std::isfinite(a.temperature)) return POLYSPEC_ERR_INVALID_ARG;
    if (!a.workspace || (reinterpret_cast<uintptr_t>(a.workspace) & 255u) != 0) return POLYSPEC_ERR_INVALID_ARG;
    for (int i = 0; i < a.n_models; ++i)
        if (!a.logits[i] || !aligned16(a.logits[i])) return POLYSPEC_ERR_INVALID_ARG;
    *pl = plan_stats(total_rows, a.V, a.dt);
    if (a.parts_override > 0) {
        pl->parts = a.parts_override;
        pl->partial_bytes = align256(static_cast<size_t>(total_rows) * a.parts_override * sizeof(float2));
    }
    if (a.workspace_bytes < pl->partial_bytes) return POLYSPEC_ERR_WORKSPACE;
    if (fill_rows(sp->t, a.logits, a.rows, a.n_models, a.B) < 0) return POLYSPEC_ERR_UNSUPPORTED;
    sp->V = a.V;
    sp->seg = pl->seg;
    sp->parts = pl->parts;
    sp->n_items = static_cast<int>(pl->n_items);
    sp->c = static_cast<float>(kLog2e / static_cast<double>(a.temperature));
    sp->partials = static_cast<float2*>(a.workspace);
    return POLYSPEC_OK;
}

// First half: the softmax normaliser of every row (the only pass that touches every logit).
polyspec_status run_stats(const ChainArgs& a)
{
    StatsPlan pl;
    StatsParams sp;
    polyspec_status st = prepare_chain(a, &pl, &sp);
    if (st != POLYSPEC_OK) return st;
    if (cuda_failed(launch_stats(a.dt, sp, a.stream))) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

void fill_walk_params(const ChainArgs& a, const StatsParams& sp, int parts, WalkParams* out)
{
    WalkParams& wp = *out;
    wp.t = sp.t;
    wp.V = a.V;
    wp.parts = parts;
    wp.c = sp.c;
    wp.partials = sp.partials;
    wp.n_levels = a.n_models - 1;
    int kmax = 0;
    for (int l = 0; l < kMaxLevels; ++l) {
        wp.k[l] = l < wp.n_levels ? a.k[l] : 0;
        if (wp.k[l] > kmax) kmax = wp.k[l];
    }
    wp.kmax = kmax;
    wp.B = a.B;
    wp.draft_tokens = a.draft_tokens;
    wp.bottom_len = a.bottom_len;
    wp.uniforms = a.uniforms;
    wp.accepted_len = a.accepted_len;
    wp.block_len = a.block_len;
    wp.out_tokens = a.out_tokens;
    wp.out_len = a.out_len;
    wp.next_token = a.next_token;
    wp.p_at = a.p_at;
    wp.q_at = a.q_at;
    wp.device_status = a.device_status;
    wp.cluster = 1;
}

// Second half: accept tests, first rejection, replacement / bonus token, hand-off, level by level.
polyspec_status run_walk(const ChainArgs& a)
{
    StatsPlan pl;
    StatsParams sp;
    polyspec_status st = prepare_chain(a, &pl, &sp);
    if (st != POLYSPEC_OK) return st;
    if (!a.draft_tokens || !a.uniforms || !a.accepted_len) return POLYSPEC_ERR_INVALID_ARG;
    WalkParams wp;
    fill_walk_params(a, sp, pl.parts, &wp);
    if (cuda_failed(launch_walk(a.dt, wp, a.stream))) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

// The two halves one after the other on the caller's stream (two launches).
polyspec_status run_chain_two_launch(const ChainArgs& a)
{
    if (!a.draft_tokens || !a.uniforms || !a.accepted_len) return POLYSPEC_ERR_INVALID_ARG;
    polyspec_status st = run_stats(a);
    if (st != POLYSPEC_OK) return st;
    return run_walk(a);
}

polyspec_status run_chain(const ChainArgs& a)
{
    return run_chain_two_launch(a);
}

ChainArgs chain_args(const polyspec_model_logits* models, int n_models, const int* k, int B, int V, polyspec_dtype dt,
                     float temperature, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ChainArgs a;
    std::memset(&a, 0, sizeof a);
    for (int i = 0; i < n_models; ++i) { a.logits[i] = models[i].logits; a.rows[i] = models[i].rows; }
    a.n_models = n_models;
    for (int l = 0; l < n_models - 1; ++l) a.k[l] = k[l];
    a.B = B; a.V = V; a.dt = dt; a.temperature = temperature;
    a.workspace = workspace; a.workspace_bytes = workspace_bytes;
    a.stream = static_cast<cudaStream_t>(cuda_stream);
    return a;
}

}  // namespace

bool polyspec::cuda_failed(cudaError_t e)
{
    if (e == cudaSuccess) return false;
    g_last_cuda_error = e;
    return true;
}

extern "C" {

const char* polyspec_status_string(polyspec_status s)
{
    switch (s) {
        case POLYSPEC_OK: return "ok";
        case POLYSPEC_ERR_INVALID_ARG: return "invalid argument";
        case POLYSPEC_ERR_UNSUPPORTED: return "unsupported size or layout";
        case POLYSPEC_ERR_WORKSPACE: return "workspace too small";
        case POLYSPEC_ERR_CUDA: return "CUDA error";
        case POLYSPEC_ERR_TIMEOUT: return "bounded wait expired on the device";
        case POLYSPEC_ERR_BAD_INPUT_ON_DEVICE: return "unusable input found on the device (token out of range or unusable logits row)";
        case POLYSPEC_ERR_SCRATCH_LIMIT: return "problem too large for the built-in scratch of a *_static call";
    }
    return "unknown status";
}

int polyspec_version(void) { return 310; }      // 0.3.1: staged verification and the second insertion condition in the ABI

const char* polyspec_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda_error); }

polyspec_status polyspec_verify_level_workspace(int B, int k, int V, polyspec_dtype dt, size_t* bytes)
{
    if (!bytes) return POLYSPEC_ERR_INVALID_ARG;
    const int kk[1] = {k};
    const int rows[2] = {k + 1, k};
    long long total = 0;
    polyspec_status st = check_chain_shape(2, kk, rows, B, V, dt, &total);
    if (st != POLYSPEC_OK) return st;
    *bytes = chain_workspace_bytes(total, 2, B, V, dt);
    return POLYSPEC_OK;
}

namespace {
ChainArgs level_args(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms,
    const int32_t* block_len, int B, int k, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ChainArgs a;
    std::memset(&a, 0, sizeof a);
    a.logits[0] = logits_p; a.logits[1] = logits_q;
    a.rows[0] = k + 1; a.rows[1] = k;
    a.n_models = 2;
    a.k[0] = k;
    a.draft_tokens = draft_tokens; a.bottom_len = block_len; a.uniforms = uniforms;
    a.B = B; a.V = V; a.dt = dt; a.temperature = temperature;
    a.accepted_len = accepted_len; a.next_token = next_token;
    a.p_at = p_at_draft; a.q_at = q_at_draft;
    a.device_status = device_status;
    a.workspace = workspace; a.workspace_bytes = workspace_bytes;
    a.stream = static_cast<cudaStream_t>(cuda_stream);
    return a;
}
}  // namespace

polyspec_status polyspec_verify_level(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms,
    const int32_t* block_len, int B, int k, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!next_token) return POLYSPEC_ERR_INVALID_ARG;
    return run_chain(level_args(logits_p, logits_q, draft_tokens, uniforms, block_len, B, k, V, dt, temperature, accepted_len,
                                next_token, p_at_draft, q_at_draft, device_status, workspace, workspace_bytes, cuda_stream));
}

}  // extern "C"

// The level call as two launches (row statistics, then the walk) on a workspace that holds the partials only: what
// polyspec_verify_level_static runs on its built-in scratch.
polyspec_status polyspec::verify_level_two_launch_workspace(int B, int k, int V, polyspec_dtype dt, size_t* bytes)
{
    const int kk[1] = {k};
    const int rows[2] = {k + 1, k};
    long long total = 0;
    polyspec_status st = check_chain_shape(2, kk, rows, B, V, dt, &total);
    if (st != POLYSPEC_OK) return st;
    *bytes = plan_stats(total, V, dt).partial_bytes;
    return POLYSPEC_OK;
}

polyspec_status polyspec::verify_level_two_launch(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms,
    const int32_t* block_len, int B, int k, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!next_token) return POLYSPEC_ERR_INVALID_ARG;
    return run_chain_two_launch(level_args(logits_p, logits_q, draft_tokens, uniforms, block_len, B, k, V, dt, temperature, accepted_len,
                                           next_token, p_at_draft, q_at_draft, device_status, workspace, workspace_bytes, cuda_stream));
}

extern "C" {

polyspec_status polyspec_verify_chain_workspace(int n_models, const int* k, const int* rows, int B, int V,
                                                polyspec_dtype dt, size_t* bytes)
{
    if (!bytes) return POLYSPEC_ERR_INVALID_ARG;
    long long total = 0;
    polyspec_status st = check_chain_shape(n_models, k, rows, B, V, dt, &total);
    if (st != POLYSPEC_OK) return st;
    *bytes = chain_workspace_bytes(total, n_models, B, V, dt);
    return POLYSPEC_OK;
}

polyspec_status polyspec_verify_chain(
    const polyspec_model_logits* models, int n_models, const int* k,
    const int32_t* draft_tokens, const float* uniforms, int B, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens, int32_t* out_len,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!models || !k || n_models < 2 || n_models > kMaxModels) return POLYSPEC_ERR_INVALID_ARG;
    if (!block_len || !out_tokens || !out_len) return POLYSPEC_ERR_INVALID_ARG;
    ChainArgs a = chain_args(models, n_models, k, B, V, dt, temperature, workspace, workspace_bytes, cuda_stream);
    a.draft_tokens = draft_tokens; a.uniforms = uniforms;
    a.accepted_len = accepted_len; a.block_len = block_len; a.out_tokens = out_tokens; a.out_len = out_len;
    a.device_status = device_status;
    return run_chain(a);
}

polyspec_status polyspec_chain_row_stats(
    const polyspec_model_logits* models, int n_models, const int* k, int B, int V, polyspec_dtype dt,
    float temperature, int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!models || !k || n_models < 2 || n_models > kMaxModels) return POLYSPEC_ERR_INVALID_ARG;
    ChainArgs a = chain_args(models, n_models, k, B, V, dt, temperature, workspace, workspace_bytes, cuda_stream);
    a.device_status = device_status;
    return run_stats(a);
}

polyspec_status polyspec_chain_walk(
    const polyspec_model_logits* models, int n_models, const int* k,
    const int32_t* draft_tokens, const float* uniforms, int B, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens, int32_t* out_len,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!models || !k || n_models < 2 || n_models > kMaxModels) return POLYSPEC_ERR_INVALID_ARG;
    if (!block_len || !out_tokens || !out_len) return POLYSPEC_ERR_INVALID_ARG;
    ChainArgs a = chain_args(models, n_models, k, B, V, dt, temperature, workspace, workspace_bytes, cuda_stream);
    a.draft_tokens = draft_tokens; a.uniforms = uniforms;
    a.accepted_len = accepted_len; a.block_len = block_len; a.out_tokens = out_tokens; a.out_len = out_len;
    a.device_status = device_status;
    return run_walk(a);
}

// ---- cost model of Section 3.2 (host arithmetic)
double polyspec_cost_total_time(int n, const double* T, const double* L, double beta, double N)
{
    if (n < 2 || !T || !L) return std::nan("");
    double total = 0.0;
    for (int i = 0; i < n - 1; ++i) {
        if (!(L[i] > 0.0)) return std::nan("");
        total += N / L[i] * T[i];
    }
    return total + beta * (N / L[n - 2]) * T[n - 1];
}

int polyspec_cost_insertion(double T_new, double T_i, double L_new, double L_i, double L_i_new, double* lhs, double* rhs)
{
    if (!(T_i > 0.0) || !(T_new > 0.0) || !(L_new > 0.0) || !(L_i > 0.0) || !(L_i_new > 0.0)) return -1;
    const double a = T_new / T_i;
    const double b = L_new * (1.0 / L_i - 1.0 / L_i_new);
    if (lhs) *lhs = a;
    if (rhs) *rhs = b;
    return a < b ? 1 : 0;
}

int polyspec_cost_insertion_drafter(double T_new, double T_next, double L_new, double L_i, double beta, double* lhs, double* rhs)
{
    if (!(T_next > 0.0) || !(T_new > 0.0) || !(L_new > 0.0) || !(L_i > 0.0) || !(beta > 0.0)) return -1;
    const double a = T_new / T_next;
    const double b = beta * (L_new / L_i - 1.0);
    if (lhs) *lhs = a;
    if (rhs) *rhs = b;
    return a < b ? 1 : 0;
}

// ---- greedy matching: only the verifiers' rows are read (arg max), the drafter contributes its tokens
namespace {
polyspec_status greedy_shape(int n_models, const int* k, const int* rows, int B, int V, polyspec_dtype dt, long long* total_rows)
{
    if (n_models < 2 || n_models > kMaxModels || !k || !rows) return POLYSPEC_ERR_INVALID_ARG;
    if (B <= 0 || V <= 0) return POLYSPEC_ERR_INVALID_ARG;
    if (dt != POLYSPEC_F32 && dt != POLYSPEC_BF16) return POLYSPEC_ERR_INVALID_ARG;
    if (V % 8 != 0 || V > kMaxV) return POLYSPEC_ERR_UNSUPPORTED;
    long long acc = 0;
    for (int l = 0; l < n_models - 1; ++l) {
        if (k[l] < 1 || k[l] > kMaxK || rows[l] < k[l] + 1) return POLYSPEC_ERR_INVALID_ARG;
        acc += static_cast<long long>(B) * rows[l];
        if (acc > 0x3fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    }
    if (plan_stats(acc, V, dt).n_items > 0x7fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    *total_rows = acc;
    return POLYSPEC_OK;
}
}  // namespace

polyspec_status polyspec_verify_chain_greedy_workspace(int n_models, const int* k, const int* rows, int B, int V,
                                                       polyspec_dtype dt, size_t* bytes)
{
    if (!bytes) return POLYSPEC_ERR_INVALID_ARG;
    long long total = 0;
    polyspec_status st = greedy_shape(n_models, k, rows, B, V, dt, &total);
    if (st != POLYSPEC_OK) return st;
    *bytes = plan_stats(total, V, dt).partial_bytes;
    return POLYSPEC_OK;
}

polyspec_status polyspec_verify_chain_greedy(
    const polyspec_model_logits* models, int n_models, const int* k, const int32_t* draft_tokens,
    int B, int V, polyspec_dtype dt,
    int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens, int32_t* out_len,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!models || !k || n_models < 2 || n_models > kMaxModels) return POLYSPEC_ERR_INVALID_ARG;
    if (!draft_tokens || !accepted_len || !block_len || !out_tokens || !out_len) return POLYSPEC_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return POLYSPEC_ERR_INVALID_ARG;
    const int nv = n_models - 1;                    // verifiers; the drafter's logits are never read
    int rows[kMaxModels];
    const void* logits[kMaxModels];
    for (int i = 0; i < n_models; ++i) { rows[i] = models[i].rows; logits[i] = models[i].logits; }
    for (int l = 0; l < nv; ++l)
        if (!logits[l] || !aligned16(logits[l])) return POLYSPEC_ERR_INVALID_ARG;
    long long total = 0;
    polyspec_status st = greedy_shape(n_models, k, rows, B, V, dt, &total);
    if (st != POLYSPEC_OK) return st;
    const StatsPlan pl = plan_stats(total, V, dt);
    if (workspace_bytes < pl.partial_bytes) return POLYSPEC_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

    StatsParams sp;
    if (fill_rows(sp.t, logits, rows, nv, B) < 0) return POLYSPEC_ERR_UNSUPPORTED;
    sp.V = V;
    sp.seg = pl.seg;
    sp.parts = pl.parts;
    sp.n_items = static_cast<int>(pl.n_items);
    sp.c = 1.0f;
    sp.partials = static_cast<float2*>(workspace);
    if (cuda_failed(launch_stats(dt, sp, s, /*argmax=*/true))) return POLYSPEC_ERR_CUDA;

    WalkParams wp;
    std::memset(&wp, 0, sizeof wp);
    wp.t = sp.t;
    wp.V = V;
    wp.parts = pl.parts;
    wp.partials = sp.partials;
    wp.n_levels = nv;
    int kmax = 0;
    for (int l = 0; l < kMaxLevels; ++l) {
        wp.k[l] = l < nv ? k[l] : 0;
        if (wp.k[l] > kmax) kmax = wp.k[l];
    }
    wp.kmax = kmax;
    wp.B = B;
    wp.draft_tokens = draft_tokens;
    wp.accepted_len = accepted_len;
    wp.block_len = block_len;
    wp.out_tokens = out_tokens;
    wp.out_len = out_len;
    wp.device_status = device_status;
    if (cuda_failed(launch_greedy_walk(wp, s))) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

// Staging layout of the host-buffer call, after the partials: logits of each model, draft
// tokens, uniforms, the four outputs, the status word; every piece 256-byte aligned.
namespace {
struct HostLayout {
    size_t partials, logits[kMaxModels], tokens, uniforms, acc, blk, otok, olen, status, total;
    size_t logits_bytes[kMaxModels], tokens_bytes, uniforms_bytes, lb_bytes, otok_bytes;
};
polyspec_status host_layout(int n_models, const int* k, const int* rows, int B, int V, polyspec_dtype dt, HostLayout* h)
{
    long long total = 0;
    polyspec_status st = check_chain_shape(n_models, k, rows, B, V, dt, &total);
    if (st != POLYSPEC_OK) return st;
    const int L = n_models - 1;
    int kmax = 0;
    for (int l = 0; l < L; ++l) kmax = k[l] > kmax ? k[l] : kmax;
    size_t off = 0;
    h->partials = off; off += align256(chain_workspace_bytes(total, n_models, B, V, dt));
    for (int i = 0; i < n_models; ++i) {
        h->logits_bytes[i] = static_cast<size_t>(B) * rows[i] * V * elem_size(dt);
        h->logits[i] = off; off += align256(h->logits_bytes[i]);
    }
    h->tokens_bytes = static_cast<size_t>(B) * k[L - 1] * 4;      h->tokens = off;   off += align256(h->tokens_bytes);
    h->uniforms_bytes = static_cast<size_t>(L) * B * (kmax + 1) * 4; h->uniforms = off; off += align256(h->uniforms_bytes);
    h->lb_bytes = static_cast<size_t>(L) * B * 4;
    h->otok_bytes = static_cast<size_t>(L) * B * (kmax + 1) * 4;
    h->acc = off;  off += align256(h->lb_bytes);
    h->blk = off;  off += align256(h->lb_bytes);
    h->olen = off; off += align256(h->lb_bytes);
    h->otok = off; off += align256(h->otok_bytes);
    h->status = off; off += 256;
    h->total = off;
    return POLYSPEC_OK;
}
}  // namespace

polyspec_status polyspec_verify_chain_host_workspace(int n_models, const int* k, const int* rows, int B, int V,
                                                     polyspec_dtype dt, size_t* bytes)
{
    if (!bytes) return POLYSPEC_ERR_INVALID_ARG;
    HostLayout h;
    polyspec_status st = host_layout(n_models, k, rows, B, V, dt, &h);
    if (st != POLYSPEC_OK) return st;
    *bytes = h.total;
    return POLYSPEC_OK;
}

polyspec_status polyspec_verify_chain_host(
    const polyspec_model_logits* models_host, int n_models, const int* k,
    const int32_t* draft_tokens_host, const float* uniforms_host, int B, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len_host, int32_t* block_len_host, int32_t* out_tokens_host, int32_t* out_len_host,
    int32_t* host_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!models_host || !k || n_models < 2 || n_models > kMaxModels) return POLYSPEC_ERR_INVALID_ARG;
    if (!draft_tokens_host || !uniforms_host || !accepted_len_host || !block_len_host || !out_tokens_host || !out_len_host)
        return POLYSPEC_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return POLYSPEC_ERR_INVALID_ARG;
    int rows[kMaxModels];
    for (int i = 0; i < n_models; ++i) {
        if (!models_host[i].logits) return POLYSPEC_ERR_INVALID_ARG;
        rows[i] = models_host[i].rows;
    }
    HostLayout h;
    polyspec_status st = host_layout(n_models, k, rows, B, V, dt, &h);
    if (st != POLYSPEC_OK) return st;
    if (workspace_bytes < h.total) return POLYSPEC_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);

    polyspec_model_logits dev_models[kMaxModels];
    // bottom-up order: the drafter's rows are the first the kernels touch
    for (int i = n_models - 1; i >= 0; --i) {
        if (cuda_failed(cudaMemcpyAsync(ws + h.logits[i], models_host[i].logits, h.logits_bytes[i], cudaMemcpyHostToDevice, s)))
            return POLYSPEC_ERR_CUDA;
        dev_models[i].logits = ws + h.logits[i];
        dev_models[i].rows = rows[i];
    }
    if (cuda_failed(cudaMemcpyAsync(ws + h.tokens, draft_tokens_host, h.tokens_bytes, cudaMemcpyHostToDevice, s))) return POLYSPEC_ERR_CUDA;
    if (cuda_failed(cudaMemcpyAsync(ws + h.uniforms, uniforms_host, h.uniforms_bytes, cudaMemcpyHostToDevice, s))) return POLYSPEC_ERR_CUDA;
    if (cuda_failed(cudaMemsetAsync(ws + h.status, 0, 4, s))) return POLYSPEC_ERR_CUDA;

    st = polyspec_verify_chain(dev_models, n_models, k,
                               reinterpret_cast<const int32_t*>(ws + h.tokens), reinterpret_cast<const float*>(ws + h.uniforms),
                               B, V, dt, temperature,
                               reinterpret_cast<int32_t*>(ws + h.acc), reinterpret_cast<int32_t*>(ws + h.blk),
                               reinterpret_cast<int32_t*>(ws + h.otok), reinterpret_cast<int32_t*>(ws + h.olen),
                               reinterpret_cast<int32_t*>(ws + h.status), ws + h.partials, h.logits[0] - h.partials, s);
    if (st != POLYSPEC_OK) return st;
    if (cuda_failed(cudaMemcpyAsync(accepted_len_host, ws + h.acc, h.lb_bytes, cudaMemcpyDeviceToHost, s))) return POLYSPEC_ERR_CUDA;
    if (cuda_failed(cudaMemcpyAsync(block_len_host, ws + h.blk, h.lb_bytes, cudaMemcpyDeviceToHost, s))) return POLYSPEC_ERR_CUDA;
    if (cuda_failed(cudaMemcpyAsync(out_len_host, ws + h.olen, h.lb_bytes, cudaMemcpyDeviceToHost, s))) return POLYSPEC_ERR_CUDA;
    if (cuda_failed(cudaMemcpyAsync(out_tokens_host, ws + h.otok, h.otok_bytes, cudaMemcpyDeviceToHost, s))) return POLYSPEC_ERR_CUDA;
    if (host_status && cuda_failed(cudaMemcpyAsync(host_status, ws + h.status, 4, cudaMemcpyDeviceToHost, s))) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

polyspec_status polyspec_lm_head(const void* hidden, const void* W, int rows, int V, int d, float* logits,
                                 int32_t* device_status, void* cuda_stream)
{
    if (!hidden || !W || !logits || rows <= 0 || V <= 0 || d <= 0) return POLYSPEC_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(W) || !aligned16(logits)) return POLYSPEC_ERR_INVALID_ARG;
    if (d % 64 != 0 || V % 4 != 0 || static_cast<long long>(rows) * V > 0x7fffffffLL * 16) return POLYSPEC_ERR_UNSUPPORTED;
    const LmHeadProblem pr = {hidden, W, rows, d, logits, nullptr};
    if (cuda_failed(launch_lmhead(&pr, 1, V, 0.0f, device_status, static_cast<cudaStream_t>(cuda_stream)))) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

// Workspace of the fused call: fp32 logits of both models (written by the projection, read
// back for the gathers and, for one row pair per sequence, by the sampling pass), then the
// row-statistics partials, which the projection's epilogue writes as well.
namespace {
struct FusedLayout { size_t logits_p, logits_q, partials, total; long long total_rows; };
polyspec_status fused_layout(int B, int k, int rows_q, int V, int d_p, int d_q, FusedLayout* f)
{
    if (B <= 0 || k < 1 || k > kMaxK || V <= 0 || d_p <= 0 || d_q <= 0 || rows_q < k) return POLYSPEC_ERR_INVALID_ARG;
    if (V % 8 != 0 || V > kMaxV || d_p % 64 != 0 || d_q % 64 != 0) return POLYSPEC_ERR_UNSUPPORTED;
    const int kk[1] = {k};
    const int rows[2] = {k + 1, rows_q};
    long long total = 0;
    polyspec_status st = check_chain_shape(2, kk, rows, B, V, POLYSPEC_F32, &total);
    if (st != POLYSPEC_OK) return st;
    size_t off = 0;
    f->logits_p = off; off += align256(static_cast<size_t>(B) * (k + 1) * V * 4);
    f->logits_q = off; off += align256(static_cast<size_t>(B) * rows_q * V * 4);
    f->partials = off; off += align256(static_cast<size_t>(total) * lmhead_parts(V) * sizeof(float2));
    f->total = off;
    f->total_rows = total;
    return POLYSPEC_OK;
}
}  // namespace

polyspec_status polyspec_verify_from_hidden_workspace(int B, int k, int V, int d_p, int d_q, size_t* bytes)
{
    if (!bytes) return POLYSPEC_ERR_INVALID_ARG;
    FusedLayout f;
    // sized for the largest rows_q a caller may pass alongside k: k + 1
    polyspec_status st = fused_layout(B, k, k + 1, V, d_p, d_q, &f);
    if (st != POLYSPEC_OK) return st;
    *bytes = f.total;
    return POLYSPEC_OK;
}

namespace {
struct FusedCall {
    FusedLayout f;
    float *lp, *lq;
    char* ws;
    cudaStream_t s;
};
polyspec_status fused_prepare(int rows_q, int B, int k, int V, int d_p, int d_q, void* workspace, size_t workspace_bytes,
                              void* cuda_stream, FusedCall* c)
{
    if (!workspace) return POLYSPEC_ERR_INVALID_ARG;
    if (rows_q > k + 1) return POLYSPEC_ERR_INVALID_ARG;
    polyspec_status st = fused_layout(B, k, rows_q, V, d_p, d_q, &c->f);
    if (st != POLYSPEC_OK) return st;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return POLYSPEC_ERR_INVALID_ARG;
    if (workspace_bytes < c->f.total) return POLYSPEC_ERR_WORKSPACE;
    c->s = static_cast<cudaStream_t>(cuda_stream);
    c->ws = static_cast<char*>(workspace);
    c->lp = reinterpret_cast<float*>(c->ws + c->f.logits_p);
    c->lq = reinterpret_cast<float*>(c->ws + c->f.logits_q);
    return POLYSPEC_OK;
}
}  // namespace

polyspec_status polyspec_from_hidden_project(
    const void* hidden_p, const void* W_p, const void* hidden_q, const void* W_q, int rows_q,
    int B, int k, int V, int d_p, int d_q, float temperature, int32_t* device_status, void* workspace, size_t workspace_bytes,
    void* cuda_stream)
{
    if (!hidden_p || !W_p || !hidden_q || !W_q) return POLYSPEC_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !std::isfinite(temperature)) return POLYSPEC_ERR_INVALID_ARG;
    if (!aligned16(hidden_p) || !aligned16(W_p) || !aligned16(hidden_q) || !aligned16(W_q)) return POLYSPEC_ERR_INVALID_ARG;
    FusedCall c;
    polyspec_status st = fused_prepare(rows_q, B, k, V, d_p, d_q, workspace, workspace_bytes, cuda_stream, &c);
    if (st != POLYSPEC_OK) return st;
    float2* partials = reinterpret_cast<float2*>(c.ws + c.f.partials);
    const int parts = lmhead_parts(V);
    const LmHeadProblem probs[2] = {{hidden_p, W_p, B * (k + 1), d_p, c.lp, partials},
                                    {hidden_q, W_q, B * rows_q, d_q, c.lq, partials + static_cast<size_t>(B) * (k + 1) * parts}};
    const float scale = static_cast<float>(kLog2e / static_cast<double>(temperature));
    if (cuda_failed(launch_lmhead(probs, 2, V, scale, device_status, c.s))) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

polyspec_status polyspec_from_hidden_verify(
    int rows_q, const int32_t* draft_tokens, const float* uniforms, const int32_t* block_len,
    int B, int k, int V, int d_p, int d_q, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!next_token || !accepted_len) return POLYSPEC_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !std::isfinite(temperature)) return POLYSPEC_ERR_INVALID_ARG;
    FusedCall c;
    polyspec_status st = fused_prepare(rows_q, B, k, V, d_p, d_q, workspace, workspace_bytes, cuda_stream, &c);
    if (st != POLYSPEC_OK) return st;
    ChainArgs a;
    std::memset(&a, 0, sizeof a);
    a.logits[0] = c.lp; a.logits[1] = c.lq;
    a.rows[0] = k + 1; a.rows[1] = rows_q;
    a.n_models = 2;
    a.k[0] = k;
    a.draft_tokens = draft_tokens; a.bottom_len = block_len; a.uniforms = uniforms;
    a.B = B; a.V = V; a.dt = POLYSPEC_F32; a.temperature = temperature;
    a.accepted_len = accepted_len; a.next_token = next_token;
    a.p_at = p_at_draft; a.q_at = q_at_draft;
    a.device_status = device_status;
    a.workspace = c.ws + c.f.partials; a.workspace_bytes = c.f.total - c.f.partials;
    a.stream = c.s;
    a.parts_override = lmhead_parts(V);      // the projection already left every row's partials there
    if (!draft_tokens || !uniforms) return POLYSPEC_ERR_INVALID_ARG;
    return run_walk(a);
}

polyspec_status polyspec_verify_from_hidden(
    const void* hidden_p, const void* W_p, const void* hidden_q, const void* W_q, int rows_q,
    const int32_t* draft_tokens, const float* uniforms, const int32_t* block_len,
    int B, int k, int V, int d_p, int d_q, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    // nothing may be launched unless both halves will accept their arguments
    if (!next_token || !accepted_len || !draft_tokens || !uniforms) return POLYSPEC_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !std::isfinite(temperature)) return POLYSPEC_ERR_INVALID_ARG;
    polyspec_status st = polyspec_from_hidden_project(hidden_p, W_p, hidden_q, W_q, rows_q, B, k, V, d_p, d_q, temperature,
                                                      device_status, workspace, workspace_bytes, cuda_stream);
    if (st != POLYSPEC_OK) return st;
    return polyspec_from_hidden_verify(rows_q, draft_tokens, uniforms, block_len, B, k, V, d_p, d_q, temperature,
                                       accepted_len, next_token, p_at_draft, q_at_draft, device_status,
                                       workspace, workspace_bytes, cuda_stream);
}

}  // extern "C"
