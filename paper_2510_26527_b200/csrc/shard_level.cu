// One verification level (Algorithm 1's Verify loop and the replacement / bonus token) when the
// vocabulary of both models is sharded over several ranks, as a tensor-parallel LM head leaves it:
// rank r holds entries [r * V_local, (r + 1) * V_local) of every logits row.  The softmax normaliser,
// the accept tests and the inverse-CDF search all need sums over the whole vocabulary, so the level
// becomes three local phases with a small exchange between them (the caller's all-gathers; nothing
// here talks to another rank):
//   stats   each rank: the normaliser partials of its slice of every row, merged to one (E, Z) per row,
//           and the logits at the block tokens it owns                      -> exchange 1: all ranks' records
//   decide  every rank, identically: whole-row normalisers from all records, accept tests, accepted
//           length a; then, on its own slice, the mass of the residual max(0, P - Q) of row a (of P for
//           the bonus row), tile by tile                                     -> exchange 2: all ranks' masses
//   pick    every rank, identically: the rank whose slice contains u * total mass; that rank alone
//           finds the token in its slice                                     -> reduce: the one token that is not -1
// The arithmetic is that of the unsharded walk (same residual, same tile sums, same search), so with
// one rank the result is bit-identical to polyspec_verify_level.
// A chain of models repeats decide / pick level by level, bottom-up (Section 3.1), on normalisers that one
// stats call computed for every row of every model; the logits at the block tokens are then a small
// exchange of their own per level (the block of a level is only known once the level below is done), and
// a hand-off kernel turns (accepted length, token) into the block of the level above.
#include <cmath>

#include "polyspec_kernels.cuh"
#include "walk_device.cuh"

namespace polyspec {
namespace {

using namespace walkdev;

constexpr int kMaxRanks = 64;
constexpr double kLog2eS = 1.4426950408889634074;

inline size_t align256s(size_t x) { return (x + 255) / 256 * 256; }
inline bool aligned16s(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A stats record holds, for `rows` logits rows in the row numbering of the row-statistics pass (model after
// model, sequence after sequence), double Z[rows] then float E[rows]: the normaliser of the rank's slice of
// each row.  The single-level call appends the logits at the block tokens the rank owns, float zp[B][k] and
// zq[B][k] (0 for tokens of other ranks); the chain sends those as a gather record of their own.
__host__ __device__ inline size_t stats_part_bytes(long long rows) { return static_cast<size_t>(rows) * 12; }
__host__ __device__ inline size_t gather_part_bytes(int B, int slots) { return static_cast<size_t>(B) * slots * 8; }
// Mass record: double mass[B] (what the slice holds of the distribution being sampled), double pmass[B]
// (what it holds of P at the same row, filled in when it holds nothing of the residual: needed if no rank does);
// both carry the row's common factor Z_p (see resid()), the same on every rank, which the search never needs.
__host__ __device__ inline size_t mass_record_bytes(int B) { return (static_cast<size_t>(B) * 16 + 255) / 256 * 256; }

// What `decide` leaves for `pick`, per sequence.
struct Decision {
    double Zp, Zq;
    float Ep, Eq;
    int a;          // accepted length, -1: unusable input
    int use_q;      // row a is a rejection (sample the residual) rather than the bonus row
};

struct ShardParams {
    // this level's verifier (p) and drafter-side (q) slices, [B, rows_*, V_local]
    const void* logits_p;
    const void* logits_q;
    int rows_p, rows_q;
    int rec_p, rec_q;           // stats-record index of (sequence 0, row 0) of each
    long long rec_rows;         // rows per stats record
    size_t rec_stride;          // bytes from one rank's stats record to the next
    const unsigned char* records;       // all ranks' stats records
    // logits at the block tokens: rank r's floats zp[B][tok_stride] at gathers + r * gather_stride + gather_zp, zq likewise
    const unsigned char* gathers;
    size_t gather_stride, gather_zp, gather_zq;
    const int32_t* tokens;      // [B, tok_stride] block tokens (indices in the whole vocabulary)
    int tok_stride;
    const float* uniforms;      // [B, u_stride]: accept uniform of position j at [b, j], sampling uniform at [b, u_sample]
    int u_stride, u_sample;
    const int32_t* block_len;   // [B] or nullptr
    int chain;                  // block_len < 0 marks a sequence that went wrong at a level below
    int B, k, V_local, rank, n_ranks;
    float c;
    int parts;
    const float2* partials;
    unsigned char* own_record;  // merge / gather: out
    double* own_mass;           // decide: out (mass[B], pmass[B])
    const unsigned char* masses;        // pick: all ranks' mass records
    Decision* decision;         // [B]
    float* tile_sums;           // [B][ntiles]
    int32_t* accepted_len;      // [B]
    int32_t* block_len_out;     // [B] or nullptr
    int32_t* next_token;        // [B]
    float* p_at;
    float* q_at;
    int32_t* device_status;
};

// One warp per row: the partials of the rank's slice of the row, merged.
__global__ void __launch_bounds__(256) shard_merge_kernel(const float2* partials, int parts, long long rows, unsigned char* record)
{
    const long long r = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
    if (r >= rows) return;
    const int lane = threadIdx.x & 31;
    const RowStat st = merge_partials(partials + static_cast<size_t>(r) * parts, parts, lane);
    if (lane == 0) {
        reinterpret_cast<double*>(record)[r] = st.Z;
        reinterpret_cast<float*>(record + static_cast<size_t>(rows) * 8)[r] = st.E;
    }
}

// The logits at the block tokens this rank owns (0 for the others): zp from p's row j, zq from q's row j.
template <int DT>
__global__ void __launch_bounds__(32) shard_gather_kernel(const ShardParams p)
{
    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    const int b = blockIdx.x, j = threadIdx.x;
    if (j >= p.tok_stride) return;
    const size_t row_bytes = static_cast<size_t>(p.V_local) * ELEM;
    int m = p.k;
    if (p.block_len) m = max(0, min(p.k, p.block_len[b]));
    float zp = 0.0f, zq = 0.0f;
    if (j < m) {
        const int x = p.tokens[static_cast<size_t>(b) * p.tok_stride + j] - p.rank * p.V_local;
        if (x >= 0 && x < p.V_local) {
            zp = load_logit<DT>(static_cast<const char*>(p.logits_p) + (static_cast<size_t>(b) * p.rows_p + j) * row_bytes, x);
            zq = load_logit<DT>(static_cast<const char*>(p.logits_q) + (static_cast<size_t>(b) * p.rows_q + j) * row_bytes, x);
        }
    }
    reinterpret_cast<float*>(p.own_record + p.gather_zp)[static_cast<size_t>(b) * p.tok_stride + j] = zp;
    reinterpret_cast<float*>(p.own_record + p.gather_zq)[static_cast<size_t>(b) * p.tok_stride + j] = zq;
}

// The mass of tiles [0, nt) as warp 0 adds it up: lane i owns a contiguous run of tiles, tile sums are
// added in double, in order (the same runs and order as in the search).  Returns the total in every lane.
__device__ __forceinline__ double share_of_tiles(const float* tile_sum, int nt, int lane, int* t0_out, int* t1_out,
                                                 double* mine_out, double* incl_out)
{
    const int per = (nt + 31) / 32;
    const int t0 = min(lane * per, nt), t1 = min(t0 + per, nt);
    double mine = 0.0;
    for (int t = t0; t < t1; ++t) mine += static_cast<double>(tile_sum[t]);
    const double incl = warp_incl_scan(mine, lane);
    *t0_out = t0; *t1_out = t1; *mine_out = mine; *incl_out = incl;
    return __shfl_sync(0xffffffffu, incl, 31);
}

template <int DT>
__global__ void __launch_bounds__(kWalkThreads, POLYSPEC_WALK_CTAS_PER_SM) shard_decide_kernel(const ShardParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* tile_sum = reinterpret_cast<float*>(smem_raw);
    __shared__ RowStat st_p[kMaxK + 1];
    __shared__ RowStat st_q[kMaxK + 1];
    __shared__ int sh_a, sh_bad;
    __shared__ double sh_share, sh_pshare;

    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int k = p.k, R = p.n_ranks;
    const size_t row_bytes = static_cast<size_t>(p.V_local) * ELEM;
    const double cd = static_cast<double>(p.c);
    double* mass_out = p.own_mass;
    Decision* dec = p.decision + b;
    int m = k;
    if (p.block_len) {
        const int bl = p.block_len[b];
        if (p.chain && bl < 0) {            // an unusable input at a level below: this level reports -1 as well
            if (tid == 0) {
                p.accepted_len[b] = -1;
                if (p.block_len_out) p.block_len_out[b] = -1;
                dec->a = -1; dec->use_q = 0; dec->Ep = dec->Eq = 0.0f; dec->Zp = dec->Zq = 1.0;
                mass_out[b] = 0.0;
                mass_out[p.B + b] = 0.0;
            }
            return;
        }
        m = max(0, min(k, bl));
    }
    const int V_all = p.V_local * R;

    // whole-row normalisers of p rows 0..k and q rows 0..k-1: the ranks' (E, Z) rebased to the largest E (an exact
    // scaling) and added in rank order
    if (tid < 2 * k + 1) {
        const bool is_q = tid > k;
        const int j = is_q ? tid - (k + 1) : tid;
        const size_t idx = is_q ? static_cast<size_t>(p.rec_q) + static_cast<size_t>(b) * p.rows_q + j
                                : static_cast<size_t>(p.rec_p) + static_cast<size_t>(b) * p.rows_p + j;
        const size_t e_off = static_cast<size_t>(p.rec_rows) * 8;
        float E = kEmptyRef;
        for (int r = 0; r < R; ++r) E = fmaxf(E, reinterpret_cast<const float*>(p.records + r * p.rec_stride + e_off)[idx]);
        double Z = 0.0;
        for (int r = 0; r < R; ++r) {
            const unsigned char* rec = p.records + r * p.rec_stride;
            Z += scale_pow2(reinterpret_cast<const double*>(rec)[idx], reinterpret_cast<const float*>(rec + e_off)[idx] - E);
        }
        RowStat& dst = is_q ? st_q[j] : st_p[j];
        dst.E = E;
        dst.Z = Z;
    }
    __syncthreads();

    // accept tests (warp 0; m <= 32), exactly as in the unsharded walk
    if (tid < 32) {
        bool rej = false, bad = false;
        float pf = 0.0f, qf = 0.0f;
        if (tid < m) {
            const int x = p.tokens[static_cast<size_t>(b) * p.tok_stride + tid];
            const RowStat sp = st_p[tid], sq = st_q[tid];
            if (x < 0 || x >= V_all || !stat_ok(sp) || !stat_ok(sq)) {
                bad = true;
            } else {
                const unsigned char* g = p.gathers + (x / p.V_local) * p.gather_stride;       // the rank that owns the token
                const float zp = reinterpret_cast<const float*>(g + p.gather_zp)[static_cast<size_t>(b) * p.tok_stride + tid];
                const float zq = reinterpret_cast<const float*>(g + p.gather_zq)[static_cast<size_t>(b) * p.tok_stride + tid];
                const double P = exp2(static_cast<double>(zp) * cd - static_cast<double>(sp.E)) / sp.Z;
                const double Q = exp2(static_cast<double>(zq) * cd - static_cast<double>(sq.E)) / sq.Z;
                const double u = static_cast<double>(p.uniforms[static_cast<size_t>(b) * p.u_stride + tid]);
                rej = !(u * Q <= P);
                pf = static_cast<float>(P);
                qf = static_cast<float>(Q);
            }
        }
        if (p.p_at && tid < k) p.p_at[static_cast<size_t>(b) * k + tid] = pf;
        if (p.q_at && tid < k) p.q_at[static_cast<size_t>(b) * k + tid] = qf;
        const unsigned rej_mask = __ballot_sync(0xffffffffu, rej);
        const unsigned bad_mask = __ballot_sync(0xffffffffu, bad);
        const int first_rej = rej_mask ? (__ffs(rej_mask) - 1) : m;
        const int first_bad = bad_mask ? (__ffs(bad_mask) - 1) : m + 1;
        if (tid == 0) {
            int isbad = first_bad < first_rej;
            if (!isbad && first_rej == m && !stat_ok(st_p[m])) isbad = 1;     // bonus row unusable
            sh_a = first_rej;
            sh_bad = isbad;
        }
    }
    __syncthreads();
    const int a = sh_a;
    if (sh_bad) {
        if (tid == 0) {
            p.accepted_len[b] = -1;
            if (p.block_len_out) p.block_len_out[b] = -1;
            dec->a = -1; dec->use_q = 0; dec->Ep = dec->Eq = 0.0f; dec->Zp = dec->Zq = 1.0;
            mass_out[b] = 0.0;
            mass_out[p.B + b] = 0.0;
            if (p.device_status) atomicCAS(p.device_status, 0, static_cast<int>(POLYSPEC_ERR_BAD_INPUT_ON_DEVICE));
        }
        return;
    }

    // this slice's share of row a: tile sums of the residual (or of P for the bonus row), kept for the search
    const bool use_q = a < m;
    const RowStat sp = st_p[a];
    const RowStat sq = use_q ? st_q[a] : sp;
    const void* prow = static_cast<const char*>(p.logits_p) + (static_cast<size_t>(b) * p.rows_p + a) * row_bytes;
    const void* qrow = static_cast<const char*>(p.logits_q) + (static_cast<size_t>(b) * p.rows_q + (use_q ? a : 0)) * row_bytes;
    const int ntiles = (p.V_local + kTile - 1) / kTile;
    const RowScale sc = row_scale(sp.E, sp.Z, sq.E, sq.Z, use_q);
    tiles_pass<DT>(prow, qrow, p.V_local, p.c, sc, use_q, tile_sum, 0, ntiles);
    __syncthreads();
    int t0, t1;
    double mine, incl;
    if (tid < 32) {
        const double share = share_of_tiles(tile_sum, ntiles, lane, &t0, &t1, &mine, &incl);
        if (lane == 0) sh_share = share;
    }
    __syncthreads();
    // No residual mass in this slice: should that be so on every rank, P is sampled instead (as in the unsharded walk),
    // so the slice's tile sums and mass of P are what `pick` will need; a rank without mass is never searched otherwise.
    const bool no_mass = use_q && !(sh_share > 0.0);
    if (no_mass) {
        __syncthreads();
        tiles_pass<DT>(prow, qrow, p.V_local, p.c, sc, false, tile_sum, 0, ntiles);
        __syncthreads();
        if (tid < 32) {
            const double pshare = share_of_tiles(tile_sum, ntiles, lane, &t0, &t1, &mine, &incl);
            if (lane == 0) sh_pshare = pshare;
        }
        __syncthreads();
    }
    float* keep = p.tile_sums + static_cast<size_t>(b) * ntiles;
    for (int t = tid; t < ntiles; t += kWalkThreads) keep[t] = tile_sum[t];
    if (tid == 0) {
        mass_out[b] = sh_share;
        mass_out[p.B + b] = no_mass ? sh_pshare : 0.0;
        p.accepted_len[b] = a;
        if (p.block_len_out) p.block_len_out[b] = m;
        dec->a = a; dec->use_q = use_q ? 1 : 0;
        dec->Ep = sp.E; dec->Eq = sq.E; dec->Zp = sp.Z; dec->Zq = sq.Z;
    }
}

template <int DT>
__global__ void __launch_bounds__(kWalkThreads, POLYSPEC_WALK_CTAS_PER_SM) shard_pick_kernel(const ShardParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* tile_sum = reinterpret_cast<float*>(smem_raw);
    __shared__ int sh_fallback;

    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int R = p.n_ranks;
    const Decision dec = p.decision[b];
    if (dec.a < 0) {
        if (tid == 0) p.next_token[b] = -1;
        return;
    }
    const size_t mbytes = mass_record_bytes(p.B);
    const size_t row_bytes = static_cast<size_t>(p.V_local) * ELEM;
    const int ntiles = (p.V_local + kTile - 1) / kTile;
    bool use_q = dec.use_q != 0;
    const void* prow = static_cast<const char*>(p.logits_p) + (static_cast<size_t>(b) * p.rows_p + dec.a) * row_bytes;
    const void* qrow = static_cast<const char*>(p.logits_q) + (static_cast<size_t>(b) * p.rows_q + (use_q ? dec.a : 0)) * row_bytes;
    const RowScale sc = row_scale(dec.Ep, dec.Zp, dec.Eq, dec.Zq, use_q);

    // the residual vanished in floating point on every rank: sample P instead (its masses are in the records too)
    if (tid == 0) {
        double total = 0.0;
        for (int r = 0; r < R; ++r) total += reinterpret_cast<const double*>(p.masses + r * mbytes)[b];
        sh_fallback = (use_q && !(total > 0.0)) ? 1 : 0;
    }
    __syncthreads();
    const bool fallback = sh_fallback != 0;
    if (fallback) use_q = false;        // every rank kept the tile sums of P in that case
    const float* keep = p.tile_sums + static_cast<size_t>(b) * ntiles;
    for (int t = tid; t < ntiles; t += kWalkThreads) tile_sum[t] = keep[t];
    __syncthreads();

    if (tid < 32) {
        const float u = p.uniforms[static_cast<size_t>(b) * p.u_stride + p.u_sample];
        const size_t off = fallback ? static_cast<size_t>(p.B) + b : static_cast<size_t>(b);
        // total mass and the rank whose slice contains u * total (the same arithmetic on every rank)
        double total = 0.0;
        for (int r = 0; r < R; ++r) total += reinterpret_cast<const double*>(p.masses + r * mbytes)[off];
        const double target = static_cast<double>(u) * total;
        int owner_rank = -1, last_mass = -1;
        double base = 0.0, last_base = 0.0, cum = 0.0;
        for (int r = 0; r < R; ++r) {
            const double mr = reinterpret_cast<const double*>(p.masses + r * mbytes)[off];
            const double nxt = cum + mr;
            if (owner_rank < 0 && nxt > target) { owner_rank = r; base = cum; }
            if (mr > 0.0) { last_mass = r; last_base = cum; }
            cum = nxt;
        }
        if (owner_rank < 0) { owner_rank = last_mass; base = last_base; }      // u not below 1, or rounding
        int token = -1;
        if (owner_rank == p.rank) {
            int t0, t1;
            double mine, incl;
            (void)share_of_tiles(tile_sum, ntiles, lane, &t0, &t1, &mine, &incl);
            token = pick_in_share<DT>(prow, qrow, p.V_local, p.c, sc, use_q, tile_sum, t0, t1, mine, incl,
                                      base, target, lane);
            if (token >= 0) token += p.rank * p.V_local;
        }
        if (lane == 0) p.next_token[b] = token;
    }
}

// After the ranks have agreed on the token: the stream this level emits (accepted prefix + token) becomes the block
// of the level above (Section 3.1's hand-off), and is recorded as the level's output.
__global__ void shard_handoff_kernel(const int32_t* accepted_len, const int32_t* next_token, int32_t* tokens, int32_t* block_len,
                                     int32_t* out_tokens, int32_t* out_len, int B, int slots)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int a = accepted_len[b];
    int32_t* tk = tokens + static_cast<size_t>(b) * slots;
    if (a < 0) {
        block_len[b] = -1;
        if (out_len) out_len[b] = -1;
        if (out_tokens) for (int j = 0; j < slots; ++j) out_tokens[static_cast<size_t>(b) * slots + j] = -1;
        return;
    }
    tk[a] = next_token[b];
    block_len[b] = a + 1;
    if (out_len) out_len[b] = a + 1;
    if (out_tokens)
        for (int j = 0; j < slots; ++j) out_tokens[static_cast<size_t>(b) * slots + j] = j <= a ? tk[j] : -1;
}

// ---------------------------------------------------------------------------------------------- host side
struct ShardSizes {
    StatsPlan plan;
    long long rec_rows;
    size_t partials, decision, tiles, total;
    int ntiles;
};

polyspec_status common_checks(int B, int V_local, polyspec_dtype dt, int n_ranks)
{
    if (B <= 0 || V_local <= 0 || n_ranks < 1 || n_ranks > kMaxRanks) return POLYSPEC_ERR_INVALID_ARG;
    if (dt != POLYSPEC_F32 && dt != POLYSPEC_BF16) return POLYSPEC_ERR_INVALID_ARG;
    if (V_local % 8 != 0 || V_local > kMaxV) return POLYSPEC_ERR_UNSUPPORTED;
    if (static_cast<long long>(V_local) * n_ranks > 0x7fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    return POLYSPEC_OK;
}

polyspec_status shard_sizes_rows(long long rows, int B, int V_local, polyspec_dtype dt, ShardSizes* s)
{
    if (rows > 0x3fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    s->rec_rows = rows;
    s->plan = plan_stats(rows, V_local, dt);
    if (s->plan.n_items > 0x7fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    s->ntiles = (V_local + kTile - 1) / kTile;
    size_t off = 0;
    s->partials = off; off += align256s(s->plan.partial_bytes);
    s->decision = off; off += align256s(static_cast<size_t>(B) * sizeof(Decision));
    s->tiles = off; off += align256s(static_cast<size_t>(B) * s->ntiles * sizeof(float));
    s->total = off;
    return POLYSPEC_OK;
}

polyspec_status level_sizes(int B, int k, int V_local, polyspec_dtype dt, int n_ranks, ShardSizes* s)
{
    const polyspec_status st = common_checks(B, V_local, dt, n_ranks);
    if (st != POLYSPEC_OK) return st;
    if (k < 1 || k > kMaxK) return POLYSPEC_ERR_INVALID_ARG;
    return shard_sizes_rows(static_cast<long long>(B) * (2 * k + 1), B, V_local, dt, s);
}

struct ChainShape {
    int n_models, L, kmax;
    int k[kMaxLevels];
    int rows[kMaxModels];
    int row_begin[kMaxModels + 1];
};

polyspec_status chain_sizes(int n_models, const int* k, const int* rows, int B, int V_local, polyspec_dtype dt, int n_ranks,
                            ShardSizes* s, ChainShape* c)
{
    const polyspec_status st = common_checks(B, V_local, dt, n_ranks);
    if (st != POLYSPEC_OK) return st;
    if (n_models < 2 || n_models > kMaxModels || !k || !rows) return POLYSPEC_ERR_INVALID_ARG;
    c->n_models = n_models; c->L = n_models - 1; c->kmax = 0;
    for (int l = 0; l < c->L; ++l) {
        if (k[l] < 1 || k[l] > kMaxK || rows[l] < k[l] + 1) return POLYSPEC_ERR_INVALID_ARG;
        c->k[l] = k[l];
        if (k[l] > c->kmax) c->kmax = k[l];
    }
    if (rows[n_models - 1] < k[c->L - 1]) return POLYSPEC_ERR_INVALID_ARG;
    long long acc = 0;
    for (int i = 0; i < n_models; ++i) {
        c->rows[i] = rows[i];
        c->row_begin[i] = static_cast<int>(acc);
        acc += static_cast<long long>(B) * rows[i];
        if (acc > 0x3fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    }
    for (int i = n_models; i <= kMaxModels; ++i) c->row_begin[i] = static_cast<int>(acc);
    return shard_sizes_rows(acc, B, V_local, dt, s);
}

polyspec_status base_params(int B, int V_local, int rank, int n_ranks, float temperature, void* workspace, size_t workspace_bytes,
                            const ShardSizes& sz, ShardParams* p)
{
    if (rank < 0 || rank >= n_ranks) return POLYSPEC_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !std::isfinite(temperature)) return POLYSPEC_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return POLYSPEC_ERR_INVALID_ARG;
    if (workspace_bytes < sz.total) return POLYSPEC_ERR_WORKSPACE;
    *p = ShardParams{};
    p->B = B; p->V_local = V_local; p->rank = rank; p->n_ranks = n_ranks;
    p->c = static_cast<float>(kLog2eS / static_cast<double>(temperature));
    p->parts = sz.plan.parts;
    p->rec_rows = sz.rec_rows;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    p->partials = reinterpret_cast<const float2*>(ws + sz.partials);
    p->decision = reinterpret_cast<Decision*>(ws + sz.decision);
    p->tile_sums = reinterpret_cast<float*>(ws + sz.tiles);
    return POLYSPEC_OK;
}

// The row-statistics pass over this rank's slices and the merge of its partials into the stats record.
polyspec_status run_stats_and_merge(const void* const* logits, const int* rows, const int* row_begin, int n_models, int B, int V_local,
                                    polyspec_dtype dt, const ShardSizes& sz, const ShardParams& p, void* record, int32_t* device_status,
                                    cudaStream_t stream)
{
    StatsParams sp;
    sp.t.n_models = n_models;
    for (int i = 0; i < kMaxModels; ++i) { sp.t.logits[i] = nullptr; sp.t.rows[i] = 0; sp.t.row_begin[i] = 0; }
    for (int i = 0; i < n_models; ++i) { sp.t.logits[i] = logits[i]; sp.t.rows[i] = rows[i]; sp.t.row_begin[i] = row_begin[i]; }
    for (int i = n_models; i <= kMaxModels; ++i) sp.t.row_begin[i] = static_cast<int>(sz.rec_rows);
    sp.V = V_local;
    sp.seg = sz.plan.seg;
    sp.parts = sz.plan.parts;
    sp.n_items = static_cast<int>(sz.plan.n_items);
    sp.c = p.c;
    sp.partials = const_cast<float2*>(p.partials);
    if (cuda_failed(launch_stats(dt, sp, stream))) return POLYSPEC_ERR_CUDA;
    const unsigned blocks = static_cast<unsigned>((sz.rec_rows + 7) / 8);
    shard_merge_kernel<<<blocks, 256, 0, stream>>>(p.partials, p.parts, sz.rec_rows, static_cast<unsigned char*>(record));
    if (cuda_failed(cudaGetLastError())) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

template <typename K32, typename KBF>
polyspec_status launch_by_dtype(polyspec_dtype dt, K32 f32, KBF bf16, dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                const ShardParams& p)
{
    if (dt == POLYSPEC_BF16) bf16<<<grid, block, smem, stream>>>(p);
    else f32<<<grid, block, smem, stream>>>(p);
    return cuda_failed(cudaGetLastError()) ? POLYSPEC_ERR_CUDA : POLYSPEC_OK;
}

// The level a chain call works on: models[level] verifies, models[level + 1] is the drafter side.
polyspec_status chain_level_params(const polyspec_model_logits* models, const ChainShape& c, int level, ShardParams* p)
{
    if (level < 0 || level >= c.L) return POLYSPEC_ERR_INVALID_ARG;
    for (int i = 0; i < c.n_models; ++i)
        if (!models[i].logits || !aligned16s(models[i].logits)) return POLYSPEC_ERR_INVALID_ARG;
    p->logits_p = models[level].logits; p->rows_p = c.rows[level]; p->rec_p = c.row_begin[level];
    p->logits_q = models[level + 1].logits; p->rows_q = c.rows[level + 1]; p->rec_q = c.row_begin[level + 1];
    p->k = c.k[level];
    p->tok_stride = c.kmax + 1;
    p->u_stride = c.kmax + 1;
    p->u_sample = c.kmax;
    p->chain = 1;
    return POLYSPEC_OK;
}

}  // namespace
}  // namespace polyspec

using namespace polyspec;

extern "C" {

// ------------------------------------------------------------------------------------------------ one level
polyspec_status polyspec_sharded_level_sizes(int B, int k, int V_local, polyspec_dtype dt, int n_ranks,
                                             size_t* workspace_bytes, size_t* stats_record_bytes, size_t* mass_record_bytes_out)
{
    if (!workspace_bytes || !stats_record_bytes || !mass_record_bytes_out) return POLYSPEC_ERR_INVALID_ARG;
    ShardSizes sz;
    const polyspec_status st = level_sizes(B, k, V_local, dt, n_ranks, &sz);
    if (st != POLYSPEC_OK) return st;
    *workspace_bytes = sz.total;
    *stats_record_bytes = align256s(stats_part_bytes(sz.rec_rows) + gather_part_bytes(B, k));
    *mass_record_bytes_out = mass_record_bytes(B);
    return POLYSPEC_OK;
}

namespace {
// Geometry of the single-level call: p rows first in the record, then q rows; the gather part follows the stats part.
polyspec_status level_params(const void* logits_p, const void* logits_q, int B, int k, int V_local, int rank, int n_ranks,
                             polyspec_dtype dt, float temperature, void* workspace, size_t workspace_bytes, ShardSizes* sz, ShardParams* p)
{
    polyspec_status st = level_sizes(B, k, V_local, dt, n_ranks, sz);
    if (st != POLYSPEC_OK) return st;
    if (!logits_p || !logits_q || !aligned16s(logits_p) || !aligned16s(logits_q)) return POLYSPEC_ERR_INVALID_ARG;
    st = base_params(B, V_local, rank, n_ranks, temperature, workspace, workspace_bytes, *sz, p);
    if (st != POLYSPEC_OK) return st;
    p->logits_p = logits_p; p->rows_p = k + 1; p->rec_p = 0;
    p->logits_q = logits_q; p->rows_q = k; p->rec_q = B * (k + 1);
    p->k = k;
    p->tok_stride = k;
    p->u_stride = k + 1;
    p->u_sample = k;
    p->rec_stride = align256s(stats_part_bytes(sz->rec_rows) + gather_part_bytes(B, k));
    p->gather_stride = p->rec_stride;
    p->gather_zp = stats_part_bytes(sz->rec_rows);
    p->gather_zq = p->gather_zp + static_cast<size_t>(B) * k * sizeof(float);
    return POLYSPEC_OK;
}
}  // namespace

polyspec_status polyspec_sharded_level_stats(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, int B, int k, int V_local, int rank, int n_ranks,
    polyspec_dtype dt, float temperature, void* stats_record, int32_t* device_status, void* workspace, size_t workspace_bytes,
    void* cuda_stream)
{
    ShardSizes sz;
    ShardParams p;
    polyspec_status st = level_params(logits_p, logits_q, B, k, V_local, rank, n_ranks, dt, temperature, workspace, workspace_bytes, &sz, &p);
    if (st != POLYSPEC_OK) return st;
    if (!draft_tokens || !stats_record || !aligned16s(stats_record)) return POLYSPEC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const void* logits[2] = {logits_p, logits_q};
    const int rows[2] = {k + 1, k}, row_begin[2] = {0, B * (k + 1)};
    st = run_stats_and_merge(logits, rows, row_begin, 2, B, V_local, dt, sz, p, stats_record, device_status, stream);
    if (st != POLYSPEC_OK) return st;
    p.tokens = draft_tokens;
    p.own_record = static_cast<unsigned char*>(stats_record);
    return launch_by_dtype(dt, shard_gather_kernel<POLYSPEC_F32>, shard_gather_kernel<POLYSPEC_BF16>, dim3(B), dim3(32), 0, stream, p);
}

polyspec_status polyspec_sharded_level_decide(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms, const int32_t* block_len,
    int B, int k, int V_local, int rank, int n_ranks, polyspec_dtype dt, float temperature, const void* stats_records,
    int32_t* accepted_len, float* p_at_draft, float* q_at_draft, void* mass_record, int32_t* device_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ShardSizes sz;
    ShardParams p;
    const polyspec_status st = level_params(logits_p, logits_q, B, k, V_local, rank, n_ranks, dt, temperature, workspace, workspace_bytes, &sz, &p);
    if (st != POLYSPEC_OK) return st;
    if (!draft_tokens || !uniforms || !stats_records || !accepted_len || !mass_record) return POLYSPEC_ERR_INVALID_ARG;
    if (!aligned16s(stats_records) || !aligned16s(mass_record)) return POLYSPEC_ERR_INVALID_ARG;
    p.tokens = draft_tokens; p.uniforms = uniforms; p.block_len = block_len;
    p.records = static_cast<const unsigned char*>(stats_records);
    p.gathers = p.records;
    p.own_mass = static_cast<double*>(mass_record);
    p.accepted_len = accepted_len; p.p_at = p_at_draft; p.q_at = q_at_draft;
    p.device_status = device_status;
    return launch_by_dtype(dt, shard_decide_kernel<POLYSPEC_F32>, shard_decide_kernel<POLYSPEC_BF16>, dim3(B), dim3(kWalkThreads),
                           static_cast<size_t>(sz.ntiles) * sizeof(float), static_cast<cudaStream_t>(cuda_stream), p);
}

polyspec_status polyspec_sharded_level_pick(
    const void* logits_p, const void* logits_q, const float* uniforms, int B, int k, int V_local, int rank, int n_ranks,
    polyspec_dtype dt, float temperature, const void* mass_records, int32_t* next_token, int32_t* device_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ShardSizes sz;
    ShardParams p;
    const polyspec_status st = level_params(logits_p, logits_q, B, k, V_local, rank, n_ranks, dt, temperature, workspace, workspace_bytes, &sz, &p);
    if (st != POLYSPEC_OK) return st;
    if (!uniforms || !mass_records || !next_token || !aligned16s(mass_records)) return POLYSPEC_ERR_INVALID_ARG;
    p.uniforms = uniforms;
    p.masses = static_cast<const unsigned char*>(mass_records);
    p.next_token = next_token;
    p.device_status = device_status;
    return launch_by_dtype(dt, shard_pick_kernel<POLYSPEC_F32>, shard_pick_kernel<POLYSPEC_BF16>, dim3(B), dim3(kWalkThreads),
                           static_cast<size_t>(sz.ntiles) * sizeof(float), static_cast<cudaStream_t>(cuda_stream), p);
}

// ------------------------------------------------------------------------------------------------ a chain
polyspec_status polyspec_sharded_chain_sizes(int n_models, const int* k, const int* rows, int B, int V_local, polyspec_dtype dt,
                                             int n_ranks, size_t* workspace_bytes, size_t* stats_record_bytes,
                                             size_t* gather_record_bytes, size_t* mass_record_bytes_out)
{
    if (!workspace_bytes || !stats_record_bytes || !gather_record_bytes || !mass_record_bytes_out) return POLYSPEC_ERR_INVALID_ARG;
    ShardSizes sz;
    ChainShape c;
    const polyspec_status st = chain_sizes(n_models, k, rows, B, V_local, dt, n_ranks, &sz, &c);
    if (st != POLYSPEC_OK) return st;
    *workspace_bytes = sz.total;
    *stats_record_bytes = align256s(stats_part_bytes(sz.rec_rows));
    *gather_record_bytes = align256s(gather_part_bytes(B, c.kmax + 1));
    *mass_record_bytes_out = mass_record_bytes(B);
    return POLYSPEC_OK;
}

namespace {
polyspec_status chain_params(const polyspec_model_logits* models, int n_models, const int* k, int level, int B, int V_local, int rank,
                             int n_ranks, polyspec_dtype dt, float temperature, void* workspace, size_t workspace_bytes,
                             ShardSizes* sz, ChainShape* c, ShardParams* p)
{
    if (!models || !k || n_models < 2 || n_models > kMaxModels) return POLYSPEC_ERR_INVALID_ARG;
    int rows[kMaxModels];
    for (int i = 0; i < n_models; ++i) rows[i] = models[i].rows;
    polyspec_status st = chain_sizes(n_models, k, rows, B, V_local, dt, n_ranks, sz, c);
    if (st != POLYSPEC_OK) return st;
    st = base_params(B, V_local, rank, n_ranks, temperature, workspace, workspace_bytes, *sz, p);
    if (st != POLYSPEC_OK) return st;
    p->rec_stride = align256s(stats_part_bytes(sz->rec_rows));
    p->gather_stride = align256s(gather_part_bytes(B, c->kmax + 1));
    p->gather_zp = 0;
    p->gather_zq = static_cast<size_t>(B) * (c->kmax + 1) * sizeof(float);
    return chain_level_params(models, *c, level, p);
}
}  // namespace

polyspec_status polyspec_sharded_chain_stats(
    const polyspec_model_logits* models, int n_models, const int* k, int B, int V_local, int rank, int n_ranks, polyspec_dtype dt,
    float temperature, void* stats_record, int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ShardSizes sz;
    ChainShape c;
    ShardParams p;
    polyspec_status st = chain_params(models, n_models, k, 0, B, V_local, rank, n_ranks, dt, temperature, workspace, workspace_bytes, &sz, &c, &p);
    if (st != POLYSPEC_OK) return st;
    if (!stats_record || !aligned16s(stats_record)) return POLYSPEC_ERR_INVALID_ARG;
    const void* logits[kMaxModels];
    for (int i = 0; i < n_models; ++i) logits[i] = models[i].logits;
    return run_stats_and_merge(logits, c.rows, c.row_begin, n_models, B, V_local, dt, sz, p, stats_record, device_status,
                               static_cast<cudaStream_t>(cuda_stream));
}

polyspec_status polyspec_sharded_chain_gather(
    const polyspec_model_logits* models, int n_models, const int* k, int level, const int32_t* block_tokens, const int32_t* block_len,
    int B, int V_local, int rank, int n_ranks, polyspec_dtype dt, void* gather_record, void* workspace, size_t workspace_bytes,
    void* cuda_stream)
{
    ShardSizes sz;
    ChainShape c;
    ShardParams p;
    const polyspec_status st = chain_params(models, n_models, k, level, B, V_local, rank, n_ranks, dt, 1.0f, workspace, workspace_bytes, &sz, &c, &p);
    if (st != POLYSPEC_OK) return st;
    if (!block_tokens || !block_len || !gather_record || !aligned16s(gather_record)) return POLYSPEC_ERR_INVALID_ARG;
    p.tokens = block_tokens; p.block_len = block_len;
    p.own_record = static_cast<unsigned char*>(gather_record);
    return launch_by_dtype(dt, shard_gather_kernel<POLYSPEC_F32>, shard_gather_kernel<POLYSPEC_BF16>, dim3(B), dim3(32), 0,
                           static_cast<cudaStream_t>(cuda_stream), p);
}

polyspec_status polyspec_sharded_chain_decide(
    const polyspec_model_logits* models, int n_models, const int* k, int level, const int32_t* block_tokens, const int32_t* block_len,
    const float* uniforms, int B, int V_local, int rank, int n_ranks, polyspec_dtype dt, float temperature,
    const void* stats_records, const void* gather_records, int32_t* accepted_len, int32_t* block_len_out, void* mass_record,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ShardSizes sz;
    ChainShape c;
    ShardParams p;
    const polyspec_status st = chain_params(models, n_models, k, level, B, V_local, rank, n_ranks, dt, temperature, workspace, workspace_bytes, &sz, &c, &p);
    if (st != POLYSPEC_OK) return st;
    if (!block_tokens || !block_len || !uniforms || !stats_records || !gather_records || !accepted_len || !mass_record)
        return POLYSPEC_ERR_INVALID_ARG;
    if (!aligned16s(stats_records) || !aligned16s(gather_records) || !aligned16s(mass_record)) return POLYSPEC_ERR_INVALID_ARG;
    p.tokens = block_tokens; p.block_len = block_len;
    p.uniforms = uniforms + static_cast<size_t>(level) * B * (c.kmax + 1);
    p.records = static_cast<const unsigned char*>(stats_records);
    p.gathers = static_cast<const unsigned char*>(gather_records);
    p.own_mass = static_cast<double*>(mass_record);
    p.accepted_len = accepted_len + static_cast<size_t>(level) * B;
    p.block_len_out = block_len_out ? block_len_out + static_cast<size_t>(level) * B : nullptr;
    p.device_status = device_status;
    return launch_by_dtype(dt, shard_decide_kernel<POLYSPEC_F32>, shard_decide_kernel<POLYSPEC_BF16>, dim3(B), dim3(kWalkThreads),
                           static_cast<size_t>(sz.ntiles) * sizeof(float), static_cast<cudaStream_t>(cuda_stream), p);
}

polyspec_status polyspec_sharded_chain_pick(
    const polyspec_model_logits* models, int n_models, const int* k, int level, const float* uniforms, int B, int V_local, int rank,
    int n_ranks, polyspec_dtype dt, float temperature, const void* mass_records, int32_t* next_token, int32_t* device_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ShardSizes sz;
    ChainShape c;
    ShardParams p;
    const polyspec_status st = chain_params(models, n_models, k, level, B, V_local, rank, n_ranks, dt, temperature, workspace, workspace_bytes, &sz, &c, &p);
    if (st != POLYSPEC_OK) return st;
    if (!uniforms || !mass_records || !next_token || !aligned16s(mass_records)) return POLYSPEC_ERR_INVALID_ARG;
    p.uniforms = uniforms + static_cast<size_t>(level) * B * (c.kmax + 1);
    p.masses = static_cast<const unsigned char*>(mass_records);
    p.next_token = next_token;
    p.device_status = device_status;
    return launch_by_dtype(dt, shard_pick_kernel<POLYSPEC_F32>, shard_pick_kernel<POLYSPEC_BF16>, dim3(B), dim3(kWalkThreads),
                           static_cast<size_t>(sz.ntiles) * sizeof(float), static_cast<cudaStream_t>(cuda_stream), p);
}

polyspec_status polyspec_sharded_chain_handoff(
    int n_models, const int* k, int level, int B, const int32_t* accepted_len, const int32_t* next_token, int32_t* block_tokens,
    int32_t* block_len, int32_t* out_tokens, int32_t* out_len, void* cuda_stream)
{
    if (n_models < 2 || n_models > kMaxModels || !k || level < 0 || level >= n_models - 1 || B <= 0) return POLYSPEC_ERR_INVALID_ARG;
    if (!accepted_len || !next_token || !block_tokens || !block_len) return POLYSPEC_ERR_INVALID_ARG;
    int kmax = 0;
    for (int l = 0; l < n_models - 1; ++l) {
        if (k[l] < 1 || k[l] > kMaxK) return POLYSPEC_ERR_INVALID_ARG;
        if (k[l] > kmax) kmax = k[l];
    }
    const int slots = kmax + 1;
    shard_handoff_kernel<<<(B + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        accepted_len + static_cast<size_t>(level) * B, next_token, block_tokens, block_len,
        out_tokens ? out_tokens + static_cast<size_t>(level) * B * slots : nullptr,
        out_len ? out_len + static_cast<size_t>(level) * B : nullptr, B, slots);
    if (cuda_failed(cudaGetLastError())) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

}  // extern "C"
