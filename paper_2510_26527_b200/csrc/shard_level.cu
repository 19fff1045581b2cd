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
#include <cmath>

#include "polyspec_kernels.cuh"
#include "walk_device.cuh"

namespace polyspec {
namespace {

using namespace walkdev;

constexpr int kMaxRanks = 64;
constexpr double kLog2eS = 1.4426950408889634074;

inline size_t align256s(size_t x) { return (x + 255) / 256 * 256; }

// What one rank contributes to exchange 1, for B sequences and blocks of k:
//   double Z[B][2k+1], float E[B][2k+1]   normaliser of its slice of p rows 0..k, then q rows 0..k-1
//   float zp[B][k], zq[B][k]              logits at the block tokens it owns (0 for the others)
struct StatsRecordLayout {
    size_t Z, E, zp, zq, total;
};
__host__ __device__ inline StatsRecordLayout stats_record_layout(int B, int k)
{
    StatsRecordLayout l;
    const size_t rows = static_cast<size_t>(B) * (2 * k + 1);
    l.Z = 0;
    l.E = l.Z + rows * sizeof(double);
    l.zp = l.E + rows * sizeof(float);
    l.zq = l.zp + static_cast<size_t>(B) * k * sizeof(float);
    l.total = (l.zq + static_cast<size_t>(B) * k * sizeof(float) + 255) / 256 * 256;
    return l;
}
// Exchange 2: double mass[B] (what the slice holds of the distribution being sampled), double pmass[B]
// (what it holds of P at the same row, filled in when it holds nothing of the residual: needed if no rank does).
__host__ __device__ inline size_t mass_record_bytes(int B) { return (static_cast<size_t>(B) * 16 + 255) / 256 * 256; }

// What `decide` leaves for `pick`, per sequence.
struct Decision {
    double Zp, Zq;
    float Ep, Eq;
    int a;          // accepted length, -1: unusable input
    int use_q;      // row a is a rejection (sample the residual) rather than the bonus row
};

struct ShardParams {
    const void* logits_p;       // [B, k+1, V_local]
    const void* logits_q;       // [B, k, V_local]
    const int32_t* draft_tokens;
    const float* uniforms;      // [B, k+1]
    const int32_t* block_len;   // [B] or nullptr
    int B, k, V_local, rank, n_ranks;
    float c;
    int parts;
    const float2* partials;     // [(B (k+1) + B k), parts]
    unsigned char* own_record;          // stats: out
    const unsigned char* records;       // decide: [n_ranks][record bytes]
    double* own_mass;                   // decide: out (mass[B], pmass[B])
    const unsigned char* masses;        // pick: [n_ranks][mass bytes]
    Decision* decision;         // [B]
    float* tile_sums;           // [B][ntiles]
    int32_t* accepted_len;
    int32_t* next_token;
    float* p_at;
    float* q_at;
    int32_t* device_status;
};

template <int DT>
__global__ void __launch_bounds__(256) shard_record_kernel(const ShardParams p)
{
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k = p.k, nrow = 2 * k + 1;
    const StatsRecordLayout L = stats_record_layout(p.B, k);
    double* Zs = reinterpret_cast<double*>(p.own_record + L.Z) + static_cast<size_t>(b) * nrow;
    float* Es = reinterpret_cast<float*>(p.own_record + L.E) + static_cast<size_t>(b) * nrow;
    const int grow_p = b * (k + 1), grow_q = p.B * (k + 1) + b * k;
    for (int r = warp; r < nrow; r += 8) {
        const int g = r <= k ? grow_p + r : grow_q + (r - k - 1);
        const RowStat st = merge_partials(p.partials + static_cast<size_t>(g) * p.parts, p.parts, lane);
        if (lane == 0) { Zs[r] = st.Z; Es[r] = st.E; }
    }
    if (tid < k) {
        constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
        const size_t row_bytes = static_cast<size_t>(p.V_local) * ELEM;
        const int x = p.draft_tokens[static_cast<size_t>(b) * k + tid] - p.rank * p.V_local;
        float zp = 0.0f, zq = 0.0f;
        if (x >= 0 && x < p.V_local) {
            zp = load_logit<DT>(static_cast<const char*>(p.logits_p) + (static_cast<size_t>(b) * (k + 1) + tid) * row_bytes, x);
            zq = load_logit<DT>(static_cast<const char*>(p.logits_q) + (static_cast<size_t>(b) * k + tid) * row_bytes, x);
        }
        reinterpret_cast<float*>(p.own_record + L.zp)[static_cast<size_t>(b) * k + tid] = zp;
        reinterpret_cast<float*>(p.own_record + L.zq)[static_cast<size_t>(b) * k + tid] = zq;
    }
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
    __shared__ RowStat st[2 * kMaxK + 1];
    __shared__ int sh_a, sh_bad;
    __shared__ double sh_share, sh_pshare;

    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int k = p.k, nrow = 2 * k + 1, R = p.n_ranks;
    const StatsRecordLayout L = stats_record_layout(p.B, k);
    const size_t row_bytes = static_cast<size_t>(p.V_local) * ELEM;
    const double cd = static_cast<double>(p.c);
    int m = k;
    if (p.block_len) m = max(0, min(k, p.block_len[b]));
    const int V_all = p.V_local * R;
    double* mass_out = p.own_mass;
    Decision* dec = p.decision + b;

    // whole-row normalisers: the ranks' (E, Z) rebased to the largest E (an exact scaling) and added in rank order
    if (tid < nrow) {
        float E = kEmptyRef;
        for (int r = 0; r < R; ++r)
            E = fmaxf(E, reinterpret_cast<const float*>(p.records + r * L.total + L.E)[static_cast<size_t>(b) * nrow + tid]);
        double Z = 0.0;
        for (int r = 0; r < R; ++r) {
            const unsigned char* rec = p.records + r * L.total;
            const float Er = reinterpret_cast<const float*>(rec + L.E)[static_cast<size_t>(b) * nrow + tid];
            Z += scale_pow2(reinterpret_cast<const double*>(rec + L.Z)[static_cast<size_t>(b) * nrow + tid], Er - E);
        }
        st[tid].E = E;
        st[tid].Z = Z;
    }
    __syncthreads();

    // accept tests (warp 0; m <= 32), exactly as in the unsharded walk
    if (tid < 32) {
        bool rej = false, bad = false;
        float pf = 0.0f, qf = 0.0f;
        if (tid < m) {
            const int x = p.draft_tokens[static_cast<size_t>(b) * k + tid];
            const RowStat sp = st[tid], sq = st[k + 1 + tid];
            if (x < 0 || x >= V_all || !stat_ok(sp) || !stat_ok(sq)) {
                bad = true;
            } else {
                const unsigned char* rec = p.records + (x / p.V_local) * L.total;       // the rank that owns the token
                const float zp = reinterpret_cast<const float*>(rec + L.zp)[static_cast<size_t>(b) * k + tid];
                const float zq = reinterpret_cast<const float*>(rec + L.zq)[static_cast<size_t>(b) * k + tid];
                const double P = exp2(static_cast<double>(zp) * cd - static_cast<double>(sp.E)) / sp.Z;
                const double Q = exp2(static_cast<double>(zq) * cd - static_cast<double>(sq.E)) / sq.Z;
                const double u = static_cast<double>(p.uniforms[static_cast<size_t>(b) * (k + 1) + tid]);
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
            if (!isbad && first_rej == m && !stat_ok(st[m])) isbad = 1;     // bonus row unusable
            sh_a = first_rej;
            sh_bad = isbad;
        }
    }
    __syncthreads();
    const int a = sh_a;
    if (sh_bad) {
        if (tid == 0) {
            p.accepted_len[b] = -1;
            dec->a = -1; dec->use_q = 0; dec->Ep = dec->Eq = 0.0f; dec->Zp = dec->Zq = 1.0;
            mass_out[b] = 0.0;
            mass_out[p.B + b] = 0.0;
            if (p.device_status) atomicCAS(p.device_status, 0, static_cast<int>(POLYSPEC_ERR_BAD_INPUT_ON_DEVICE));
        }
        return;
    }

    // this slice's share of row a: tile sums of the residual (or of P for the bonus row), kept for the search
    const bool use_q = a < m;
    const RowStat sp = st[a];
    const RowStat sq = use_q ? st[k + 1 + a] : sp;
    const void* prow = static_cast<const char*>(p.logits_p) + (static_cast<size_t>(b) * (k + 1) + a) * row_bytes;
    const void* qrow = static_cast<const char*>(p.logits_q) + (static_cast<size_t>(b) * k + (use_q ? a : 0)) * row_bytes;
    const int ntiles = (p.V_local + kTile - 1) / kTile;
    const float iZp = static_cast<float>(1.0 / sp.Z);
    const float iZq = use_q ? static_cast<float>(1.0 / sq.Z) : 0.0f;
    tiles_pass<DT>(prow, qrow, p.V_local, p.c, sp.E, iZp, sq.E, iZq, use_q, tile_sum, 0, ntiles);
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
        tiles_pass<DT>(prow, qrow, p.V_local, p.c, sp.E, iZp, sq.E, 0.0f, false, tile_sum, 0, ntiles);
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
    const int k = p.k, R = p.n_ranks;
    const Decision dec = p.decision[b];
    if (dec.a < 0) {
        if (tid == 0) p.next_token[b] = -1;
        return;
    }
    const size_t mbytes = mass_record_bytes(p.B);
    const size_t row_bytes = static_cast<size_t>(p.V_local) * ELEM;
    const int ntiles = (p.V_local + kTile - 1) / kTile;
    bool use_q = dec.use_q != 0;
    const void* prow = static_cast<const char*>(p.logits_p) + (static_cast<size_t>(b) * (k + 1) + dec.a) * row_bytes;
    const void* qrow = static_cast<const char*>(p.logits_q) + (static_cast<size_t>(b) * k + (use_q ? dec.a : 0)) * row_bytes;
    const float iZp = static_cast<float>(1.0 / dec.Zp);
    const float iZq = use_q ? static_cast<float>(1.0 / dec.Zq) : 0.0f;

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
        const float u = p.uniforms[static_cast<size_t>(b) * (k + 1) + k];
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
            token = pick_in_share<DT>(prow, qrow, p.V_local, p.c, dec.Ep, iZp, dec.Eq, iZq, use_q, tile_sum, t0, t1, mine, incl,
                                      base, target, lane);
            if (token >= 0) token += p.rank * p.V_local;
        }
        if (lane == 0) p.next_token[b] = token;
    }
}

struct ShardSizes {
    StatsPlan plan;
    size_t partials, decision, tiles, total;
    int ntiles;
};

polyspec_status shard_sizes(int B, int k, int V_local, polyspec_dtype dt, int n_ranks, ShardSizes* s)
{
    if (B <= 0 || k < 1 || k > kMaxK || V_local <= 0 || n_ranks < 1 || n_ranks > kMaxRanks) return POLYSPEC_ERR_INVALID_ARG;
    if (dt != POLYSPEC_F32 && dt != POLYSPEC_BF16) return POLYSPEC_ERR_INVALID_ARG;
    if (V_local % 8 != 0 || V_local > kMaxV) return POLYSPEC_ERR_UNSUPPORTED;
    if (static_cast<long long>(V_local) * n_ranks > 0x7fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
    const long long rows = static_cast<long long>(B) * (2 * k + 1);
    if (rows > 0x3fffffffLL) return POLYSPEC_ERR_UNSUPPORTED;
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

bool aligned16s(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

polyspec_status shard_params(const void* logits_p, const void* logits_q, int B, int k, int V_local, int rank, int n_ranks,
                             polyspec_dtype dt, float temperature, void* workspace, size_t workspace_bytes,
                             ShardSizes* sz, ShardParams* p)
{
    polyspec_status st = shard_sizes(B, k, V_local, dt, n_ranks, sz);
    if (st != POLYSPEC_OK) return st;
    if (rank < 0 || rank >= n_ranks) return POLYSPEC_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !std::isfinite(temperature)) return POLYSPEC_ERR_INVALID_ARG;
    if (!logits_p || !logits_q || !aligned16s(logits_p) || !aligned16s(logits_q)) return POLYSPEC_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return POLYSPEC_ERR_INVALID_ARG;
    if (workspace_bytes < sz->total) return POLYSPEC_ERR_WORKSPACE;
    *p = ShardParams{};
    p->logits_p = logits_p; p->logits_q = logits_q;
    p->B = B; p->k = k; p->V_local = V_local; p->rank = rank; p->n_ranks = n_ranks;
    p->c = static_cast<float>(kLog2eS / static_cast<double>(temperature));
    p->parts = sz->plan.parts;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    p->partials = reinterpret_cast<const float2*>(ws + sz->partials);
    p->decision = reinterpret_cast<Decision*>(ws + sz->decision);
    p->tile_sums = reinterpret_cast<float*>(ws + sz->tiles);
    return POLYSPEC_OK;
}

}  // namespace
}  // namespace polyspec

using namespace polyspec;

extern "C" {

polyspec_status polyspec_sharded_level_sizes(int B, int k, int V_local, polyspec_dtype dt, int n_ranks,
                                             size_t* workspace_bytes, size_t* stats_record_bytes, size_t* mass_record_bytes_out)
{
    if (!workspace_bytes || !stats_record_bytes || !mass_record_bytes_out) return POLYSPEC_ERR_INVALID_ARG;
    ShardSizes sz;
    const polyspec_status st = shard_sizes(B, k, V_local, dt, n_ranks, &sz);
    if (st != POLYSPEC_OK) return st;
    *workspace_bytes = sz.total;
    *stats_record_bytes = stats_record_layout(B, k).total;
    *mass_record_bytes_out = mass_record_bytes(B);
    return POLYSPEC_OK;
}

polyspec_status polyspec_sharded_level_stats(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, int B, int k, int V_local, int rank, int n_ranks,
    polyspec_dtype dt, float temperature, void* stats_record, int32_t* device_status, void* workspace, size_t workspace_bytes,
    void* cuda_stream)
{
    ShardSizes sz;
    ShardParams p;
    const polyspec_status st = shard_params(logits_p, logits_q, B, k, V_local, rank, n_ranks, dt, temperature, workspace,
                                            workspace_bytes, &sz, &p);
    if (st != POLYSPEC_OK) return st;
    if (!draft_tokens || !stats_record || (reinterpret_cast<uintptr_t>(stats_record) & 15u) != 0) return POLYSPEC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the row-statistics pass over this rank's slices: p rows first, then q rows
    StatsParams sp;
    sp.t.n_models = 2;
    for (int i = 0; i < kMaxModels; ++i) { sp.t.logits[i] = nullptr; sp.t.rows[i] = 0; sp.t.row_begin[i] = 0; }
    sp.t.logits[0] = logits_p; sp.t.rows[0] = k + 1; sp.t.row_begin[0] = 0;
    sp.t.logits[1] = logits_q; sp.t.rows[1] = k; sp.t.row_begin[1] = B * (k + 1);
    for (int i = 2; i <= kMaxModels; ++i) sp.t.row_begin[i] = B * (2 * k + 1);
    sp.V = V_local;
    sp.seg = sz.plan.seg;
    sp.parts = sz.plan.parts;
    sp.n_items = static_cast<int>(sz.plan.n_items);
    sp.c = p.c;
    sp.partials = const_cast<float2*>(p.partials);
    sp.status = device_status;
    if (cuda_failed(launch_stats(dt, sp, stream))) return POLYSPEC_ERR_CUDA;
    p.draft_tokens = draft_tokens;
    p.own_record = static_cast<unsigned char*>(stats_record);
    p.device_status = device_status;
    if (dt == POLYSPEC_BF16) shard_record_kernel<POLYSPEC_BF16><<<B, 256, 0, stream>>>(p);
    else shard_record_kernel<POLYSPEC_F32><<<B, 256, 0, stream>>>(p);
    if (cuda_failed(cudaGetLastError())) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

polyspec_status polyspec_sharded_level_decide(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms, const int32_t* block_len,
    int B, int k, int V_local, int rank, int n_ranks, polyspec_dtype dt, float temperature, const void* stats_records,
    int32_t* accepted_len, float* p_at_draft, float* q_at_draft, void* mass_record, int32_t* device_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ShardSizes sz;
    ShardParams p;
    const polyspec_status st = shard_params(logits_p, logits_q, B, k, V_local, rank, n_ranks, dt, temperature, workspace,
                                            workspace_bytes, &sz, &p);
    if (st != POLYSPEC_OK) return st;
    if (!draft_tokens || !uniforms || !stats_records || !accepted_len || !mass_record) return POLYSPEC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(stats_records) & 15u) != 0 || (reinterpret_cast<uintptr_t>(mass_record) & 15u) != 0)
        return POLYSPEC_ERR_INVALID_ARG;
    p.draft_tokens = draft_tokens; p.uniforms = uniforms; p.block_len = block_len;
    p.records = static_cast<const unsigned char*>(stats_records);
    p.own_mass = static_cast<double*>(mass_record);
    p.accepted_len = accepted_len; p.p_at = p_at_draft; p.q_at = q_at_draft;
    p.device_status = device_status;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t smem = static_cast<size_t>(sz.ntiles) * sizeof(float);
    if (dt == POLYSPEC_BF16) shard_decide_kernel<POLYSPEC_BF16><<<B, kWalkThreads, smem, stream>>>(p);
    else shard_decide_kernel<POLYSPEC_F32><<<B, kWalkThreads, smem, stream>>>(p);
    if (cuda_failed(cudaGetLastError())) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

polyspec_status polyspec_sharded_level_pick(
    const void* logits_p, const void* logits_q, const float* uniforms, int B, int k, int V_local, int rank, int n_ranks,
    polyspec_dtype dt, float temperature, const void* mass_records, int32_t* next_token, int32_t* device_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    ShardSizes sz;
    ShardParams p;
    const polyspec_status st = shard_params(logits_p, logits_q, B, k, V_local, rank, n_ranks, dt, temperature, workspace,
                                            workspace_bytes, &sz, &p);
    if (st != POLYSPEC_OK) return st;
    if (!uniforms || !mass_records || !next_token) return POLYSPEC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(mass_records) & 15u) != 0) return POLYSPEC_ERR_INVALID_ARG;
    p.uniforms = uniforms;
    p.masses = static_cast<const unsigned char*>(mass_records);
    p.next_token = next_token;
    p.device_status = device_status;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t smem = static_cast<size_t>(sz.ntiles) * sizeof(float);
    if (dt == POLYSPEC_BF16) shard_pick_kernel<POLYSPEC_BF16><<<B, kWalkThreads, smem, stream>>>(p);
    else shard_pick_kernel<POLYSPEC_F32><<<B, kWalkThreads, smem, stream>>>(p);
    if (cuda_failed(cudaGetLastError())) return POLYSPEC_ERR_CUDA;
    return POLYSPEC_OK;
}

}  // extern "C"
