// The whole chain in ONE launch: the temperature-softmax normaliser of every logits row of every model
// (Section 3.1's p_i over the vocabulary), read once from HBM, and -- trailing that stream by a few
// microseconds -- every sequence's decisions: Algorithm 1's Verify loop with its break at the first failure,
// the replacement / bonus token, and the hand-off from level to level (the block is checked bottom-up, by
// M_{n-1} first and M_1 last).
//
// Why one launch.  The second pass over a row pair (the residual max(0, P - Q) needs both normalisers first)
// re-reads two rows per level and sequence.  After a separate statistics launch those rows have long left L2
// and come from HBM again (up to 18 % more traffic on the four-level workload, on top of a dependent chain of
// memory round trips per level).  Here rows are streamed in POSITION-MAJOR order -- position 0 of every
// sequence and model, then position 1, ... -- and a sequence's decision at a position is taken as soon as the
// rows of that position are complete, so the rows it re-reads were read microseconds earlier and are still in L2.
//
// How.  A persistent grid, one CTA per SM, every warp a self-contained pipeline as in the row-statistics kernel
// (1-D bulk TMA copies into a private shared-memory ring, completion on an mbarrier).  Nothing ever waits for
// another warp.  Progress is continuation passing with counters:
//   - a warp that finishes the last segment of a row (atomic counter per row) runs that sequence's state machine
//     as far as the completed rows allow: merge the partials, gather the logits at the block token, accept test
//     in double precision; positions are visited in order and, inside a position, levels bottom-up, which is
//     exactly the order the rows arrive in;
//   - when a level needs its token, the pass over the row pair is cut into jobs that go to a queue in global
//     memory; every warp looks there before it claims its next row segment; the warp that finishes the last job
//     (atomic counter) resumes the state machine: scan of the tile sums, rescan of one tile, token, hand-off;
//   - the state machine of a sequence is serialised by a try-lock with a wake-up count (a warp that finds it
//     taken leaves a note and goes on; the holder runs again before it lets go).
// All arithmetic is that of the two-launch path (same partials, same merge, same residual, same scan order), so
// the results are bit-identical to polyspec_chain_row_stats + polyspec_chain_walk and independent of scheduling.
//
// Waits: only the bounded mbarrier waits of the copies.  After the stream has ended a few warps per CTA keep
// looking for residual jobs until every sequence is finished, for a bounded number of polls; correctness never
// depends on them (a warp that enqueues jobs is itself about to look into the queue).
#include <mutex>

#include "polyspec_kernels.cuh"
#include "stream_device.cuh"
#include "walk_device.cuh"

namespace polyspec {

// One sequence's progress.  Zeroed before the launch; read and written through volatile accesses only (the
// warps that touch it sit on different SMs), by the warp that holds `lock`.
struct ChainSeqState {
    int lock;                      // 0 free, 1 held
    int pending;                   // wake-ups since the holder last looked
    int started, finished;
    int pos, lvl;                  // next step: position, then level (bottom-up inside a position)
    int sampling;                  // 1 while the jobs of the sample of level `lvl` at position `pos` are in flight
    int jobs_left;
    int len_bottom;                // tokens the bottom level is presented
    int status[kMaxLevels];        // 0 running, 1 done, 2 unusable input at this level or below
    int acc[kMaxLevels];           // positions accepted so far; the accepted length once done
    int s_use_q;                   // the sample in flight: residual of (p, q) or p alone, and the two normalisers
    float s_Ep, s_Eq, s_iZp, s_iZq;
    int tok[kMaxK + 1];            // the stream as the level about to look at a position sees it
    int pad[3];
};
static_assert(sizeof(ChainSeqState) % 16 == 0, "state records are laid out back to back");

namespace {

using namespace streamdev;
using walkdev::RowStat;

constexpr int kRun = 0, kDone = 1, kDead = 2;
constexpr int kFifo = 8;                       // claimed-item slots per warp (needs kStages + 1)
constexpr int kLingerWarps = 4;                // warps per CTA that keep serving residual jobs after the stream
constexpr int kLingerPolls = 1 << 15;
static_assert(kStages + 1 <= kFifo, "claim fifo too small");

// Position-major order: work item -> (row segment, global row, sequence).
template <int DT>
__device__ __forceinline__ void decode_item(const ChainParams& p, int item, const char** src, uint32_t* bytes, int* grow, int* seq, int* part_out)
{
    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    const RowTable& t = p.w.t;
    const int parts = p.w.parts;
    const int slot = item / parts;
    const int part = item - slot * parts;
    int j = 0;
    while (j + 1 < p.max_rows && slot >= p.pos_begin[j + 1]) ++j;
    int nmod = 0;
    for (int i = 0; i < t.n_models; ++i) nmod += t.rows[i] > j;
    const int rs = slot - p.pos_begin[j];
    const int b = rs / nmod;
    int r = rs - b * nmod;
    int mi = t.n_models - 1;                    // the r-th model, bottom-up, that has a row j
    for (; mi > 0; --mi) {
        if (t.rows[mi] > j) {
            if (r == 0) break;
            --r;
        }
    }
    const int v0 = part * p.seg;
    const int v1 = min(p.w.V, v0 + p.seg);
    *src = static_cast<const char*>(t.logits[mi]) + ((static_cast<size_t>(b) * t.rows[mi] + j) * p.w.V + v0) * ELEM;
    *bytes = static_cast<uint32_t>((v1 - v0) * ELEM);
    *grow = t.row_begin[mi] + b * t.rows[mi] + j;
    *seq = b;
    *part_out = part;
}

// ---------------------------------------------------------------------------------- residual job queue
// Slots are written once per launch (capacity = the most jobs a launch can enqueue), as one 64-bit word
// (ticket + 1) << 32 | payload, so a reader sees a slot either empty or complete.
__device__ __forceinline__ bool queue_pop(const ChainParams& p, int lane, unsigned int* payload)
{
    unsigned int got = 0xffffffffu;
    if (lane == 0) {
        unsigned int h = *reinterpret_cast<volatile unsigned int*>(&p.ctl->q_head);
        for (int tries = 0; tries < 4 && h < p.q_cap; ++tries) {
            const unsigned long long s = *reinterpret_cast<volatile unsigned long long*>(p.queue + h);
            if (static_cast<unsigned int>(s >> 32) != h + 1u) break;             // nothing published there (yet)
            const unsigned int seen = atomicCAS(&p.ctl->q_head, h, h + 1u);
            if (seen == h) {
                got = static_cast<unsigned int>(s & 0xffffffffull);
                break;
            }
            h = seen;                                                             // another warp took it: look at the next one
        }
    }
    got = __shfl_sync(0xffffffffu, got, 0);
    if (got == 0xffffffffu) return false;
    *payload = got;
    return true;
}

__device__ __forceinline__ void queue_push(const ChainParams& p, int lane, int b, int n)
{
    unsigned int base = 0;
    if (lane == 0) base = atomicAdd(&p.ctl->q_tail, static_cast<unsigned int>(n));
    base = __shfl_sync(0xffffffffu, base, 0);
    if (base + static_cast<unsigned int>(n) > p.q_cap) {          // cannot happen: the capacity covers every job of a launch
        if (lane == 0 && p.w.device_status) atomicCAS(p.w.device_status, 0, static_cast<int>(POLYSPEC_ERR_TIMEOUT));
        return;
    }
    for (int i = lane; i < n; i += 32) {
        const unsigned long long word = (static_cast<unsigned long long>(base + i + 1u) << 32) |
                                        static_cast<unsigned int>(b * p.n_rsegs + i);
        *reinterpret_cast<volatile unsigned long long*>(p.queue + base + i) = word;
    }
}

// ---------------------------------------------------------------------------------- the per-sequence state machine
template <int DT> __device__ __noinline__ void advance(const ChainParams& p, int b);

template <int DT>
__device__ __forceinline__ const char* row_ptr(const ChainParams& p, int model, int b, int j)
{
    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    return static_cast<const char*>(p.w.t.logits[model]) + (static_cast<size_t>(b) * p.w.t.rows[model] + j) * p.w.V * ELEM;
}

// The sums of the residual (or of P) over tiles [tlo, thi) of one row pair, by one warp; each tile's sum is computed
// exactly as in walkdev::tiles_pass and in the rescan of pick_in_share.
template <int DT>
__device__ __forceinline__ void warp_tiles_pass(const void* prow, const void* qrow, int V, float c, float Ep, float iZp, float Eq,
                                                float iZq, bool use_q, float* tile_sum, int tlo, int thi, int lane)
{
    constexpr int kU = (DT == POLYSPEC_BF16) ? 2 : 1;
    for (int t0 = tlo; t0 < thi; t0 += kU) {
        walkdev::RawTile<DT> rp[kU], rq[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int v = (t0 + u) * kTile + lane * 8;
            if (t0 + u < thi && v < V) {
                rp[u].load(prow, v);
                if (use_q) rq[u].load(qrow, v);
            }
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            if (t0 + u < thi) {                     // warp-uniform
                const int v = (t0 + u) * kTile + lane * 8;
                float r[8];
                if (v < V) {
                    float zp[8], zq[8];
                    rp[u].unpack(zp);
                    if (use_q) rq[u].unpack(zq);
#pragma unroll
                    for (int e = 0; e < 8; ++e) r[e] = walkdev::resid(zp[e], use_q ? zq[e] : 0.0f, c, Ep, iZp, Eq, iZq, use_q);
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) r[e] = 0.0f;
                }
                float x = walkdev::sum8(r);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) x = __fadd_rn(x, __shfl_xor_sync(0xffffffffu, x, o));
                if (lane == 0) tile_sum[t0 + u] = x;
            }
        }
    }
}

// One residual job: the tile sums of one stretch of the row pair a sequence is sampling from.
template <int DT>
__device__ __noinline__ void run_resid_job(const ChainParams& p, unsigned int payload)
{
    const int lane = threadIdx.x & 31;
    const int b = static_cast<int>(payload / static_cast<unsigned int>(p.n_rsegs));
    const int seg = static_cast<int>(payload - static_cast<unsigned int>(b) * p.n_rsegs);
    __threadfence();                                    // the state below was written before the job was published
    volatile ChainSeqState* st = p.seq + b;
    const int l = st->lvl, j = st->pos;
    const bool use_q = st->s_use_q != 0;
    const float Ep = st->s_Ep, Eq = st->s_Eq, iZp = st->s_iZp, iZq = st->s_iZq;
    const char* prow = row_ptr<DT>(p, l, b, j);
    const char* qrow = use_q ? row_ptr<DT>(p, l + 1, b, j) : prow;
    const int tlo = seg * p.rseg_tiles, thi = min(tlo + p.rseg_tiles, p.ntiles);
    warp_tiles_pass<DT>(prow, qrow, p.w.V, p.w.c, Ep, iZp, Eq, iZq, use_q, p.tile_sum + static_cast<size_t>(b) * p.ntiles, tlo, thi, lane);
    __syncwarp();
    int last = 0;
    if (lane == 0) {
        __threadfence();
        last = atomicSub(const_cast<int*>(&st->jobs_left), 1) == 1;
    }
    if (__shfl_sync(0xffffffffu, last, 0)) advance<DT>(p, b);
}

template <int DT>
__device__ __noinline__ void run_machine(const ChainParams& p, int b, volatile ChainSeqState* st)
{
    const WalkParams& w = p.w;
    const RowTable& t = w.t;
    const int lane = threadIdx.x & 31;
    const int L = w.n_levels;
    const double cd = static_cast<double>(w.c);
    const bool probes = (w.p_at != nullptr) || (w.q_at != nullptr);        // single-level calls only
    float* ts = p.tile_sum + static_cast<size_t>(b) * p.ntiles;

    if (st->finished) return;
    if (!st->started) {
        const int kb = w.k[L - 1];
        int len = kb;
        if (w.bottom_len) len = max(0, min(len, w.bottom_len[b]));
        for (int j = lane; j < kb; j += 32) st->tok[j] = w.draft_tokens[static_cast<size_t>(b) * kb + j];
        if (probes)
            for (int j = lane; j < w.k[0]; j += 32) {
                if (w.p_at) w.p_at[static_cast<size_t>(b) * w.k[0] + j] = 0.0f;
                if (w.q_at) w.q_at[static_cast<size_t>(b) * w.k[0] + j] = 0.0f;
            }
        if (lane == 0) {
            st->len_bottom = len;
            st->pos = 0;
            st->lvl = L - 1;
            st->started = 1;
        }
        __syncwarp();
    }

    // a level (and every level above it) met unusable input: they report -1
    auto kill = [&](int l) {
        for (int ll = l; ll >= 0; --ll) {
            const size_t lb = static_cast<size_t>(ll) * w.B + b;
            if (lane == 0) {
                st->status[ll] = kDead;
                w.accepted_len[lb] = -1;
                if (w.block_len) w.block_len[lb] = -1;
                if (w.out_len) w.out_len[lb] = -1;
            }
            if (w.out_tokens)
                for (int i = lane; i <= w.kmax; i += 32) w.out_tokens[lb * (w.kmax + 1) + i] = -1;
        }
        if (lane == 0) {
            if (w.next_token) w.next_token[b] = -1;
            if (w.device_status) atomicCAS(w.device_status, 0, static_cast<int>(POLYSPEC_ERR_BAD_INPUT_ON_DEVICE));
        }
        __syncwarp();
    };
    auto step_on = [&](int l, int j) {
        if (lane == 0) {
            if (l > 0) st->lvl = l - 1;
            else { st->lvl = L - 1; st->pos = j + 1; }
        }
        __syncwarp();
    };
    auto complete = [&](int grow) { return __ldcg(p.row_done + grow) >= w.parts; };
    // The pass over the row pair of the sample at (level l, position j).  A row of one job's length is summed here and
    // now (returns false: carry on); a longer one is cut into jobs for the queue (returns true: the last job to finish
    // resumes this state machine).
    auto run_or_queue = [&](int l, int j) {
        if (p.n_rsegs > 1) {
            __threadfence();                        // every lane publishes slots: each orders the state before its own
            queue_push(p, lane, b, p.n_rsegs);
            return true;
        }
        const bool use_q = st->s_use_q != 0;
        const char* prow = row_ptr<DT>(p, l, b, j);
        warp_tiles_pass<DT>(prow, use_q ? row_ptr<DT>(p, l + 1, b, j) : prow, w.V, w.c, st->s_Ep, st->s_iZp, st->s_Eq, st->s_iZq,
                            use_q, ts, 0, p.ntiles, lane);
        if (lane == 0) st->jobs_left = 0;
        __threadfence();
        __syncwarp();
        return false;
    };
    auto start_sample = [&](int l, int j, bool use_q, const RowStat& sp, const RowStat& sq) {
        if (lane == 0) {
            st->s_use_q = use_q ? 1 : 0;
            st->s_Ep = sp.E;
            st->s_Eq = sq.E;
            st->s_iZp = static_cast<float>(1.0 / sp.Z);
            st->s_iZq = use_q ? static_cast<float>(1.0 / sq.Z) : 0.0f;
            st->jobs_left = p.n_rsegs;
            st->sampling = 1;
        }
        __syncwarp();
        return run_or_queue(l, j);
    };

    for (;;) {
        const int j = st->pos, l = st->lvl;
        const size_t lb = static_cast<size_t>(l) * w.B + b;

        if (st->sampling) {
            if (*const_cast<volatile int*>(&st->jobs_left) > 0) return;          // the last job to finish comes back here
            __threadfence();
            const bool use_q = st->s_use_q != 0;
            const float Ep = st->s_Ep, Eq = st->s_Eq, iZp = st->s_iZp, iZq = st->s_iZq;
            const char* prow = row_ptr<DT>(p, l, b, j);
            const char* qrow = use_q ? row_ptr<DT>(p, l + 1, b, j) : prow;
            // each lane owns a contiguous run of tiles; tile sums are added in double, in order
            const int nt = p.ntiles, per = (nt + 31) / 32;
            const int t0 = min(lane * per, nt), t1 = min(t0 + per, nt);
            double mine = 0.0;
            for (int tt = t0; tt < t1; ++tt) mine += static_cast<double>(__ldcg(ts + tt));
            const double incl = walkdev::warp_incl_scan(mine, lane);
            const double share = __shfl_sync(0xffffffffu, incl, 31);
            double total = 0.0;
            total += share;
            const float u = w.uniforms[lb * (w.kmax + 1) + w.kmax];
            const double target = static_cast<double>(u) * total;
            const bool has_owner = (0.0 + share > target) || (share > 0.0);
            int token = -1;
            if (has_owner)
                token = walkdev::pick_in_share<DT, true>(prow, qrow, w.V, w.c, Ep, iZp, Eq, iZq, use_q, ts, t0, t1, mine, incl, 0.0, target, lane);
            if (use_q && !(total > 0.0)) {          // residual vanished in floating point: sample P instead
                if (lane == 0) {
                    st->s_use_q = 0;
                    st->s_iZq = 0.0f;
                    st->jobs_left = p.n_rsegs;
                }
                __syncwarp();
                if (run_or_queue(l, j)) return;
                continue;
            }
            // the level ends here: a = j accepted, `token` follows them; the stream is handed to the level above
            if (lane == 0) {
                st->sampling = 0;
                st->status[l] = kDone;
                st->acc[l] = j;
                st->tok[j] = token;
                w.accepted_len[lb] = j;
                if (w.out_len) w.out_len[lb] = j + 1;
                if (w.next_token) w.next_token[b] = token;
            }
            if (w.out_tokens)
                for (int i = j + lane; i <= w.kmax; i += 32) w.out_tokens[lb * (w.kmax + 1) + i] = (i == j) ? token : -1;
            __syncwarp();
            step_on(l, j);
            continue;
        }

        // every level settled (and, for a single-level call that wants them, every probability written)?
        bool all_settled = true;
        for (int ll = 0; ll < L; ++ll) all_settled = all_settled && (st->status[ll] != kRun);
        const int m0 = min(w.k[0], st->len_bottom);
        if (all_settled && (!probes || j >= m0)) {
            if (lane == 0) {
                if (w.block_len) {
                    for (int ll = L - 1; ll >= 0; --ll) {
                        if (st->status[ll] != kDone) continue;              // -1 already written
                        const int len = (ll == L - 1) ? st->len_bottom : st->acc[ll + 1] + 1;
                        w.block_len[static_cast<size_t>(ll) * w.B + b] = min(w.k[ll], len);
                    }
                }
                st->finished = 1;
                __threadfence();
                atomicAdd(&p.ctl->finished, 1);
            }
            __syncwarp();
            return;
        }

        const int grow_p = t.row_begin[l] + b * t.rows[l] + j;
        const int grow_q = t.row_begin[l + 1] + b * t.rows[l + 1] + j;

        if (st->status[l] != kRun) {
            // a single-level call reports P and Q at every presented position, also past the first rejection
            if (probes && l == 0 && j < m0) {
                if (!complete(grow_p) || !complete(grow_q)) return;
                __threadfence();
                const RowStat sp = walkdev::merge_partials<true>(p.partials + static_cast<size_t>(grow_p) * w.parts, w.parts, lane);
                const RowStat sq = walkdev::merge_partials<true>(p.partials + static_cast<size_t>(grow_q) * w.parts, w.parts, lane);
                const int x = st->tok[j];
                if (lane == 0 && x >= 0 && x < w.V && walkdev::stat_ok(sp) && walkdev::stat_ok(sq)) {
                    const float zp = walkdev::load_logit<DT>(row_ptr<DT>(p, 0, b, j), x), zq = walkdev::load_logit<DT>(row_ptr<DT>(p, 1, b, j), x);
                    if (w.p_at) w.p_at[static_cast<size_t>(b) * w.k[0] + j] = static_cast<float>(exp2(static_cast<double>(zp) * cd - static_cast<double>(sp.E)) / sp.Z);
                    if (w.q_at) w.q_at[static_cast<size_t>(b) * w.k[0] + j] = static_cast<float>(exp2(static_cast<double>(zq) * cd - static_cast<double>(sq.E)) / sq.Z);
                }
            }
            step_on(l, j);
            continue;
        }

        // does the stream below hold a token at position j?
        bool has_tok;
        if (l == L - 1) has_tok = j < st->len_bottom;
        else has_tok = (st->status[l + 1] == kRun) || (st->status[l + 1] == kDone && j <= st->acc[l + 1]);
        const bool bonus = (j >= w.k[l]) || !has_tok;

        if (!complete(grow_p)) return;
        if (!bonus && !complete(grow_q)) return;
        __threadfence();
        const RowStat sp = walkdev::merge_partials<true>(p.partials + static_cast<size_t>(grow_p) * w.parts, w.parts, lane);
        if (bonus) {                                     // the block is exhausted and fully accepted: token from the next row of p
            if (!walkdev::stat_ok(sp)) {
                kill(l);
                step_on(l, j);
                continue;
            }
            if (start_sample(l, j, false, sp, sp)) return;
            continue;
        }
        const RowStat sq = walkdev::merge_partials<true>(p.partials + static_cast<size_t>(grow_q) * w.parts, w.parts, lane);
        const int x = st->tok[j];
        if (x < 0 || x >= w.V || !walkdev::stat_ok(sp) || !walkdev::stat_ok(sq)) {
            kill(l);
            step_on(l, j);
            continue;
        }
        const float zp = walkdev::load_logit<DT>(row_ptr<DT>(p, l, b, j), x);
        const float zq = walkdev::load_logit<DT>(row_ptr<DT>(p, l + 1, b, j), x);
        const double P = exp2(static_cast<double>(zp) * cd - static_cast<double>(sp.E)) / sp.Z;
        const double Q = exp2(static_cast<double>(zq) * cd - static_cast<double>(sq.E)) / sq.Z;
        const double u = static_cast<double>(w.uniforms[lb * (w.kmax + 1) + j]);
        const bool rej = !(u * Q <= P);
        if (lane == 0 && l == 0) {
            if (w.p_at) w.p_at[static_cast<size_t>(b) * w.k[0] + j] = static_cast<float>(P);
            if (w.q_at) w.q_at[static_cast<size_t>(b) * w.k[0] + j] = static_cast<float>(Q);
        }
        if (!rej) {
            if (lane == 0) {
                st->acc[l] = j + 1;
                if (w.out_tokens) w.out_tokens[lb * (w.kmax + 1) + j] = x;
            }
            __syncwarp();
            step_on(l, j);
            continue;
        }
        if (start_sample(l, j, true, sp, sq)) return;
    }
}

// Runs the state machine of sequence b unless another warp is running it; then that warp is told to look again.
template <int DT>
__device__ void advance(const ChainParams& p, int b)
{
    ChainSeqState* raw = p.seq + b;
    volatile ChainSeqState* st = raw;
    const int lane = threadIdx.x & 31;
    int got = 0;
    if (lane == 0) {
        atomicAdd(&raw->pending, 1);
        got = atomicCAS(&raw->lock, 0, 1) == 0;
    }
    got = __shfl_sync(0xffffffffu, got, 0);
    while (got) {
        if (lane == 0) {
            __threadfence();
            atomicExch(&raw->pending, 0);
        }
        __syncwarp();
        run_machine<DT>(p, b, st);
        __syncwarp();
        int again = 0;
        if (lane == 0) {
            __threadfence();
            atomicExch(&raw->lock, 0);
            if (atomicAdd(&raw->pending, 0) > 0) again = atomicCAS(&raw->lock, 0, 1) == 0;
        }
        got = __shfl_sync(0xffffffffu, again, 0);
    }
}

// ---------------------------------------------------------------------------------- the kernel
template <int DT>
__global__ void __launch_bounds__(kStatsThreads, 1) chain_kernel(const ChainParams p)
{
    using EL = Elems<DT>;
    constexpr int EPV = EL::per_vec;
    extern __shared__ __align__(128) unsigned char smem_raw[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* ring = smem_raw + static_cast<size_t>(warp) * kStages * kChunkBytes;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + static_cast<size_t>(kWarps) * kStages * kChunkBytes)
                               + warp * kStages;
    int* fifo = reinterpret_cast<int*>(smem_raw + static_cast<size_t>(kWarps) * kStages * (kChunkBytes + sizeof(unsigned long long)))
                + warp * kFifo;
    if (lane == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    const float c = p.w.c;
    const uint32_t spin = p.spin_limit;

    // row segments are claimed one at a time from a global counter, so that warps that spend time on residual jobs
    // or on a state machine simply claim fewer; the copy cursor runs ahead of the arithmetic, hence a small fifo
    int f_head = 0, f_tail = 0;
    bool drained = false;                       // a claim came back past the end: nothing left to claim
    auto claim = [&]() {
        int it = p.n_items;
        if (!drained) {
            if (lane == 0) it = atomicAdd(&p.ctl->next_item, 1);
            it = __shfl_sync(0xffffffffu, it, 0);
            if (it >= p.n_items) { it = p.n_items; drained = true; }
        }
        if (lane == 0) fifo[f_tail % kFifo] = it;
        ++f_tail;
        __syncwarp();
        return it;
    };

    struct Cursor { int item; uint32_t off, bytes; const char* src; } ahead;
    auto open = [&](Cursor& cur) {
        if (cur.item < p.n_items) {
            int g, s, pt;
            decode_item<DT>(p, cur.item, &cur.src, &cur.bytes, &g, &s, &pt);
        }
        cur.off = 0;
    };
    ahead.item = claim();
    open(ahead);
    uint32_t issued = 0, done = 0;

    auto issue_one = [&]() {
        if (ahead.item >= p.n_items) return;
        const uint32_t n = min(static_cast<uint32_t>(kChunkBytes), ahead.bytes - ahead.off);
        if (lane == 0) {
            const uint32_t stage = issued % kStages;
            const uint32_t bar = smem_u32(&bars[stage]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic reads of this stage are done
            mbar_arrive_expect_tx(bar, n);
            bulk_copy_g2s(smem_u32(ring + stage * kChunkBytes), ahead.src + ahead.off, n, bar);
        }
        ++issued;
        ahead.off += n;
        if (ahead.off >= ahead.bytes) {
            ahead.item = claim();
            open(ahead);
        }
    };

#pragma unroll 1
    for (int s = 0; s < kStages - 1; ++s) issue_one();

    for (;;) {
        // residual jobs first: the rows they re-read are still in L2
        unsigned int job;
        while (queue_pop(p, lane, &job)) run_resid_job<DT>(p, job);

        const int item = fifo[f_head % kFifo];
        if (item >= p.n_items) break;
        const char* src;
        uint32_t bytes;
        int grow, seq, part;
        decode_item<DT>(p, item, &src, &bytes, &grow, &seq, &part);

        float E = kEmptyRef;
        float s[kVecPerLane];
#pragma unroll
        for (int u = 0; u < kVecPerLane; ++u) s[u] = 0.0f;

        for (uint32_t off = 0; off < bytes; off += kChunkBytes, ++done) {
            __syncwarp();          // every lane has finished reading the stage the next copy will overwrite
            issue_one();
            const uint32_t stage = done % kStages;
            const bool ok = wait_bounded(smem_u32(&bars[stage]), (done / kStages) & 1u, spin);
            if (!__all_sync(0xffffffffu, ok)) {
                if (lane == 0) {
                    if (p.w.device_status) atomicCAS(p.w.device_status, 0, static_cast<int>(POLYSPEC_ERR_TIMEOUT));
                    for (uint32_t jj = done; jj < issued; ++jj)      // let the copies in flight land
                        wait_bounded(smem_u32(&bars[jj % kStages]), (jj / kStages) & 1u);
                }
                return;
            }
            const int nvec = static_cast<int>(min(static_cast<uint32_t>(kChunkBytes), bytes - off) >> 4);
            const uint32_t base = smem_u32(ring + stage * kChunkBytes);
            uint4 r[kVecPerLane];
#pragma unroll
            for (int u = 0; u < kVecPerLane; ++u) {
                const int idx = lane + u * 32;
                r[u] = (idx < nvec) ? ld_shared_v4(base + idx * 16) : EL::neg_inf();
            }
            float z[kVecPerLane][EPV];
            const float M = EL::vec_max(r);
#pragma unroll
            for (int u = 0; u < kVecPerLane; ++u) EL::unpack(r[u], z[u]);
            const float En = (M == -INFINITY) ? kEmptyRef : ceilf(M * c);
            if (En > E) {
                const float sc = pow2_neg(E - En);
#pragma unroll
                for (int u = 0; u < kVecPerLane; ++u) s[u] *= sc;
                E = En;
            }
#pragma unroll
            for (int u = 0; u < kVecPerLane; ++u)
#pragma unroll
                for (int e = 0; e < EPV; ++e) s[u] += streamdev::ex2f(__fmaf_rn(z[u][e], c, -E));
        }

        // lanes -> warp: rebase every lane to the warp's largest reference (exact), then add
        float Ew = E;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) Ew = fmaxf(Ew, __shfl_xor_sync(0xffffffffu, Ew, o));
        float sw = ((s[0] + s[1]) + (s[2] + s[3])) * pow2_neg(E - Ew);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sw += __shfl_xor_sync(0xffffffffu, sw, o);
        int row_complete = 0;
        if (lane == 0) {
            p.partials[static_cast<size_t>(grow) * p.w.parts + part] = make_float2(Ew, sw);
            __threadfence();
            row_complete = atomicAdd(p.row_done + grow, 1) == p.w.parts - 1;
        }
        ++f_head;
        if (__shfl_sync(0xffffffffu, row_complete, 0)) advance<DT>(p, seq);
    }

    // The stream has ended.  Residual jobs may still be enqueued by the state machines that the last rows set off:
    // a few warps per CTA keep serving them until every sequence is finished (bounded; nothing depends on it).
    if (warp < kLingerWarps) {
        for (int polls = 0; polls < kLingerPolls; ++polls) {
            unsigned int job;
            if (queue_pop(p, lane, &job)) {
                run_resid_job<DT>(p, job);
                continue;
            }
            int fin = 0;
            if (lane == 0) fin = *reinterpret_cast<volatile int*>(&p.ctl->finished);
            if (__shfl_sync(0xffffffffu, fin, 0) >= p.w.B) break;
            __nanosleep(500);
        }
    }
}

constexpr int kMaxDevices = 64;
std::mutex g_chain_mutex;
int g_chain_sms[kMaxDevices] = {0};
constexpr size_t kChainSmemBytes = static_cast<size_t>(kWarps) * kStages * (kChunkBytes + sizeof(unsigned long long)) +
                                   static_cast<size_t>(kWarps) * kFifo * sizeof(int);

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

ChainPlan plan_chain(long long total_rows, int B, int V, int n_levels, polyspec_dtype dt)
{
    ChainPlan pl;
    pl.stats = plan_stats(total_rows, V, dt);
    pl.ntiles = (V + kTile - 1) / kTile;
    pl.rseg_tiles = 32;                                  // 8192 elements per residual job
    pl.n_rsegs = (pl.ntiles + pl.rseg_tiles - 1) / pl.rseg_tiles;
    const unsigned long long cap = 2ull * static_cast<unsigned long long>(B) * n_levels * pl.n_rsegs;   // residual + fallback per level
    pl.q_cap = cap > 0xfffffff0ull ? 0u : static_cast<unsigned int>(cap);                               // 0: too large, not supported
    size_t off = pl.stats.partial_bytes;
    pl.zero_begin = off;
    pl.row_done = off; off += align256(static_cast<size_t>(total_rows) * sizeof(int));
    pl.seq = off;      off += align256(static_cast<size_t>(B) * sizeof(ChainSeqState));
    pl.queue = off;    off += align256(static_cast<size_t>(pl.q_cap) * sizeof(unsigned long long));
    pl.ctl = off;      off += align256(sizeof(ChainCtl));
    pl.zero_end = off;
    pl.tile_sum = off; off += align256(static_cast<size_t>(B) * pl.ntiles * sizeof(float));
    pl.total = off;
    return pl;
}

cudaError_t launch_chain(polyspec_dtype dt, ChainParams& p, const ChainPlan& plan, void* workspace, cudaStream_t stream)
{
    if (p.w.B <= 0) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int sm_count = 0;
    {
        std::lock_guard<std::mutex> lock(g_chain_mutex);
        if (g_chain_sms[dev] == 0) {
            int sms = 0;
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return e;
            const void* kernels[2] = {reinterpret_cast<const void*>(chain_kernel<POLYSPEC_F32>),
                                      reinterpret_cast<const void*>(chain_kernel<POLYSPEC_BF16>)};
            for (const void* k : kernels) {
                e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kChainSmemBytes));
                if (e != cudaSuccess) return e;
            }
            g_chain_sms[dev] = sms > 0 ? sms : 148;
        }
        sm_count = g_chain_sms[dev];
    }
    char* ws = static_cast<char*>(workspace);
    const RowTable& t = p.w.t;
    p.seg = plan.stats.seg;
    p.n_items = static_cast<int>(plan.stats.n_items);
    p.max_rows = 0;
    for (int i = 0; i < t.n_models; ++i) p.max_rows = t.rows[i] > p.max_rows ? t.rows[i] : p.max_rows;
    if (p.max_rows > kMaxK + 1) return cudaErrorInvalidValue;
    int acc = 0;
    for (int j = 0; j <= p.max_rows; ++j) {
        p.pos_begin[j] = acc;
        int nmod = 0;
        for (int i = 0; i < t.n_models; ++i) nmod += t.rows[i] > j;
        acc += p.w.B * nmod;
    }
    for (int j = p.max_rows + 1; j < kMaxK + 3; ++j) p.pos_begin[j] = acc;
    p.ntiles = plan.ntiles;
    p.rseg_tiles = plan.rseg_tiles;
    p.n_rsegs = plan.n_rsegs;
    p.partials = reinterpret_cast<float2*>(ws);
    p.w.partials = p.partials;
    p.row_done = reinterpret_cast<int*>(ws + plan.row_done);
    p.seq = reinterpret_cast<ChainSeqState*>(ws + plan.seq);
    p.queue = reinterpret_cast<unsigned long long*>(ws + plan.queue);
    p.q_cap = plan.q_cap;
    p.ctl = reinterpret_cast<ChainCtl*>(ws + plan.ctl);
    p.tile_sum = reinterpret_cast<float*>(ws + plan.tile_sum);
    if (p.spin_limit == 0) p.spin_limit = kSpinLimit;
    e = cudaMemsetAsync(ws + plan.zero_begin, 0, plan.zero_end - plan.zero_begin, stream);
    if (e != cudaSuccess) return e;
    const int grid = p.n_items < sm_count ? p.n_items : sm_count;       // one CTA per SM
    if (dt == POLYSPEC_BF16) chain_kernel<POLYSPEC_BF16><<<grid, kStatsThreads, kChainSmemBytes, stream>>>(p);
    else chain_kernel<POLYSPEC_F32><<<grid, kStatsThreads, kChainSmemBytes, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace polyspec
