// Decision and sampling: one CTA walks one sequence up the chain, level by level
// (Section 3.1: the drafted block is checked bottom-up, by M_{n-1} first and M_1 last).
// Per level (Algorithm 1: Verify with a break at the first failure, then the token that
// replaces the first rejected one, or the bonus token after a fully accepted block):
//   1. merge the row-statistics partials of the rows this level needs;
//   2. gather P_j(x_j), Q_j(x_j), test u_j * Q <= P in double precision, ballot for the
//      first rejection -> accepted length a;
//   3. one pass over row a of p (and of q unless this is the bonus row): residual
//      max(0, P - Q) per element, per-tile sums, a scan of the tile sums, then a rescan of
//      the one tile that contains u_s * total -> next token (inverse CDF, ascending order);
//   4. the emitted stream (x_1..x_a, next) becomes the block of the level above.
// Levels of one sequence depend on each other; sequences do not.  With few sequences a cluster of
// CTAs shares one sequence: every CTA of the cluster runs the same steps on the same inputs, only the
// row pass of step 3 is divided by tile ranges, the shares' sums and the chosen token being exchanged
// through distributed shared memory around two cluster barriers (hardware barriers that every CTA
// reaches unconditionally; nothing else waits).
#include <mutex>

#include "polyspec_kernels.cuh"
#include "walk_device.cuh"

namespace polyspec {
namespace {

using namespace walkdev;

template <int DT>
__global__ void __launch_bounds__(kWalkThreads, POLYSPEC_WALK_CTAS_PER_SM) walk_kernel(const WalkParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* tile_sum = reinterpret_cast<float*>(smem_raw);

    __shared__ int tok[kMaxK + 2];
    __shared__ RowStat st_p[kMaxK + 1];
    __shared__ RowStat st_q[kMaxK + 1];
    __shared__ int sh_a, sh_bad;
    __shared__ float g_zp[32], g_zq[32], g_u[32];       // logits at the block tokens, accept uniforms
    __shared__ SampleShared sh_sample;

    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    // Launched with programmatic stream serialisation: the CTAs may be placed while the kernel before
    // (row statistics or the LM-head projection) is still finishing; nothing it wrote is touched before
    // this point.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // A CTA may only touch a peer's shared memory once that peer is known to have started: one cluster
    // barrier up front, reached by every CTA of the cluster unconditionally.
    if (p.cluster > 1) {
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    // blockIdx.x = sequence * cluster size + rank in the cluster; only rank 0 writes results
    ClusterCtx cl;
    cl.size = p.cluster;
    cl.rank = static_cast<int>(blockIdx.x) % p.cluster;
    const bool writer = cl.rank == 0;
    const int b = static_cast<int>(blockIdx.x) / p.cluster;
    const int tid = threadIdx.x;
    const int L = p.n_levels;
    const size_t row_bytes = static_cast<size_t>(p.V) * ELEM;
    const double cd = static_cast<double>(p.c);

    int stream_len = p.k[L - 1];
    if (p.bottom_len) stream_len = max(0, min(stream_len, p.bottom_len[b]));
    if (tid < p.k[L - 1]) tok[tid] = p.draft_tokens[static_cast<size_t>(b) * p.k[L - 1] + tid];
    __syncthreads();

    bool dead = false;
    for (int l = L - 1; l >= 0; --l) {
        const int kl = p.k[l];
        const size_t lb = static_cast<size_t>(l) * p.B + b;
        if (dead) {               // an unusable input below: this level reports -1 as well
            if (writer && tid == 0) {
                p.accepted_len[lb] = -1;
                if (p.block_len) p.block_len[lb] = -1;
                if (p.out_len) p.out_len[lb] = -1;
            }
            if (writer && p.out_tokens && tid <= p.kmax) p.out_tokens[lb * (p.kmax + 1) + tid] = -1;
            continue;
        }
        const int m = min(kl, stream_len);
        const int grow_p = p.t.row_begin[l] + b * p.t.rows[l];
        const int grow_q = p.t.row_begin[l + 1] + b * p.t.rows[l + 1];
        const char* base_p = static_cast<const char*>(p.t.logits[l]) + static_cast<size_t>(b) * p.t.rows[l] * row_bytes;
        const char* base_q = static_cast<const char*>(p.t.logits[l + 1]) + static_cast<size_t>(b) * p.t.rows[l + 1] * row_bytes;

        // 1. normalisers of p rows 0..m and q rows 0..m-1; the last warp first requests the logits at the
        // block tokens and the accept uniforms, so that those loads are in flight during the merges
        if ((tid >> 5) == kWalkWarps - 1) {
            const int j = tid & 31;
            float zp = 0.0f, zq = 0.0f, uu = 0.0f;
            if (j < m) {
                const int x = tok[j];
                if (x >= 0 && x < p.V) {
                    zp = load_logit<DT>(base_p + j * row_bytes, x);
                    zq = load_logit<DT>(base_q + j * row_bytes, x);
                }
                uu = p.uniforms[lb * (p.kmax + 1) + j];
            }
            g_zp[j] = zp;
            g_zq[j] = zq;
            g_u[j] = uu;
        }
        for (int r = tid >> 5; r < 2 * m + 1; r += kWalkWarps) {          // one warp per row
            const bool is_q = r > m;
            const int j = is_q ? r - (m + 1) : r;
            const RowStat st = merge_partials(p.partials + static_cast<size_t>((is_q ? grow_q : grow_p) + j) * p.parts, p.parts, tid & 31);
            if ((tid & 31) == 0) (is_q ? st_q : st_p)[j] = st;
        }
        __syncthreads();

        // 2. accept tests (warp 0; m <= 32)
        if (tid < 32) {
            bool rej = false, bad = false;
            float pf = 0.0f, qf = 0.0f;
            const bool want_pq = writer && l == 0 && (p.p_at || p.q_at);      // the probabilities are a diagnostic output
            if (tid < m) {
                const int x = tok[tid];
                const RowStat sp = st_p[tid], sq = st_q[tid];
                if (x < 0 || x >= p.V || !stat_ok(sp) || !stat_ok(sq)) {
                    bad = true;
                } else {
                    // u Q <= P with P = 2^xp / Z_p and Q = 2^xq / Z_q, taken as u Z_p 2^(xq - xp) <= Z_q: one
                    // double-precision exponential and no division on the path every level waits for (the two
                    // exponentials and divisions of the plain form are 1.5 us of dependent arithmetic).  Q = 0 or
                    // u = 0 make the left side zero whatever the gap of the exponents: accepted.
                    const float zp = g_zp[tid], zq = g_zq[tid];
                    const double xp = static_cast<double>(zp) * cd - static_cast<double>(sp.E);
                    const double xq = static_cast<double>(zq) * cd - static_cast<double>(sq.E);
                    const double u = static_cast<double>(g_u[tid]);
                    const bool left_zero = zq == -INFINITY || !(u > 0.0);
                    rej = !(left_zero || u * sp.Z * exp2(xq - xp) <= sq.Z);
                    if (want_pq) {
                        pf = static_cast<float>(exp2(xp) / sp.Z);
                        qf = static_cast<float>(exp2(xq) / sq.Z);
                    }
                }
            }
            if (writer && l == 0 && p.p_at && tid < kl) p.p_at[static_cast<size_t>(b) * kl + tid] = pf;
            if (writer && l == 0 && p.q_at && tid < kl) p.q_at[static_cast<size_t>(b) * kl + tid] = qf;
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
            dead = true;
            if (writer && tid == 0) {
                p.accepted_len[lb] = -1;
                if (p.block_len) p.block_len[lb] = -1;
                if (p.out_len) p.out_len[lb] = -1;
                if (p.next_token) p.next_token[b] = -1;
                if (p.device_status) atomicCAS(p.device_status, 0, static_cast<int>(POLYSPEC_ERR_BAD_INPUT_ON_DEVICE));
            }
            if (writer && p.out_tokens && tid <= p.kmax) p.out_tokens[lb * (p.kmax + 1) + tid] = -1;
            __syncthreads();
            continue;
        }

        // 3. replacement (a < m) or bonus (a == m) token
        const float u_s = p.uniforms[lb * (p.kmax + 1) + p.kmax];
        const void* prow = base_p + a * row_bytes;
        const void* qrow = base_q + a * row_bytes;
        bool use_q = a < m;
        const RowStat sp = st_p[a];
        const RowStat sq = use_q ? st_q[a] : sp;
        double total = 0.0;
        int next = sample_row<DT>(prow, qrow, p.V, p.c, sp, sq, use_q, u_s, tile_sum, &sh_sample, &total, cl);
        if (use_q && !(total > 0.0)) {          // residual vanished in floating point: sample P instead
            next = sample_row<DT>(prow, qrow, p.V, p.c, sp, sq, false, u_s, tile_sum, &sh_sample, &total, cl);
        }

        // 4. outputs and hand-off
        if (writer && tid == 0) {
            p.accepted_len[lb] = a;
            if (p.block_len) p.block_len[lb] = m;
            if (p.out_len) p.out_len[lb] = a + 1;
            if (p.next_token) p.next_token[b] = next;
        }
        if (writer && p.out_tokens && tid <= p.kmax)
            p.out_tokens[lb * (p.kmax + 1) + tid] = (tid < a) ? tok[tid] : (tid == a ? next : -1);
        __syncthreads();
        if (tid == 0) tok[a] = next;
        stream_len = a + 1;
        __syncthreads();
    }
}

}  // namespace

namespace {
std::mutex g_walk_mutex;
int g_walk_sms[64] = {0};     // per device, filled once under g_walk_mutex
}

cudaError_t launch_walk(polyspec_dtype dt, const WalkParams& p_in, cudaStream_t stream)
{
    if (p_in.B <= 0) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int walk_sms = 0;
    {
        std::lock_guard<std::mutex> lock(g_walk_mutex);
        if (g_walk_sms[dev] == 0) {
            int sms = 0;
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return e;
            g_walk_sms[dev] = sms > 0 ? sms : 148;
        }
        walk_sms = g_walk_sms[dev];
    }
    const int ntiles = (p_in.V + kTile - 1) / kTile;
    // Few sequences: a cluster of up to 8 CTAs walks each one, so that the row passes use more SMs.
    // The largest power of two that still lets every CTA be resident at once (two per SM).
    WalkParams p = p_in;
    p.cluster = 1;
    while (p.cluster < 8 && static_cast<long long>(p.B) * (2 * p.cluster) <= 2LL * walk_sms && 2 * p.cluster <= ntiles)
        p.cluster *= 2;
    const size_t smem = static_cast<size_t>(ntiles) * sizeof(float);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(p.B) * p.cluster);
    cfg.blockDim = dim3(kWalkThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(p.cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // see griddepcontrol.wait in the kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (dt == POLYSPEC_BF16) return cudaLaunchKernelEx(&cfg, walk_kernel<POLYSPEC_BF16>, p);
    return cudaLaunchKernelEx(&cfg, walk_kernel<POLYSPEC_F32>, p);
}

}  // namespace polyspec
