// Device code shared by the kernels that decide and sample (the per-sequence walk and the
// vocabulary-sharded level): loads, the merge of row-statistics partials, the residual of
// Section 3.1's rejection rule in a fixed operation order, and the inverse-CDF search.
#pragma once

#include "polyspec_kernels.cuh"

namespace polyspec {
namespace walkdev {

constexpr int kWalkThreads = 512;
constexpr int kWalkWarps = kWalkThreads / 32;
// tiles a warp loads before it computes (a float32 tile is two vectors per lane and row), and how
// many CTAs the register budget must let an SM hold
#ifndef POLYSPEC_WALK_UNROLL
#define POLYSPEC_WALK_UNROLL 2
#endif
#ifndef POLYSPEC_WALK_CTAS_PER_SM
#define POLYSPEC_WALK_CTAS_PER_SM 2
#endif
template <int DT> struct Unroll { static constexpr int value = (DT == POLYSPEC_BF16) ? POLYSPEC_WALK_UNROLL : (POLYSPEC_WALK_UNROLL + 1) / 2; };

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 ld_nc(const void* p)
{
    uint4 r;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

template <int DT> __device__ __forceinline__ float load_logit(const void* row, int v)
{
    if (DT == POLYSPEC_BF16)
        return __uint_as_float(static_cast<uint32_t>(static_cast<const unsigned short*>(row)[v]) << 16);
    return static_cast<const float*>(row)[v];
}

// Eight consecutive logits starting at element v (v a multiple of 8, inside the row).
template <int DT> __device__ __forceinline__ void load8(const void* row, int v, float* z)
{
    if (DT == POLYSPEC_BF16) {
        const uint4 r = ld_nc(static_cast<const unsigned short*>(row) + v);
        z[0] = __uint_as_float(r.x << 16); z[1] = __uint_as_float(r.x & 0xffff0000u);
        z[2] = __uint_as_float(r.y << 16); z[3] = __uint_as_float(r.y & 0xffff0000u);
        z[4] = __uint_as_float(r.z << 16); z[5] = __uint_as_float(r.z & 0xffff0000u);
        z[6] = __uint_as_float(r.w << 16); z[7] = __uint_as_float(r.w & 0xffff0000u);
    } else {
        const uint4 a = ld_nc(static_cast<const float*>(row) + v);
        const uint4 b = ld_nc(static_cast<const float*>(row) + v + 4);
        z[0] = __uint_as_float(a.x); z[1] = __uint_as_float(a.y); z[2] = __uint_as_float(a.z); z[3] = __uint_as_float(a.w);
        z[4] = __uint_as_float(b.x); z[5] = __uint_as_float(b.y); z[6] = __uint_as_float(b.z); z[7] = __uint_as_float(b.w);
    }
}

// Eight consecutive logits as loaded (one or two 16-byte vectors), unpacked later.
template <int DT> struct RawTile;
template <> struct RawTile<POLYSPEC_BF16> {
    uint4 a;
    __device__ __forceinline__ void load(const void* row, int v) { a = ld_nc(static_cast<const unsigned short*>(row) + v); }
    __device__ __forceinline__ void unpack(float* z) const
    {
        z[0] = __uint_as_float(a.x << 16); z[1] = __uint_as_float(a.x & 0xffff0000u);
        z[2] = __uint_as_float(a.y << 16); z[3] = __uint_as_float(a.y & 0xffff0000u);
        z[4] = __uint_as_float(a.z << 16); z[5] = __uint_as_float(a.z & 0xffff0000u);
        z[6] = __uint_as_float(a.w << 16); z[7] = __uint_as_float(a.w & 0xffff0000u);
    }
};
template <> struct RawTile<POLYSPEC_F32> {
    uint4 a, b;
    __device__ __forceinline__ void load(const void* row, int v)
    {
        a = ld_nc(static_cast<const float*>(row) + v);
        b = ld_nc(static_cast<const float*>(row) + v + 4);
    }
    __device__ __forceinline__ void unpack(float* z) const
    {
        z[0] = __uint_as_float(a.x); z[1] = __uint_as_float(a.y); z[2] = __uint_as_float(a.z); z[3] = __uint_as_float(a.w);
        z[4] = __uint_as_float(b.x); z[5] = __uint_as_float(b.y); z[6] = __uint_as_float(b.z); z[7] = __uint_as_float(b.w);
    }
};

struct RowStat {      // sum_v 2^(z_v * c - E) = Z
    float E;
    double Z;
};

// Z * 2^d for an integer-valued d <= 0: an exact rescaling (0 once the gap is huge; NaN stays NaN).
__device__ __forceinline__ double scale_pow2(double Z, float d)
{
    // 2^d built from its bit pattern: d is an integer in [-1000, 0] here, so the factor is a normal double
    const double f = (d < -1000.0f) ? 0.0 : __longlong_as_double(static_cast<long long>(1023 + static_cast<int>(d)) << 52);
    return Z * f;
}

// One warp merges the partials of one row: lanes take partials in parallel, four loads in flight
// each, keeping a running (E, Z) that is rebased whenever a larger reference turns up; then the
// lanes are rebased to the warp's largest reference and added.  Rebasing is an exact power-of-two
// scaling, the sums are in double.  Every lane returns the same result.
// COHERENT: the partials were written by other SMs during this very launch, so they are read from L2
// (ld.global.cg) instead of through this SM's L1.
template <bool COHERENT = false>
__device__ __forceinline__ RowStat merge_partials(const float2* part, int parts, int lane)
{
    float E = kEmptyRef;
    double Z = 0.0;
    for (int i0 = lane; i0 < parts; i0 += 4 * 32) {
        float2 ps[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * 32;
            ps[u] = (i < parts) ? (COHERENT ? __ldcg(part + i) : part[i]) : make_float2(kEmptyRef, 0.0f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (ps[u].x > E) {
                Z = scale_pow2(Z, E - ps[u].x);
                E = ps[u].x;
            }
            Z += scale_pow2(static_cast<double>(ps[u].y), ps[u].x - E);
        }
    }
    float Ew = E;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Ew = fmaxf(Ew, __shfl_xor_sync(0xffffffffu, Ew, o));
    Z = scale_pow2(Z, E - Ew);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, o);
    RowStat r;
    r.E = Ew;
    r.Z = Z;
    return r;
}

__device__ __forceinline__ bool stat_ok(const RowStat& s) { return s.Z > 0.0 && s.Z < 1.0e300; }   // false for NaN too

// The residual (or, without q, the probability) of one element, up to the row's common factor: with
// a = 2^(z_p c - E_p) = P Z_p and b = 2^(z_q c - E_q) = Q Z_q the value is max(0, a - rho b) = Z_p max(0, P - Q) for
// rho = Z_p / Z_q.  The inverse-CDF search only ever compares partial sums with u times the total, so the factor
// Z_p never has to be divided out.  One fixed operation order, so that the sum pass and the rescan produce
// identical values.
template <bool USE_Q>
__device__ __forceinline__ float resid(float zp, float zq, float c, float nEp, float nEq, float nrho)
{
    const float a = ex2f(__fmaf_rn(zp, c, nEp));
    if (!USE_Q) return a;
    const float b = ex2f(__fmaf_rn(zq, c, nEq));
    return fmaxf(0.0f, __fmaf_rn(nrho, b, a));
}

// The per-row constants of resid(): the negated references and the negated ratio of the normalisers.
struct RowScale {
    float nEp, nEq, nrho;
};
__device__ __forceinline__ RowScale row_scale(float Ep, double Zp, float Eq, double Zq, bool use_q)
{
    RowScale s;
    s.nEp = -Ep;
    s.nEq = -Eq;
    s.nrho = use_q ? -static_cast<float>(Zp / Zq) : 0.0f;
    return s;
}

__device__ __forceinline__ float sum8(const float* r)
{
    return __fadd_rn(__fadd_rn(__fadd_rn(r[0], r[1]), __fadd_rn(r[2], r[3])),
                     __fadd_rn(__fadd_rn(r[4], r[5]), __fadd_rn(r[6], r[7])));
}

template <int DT, bool USE_Q>
__device__ __forceinline__ void tile_resid_q(const void* prow, const void* qrow, int v, int V, float c, const RowScale sc, float* r)
{
    if (v < V) {
        float zp[8], zq[8];
        load8<DT>(prow, v, zp);
        if (USE_Q) load8<DT>(qrow, v, zq);
#pragma unroll
        for (int e = 0; e < 8; ++e) r[e] = resid<USE_Q>(zp[e], USE_Q ? zq[e] : 0.0f, c, sc.nEp, sc.nEq, sc.nrho);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) r[e] = 0.0f;
    }
}
template <int DT>
__device__ __forceinline__ void tile_resid(const void* prow, const void* qrow, int v, int V, float c, const RowScale sc, bool use_q,
                                           float* r)
{
    if (use_q) tile_resid_q<DT, true>(prow, qrow, v, V, c, sc, r);
    else tile_resid_q<DT, false>(prow, qrow, v, V, c, sc, r);
}

__device__ __forceinline__ double warp_incl_scan(double x, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    return x;
}

struct SampleShared {
    double total;
    double rank_total[8];   // mass of each CTA's share of the row (filled by the CTAs of the cluster)
    int token;
};

// A sequence may be walked by a cluster of CTAs (small batches: more SMs per sequence).  Every CTA
// runs the same control flow on the same inputs; only the row pass is divided, by tile ranges.
struct ClusterCtx {
    int size;       // CTAs per sequence: 1, 2, 4 or 8
    int rank;
};

__device__ __forceinline__ uint32_t peer_addr(const void* local, int rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(local))), "r"(rank));
    return r;
}
// All threads of all CTAs of the cluster; also orders their shared-memory traffic (release / acquire).
__device__ __forceinline__ void cluster_barrier(const ClusterCtx& cl)
{
    if (cl.size > 1) {
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        __syncthreads();
    }
}

// The sum of one lane's eight elements of a tile, added as a fixed tree.
template <int DT, bool USE_Q>
__device__ __forceinline__ float lane_sum(const RawTile<DT>& rp, const RawTile<DT>& rq, float c, const RowScale sc)
{
    float zp[8], zq[8], r[8];
    rp.unpack(zp);
    if (USE_Q) rq.unpack(zq);
#pragma unroll
    for (int e = 0; e < 8; ++e) r[e] = resid<USE_Q>(zp[e], USE_Q ? zq[e] : 0.0f, c, sc.nEp, sc.nEq, sc.nrho);
    return sum8(r);
}

// Tiles handled together by one warp in the row pass: their four per-lane sums are reduced over the warp in one
// transposed butterfly (6 shuffles for four tiles instead of 20).
constexpr int kTileGroup = 4;

// x0..x3 are a lane's sums of four tiles.  Returns, in the lanes with (lane >> 3) == i, the sum of x_i over the warp,
// added in the order of a plain xor-butterfly (16, 8, 4, 2, 1), so a tile's sum does not depend on whether it was
// reduced alone or in a group.
__device__ __forceinline__ float reduce_four_tiles(float x0, float x1, float x2, float x3, int lane)
{
    const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0;
    float k0 = up16 ? x2 : x0, k1 = up16 ? x3 : x1;
    const float g0 = up16 ? x0 : x2, g1 = up16 ? x1 : x3;
    k0 = __fadd_rn(k0, __shfl_xor_sync(0xffffffffu, g0, 16));
    k1 = __fadd_rn(k1, __shfl_xor_sync(0xffffffffu, g1, 16));
    float k = up8 ? k1 : k0;
    const float g = up8 ? k0 : k1;
    k = __fadd_rn(k, __shfl_xor_sync(0xffffffffu, g, 8));
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) k = __fadd_rn(k, __shfl_xor_sync(0xffffffffu, k, o));
    return k;
}

// The sums of the residual (or of P) over tiles [tlo, thi) of one row, one float per tile in tile_sum[t]; all warps
// of the CTA take part, no synchronisation inside.  Whole tiles go in groups of four per warp while there are
// enough groups to occupy every warp; what is left (and the ragged last tile) goes one tile per warp.
template <int DT, bool USE_Q>
__device__ __forceinline__ void tiles_pass_q(const void* prow, const void* qrow, int V, float c, const RowScale sc, float* tile_sum,
                                             int tlo, int thi)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int whole = min(thi, V / kTile);              // tiles below this index lie wholly inside the row
    int ngroups = (whole - tlo) / kTileGroup;
    if (ngroups < kWalkWarps) ngroups = 0;
    for (int g = warp; g < ngroups; g += kWalkWarps) {
        const int t0 = tlo + g * kTileGroup;
        float x[kTileGroup];
        // tiles whose loads are in flight together per lane: two of 2-byte logits (four 16-byte vectors with q),
        // one of float32 (the same four vectors)
        constexpr int kFly = (DT == POLYSPEC_BF16) ? 2 : 1;
#pragma unroll
        for (int h = 0; h < kTileGroup; h += kFly) {
            RawTile<DT> rp[kFly], rq[kFly];
#pragma unroll
            for (int f = 0; f < kFly; ++f) {
                const int v = (t0 + h + f) * kTile + lane * 8;
                rp[f].load(prow, v);
                if (USE_Q) rq[f].load(qrow, v);
            }
#pragma unroll
            for (int f = 0; f < kFly; ++f) x[h + f] = lane_sum<DT, USE_Q>(rp[f], rq[f], c, sc);
        }
        const float k = reduce_four_tiles(x[0], x[1], x[2], x[3], lane);
        if ((lane & 7) == 0) tile_sum[t0 + (lane >> 3)] = k;
    }
    for (int t = tlo + ngroups * kTileGroup + warp; t < thi; t += kWalkWarps) {
        float r[8];
        tile_resid_q<DT, USE_Q>(prow, qrow, t * kTile + lane * 8, V, c, sc, r);
        float x = sum8(r);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x = __fadd_rn(x, __shfl_xor_sync(0xffffffffu, x, o));
        if (lane == 0) tile_sum[t] = x;
    }
}
template <int DT>
__device__ __forceinline__ void tiles_pass(const void* prow, const void* qrow, int V, float c, const RowScale sc, bool use_q,
                                           float* tile_sum, int tlo, int thi)
{
    if (use_q) tiles_pass_q<DT, true>(prow, qrow, V, c, sc, tile_sum, tlo, thi);
    else tiles_pass_q<DT, false>(prow, qrow, V, c, sc, tile_sum, tlo, thi);
}

// The token at `target` of the row's running sum, for the warp of the share that contains it: lane i of the warp
// owns tiles [t0, t1) of the share with sum `mine` and inclusive running sum `incl` over the lanes, `base` is the mass
// before the share.  Returns the token in every lane (-1 if the share holds no mass).
template <int DT, bool COHERENT = false>
__device__ __forceinline__ int pick_in_share(const void* prow, const void* qrow, int V, float c, const RowScale sc,
                                             bool use_q, const float* tile_sum, int t0, int t1, double mine, double incl,
                                             double base, double target, int lane)
{
    auto sum_of = [&](int t) { return COHERENT ? __ldcg(tile_sum + t) : tile_sum[t]; };
    int token = -1;
    const unsigned hit = __ballot_sync(0xffffffffu, base + incl > target);
    const unsigned has_mass = __ballot_sync(0xffffffffu, mine > 0.0);
    // the first lane whose running sum passes the target; if rounding leaves none, the last lane
    // that holds any mass
    const int owner = hit ? (__ffs(hit) - 1) : (has_mass ? (31 - __clz(has_mass)) : -1);
    int tile = -1;
    double prefix = 0.0;
    if (owner >= 0) {
        if (lane == owner) {
            double run = base + (incl - mine);
            for (int t = t0; t < t1; ++t) {
                const double nxt = run + static_cast<double>(sum_of(t));
                if (nxt > target) { tile = t; prefix = run; break; }
                run = nxt;
            }
            if (tile < 0) {                       // take the lane's last non-empty tile
                run = base + (incl - mine);
                for (int t = t0; t < t1; ++t) {
                    if (sum_of(t) > 0.0f) { tile = t; prefix = run; }
                    run += static_cast<double>(sum_of(t));
                }
            }
        }
        tile = __shfl_sync(0xffffffffu, tile, owner);
        prefix = __shfl_sync(0xffffffffu, prefix, owner);
    }
    if (tile >= 0) {
        float r[8];
        tile_resid<DT>(prow, qrow, tile * kTile + lane * 8, V, c, sc, use_q, r);
        double lane_sum = 0.0;
#pragma unroll
        for (int e = 0; e < 8; ++e) lane_sum += static_cast<double>(r[e]);
        const double lincl = warp_incl_scan(lane_sum, lane);
        const double tt = target - prefix;
        const unsigned lhit = __ballot_sync(0xffffffffu, lincl > tt);
        const unsigned lpos = __ballot_sync(0xffffffffu, lane_sum > 0.0);
        // the first lane whose running sum passes the target; if rounding leaves none, the last lane with mass
        const int pick = lhit ? (__ffs(lhit) - 1) : (lpos ? (31 - __clz(lpos)) : -1);
        if (pick >= 0 && lane == pick) {
            double run = lincl - lane_sum;
            int last_pos = -1;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (token < 0) {
                    run += static_cast<double>(r[e]);
                    if (r[e] > 0.0f) last_pos = e;
                    if (run > tt) token = tile * kTile + lane * 8 + e;
                }
            }
            if (token < 0 && last_pos >= 0) token = tile * kTile + lane * 8 + last_pos;
        }
        if (pick >= 0) token = __shfl_sync(0xffffffffu, token, pick);
    }
    return token;
}

// Inverse CDF of the residual (use_q) or of P (bonus / fallback) at uniform u.
// Returns the token (same value in every thread) and, through *total_out, the total mass times the row's
// common factor Z_p (only its sign is meaningful to the caller).
template <int DT>
__device__ int sample_row(const void* prow, const void* qrow, int V, float c, RowStat sp, RowStat sq, bool use_q,
                          float u, float* tile_sum, SampleShared* sh, double* total_out, const ClusterCtx cl)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ntiles = (V + kTile - 1) / kTile;
    // this CTA's share of the row: tiles [tlo, thi)
    const int tiles_per_rank = (ntiles + cl.size - 1) / cl.size;
    const int tlo = min(cl.rank * tiles_per_rank, ntiles), thi = min(tlo + tiles_per_rank, ntiles);
    const RowScale sc = row_scale(sp.E, sp.Z, sq.E, sq.Z, use_q);

    tiles_pass<DT>(prow, qrow, V, c, sc, use_q, tile_sum, tlo, thi);
    __syncthreads();

    // each lane of warp 0 owns a contiguous run of the CTA's tiles; tile sums are added in double, in order
    const int nt = thi - tlo, per = (nt + 31) / 32;
    const int t0 = tlo + min(lane * per, nt), t1 = min(t0 + per, thi);
    double mine = 0.0, incl = 0.0;
    if (warp == 0) {
        for (int t = t0; t < t1; ++t) mine += static_cast<double>(tile_sum[t]);
        incl = warp_incl_scan(mine, lane);
        const double share = __shfl_sync(0xffffffffu, incl, 31);
        if (cl.size == 1) {
            if (lane == 0) sh->rank_total[0] = share;
        } else if (lane < cl.size) {            // lane r tells CTA r this CTA's share
            asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(peer_addr(&sh->rank_total[cl.rank], lane)), "d"(share) : "memory");
        }
    }
    cluster_barrier(cl);

    if (warp == 0) {
        // total mass and the CTA whose share contains u * total (the same arithmetic in every CTA)
        double total = 0.0;
        for (int r = 0; r < cl.size; ++r) total += sh->rank_total[r];
        const double target = static_cast<double>(u) * total;
        int owner_rank = -1, last_mass = -1;
        double base = 0.0, last_base = 0.0, cum = 0.0;
        for (int r = 0; r < cl.size; ++r) {
            const double nxt = cum + sh->rank_total[r];
            if (owner_rank < 0 && nxt > target) { owner_rank = r; base = cum; }
            if (sh->rank_total[r] > 0.0) { last_mass = r; last_base = cum; }
            cum = nxt;
        }
        if (owner_rank < 0) { owner_rank = last_mass; base = last_base; }      // u not below 1, or rounding
        int token = -1;
        if (owner_rank == cl.rank) {
            token = pick_in_share<DT>(prow, qrow, V, c, sc, use_q, tile_sum, t0, t1, mine, incl, base, target, lane);
        }
        if (lane == 0) sh->total = total;
        // the CTA that holds the token tells every CTA (with no mass anywhere, CTA 0 reports -1)
        if (cl.rank == (owner_rank < 0 ? 0 : owner_rank)) {
            if (cl.size == 1) {
                if (lane == 0) sh->token = token;
            } else if (lane < cl.size) {
                asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_addr(&sh->token, lane)), "r"(token) : "memory");
            }
        }
    }
    cluster_barrier(cl);
    *total_out = sh->total;
    const int token = sh->token;
    __syncthreads();          // sh and tile_sum are reused by the next pass
    return token;
}

}  // namespace walkdev
}  // namespace polyspec
