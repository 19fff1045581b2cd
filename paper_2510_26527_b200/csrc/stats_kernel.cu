// Row statistics: the temperature-softmax normaliser of every logits row of every model,
// read exactly once (the distribution p_i(x | x_<=t) over the vocabulary of Section 3.1
// needs it for each drafted position before Algorithm 1's Verify can run).
//
// HBM-bound.  One persistent CTA per SM, and inside it every warp is a self-contained
// pipeline: lane 0 streams the warp's row segments into the warp's private ring of
// shared-memory stages with 1-D bulk TMA copies (cp.async.bulk, completion on an
// mbarrier), one stage ahead of the lanes that read them back with conflict-free
// 128-bit shared loads.  Warps never synchronise with each other, so their load, ALU and
// ex2 phases drift apart and overlap on the SM's pipes.  Each element costs one FFMA, one
// ex2 and one add.  Every thread keeps an online pair (E, s) with  sum 2^(z*c - E) = s
// and E an INTEGER-valued reference at or just above its running maximum of z*c,
// c = log2(e)/T.  Because E is an integer, rebasing s when the maximum grows, and merging
// pairs across lanes and segments, are exact multiplications by powers of two: no second
// exponential is ever spent.
//
// Every wait on an mbarrier is bounded.  If one expires the warp records
// POLYSPEC_ERR_TIMEOUT, lets the copies it has in flight land (again bounded) and returns;
// the outputs of that launch are then meaningless.
#include <algorithm>
#include <mutex>

#include "polyspec_kernels.cuh"
#include "stream_device.cuh"

namespace polyspec {
namespace {

using namespace streamdev;

// Where work item `item` lives: first byte and byte count of its row segment.
template <int DT>
__device__ __forceinline__ void item_span(const StatsParams& p, int item, const char** src, uint32_t* bytes)
{
    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    const int grow = item / p.parts;
    const int part = item - grow * p.parts;
    int mi = 0;
    while (mi + 1 < p.t.n_models && grow >= p.t.row_begin[mi + 1]) ++mi;
    const int v0 = part * p.seg;
    const int v1 = min(p.V, v0 + p.seg);
    *src = static_cast<const char*>(p.t.logits[mi]) + (static_cast<size_t>(grow - p.t.row_begin[mi]) * p.V + v0) * ELEM;
    *bytes = static_cast<uint32_t>((v1 - v0) * ELEM);
}

// A warp's position in its list of chunks: work item (row segment) and byte offset inside it.
struct ChunkCursor {
    int item;
    uint32_t off, bytes;
    const char* src;
};

template <int DT>
__device__ __forceinline__ void cursor_open(const StatsParams& p, ChunkCursor& cur)
{
    if (cur.item < p.n_items) item_span<DT>(p, cur.item, &cur.src, &cur.bytes);
    cur.off = 0;
}

// MODE 0: softmax normaliser partials (E, s).  MODE 1: arg-max partials for greedy matching
// (Section 3.1): (largest logit of the segment, index of its first occurrence as int bits; -1 if
// the segment holds NaN or +inf).  Same pipeline, different arithmetic on the staged vectors.
template <int DT, int MODE>
__global__ void __launch_bounds__(kStatsThreads, 1) stats_kernel(const StatsParams p)
{
    using EL = Elems<DT>;
    constexpr int EPV = EL::per_vec;
    extern __shared__ __align__(128) unsigned char smem_raw[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* ring = smem_raw + static_cast<size_t>(warp) * kStages * kChunkBytes;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + static_cast<size_t>(kWarps) * kStages * kChunkBytes)
                               + warp * kStages;
    if (lane == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    // consecutive items go to different CTAs: small problems still spread over every SM
    const int stride = gridDim.x * kWarps;
    const float c = p.c;

    ChunkCursor ahead;            // next chunk to request (lane 0 runs the copies kStages-1 ahead)
    ahead.item = warp * gridDim.x + blockIdx.x;
    cursor_open<DT>(p, ahead);
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
            ahead.item += stride;
            cursor_open<DT>(p, ahead);
        }
    };

#pragma unroll 1
    for (int s = 0; s < kStages - 1; ++s) issue_one();

    for (int item = warp * gridDim.x + blockIdx.x; item < p.n_items; item += stride) {
        const char* src;
        uint32_t bytes;
        item_span<DT>(p, item, &src, &bytes);

        float E = kEmptyRef;
        float s[kVecPerLane];
#pragma unroll
        for (int u = 0; u < kVecPerLane; ++u) s[u] = 0.0f;
        // arg-max state of this lane: its elements come in ascending index order, so a strictly
        // larger value is always the first occurrence among the lane's own
        float best = -INFINITY;
        int best_at = 0x7fffffff;
        uint32_t abs_max = 0;              // largest |bits|: above 0x7f800000 means a NaN went by
        PackedArgMax packed;               // 2-byte logits take the packed form instead
        packed.init();
        const int seg_first = (item % p.parts) * p.seg;      // row index of the segment's first element

        for (uint32_t off = 0; off < bytes; off += kChunkBytes, ++done) {
            __syncwarp();          // every lane has finished reading the stage the next copy will overwrite
            issue_one();
            const uint32_t stage = done % kStages;
            const bool ok = p.spin_limit ? wait_polls(smem_u32(&bars[stage]), (done / kStages) & 1u, p.spin_limit)
                                         : wait_bounded(smem_u32(&bars[stage]), (done / kStages) & 1u);
            if (!__all_sync(0xffffffffu, ok)) {
                if (lane == 0) {
                    if (p.status) atomicCAS(p.status, 0, static_cast<int>(POLYSPEC_ERR_TIMEOUT));
                    for (uint32_t j = done; j < issued; ++j)      // let the copies in flight land
                        wait_bounded(smem_u32(&bars[j % kStages]), (j / kStages) & 1u);
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
            if (MODE == 0) {
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
                    for (int e = 0; e < EPV; ++e) s[u] += ex2f(__fmaf_rn(z[u][e], c, -E));
            } else if (DT == POLYSPEC_BF16) {
                packed.chunk(r, off / kChunkBytes);
            } else {
                constexpr int ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
#pragma unroll
                for (int u = 0; u < kVecPerLane; ++u) {
                    EL::unpack(r[u], z[u]);
                    float vm = z[u][0];
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        vm = fmaxf(vm, z[u][e]);
                        abs_max = max(abs_max, __float_as_uint(z[u][e]) & 0x7fffffffu);
                    }
                    if (vm > best) {           // rare once the running maximum has settled
                        best = vm;
                        int e_first = 0;
#pragma unroll
                        for (int e = EPV - 1; e >= 0; --e) e_first = (z[u][e] == vm) ? e : e_first;
                        best_at = seg_first + static_cast<int>(off / ELEM) + (lane + u * 32) * EPV + e_first;
                    }
                }
            }
        }

        if (MODE == 1) {
            if (DT == POLYSPEC_BF16) {
                bool nan;
                packed.finish(lane, &best, &best_at, &nan);
                // a lane that saw nothing but -inf keeps the "no index" mark, like the scalar form
                best_at = (best == -INFINITY) ? 0x7fffffff : seg_first + best_at;
                abs_max = nan ? 0x7fc00000u : 0u;
            }
            // lanes -> warp: the larger value wins, equal values go to the lower index
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best, o);
                const int oa = __shfl_xor_sync(0xffffffffu, best_at, o);
                const uint32_t om = __shfl_xor_sync(0xffffffffu, abs_max, o);
                if (ov > best || (ov == best && oa < best_at)) { best = ov; best_at = oa; }
                abs_max = max(abs_max, om);
            }
            const bool unusable = abs_max > 0x7f800000u || best == INFINITY;
            if (lane == 0) p.partials[item] = make_float2(best, __int_as_float(unusable ? -1 : best_at));
            continue;
        }

        // lanes -> warp: rebase every lane to the warp's largest reference (exact), then add
        float Ew = E;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) Ew = fmaxf(Ew, __shfl_xor_sync(0xffffffffu, Ew, o));
        float sw = ((s[0] + s[1]) + (s[2] + s[3])) * pow2_neg(E - Ew);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sw += __shfl_xor_sync(0xffffffffu, sw, o);
        if (lane == 0) p.partials[item] = make_float2(Ew, sw);
    }
}

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
int g_sm_count[kMaxDevices] = {0};     // per device: SM count, published under g_setup_mutex once the kernels' shared-memory opt-in is done
constexpr size_t kStatsSmemBytes = static_cast<size_t>(kWarps) * kStages * (kChunkBytes + sizeof(unsigned long long));

}  // namespace

StatsPlan plan_stats(long long total_rows, int V, polyspec_dtype dt)
{
    // A segment (one warp's work item) is a whole number of 2 KiB chunks, at least 2048 elements and at most 16 KiB.
    // Work items are dealt out to the 148 x kWarps warps in equal numbers, so the pass takes as long as the warp with
    // the most items: among the admissible segment lengths take the one with the smallest (items per busiest warp) x
    // (bytes per item + a fixed cost per item); on a tie the longer segment.  Few rows are thus cut finer (every SM
    // still gets work), a mid-size problem gets a length that does not leave many warps one item short (the
    // three-level workload: 7168 elements, 4.9 items per warp, instead of 8192, 4.3 per warp with a fifth item on a
    // third of the warps), and a large one keeps 16 KiB.
    const long long elem = dt == POLYSPEC_BF16 ? 2 : 4;
    const long long seg_max = 16384LL / elem;
    const long long step = kChunkBytes / elem;
    const long long warps = 148LL * kWarps;
    long long seg = 2048, best = -1;
    for (long long cand = 2048; cand <= seg_max; cand += step) {
        const long long items = total_rows * ((V + cand - 1) / cand);
        const long long per_warp = (items + warps - 1) / warps;
        const long long cost = per_warp * (std::min<long long>(cand, V) * elem + 512);
        if (best < 0 || cost <= best) { best = cost; seg = cand; }
    }
    StatsPlan pl;
    pl.seg = static_cast<int>(seg);
    pl.parts = static_cast<int>((V + seg - 1) / seg);
    pl.total_rows = total_rows;
    pl.n_items = total_rows * pl.parts;
    pl.partial_bytes = (static_cast<size_t>(pl.n_items) * sizeof(float2) + 255) / 256 * 256;
    return pl;
}

cudaError_t launch_stats(polyspec_dtype dt, const StatsParams& p, cudaStream_t stream, bool argmax)
{
    if (p.n_items <= 0) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int sm_count = 0;
    {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_sm_count[dev] == 0) {
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        const void* kernels[4] = {reinterpret_cast<const void*>(stats_kernel<POLYSPEC_F32, 0>),
                                  reinterpret_cast<const void*>(stats_kernel<POLYSPEC_BF16, 0>),
                                  reinterpret_cast<const void*>(stats_kernel<POLYSPEC_F32, 1>),
                                  reinterpret_cast<const void*>(stats_kernel<POLYSPEC_BF16, 1>)};
        for (const void* k : kernels) {
            e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kStatsSmemBytes));
            if (e != cudaSuccess) return e;
        }
        g_sm_count[dev] = sms > 0 ? sms : 148;
    }
    sm_count = g_sm_count[dev];
    }
    const int grid = p.n_items < sm_count ? p.n_items : sm_count;   // one CTA per SM
    if (dt == POLYSPEC_BF16) {
        if (argmax) stats_kernel<POLYSPEC_BF16, 1><<<grid, kStatsThreads, kStatsSmemBytes, stream>>>(p);
        else stats_kernel<POLYSPEC_BF16, 0><<<grid, kStatsThreads, kStatsSmemBytes, stream>>>(p);
    } else {
        if (argmax) stats_kernel<POLYSPEC_F32, 1><<<grid, kStatsThreads, kStatsSmemBytes, stream>>>(p);
        else stats_kernel<POLYSPEC_F32, 0><<<grid, kStatsThreads, kStatsSmemBytes, stream>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace polyspec
