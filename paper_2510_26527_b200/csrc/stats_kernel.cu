// Row statistics: the temperature-softmax normaliser of every logits row of every model,
// read exactly once (the distribution p_i(x | x_<=t) over the vocabulary of Section 3.1
// needs it for each drafted position before Algorithm 1's Verify can run).
//
// HBM-bound.  One persistent CTA of 32 warps per SM, and every warp is a stream of its own: it takes row
// segments (work items) of at most 16 KiB and reads them in 2 KiB chunks, four 128-bit read-only loads per lane
// and chunk at fixed offsets from one running pointer, the next chunk's loads always issued before the current
// chunk's arithmetic, across segment boundaries.  Warps never synchronise with each other and nothing waits on a
// barrier.  (A first form staged the chunks in per-warp shared-memory rings with 1-D bulk TMA copies; plain
// loads into registers measured 7 % faster, in a burst and sustained, and need no shared memory.)  Each element
// costs one FFMA, one ex2 and one add.  Every thread keeps an online pair (E, s) with  sum 2^(z*c - E) = s
// and E an INTEGER-valued reference at or just above its running maximum of z*c,
// c = log2(e)/T.  Because E is an integer, rebasing s when the maximum grows, and merging
// pairs across lanes and segments, are exact multiplications by powers of two: no second
// exponential is ever spent.
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

// MODE 0: softmax normaliser partials (E, s).  MODE 1: arg-max partials for greedy matching
// (Section 3.1): (largest logit of the segment, index of its first occurrence as int bits; -1 if
// the segment holds NaN or +inf).  Same stream, different arithmetic on the vectors.
template <int DT, int MODE>
__global__ void __launch_bounds__(kStatsThreads, 1) stats_kernel(const StatsParams p)
{
    using EL = Elems<DT>;
    constexpr int EPV = EL::per_vec;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // nothing the stream's earlier work wrote is read before this point (see launch_stats)
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // consecutive items go to different CTAs: small problems still spread over every SM
    const int stride = gridDim.x * kWarps;
    const float c = p.c;

    // The lane's four vectors of the next chunk are requested one chunk ahead of the arithmetic, across item boundaries.
    int a_item = warp * gridDim.x + blockIdx.x;       // item the request cursor is in
    const char* a_ptr = nullptr;                      // this lane's first vector of the next chunk to request
    uint32_t a_left = 0;                              // bytes of the cursor's item not yet requested
    auto open_item = [&]() {
        if (a_item < p.n_items) {
            const char* src;
            item_span<DT>(p, a_item, &src, &a_left);
            a_ptr = src + lane * 16;
        }
    };
    open_item();
    uint4 nxt[kVecPerLane];
    auto fetch_one = [&]() {
        if (a_item >= p.n_items) return;
        if (a_left >= kChunkBytes) {                  // a whole chunk: four unconditional loads at fixed offsets
#pragma unroll
            for (int u = 0; u < kVecPerLane; ++u) nxt[u] = ld_stream(a_ptr + u * 512);
            a_ptr += kChunkBytes;
            a_left -= kChunkBytes;
        } else {                                      // the ragged end of a segment
            const int nvec = static_cast<int>(a_left >> 4);
#pragma unroll
            for (int u = 0; u < kVecPerLane; ++u) nxt[u] = (lane + u * 32 < nvec) ? ld_stream(a_ptr + u * 512) : EL::neg_inf();
            a_left = 0;
        }
        if (a_left == 0) {
            a_item += stride;
            open_item();
        }
    };
    fetch_one();

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

        for (uint32_t off = 0; off < bytes; off += kChunkBytes) {
            uint4 r[kVecPerLane];
#pragma unroll
            for (int u = 0; u < kVecPerLane; ++u) r[u] = nxt[u];
            fetch_one();
            if (MODE == 0) {
                const float M = EL::vec_max(r);
                const float En = (M == -INFINITY) ? kEmptyRef : ceilf(M * c);
                if (En > E) {
                    const float sc = pow2_neg(E - En);
#pragma unroll
                    for (int u = 0; u < kVecPerLane; ++u) s[u] *= sc;
                    E = En;
                }
                const float nE = -E;
#pragma unroll
                for (int u = 0; u < kVecPerLane; ++u) {
                    float z[EPV];
                    EL::unpack(r[u], z);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) s[u] += ex2f(__fmaf_rn(z[e], c, nE));
                }
            } else if (DT == POLYSPEC_BF16) {
                packed.chunk(r, off / kChunkBytes);
            } else {
                constexpr int ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
                float z[kVecPerLane][EPV];
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
int g_sm_count[kMaxDevices] = {0};     // per device: SM count, looked up once under g_setup_mutex

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
        g_sm_count[dev] = sms > 0 ? sms : 148;
    }
    sm_count = g_sm_count[dev];
    }
    const int grid = p.n_items < sm_count ? p.n_items : sm_count;   // one CTA per SM
    // Programmatic stream serialisation: the launch may be set up while the kernel before it on the stream (whatever
    // wrote the logits, or the walk of the call before) is still draining; griddepcontrol.wait at the top of the kernel
    // holds every read until that kernel has completed.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(kStatsThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (dt == POLYSPEC_BF16) {
        if (argmax) return cudaLaunchKernelEx(&cfg, stats_kernel<POLYSPEC_BF16, 1>, p);
        return cudaLaunchKernelEx(&cfg, stats_kernel<POLYSPEC_BF16, 0>, p);
    }
    if (argmax) return cudaLaunchKernelEx(&cfg, stats_kernel<POLYSPEC_F32, 1>, p);
    return cudaLaunchKernelEx(&cfg, stats_kernel<POLYSPEC_F32, 0>, p);
}

}  // namespace polyspec
