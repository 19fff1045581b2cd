// Row statistics: the temperature-softmax normaliser of every logits row of every model,
// read exactly once (the distribution p_i(x | x_<=t) over the vocabulary of Section 3.1
// needs it for each drafted position before Algorithm 1's Verify can run).
//
// HBM-bound: each element costs one FFMA, one ex2 and one add.  Every thread keeps an
// online pair (E, s) with  sum 2^(z*c - E) = s  and E an INTEGER-valued reference at or
// just above its running maximum of z*c, c = log2(e)/T.  Because E is an integer,
// rebasing s when the maximum grows, and merging pairs across lanes, warps and segments,
// are exact multiplications by powers of two: no second exponential is ever spent.
#include "polyspec_kernels.cuh"

namespace polyspec {
namespace {

constexpr int kStatsThreads = 256;
constexpr int kUnroll = 4;   // 16-byte vectors in flight per thread

__device__ __forceinline__ uint4 ld_stream(const uint4* p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 2^d for an integer-valued d <= 0 (exact); 0 once below the normal range.
__device__ __forceinline__ float pow2_neg(float d)
{
    return (d < -126.0f) ? 0.0f : __int_as_float((static_cast<int>(d) + 127) << 23);
}

template <int DT> struct Elems;
template <> struct Elems<POLYSPEC_BF16> {
    static constexpr int per_vec = 8;
    static __device__ __forceinline__ void unpack(const uint4& r, float* z)
    {
        z[0] = __uint_as_float(r.x << 16); z[1] = __uint_as_float(r.x & 0xffff0000u);
        z[2] = __uint_as_float(r.y << 16); z[3] = __uint_as_float(r.y & 0xffff0000u);
        z[4] = __uint_as_float(r.z << 16); z[5] = __uint_as_float(r.z & 0xffff0000u);
        z[6] = __uint_as_float(r.w << 16); z[7] = __uint_as_float(r.w & 0xffff0000u);
    }
    static __device__ __forceinline__ uint4 neg_inf() { return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u); }
};
template <> struct Elems<POLYSPEC_F32> {
    static constexpr int per_vec = 4;
    static __device__ __forceinline__ void unpack(const uint4& r, float* z)
    {
        z[0] = __uint_as_float(r.x); z[1] = __uint_as_float(r.y);
        z[2] = __uint_as_float(r.z); z[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ uint4 neg_inf() { return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u); }
};

template <int DT>
__global__ void __launch_bounds__(kStatsThreads) stats_kernel(const StatsParams p)
{
    using EL = Elems<DT>;
    constexpr int EPV = EL::per_vec;
    constexpr size_t ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    __shared__ float2 warp_part[2][kStatsThreads / 32];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float c = p.c;
    int parity = 0;
    for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, parity ^= 1) {
        const int grow = item / p.parts;
        const int part = item - grow * p.parts;
        int mi = 0;
        while (mi + 1 < p.t.n_models && grow >= p.t.row_begin[mi + 1]) ++mi;
        const char* base = static_cast<const char*>(p.t.logits[mi]);
        const uint4* src = reinterpret_cast<const uint4*>(base + static_cast<size_t>(grow - p.t.row_begin[mi]) * p.V * ELEM)
                           + (static_cast<size_t>(part) * p.seg) / EPV;
        const int v0 = part * p.seg;
        const int v1 = min(p.V, v0 + p.seg);
        const int nvec = (v1 - v0) / EPV;

        float E = kEmptyRef;
        float s[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) s[u] = 0.0f;

        for (int i = threadIdx.x; i < nvec; i += kStatsThreads * kUnroll) {
            uint4 r[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int idx = i + u * kStatsThreads;
                r[u] = (idx < nvec) ? ld_stream(src + idx) : EL::neg_inf();
            }
            float z[kUnroll][EPV];
            float M = -INFINITY;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                EL::unpack(r[u], z[u]);
#pragma unroll
                for (int e = 0; e < EPV; ++e) M = fmaxf(M, z[u][e]);
            }
            const float En = (M == -INFINITY) ? kEmptyRef : ceilf(M * c);
            if (En > E) {
                const float sc = pow2_neg(E - En);
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) s[u] *= sc;
                E = En;
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
#pragma unroll
                for (int e = 0; e < EPV; ++e) s[u] += ex2f(__fmaf_rn(z[u][e], c, -E));
        }

        // lanes -> warp: rebase every lane to the warp's largest reference (exact), then add
        float Ew = E;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) Ew = fmaxf(Ew, __shfl_xor_sync(0xffffffffu, Ew, o));
        float sw = ((s[0] + s[1]) + (s[2] + s[3])) * pow2_neg(E - Ew);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sw += __shfl_xor_sync(0xffffffffu, sw, o);
        if (lane == 0) warp_part[parity][warp] = make_float2(Ew, sw);
        __syncthreads();
        if (threadIdx.x == 0) {
            float Eb = kEmptyRef;
#pragma unroll
            for (int w = 0; w < kStatsThreads / 32; ++w) Eb = fmaxf(Eb, warp_part[parity][w].x);
            float sb = 0.0f;
#pragma unroll
            for (int w = 0; w < kStatsThreads / 32; ++w) sb += warp_part[parity][w].y * pow2_neg(warp_part[parity][w].x - Eb);
            p.partials[item] = make_float2(Eb, sb);
        }
        // warp_part[parity] is next written two items later, after the barrier of the item in between
    }
}

int g_sm_count = 0;
int g_occ[2] = {0, 0};

}  // namespace

StatsPlan plan_stats(long long total_rows, int V, polyspec_dtype dt)
{
    (void)dt;
    // Aim for several work items per SM even when there are few rows; a segment is a
    // multiple of 2048 elements (256 threads x one 8-element vector).
    const long long total = total_rows * static_cast<long long>(V);
    long long seg = (total / (148LL * 8) + 2047) / 2048 * 2048;
    if (seg < 2048) seg = 2048;
    if (seg > 16384) seg = 16384;
    StatsPlan pl;
    pl.seg = static_cast<int>(seg);
    pl.parts = static_cast<int>((V + seg - 1) / seg);
    pl.total_rows = total_rows;
    pl.n_items = total_rows * pl.parts;
    pl.partial_bytes = (static_cast<size_t>(pl.n_items) * sizeof(float2) + 255) / 256 * 256;
    return pl;
}

cudaError_t launch_stats(polyspec_dtype dt, const StatsParams& p, cudaStream_t stream)
{
    if (p.n_items <= 0) return cudaSuccess;
    if (g_sm_count == 0) {
        int dev = 0, sms = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        int o0 = 0, o1 = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o0, stats_kernel<POLYSPEC_F32>, kStatsThreads, 0);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o1, stats_kernel<POLYSPEC_BF16>, kStatsThreads, 0);
        if (e != cudaSuccess) return e;
        g_occ[0] = o0 > 0 ? o0 : 1;
        g_occ[1] = o1 > 0 ? o1 : 1;
        g_sm_count = sms > 0 ? sms : 148;
    }
    const int resident = g_sm_count * g_occ[dt == POLYSPEC_BF16 ? 1 : 0];
    const int grid = p.n_items < resident ? p.n_items : resident;
    if (dt == POLYSPEC_BF16)
        stats_kernel<POLYSPEC_BF16><<<grid, kStatsThreads, 0, stream>>>(p);
    else
        stats_kernel<POLYSPEC_F32><<<grid, kStatsThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace polyspec
