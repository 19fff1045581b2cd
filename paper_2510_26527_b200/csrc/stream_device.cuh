// Device helpers of the row-statistics kernel: the streaming load, the unpacking of 16-byte vectors, exact
// power-of-two rescaling, the packed arg max of 2-byte logits.
#pragma once

#include "polyspec_kernels.cuh"

namespace polyspec {
namespace streamdev {

constexpr int kChunkBytes = 2048;                 // one warp-wide sweep of 4 vectors per lane
#ifndef POLYSPEC_STATS_WARPS
#define POLYSPEC_STATS_WARPS 32
#endif
// Warp counts that are not multiples of four (one per scheduler) lose 5 %.
constexpr int kWarps = POLYSPEC_STATS_WARPS;
constexpr int kStatsThreads = kWarps * 32;
constexpr int kVecPerLane = kChunkBytes / 16 / 32;   // 4

// A 16-byte vector of a row that is read once: through the read-only path, not kept in L1.
__device__ __forceinline__ uint4 ld_stream(const void* p)
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
    // Largest element of n vectors (NaNs are passed over, as fmaxf does): two elements per instruction on the packed
    // words, the exact same value as a maximum over the unpacked floats.
    static __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b)
    {
        uint32_t d;
        asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
        return d;
    }
    template <int N> static __device__ __forceinline__ float vec_max(const uint4 (&r)[N])
    {
        uint32_t m = max2(max2(r[0].x, r[0].y), max2(r[0].z, r[0].w));
#pragma unroll
        for (int u = 1; u < N; ++u) m = max2(m, max2(max2(r[u].x, r[u].y), max2(r[u].z, r[u].w)));
        return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xffff0000u));
    }
};
template <> struct Elems<POLYSPEC_F32> {
    static constexpr int per_vec = 4;
    static __device__ __forceinline__ void unpack(const uint4& r, float* z)
    {
        z[0] = __uint_as_float(r.x); z[1] = __uint_as_float(r.y);
        z[2] = __uint_as_float(r.z); z[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ uint4 neg_inf() { return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u); }
    template <int N> static __device__ __forceinline__ float vec_max(const uint4 (&r)[N])
    {
        float m = -INFINITY;
#pragma unroll
        for (int u = 0; u < N; ++u)
            m = fmaxf(m, fmaxf(fmaxf(__uint_as_float(r[u].x), __uint_as_float(r[u].y)), fmaxf(__uint_as_float(r[u].z), __uint_as_float(r[u].w))));
        return m;
    }
};

// Arg max of 2-byte logits on the packed words: the running maximum of the even and of the odd elements a lane has
// seen, two per instruction, NaN sticking once met (max.NaN); where a half's maximum moved is kept, branch-free, as
// the word's number inside its chunk (ppos) and, once per chunk, the chunk's number (pchunk), both packed like the
// maxima.  A value equal to the running maximum does not move it, so what is kept is the first occurrence.
struct PackedArgMax {
    uint32_t pm, ppos, pchunk;
    __device__ __forceinline__ void init() { pm = 0xff80ff80u; ppos = 0; pchunk = 0; }
    template <uint32_t J> __device__ __forceinline__ void word(uint32_t w)
    {
        uint32_t nm, moved;
        asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(nm) : "r"(pm), "r"(w));
        asm("set.neu.u32.bf16x2 %0, %1, %2;" : "=r"(moved) : "r"(nm), "r"(pm));        // 0xffff per half that moved
        ppos = (ppos & ~moved) | (((J << 16) | J) & moved);
        pm = nm;
    }
    // the four vectors (sixteen words) a lane holds of one chunk; `chunk` is the chunk's number in the segment
    __device__ __forceinline__ void chunk(const uint4 (&r)[kVecPerLane], uint32_t chunk_no)
    {
        const uint32_t before = pm;
        word<0>(r[0].x); word<1>(r[0].y); word<2>(r[0].z); word<3>(r[0].w);
        word<4>(r[1].x); word<5>(r[1].y); word<6>(r[1].z); word<7>(r[1].w);
        word<8>(r[2].x); word<9>(r[2].y); word<10>(r[2].z); word<11>(r[2].w);
        word<12>(r[3].x); word<13>(r[3].y); word<14>(r[3].z); word<15>(r[3].w);
        uint32_t moved;
        asm("set.neu.u32.bf16x2 %0, %1, %2;" : "=r"(moved) : "r"(pm), "r"(before));
        pchunk = (pchunk & ~moved) | (((chunk_no << 16) | chunk_no) & moved);
    }
    // The lane's best (value, element index inside the segment) and whether it met a NaN.
    __device__ __forceinline__ void finish(int lane, float* best, int* at, bool* nan) const
    {
        const uint32_t lo = pm & 0xffffu, hi = pm >> 16;
        *nan = (lo & 0x7fffu) > 0x7f80u || (hi & 0x7fffu) > 0x7f80u;
        const float vlo = __uint_as_float(lo << 16), vhi = __uint_as_float(hi << 16);
        // word j of chunk c is word (j & 3) of the lane's vector (j >> 2), which is vector (j >> 2) * 32 + lane of the chunk
        auto element = [&](uint32_t c, uint32_t j, uint32_t half) {
            return static_cast<int>(c * (kChunkBytes / 2) + ((j >> 2) * 32 + lane) * 8 + (j & 3) * 2 + half);
        };
        const int alo = element(pchunk & 0xffffu, ppos & 0xffffu, 0), ahi = element(pchunk >> 16, ppos >> 16, 1);
        const bool take_hi = vhi > vlo || (vhi == vlo && ahi < alo);
        *best = take_hi ? vhi : vlo;
        *at = take_hi ? ahi : alo;
    }
};

}  // namespace streamdev
}  // namespace polyspec
