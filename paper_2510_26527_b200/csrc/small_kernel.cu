// Small batches in one launch: the paper's own setting is batch size 1 (Section 4.1), where a verification step
// touches a megabyte or two of logits and its cost is launch and round-trip latency, not bandwidth.  When all
// rows of a sequence fit the shared memory of one cluster, a cluster of eight CTAs takes the whole sequence:
//   1. every CTA copies its slice (a contiguous range of vocabulary tiles) of EVERY row of the sequence into
//      shared memory with bulk TMA copies on one mbarrier;
//   2. its warps compute the row-statistics partials of the row segments it holds -- the same segments, the
//      same arithmetic (streamdev::SoftmaxAcc) and therefore the same bits as the row-statistics kernel --
//      and store each partial into every CTA's partial table through distributed shared memory;
//   3. one cluster barrier; then the level loop of the walk (walkdev::walk_levels) runs in every CTA as it does
//      after the row-statistics kernel, except that the partials and the rows of the sampling pass are read
//      from shared memory: no logit is read from global memory twice, and there is no second launch.
// The results are those of the two launches.  Every wait is bounded; a CTA whose copies do not arrive tells
// its cluster at the barrier, and the whole sequence then reports POLYSPEC_ERR_TIMEOUT.
#include <mutex>

#include "polyspec_kernels.cuh"
#include "stream_device.cuh"
#include "walk_device.cuh"

namespace polyspec {
namespace {

using namespace walkdev;
namespace sd = streamdev;

constexpr int kSmallCluster = 8;
constexpr int kSegEl = 2048;                    // elements per row segment (one partial): the plan of small problems
constexpr int kSegTiles = kSegEl / kTile;
constexpr size_t kSmallSmemLimit = 232448 - 2560;   // 227 KiB per CTA less the kernel's static shared memory

struct SmallParams {
    WalkParams w;
    int tiles_per_rank;             // a multiple of kSegTiles: a segment never straddles two CTAs
    int slice_bytes;                // what one CTA holds of a row: tiles_per_rank * kTile elements
    int rows_per_seq;               // rows of all models of one sequence
    int lbegin[kMaxModels + 1];     // first row of each model among those
};

__host__ __device__ inline size_t small_part_offset(int rows_per_seq, int slice_bytes)
{
    return static_cast<size_t>(rows_per_seq) * slice_bytes;
}
__host__ __device__ inline size_t small_tile_offset(int rows_per_seq, int slice_bytes, int parts)
{
    return small_part_offset(rows_per_seq, slice_bytes) + static_cast<size_t>(rows_per_seq) * parts * sizeof(float2);
}
__host__ __device__ inline size_t small_flag_offset(int rows_per_seq, int slice_bytes, int parts, int ntiles)
{
    return (small_tile_offset(rows_per_seq, slice_bytes, parts) + static_cast<size_t>(ntiles) * sizeof(float) + 15) / 16 * 16;
}
__host__ __device__ inline size_t small_smem_bytes(int rows_per_seq, int slice_bytes, int parts, int ntiles)
{
    return small_flag_offset(rows_per_seq, slice_bytes, parts, ntiles) + kSmallCluster * sizeof(int) + 16;   // flags, mbarrier
}

// The sequence's rows and partials as this CTA holds them in shared memory.
template <int DT> struct LocalRows {
    static constexpr bool kLocal = true;
    const float2* part;
    const unsigned char* rows;
    const int* lbegin;
    int parts, slice_bytes;
    size_t first_byte;          // byte offset, inside a row, of the first element this CTA holds
    __device__ __forceinline__ const float2* partials(int model, int j) const
    {
        return part + static_cast<size_t>(lbegin[model] + j) * parts;
    }
    // element v of the row is at base + v * sizeof(element) for the elements this CTA holds (the pass asks for no others)
    __device__ __forceinline__ const void* pass_row(int model, int j) const
    {
        return rows + static_cast<size_t>(lbegin[model] + j) * slice_bytes - first_byte;
    }
};

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int DT>
__global__ void __launch_bounds__(kWalkThreads, 1) small_chain_kernel(const __grid_constant__ SmallParams sp)
{
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int ELEM = (DT == POLYSPEC_BF16) ? 2 : 4;
    const WalkParams& p = sp.w;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = static_cast<int>(blockIdx.x) % kSmallCluster;
    const int b = static_cast<int>(blockIdx.x) / kSmallCluster;
    const int R = sp.rows_per_seq, parts = p.parts;
    const int ntiles = (p.V + kTile - 1) / kTile;

    unsigned char* rows = smem;
    float2* part = reinterpret_cast<float2*>(smem + small_part_offset(R, sp.slice_bytes));
    float* tile_sum = reinterpret_cast<float*>(smem + small_tile_offset(R, sp.slice_bytes, parts));
    int* flags = reinterpret_cast<int*>(smem + small_flag_offset(R, sp.slice_bytes, parts, ntiles));
    unsigned long long* bar = reinterpret_cast<unsigned long long*>(flags + kSmallCluster);

    // this CTA's slice of every row: elements [el0, el0 + el_n)
    const int el0 = rank * sp.tiles_per_rank * kTile;
    const int el_n = max(0, min(p.V, el0 + sp.tiles_per_rank * kTile) - el0);
    const uint32_t row_bytes_local = static_cast<uint32_t>(el_n) * ELEM;

    if (tid == 0) {
        sd::mbar_init(sd::smem_u32(bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0 && row_bytes_local > 0) {
        if (lane == 0) sd::mbar_arrive_expect_tx(sd::smem_u32(bar), static_cast<uint32_t>(R) * row_bytes_local);
        __syncwarp();
        for (int i = lane; i < R; i += 32) {
            int mi = 0;
            while (mi + 1 < p.t.n_models && i >= sp.lbegin[mi + 1]) ++mi;
            const int j = i - sp.lbegin[mi];
            const char* src = static_cast<const char*>(p.t.logits[mi]) +
                              ((static_cast<size_t>(b) * p.t.rows[mi] + j) * p.V + el0) * ELEM;
            sd::bulk_copy_g2s(sd::smem_u32(rows + static_cast<size_t>(i) * sp.slice_bytes), src, row_bytes_local, sd::smem_u32(bar));
        }
    }
    // A CTA may only touch a peer's shared memory once that peer is known to have started; the copies are in
    // flight meanwhile.
    cluster_sync_all();

    bool ok = row_bytes_local == 0 || sd::wait_bounded(sd::smem_u32(bar), 0);
    if (!ok) ok = sd::wait_bounded(sd::smem_u32(bar), 0);        // gave up once: let the copies in flight land before going on
    const bool cta_ok = __syncthreads_and(ok ? 1 : 0) != 0;

    // row-statistics partials of the segments held here, one warp per segment, stored into every CTA's table
    if (cta_ok) {
        const int spr = sp.tiles_per_rank / kSegTiles;       // segments per slice
        for (int it = warp; it < R * spr; it += kWalkWarps) {
            const int row = it / spr, s = it - row * spr;
            const int gp = rank * spr + s;                    // index of the segment in its row
            const int v0 = gp * kSegEl;
            if (v0 >= p.V) continue;
            const uint32_t bytes = static_cast<uint32_t>(min(kSegEl, p.V - v0)) * ELEM;
            const uint32_t base = sd::smem_u32(rows + static_cast<size_t>(row) * sp.slice_bytes + static_cast<size_t>(s) * kSegEl * ELEM);
            sd::SoftmaxAcc<DT> acc;
            acc.init();
            for (uint32_t off = 0; off < bytes; off += sd::kChunkBytes) {
                const int nvec = static_cast<int>(min(static_cast<uint32_t>(sd::kChunkBytes), bytes - off) >> 4);
                uint4 r[sd::kVecPerLane];
#pragma unroll
                for (int u = 0; u < sd::kVecPerLane; ++u) {
                    const int idx = lane + u * 32;
                    r[u] = (idx < nvec) ? sd::ld_shared_v4(base + off + idx * 16) : sd::Elems<DT>::neg_inf();
                }
                acc.add_chunk(r, p.c);
            }
            const float2 pr = acc.finish();
            if (lane < kSmallCluster) {
                const uint32_t dst = peer_addr(&part[static_cast<size_t>(row) * parts + gp], lane);
                asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dst), "f"(pr.x) : "memory");
                asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dst + 4), "f"(pr.y) : "memory");
            }
        }
    }
    if (tid < kSmallCluster)
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_addr(&flags[rank], tid)), "r"(cta_ok ? 1 : 2) : "memory");
    cluster_sync_all();

    bool all_ok = true;
#pragma unroll
    for (int r = 0; r < kSmallCluster; ++r) all_ok = all_ok && flags[r] == 1;
    if (!all_ok) {                       // the same answer in every CTA of the cluster: nobody waits for anybody below
        if (rank == 0) {
            for (int l = 0; l < p.n_levels; ++l) {
                const size_t lb = static_cast<size_t>(l) * p.B + b;
                if (tid == 0) {
                    p.accepted_len[lb] = -1;
                    if (p.block_len) p.block_len[lb] = -1;
                    if (p.out_len) p.out_len[lb] = -1;
                }
                if (p.out_tokens && tid <= p.kmax) p.out_tokens[lb * (p.kmax + 1) + tid] = -1;
            }
            if (tid == 0) {
                if (p.next_token) p.next_token[b] = -1;
                if (p.device_status) atomicCAS(p.device_status, 0, static_cast<int>(POLYSPEC_ERR_TIMEOUT));
            }
        }
        return;
    }

    ClusterCtx cl;
    cl.size = kSmallCluster;
    cl.rank = rank;
    cl.tiles_per_rank = sp.tiles_per_rank;
    LocalRows<DT> src;
    src.part = part;
    src.rows = rows;
    src.lbegin = sp.lbegin;
    src.parts = parts;
    src.slice_bytes = sp.slice_bytes;
    src.first_byte = static_cast<size_t>(el0) * ELEM;
    walk_levels<DT>(p, src, cl, b, tile_sum);
}

std::mutex g_small_mutex;
int g_small_state[64] = {0};     // per device: 0 not looked at yet, 1 the kernel can be launched, -1 it cannot

// Can a cluster of eight CTAs with the largest shared-memory request be placed on this device at all?
int small_device_state(int dev)
{
    std::lock_guard<std::mutex> lock(g_small_mutex);
    if (g_small_state[dev] != 0) return g_small_state[dev];
    int state = 1;
    const void* kernels[2] = {reinterpret_cast<const void*>(small_chain_kernel<POLYSPEC_F32>),
                              reinterpret_cast<const void*>(small_chain_kernel<POLYSPEC_BF16>)};
    for (const void* k : kernels)
        if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmallSmemLimit)) != cudaSuccess)
            state = -1;
    if (state == 1) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kSmallCluster);
        cfg.blockDim = dim3(kWalkThreads);
        cfg.dynamicSmemBytes = kSmallSmemLimit;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kSmallCluster;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, small_chain_kernel<POLYSPEC_BF16>, &cfg) != cudaSuccess || n < 1) state = -1;
    }
    if (state != 1) (void)cudaGetLastError();        // a device that cannot take the kernel is not an error of the call
    g_small_state[dev] = state;
    return state;
}

}  // namespace

bool small_chain_plan(const RowTable& t, int B, int V, polyspec_dtype dt, const StatsPlan& pl, SmallChainPlan* out)
{
    // the partials must be those of the row-statistics kernel: segments of kSegEl elements (or a row that is one segment)
    if ((pl.seg != kSegEl && V > kSegEl) || B > kSmallMaxBatch) return false;
    const int elem = dt == POLYSPEC_BF16 ? 2 : 4;
    const int ntiles = (V + kTile - 1) / kTile;
    const int per_rank = (ntiles + kSmallCluster - 1) / kSmallCluster;
    out->tiles_per_rank = (per_rank + kSegTiles - 1) / kSegTiles * kSegTiles;
    out->slice_bytes = out->tiles_per_rank * kTile * elem;
    int rows = 0;
    for (int i = 0; i < t.n_models; ++i) rows += t.rows[i];
    out->rows_per_seq = rows;
    out->smem_bytes = small_smem_bytes(rows, out->slice_bytes, pl.parts, ntiles);
    return out->smem_bytes <= kSmallSmemLimit;
}

cudaError_t launch_small_chain(polyspec_dtype dt, const WalkParams& w, const SmallChainPlan& plan, cudaStream_t stream, bool* launched)
{
    *launched = false;
    if (w.B <= 0) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || small_device_state(dev) != 1) return cudaSuccess;
    SmallParams sp;
    sp.w = w;
    sp.w.cluster = kSmallCluster;
    sp.tiles_per_rank = plan.tiles_per_rank;
    sp.slice_bytes = plan.slice_bytes;
    sp.rows_per_seq = plan.rows_per_seq;
    int acc = 0;
    for (int i = 0; i <= kMaxModels; ++i) {
        sp.lbegin[i] = acc;
        if (i < w.t.n_models) acc += w.t.rows[i];
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(w.B) * kSmallCluster);
    cfg.blockDim = dim3(kWalkThreads);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kSmallCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    *launched = true;
    if (dt == POLYSPEC_BF16) return cudaLaunchKernelEx(&cfg, small_chain_kernel<POLYSPEC_BF16>, sp);
    return cudaLaunchKernelEx(&cfg, small_chain_kernel<POLYSPEC_F32>, sp);
}

}  // namespace polyspec
