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
    const int ntiles = (p.V + kTile - 1) / kTile;
    cl.tiles_per_rank = (ntiles + cl.size - 1) / cl.size;
    const int b = static_cast<int>(blockIdx.x) / p.cluster;
    GlobalRows<DT> src;
    src.p = &p;
    src.b = b;
    walk_levels<DT>(p, src, cl, b, tile_sum);
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
