// LM-head projection on the tensor cores: logits[r, v] = sum_d hidden[r, d] * W[v, d]
// (the last op of the model forwards in Algorithm 1, "p_{1:K} <- M_2(...)" and
// "v <- M_1(...)"), bf16 inputs, fp32 accumulation, fp32 logits out.
//
// The contraction is dense, so it runs on tcgen05: the vocabulary is the MMA's M axis (a
// CTA owns 128 vocabulary entries at a time), the (sequence, position) rows of the hidden
// states are the N axis (up to 288 columns per accumulator, issued as one or two MMAs of
// N <= 256), and d is the K loop in blocks of 64 elements = one 128-byte swizzle row.
// Both operands are K-major in shared memory exactly as 2-D TMA with 128-byte swizzle
// writes them.  The accumulator lives in TMEM (lane = vocabulary entry, column = hidden
// row) and is read back with tcgen05.ld by four epilogue warps.
//
// One persistent CTA per SM walks a static list of work items (model, vocabulary tile,
// column block), costliest model first, so the target's and the drafter's projections
// share one launch and the tail of one fills the other's idle SMs.  Warp roles:
//   warp 0      TMA producer (one lane): W tile + hidden tile per K block into a 4-stage ring
//   warp 1      MMA issuer (one lane); also allocates / frees TMEM
//   warps 2..5  epilogue: TMEM -> registers -> global, 128-byte coalesced stores per column
// When a column block needs at most 256 TMEM columns two accumulators alternate, so the
// epilogue of one tile overlaps the K loop of the next.
//
// Every wait is bounded.  A wait that runs out raises an abort flag that all roles poll,
// sets POLYSPEC_ERR_TIMEOUT in the status word, lets copies and MMAs in flight finish
// (bounded again), frees TMEM and returns.
#include <cuda.h>

#include "polyspec_kernels.cuh"

namespace polyspec {
namespace {

constexpr int kTileV = 128;                 // vocabulary entries per tile (MMA M)
constexpr int kBlockK = 64;                 // bf16 elements per K block (one 128-byte swizzle row)
constexpr int kMmaK = 16;                   // K of one tcgen05.mma for 16-bit inputs
constexpr int kMaxCols = 288;               // widest column block (TMEM columns per accumulator)
constexpr int kStagesG = 4;
constexpr int kBytesA = kTileV * kBlockK * 2;          // 16 KiB
constexpr int kBytesBMax = kMaxCols * kBlockK * 2;     // 36 KiB
constexpr int kStageBytes = kBytesA + kBytesBMax;
constexpr int kGemmThreads = 192;
constexpr int kTmemCols = 512;
constexpr uint32_t kSpinLimitG = 1u << 22;
constexpr size_t kGemmSmemBytes = 1024 /* alignment slack */ + static_cast<size_t>(kStagesG) * kStageBytes + 256 /* barriers */;

struct GemmJob {
    CUtensorMap map_w;      // [V, d] bf16, box {64, 128}
    CUtensorMap map_h;      // [rows, d] bf16, box {64, chunk}
    float* out;             // [rows, V]
    int rows;
    int kblocks;            // d / 64
    int block_cols;         // columns (hidden rows) per work item, multiple of 16, <= 288
    int chunk;              // columns per MMA / per hidden TMA box, multiple of 16, <= 256
    int nchunks;            // block_cols / chunk
    int nblocks;            // column blocks covering `rows`
    int items;              // vocabulary tiles * nblocks
};

struct GemmParams {
    GemmJob job[2];
    int n_jobs;
    int V;
    int vtiles;
    int total_items;
    int acc_stages;         // 2 when every job's column block fits 256 TMEM columns (accumulators at columns 0 and 256), else 1
    int32_t* status;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait that also gives up when another role has raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (uint32_t i = 0; i < kSpinLimitG; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Shared-memory matrix descriptor of a K-major tile stored as rows of 128 bytes with the
// 128-byte swizzle: 8-row groups 1024 bytes apart (stride byte offset), descriptor
// version 1, layout type 2.  `addr` may point 32 * i bytes into the first row to select
// the i-th 16-element K slice.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    return static_cast<uint64_t>((addr & 0x3ffffu) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kTileV >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Work item -> (job, vocabulary tile, column block).  Items of job 0 come first; inside a job
// the column blocks of one vocabulary tile are neighbours, so they run at about the same time
// and share the W tile in L2.
__device__ __forceinline__ void decode_item(const GemmParams& p, int item, int* j, int* vt, int* nb)
{
    int jj = 0;
    if (item >= p.job[0].items) { jj = 1; item -= p.job[0].items; }
    const int nbk = p.job[jj].nblocks;
    *j = jj;
    *vt = item / nbk;
    *nb = item - (item / nbk) * nbk;
}

__global__ void __launch_bounds__(kGemmThreads, 1) lmhead_kernel(const __grid_constant__ GemmParams p)
{
    extern __shared__ unsigned char smem_dyn[];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // 128-byte swizzled tiles must start on a 1024-byte boundary
    const uint32_t raw = smem_addr(smem_dyn);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t bars = tiles + kStagesG * kStageBytes;      // full[4], empty[4], acc_full[2], acc_empty[2]
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kStagesG + s); };
    auto accf_bar = [&](int a) { return bars + 8u * (2 * kStagesG + a); };
    auto acce_bar = [&](int a) { return bars + 8u * (2 * kStagesG + 2 + a); };

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < kStagesG; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_base_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abort_p = &abort_flag;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;          // K blocks issued so far (ring position)
            bool ok = true;
            for (int item = blockIdx.x; ok && item < p.total_items; item += gridDim.x) {
                int j, vt, nb;
                decode_item(p, item, &j, &vt, &nb);
                const GemmJob& job = p.job[j];
                const uint32_t bytes = kBytesA + static_cast<uint32_t>(job.block_cols) * kBlockK * 2;
                for (int kb = 0; kb < job.kblocks; ++kb, ++it) {
                    const int s = it % kStagesG;
                    if (!mbar_wait(empty_bar(s), ((it / kStagesG) & 1u) ^ 1u, abort_p)) { ok = false; break; }
                    mbar_expect_tx(full_bar(s), bytes);
                    const uint32_t a_dst = tiles + s * kStageBytes;
                    tma_load_2d(a_dst, &job.map_w, kb * kBlockK, vt * kTileV, full_bar(s));
                    for (int c = 0; c < job.nchunks; ++c)
                        tma_load_2d(a_dst + kBytesA + c * job.chunk * (kBlockK * 2), &job.map_h, kb * kBlockK,
                                    nb * job.block_cols + c * job.chunk, full_bar(s));
                }
            }
            if (!ok) {
                if (!*abort_p && p.status) atomicCAS(p.status, 0, static_cast<int>(POLYSPEC_ERR_TIMEOUT));
                *abort_p = 1;
            }
            // copies still in flight must land before the CTA may exit: the last kStagesG fills
            const uint32_t first = it > static_cast<uint32_t>(kStagesG) ? it - kStagesG : 0u;
            for (uint32_t q = first; q < it; ++q) {
                const int s = q % kStagesG;
                for (uint32_t i = 0; i < kSpinLimitG; ++i)
                    if (mbar_try(full_bar(s), (q / kStagesG) & 1u)) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tile_n = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < p.total_items; item += gridDim.x, ++tile_n) {
                int j, vt, nb;
                decode_item(p, item, &j, &vt, &nb);
                const GemmJob& job = p.job[j];
                const int acc = tile_n % p.acc_stages;
                const uint32_t use = tile_n / p.acc_stages;        // how often this accumulator was used before
                if (!mbar_wait(acce_bar(acc), (use & 1u) ^ 1u, abort_p)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = instr_desc_bf16(job.chunk);
                const uint32_t d_tmem = tmem_base + acc * (kTmemCols / 2);
                for (int kb = 0; kb < job.kblocks; ++kb, ++it) {
                    const int s = it % kStagesG;
                    if (!mbar_wait(full_bar(s), (it / kStagesG) & 1u, abort_p)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = tiles + s * kStageBytes;
                    const uint32_t b_addr = a_addr + kBytesA;
#pragma unroll
                    for (int kk = 0; kk < kBlockK / kMmaK; ++kk) {
                        const uint64_t adesc = smem_desc_sw128(a_addr + kk * (kMmaK * 2));
                        for (int c = 0; c < job.nchunks; ++c) {
                            const uint64_t bdesc = smem_desc_sw128(b_addr + c * job.chunk * (kBlockK * 2) + kk * (kMmaK * 2));
                            umma_bf16(d_tmem + c * job.chunk, adesc, bdesc, idesc, (kb | kk) != 0 ? 1u : 0u);
                        }
                    }
                    umma_commit(empty_bar(s));          // frees the stage once these MMAs have read it
                }
                if (ok) umma_commit(accf_bar(acc));     // accumulator complete
            }
            if (!ok) {
                if (!*abort_p && p.status) atomicCAS(p.status, 0, static_cast<int>(POLYSPEC_ERR_TIMEOUT));
                *abort_p = 1;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;                   // the TMEM lanes this warp may read: 32 * quarter ..
        uint32_t tile_n = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < p.total_items; item += gridDim.x, ++tile_n) {
            int j, vt, nb;
            decode_item(p, item, &j, &vt, &nb);
            const GemmJob& job = p.job[j];
            const int acc = tile_n % p.acc_stages;
            const uint32_t use = tile_n / p.acc_stages;
            if (!mbar_wait(accf_bar(acc), use & 1u, abort_p)) { ok = false; break; }
            tc_fence_after();
            const int v = vt * kTileV + quarter * 32 + lane;
            const int row0 = nb * job.block_cols;
            const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * (kTmemCols / 2);
            float* out_v = job.out + v;
            for (int c0 = 0; c0 < job.block_cols; c0 += 16) {
                uint32_t r[16];
                tmem_ld16(t_addr + c0, r);
                tmem_ld_wait();
                if (v < p.V) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int row = row0 + c0 + i;
                        if (row < job.rows) out_v[static_cast<size_t>(row) * p.V] = __uint_as_float(r[i]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(acc));
        }
        if (!ok && lane == 0) {
            if (!*abort_p && p.status) atomicCAS(p.status, 0, static_cast<int>(POLYSPEC_ERR_TIMEOUT));
            *abort_p = 1;
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        // every MMA this CTA issued has been waited for through the accumulator barriers unless the
        // kernel is aborting; in that case give the tensor core a bounded moment before freeing TMEM
        if (*abort_p) __nanosleep(1000000);
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn g_encode = nullptr;
bool g_attr_set[64] = {false};
int g_sms[64] = {0};

cudaError_t get_encoder()
{
    if (g_encode) return cudaSuccess;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess) return e;
    if (q != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return cudaSuccess;
}

// [n_rows, d] bf16 row-major; box = 64 elements of d (128 bytes) by box_rows rows; 128-byte swizzle;
// rows past n_rows read as zero.
bool encode_map(CUtensorMap* map, const void* base, int n_rows, int d, int box_rows)
{
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(n_rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(d) * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBlockK), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_lmhead(const LmHeadProblem* probs, int n, int V, int32_t* device_status, cudaStream_t stream)
{
    if (n < 1 || n > 2) return cudaErrorInvalidValue;
    cudaError_t e = get_encoder();
    if (e != cudaSuccess) return e;
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!g_attr_set[dev]) {
        e = cudaFuncSetAttribute(lmhead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kGemmSmemBytes));
        if (e != cudaSuccess) return e;
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        g_sms[dev] = sms > 0 ? sms : 148;
        g_attr_set[dev] = true;
    }

    GemmParams p;
    p.n_jobs = n;
    p.V = V;
    p.vtiles = (V + kTileV - 1) / kTileV;
    p.status = device_status;
    p.total_items = 0;
    p.acc_stages = 2;
    // costliest model first
    int order[2] = {0, 1};
    if (n == 2 && static_cast<long long>(probs[1].d) * probs[1].rows > static_cast<long long>(probs[0].d) * probs[0].rows) {
        order[0] = 1; order[1] = 0;
    }
    for (int i = 0; i < 2; ++i) {
        GemmJob& job = p.job[i];
        if (i >= n) { job = p.job[0]; job.items = 0; continue; }
        const LmHeadProblem& pr = probs[order[i]];
        if (pr.rows <= 0 || pr.d <= 0 || pr.d % kBlockK != 0) return cudaErrorInvalidValue;
        int cols = (pr.rows + 15) / 16 * 16;
        if (cols > kMaxCols) cols = 256;                            // many rows: 256-column blocks, two accumulators
        else if (cols > 256) cols = (cols + 31) / 32 * 32;          // two equal MMAs, each a multiple of 16
        job.block_cols = cols;
        job.nchunks = cols > 256 ? 2 : 1;
        job.chunk = cols / job.nchunks;
        job.nblocks = (pr.rows + cols - 1) / cols;
        job.rows = pr.rows;
        job.kblocks = pr.d / kBlockK;
        job.out = pr.out;
        job.items = p.vtiles * job.nblocks;
        p.total_items += job.items;
        if (cols > kTmemCols / 2) p.acc_stages = 1;
        if (!encode_map(&job.map_w, pr.W, V, pr.d, kTileV)) return cudaErrorInvalidValue;
        if (!encode_map(&job.map_h, pr.hidden, pr.rows, pr.d, job.chunk)) return cudaErrorInvalidValue;
    }
    const int grid = p.total_items < g_sms[dev] ? p.total_items : g_sms[dev];
    lmhead_kernel<<<grid, kGemmThreads, kGemmSmemBytes, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace polyspec
