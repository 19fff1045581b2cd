// LM-head projection on the tensor cores: logits[r, v] = sum_d hidden[r, d] * W[v, d]
// (the last op of the model forwards in Algorithm 1, "p_{1:K} <- M_2(...)" and
// "v <- M_1(...)"), bf16 inputs, fp32 accumulation, fp32 logits out.
//
// The contraction is dense, so it runs on tcgen05.  It is also skinny (a few hundred hidden
// rows against the whole vocabulary), which makes it a weight-streaming problem: per flop it
// needs more shared-memory fill than a square GEMM, and W arrives at HBM latency.  Hence:
//   - the vocabulary is the MMA's M axis and two CTAs on neighbouring SMs work as a pair
//     (cta_group::2, M = 256): each CTA streams its own 128 rows of W, and the hidden tile
//     (the N axis, up to 288 columns, one or two MMAs of N <= 256) is split between the two,
//     so each SM fills and reads only half of it;
//   - d is the K loop in blocks of 64 elements = one 128-byte swizzle row; both operands are
//     K-major in shared memory exactly as 2-D TMA with 128-byte swizzle writes them; a
//     5-stage ring of (W tile, hidden half-tile) keeps about 170 KiB in flight per SM (a sixth
//     stage measured no faster);
//   - the accumulator lives in TMEM (lane = vocabulary entry, column = hidden row) and is
//     read back with tcgen05.ld by eight epilogue warps per CTA.
//
// The grid is persistent: CTA pair i walks work items i, i + pairs, ... of a static list
// (model, 256-entry vocabulary tile, column block), costliest model first, so the target's and
// the drafter's projections share one launch and the tail of one fills the other's idle SMs;
// odd pairs walk their list backwards so that neighbouring pairs are in different phases.
// Warp roles in each CTA:
//   warp 0      TMA producer (one elected lane issues).  Both CTAs load their own tiles; all copies of a stage
//               complete on the leader CTA's "full" barrier (no multicast anywhere)
//   warp 1      MMA issuer (one elected lane, leader CTA only); allocates / frees TMEM in both CTAs.
//               tcgen05.commit arrives on the "empty" / "accumulator full" barriers of both CTAs
//   warps 2..9  epilogue (two warps per TMEM lane quarter, alternate 16-column chunks): TMEM ->
//               registers -> a 2 KiB staging tile per warp -> global by 2-D TMA store; all sixteen
//               epilogue warps of the pair arrive on the leader's "slot empty" barriers.
//               On request the epilogue also emits the row statistics of the tile (the softmax
//               normaliser partial of each hidden row over the CTA's 128 vocabulary entries, in the
//               format of the row-statistics kernel), so the logits need no second pass for them
// TMEM holds more than one accumulator so that the epilogue of a tile overlaps the K loop of the
// next: two slots of 256 columns when every column block fits one, else three slots of 144 columns
// of which a tile takes two (its two MMA chunks), so the next tile can start as soon as the first
// of them has been drained.
//
// Every wait on an mbarrier is bounded.  A wait that runs out raises an abort flag in both CTAs
// that all roles poll, sets POLYSPEC_ERR_TIMEOUT in the status word, lets copies in flight land
// (bounded again), and the kernel still frees TMEM and returns.
#include <cuda.h>

#include <mutex>

#include "polyspec_kernels.cuh"

namespace polyspec {
namespace {

constexpr int kTileV = 128;                 // vocabulary entries per CTA and tile (MMA M per CTA)
constexpr int kPairV = 2 * kTileV;          // vocabulary entries per CTA pair and tile (MMA M)
constexpr int kBlockK = 64;                 // bf16 elements per K block (one 128-byte swizzle row)
constexpr int kMmaK = 16;                   // K of one tcgen05.mma for 16-bit inputs
constexpr int kMaxCols = 288;               // widest column block (TMEM columns per accumulator)
constexpr int kStagesG = 5;                   // a sixth stage measured no faster (and the space now holds the statistics)
constexpr int kBytesA = kTileV * kBlockK * 2;                // 16 KiB: this CTA's rows of W
constexpr int kBytesBMax = (kMaxCols / 2) * kBlockK * 2;     // 18 KiB: this CTA's half of the hidden tile
constexpr int kStageBytes = kBytesA + kBytesBMax;            // 34 KiB
constexpr int kEpiWarps = 8;                // warps 2..9: two per TMEM lane quarter, alternating 16-column chunks
constexpr int kGemmThreads = 32 * (2 + kEpiWarps);
constexpr int kTmemCols = 512;
constexpr uint32_t kSpinLimitG = 1u << 20;
constexpr int kScratchPitch = 32;                            // an epilogue warp's staging tile: [16 hidden rows][32 vocabulary entries] fp32
constexpr int kStatStageBytes = kEpiWarps * 16 * kScratchPitch * 4;
constexpr int kStatMergeBytes = 4 * kMaxCols * 8;            // (E, s) of every column from each of the four lane quarters
constexpr size_t kGemmSmemBytes = 1024 /* alignment slack */ + static_cast<size_t>(kStagesG) * kStageBytes + 256 /* barriers */ + kStatStageBytes + kStatMergeBytes;

struct GemmJob {
    CUtensorMap map_w;      // [V, d] bf16, box {64, 128}
    CUtensorMap map_h;      // [rows, d] bf16, box {64, chunk / 2}
    CUtensorMap map_out;    // [rows, V] fp32, box {32, 16}, no swizzle: the epilogue's stores
    float* out;             // [rows, V]
    float2* partials;       // [rows, parts] row statistics of the tile just computed, or nullptr
    int rows;
    int kblocks;            // d / 64
    int block_cols;         // columns (hidden rows) per work item, multiple of 16, <= 288
    int chunk;              // columns per MMA, multiple of 16, <= 256; each CTA holds chunk / 2 of them
    int nchunks;            // block_cols / chunk
    int nblocks;            // column blocks covering `rows`
    int items;              // vocabulary tiles * nblocks
};

struct GemmParams {
    GemmJob job[2];
    int n_jobs;
    int V;
    int vtiles;             // 256-entry vocabulary tiles
    int total_items;
    // TMEM is cut into n_slots accumulator slots of slot_cols columns; a tile takes slots_per_tile
    // consecutive ones (round robin), one per MMA chunk: 2 slots of 256, 1 per tile when every column
    // block fits 256 columns, else 3 slots of 144, 2 per tile
    int n_slots, slots_per_tile, slot_cols;
    int parts;              // 128-entry vocabulary slices per row = 2 * vtiles (row statistics)
    float c;                // log2(e) / T (row statistics)
    int32_t* status;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// The shared::cluster address of `addr` (a shared::cta address of this CTA) in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_addr(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Arrive on a barrier of any CTA of the cluster (`bar` is a shared::cluster address).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
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
// Bounded wait that also gives up when a role of either CTA has raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (uint32_t i = 0; i < kSpinLimitG; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    return false;
}

// The same for waits that are known to be long (an epilogue warp waiting for a whole K loop): the
// lanes sleep between polls instead of competing with the issuing warps for instruction slots.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (uint32_t i = 0; i < kSpinLimitG; ++i) {
        if (mbar_try(bar, parity)) return true;
        __nanosleep(256);
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    return false;
}

// 2-D tiled TMA load into this CTA's shared memory; completion is counted on `bar`, a
// shared::cluster address that may belong to the peer CTA of the pair.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// 2-D tiled TMA store of a [16][32] fp32 staging tile; elements outside the tensor are not written.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Until the stores issued by this thread have read their shared-memory source / have completed.
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Shared-memory matrix descriptor (64 bits) of a K-major tile stored as rows of 128 bytes with
// the 128-byte swizzle: start address >> 4 in bits 0..13, leading byte offset (unused here, 1) in
// bits 16..29, stride byte offset 1024 >> 4 (8-row groups 1024 bytes apart) in bits 32..45,
// descriptor version 1 in bits 46..47, layout type 2 in bits 61..63.  The address may point
// 32 * i bytes into the first row to select the i-th 16-element K slice.
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 256 over the CTA pair, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kPairV >> 4) << 24);
}

// The upper word of smem_desc_sw128 is the same for every tile; MMAs are issued from the lower words.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr) { return ((addr & 0x3ffffu) >> 4) | (1u << 16); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint32_t adesc_lo, uint32_t bdesc_lo, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(adesc_lo), "r"(bdesc_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi) : "memory");
}
// Arrives (once all MMAs issued so far have completed) on the barrier at offset `bar` in both CTAs.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    const unsigned short mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
// True in exactly one lane of a fully active warp.  The role loops are run by whole warps
// (every lane polls the barriers) and only the issue of an asynchronous instruction is
// elected, so that loop state and descriptors stay warp-uniform.
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
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
__device__ __forceinline__ void mbar_arrive_local(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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

// Sets the abort flag of both CTAs of the pair and records the timeout.
__device__ __forceinline__ void raise_abort(int* abort_flag, uint32_t peer, int32_t* status)
{
    if (!*reinterpret_cast<volatile int*>(abort_flag) && status) atomicCAS(status, 0, static_cast<int>(POLYSPEC_ERR_TIMEOUT));
    *reinterpret_cast<volatile int*>(abort_flag) = 1;
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr(smem_addr(abort_flag), peer)), "r"(1) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1) lmhead_kernel(const __grid_constant__ GemmParams p)
{
    extern __shared__ unsigned char smem_dyn[];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    // broadcast from lane 0 so that the compiler knows the role branches and everything derived
    // from them (ring positions, descriptors) are warp-uniform
    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();           // 0 = leader of the pair
    const uint32_t peer = rank ^ 1u;
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    // Pair i owns work items i, i + pairs, ...  Odd pairs walk their list backwards (cheap model
    // first): neighbouring pairs are then in different phases, so the store bursts of the epilogues
    // of some overlap the K loops of others instead of all hitting memory at once.
    const int n_mine = (p.total_items - pair + n_pairs - 1) / n_pairs;
    const bool backwards = (pair & 1) != 0;
    const int first_item = backwards ? pair + (n_mine - 1) * n_pairs : pair;
    const int item_step = backwards ? -n_pairs : n_pairs;
    // 128-byte swizzled tiles must start on a 1024-byte boundary; both CTAs use the same offsets
    const uint32_t raw = smem_addr(smem_dyn);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t bars = tiles + kStagesG * kStageBytes;
    const uint32_t full_bar = bars, empty_bar = full_bar + 8u * kStagesG;       // full: used in the leader only
    const uint32_t acc_full = empty_bar + 8u * kStagesG, slot_empty = acc_full + 16u;   // slot_empty[3]: leader only
    float* stat_scratch = reinterpret_cast<float*>(smem_dyn + (bars - raw) + 256);     // per epilogue warp [16][kScratchPitch]
    float2* stat_merge = reinterpret_cast<float2*>(smem_dyn + (bars - raw) + 256 + kStatStageBytes);   // [4][kMaxCols]
    const uint32_t epi_bar = slot_empty + 24u;      // the epilogue warps of this CTA meet here (bounded, unlike bar.sync)

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < kStagesG; ++s) { mbar_init(full_bar + 8u * s, 1); mbar_init(empty_bar + 8u * s, 1); }
        for (int a = 0; a < 2; ++a) mbar_init(acc_full + 8u * a, 1);
        for (int a = 0; a < 3; ++a) mbar_init(slot_empty + 8u * a, 2 * kEpiWarps);
        mbar_init(epi_bar, kEpiWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_base_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();             // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abort_p = &abort_flag;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        uint32_t it = 0;          // K blocks issued so far
        uint32_t stage = 0, phase = 1;      // ring position; a fresh "empty" barrier passes a wait on parity 1
        bool ok = true;
        const uint32_t leader_full = cluster_addr(full_bar, 0);
        for (int item = first_item; ok && item >= 0 && item < p.total_items; item += item_step) {
            int j, vt, nb;
            decode_item(p, item, &j, &vt, &nb);
            const GemmJob& job = p.job[j];
            const int half = job.chunk >> 1;
            const uint32_t pair_bytes = 2u * (kBytesA + static_cast<uint32_t>(job.block_cols >> 1) * (kBlockK * 2));
            const int w_row = vt * kPairV + static_cast<int>(rank) * kTileV;
            const int h_row = nb * job.block_cols + static_cast<int>(rank) * half;
            const bool two = job.nchunks == 2;
            for (int kb = 0; kb < job.kblocks; ++kb, ++it) {
                if (!mbar_wait(empty_bar + 8u * stage, phase, abort_p)) { ok = false; break; }
                const uint32_t bar = leader_full + 8u * stage;
                const uint32_t a_dst = tiles + stage * kStageBytes;
                if (elect_one()) {
                    if (rank == 0) mbar_expect_tx(full_bar + 8u * stage, pair_bytes);
                    tma_load_2d(a_dst, &job.map_w, kb * kBlockK, w_row, bar);
                    tma_load_2d(a_dst + kBytesA, &job.map_h, kb * kBlockK, h_row, bar);
                    if (two) tma_load_2d(a_dst + kBytesA + half * (kBlockK * 2), &job.map_h, kb * kBlockK, h_row + job.chunk, bar);
                }
                __syncwarp();
                if (++stage == kStagesG) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && lane == 0) raise_abort(&abort_flag, peer, p.status);
        __syncwarp();
        // this CTA's copies must have landed before it may exit.  The leader sees them on its own
        // "full" barriers; the peer learns it from the leader's commits on its "empty" barriers,
        // which follow the MMAs that read the stage.
        const uint32_t first = it > static_cast<uint32_t>(kStagesG) ? it - kStagesG : 0u;
        for (uint32_t q = first; q < it; ++q) {
            const uint32_t b = (rank == 0 ? full_bar : empty_bar) + 8u * (q % kStagesG);
            for (uint32_t i = 0; i < kSpinLimitG; ++i)
                if (mbar_try(b, (q / kStagesG) & 1u) || *abort_p) break;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA)
        if (rank == 0) {
            uint32_t stage = 0, phase = 0, tile_n = 0;
            bool ok = true;
            for (int item = first_item; ok && item >= 0 && item < p.total_items; item += item_step, ++tile_n) {
                int j, vt, nb;
                decode_item(p, item, &j, &vt, &nb);
                const GemmJob& job = p.job[j];
                // chunk i of tile t is the (slots_per_tile * t + i)-th accumulator ever used: slot = that number
                // modulo n_slots, and the slot has been used (that number / n_slots) times before
                const uint32_t pos0 = tile_n * p.slots_per_tile, pos1 = pos0 + p.slots_per_tile - 1;
                const uint32_t slot0 = pos0 % p.n_slots, slot1 = pos1 % p.n_slots;
                if (!mbar_wait(slot_empty + 8u * slot0, ((pos0 / p.n_slots) & 1u) ^ 1u, abort_p)) { ok = false; break; }
                if (!mbar_wait(slot_empty + 8u * slot1, ((pos1 / p.n_slots) & 1u) ^ 1u, abort_p)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = instr_desc_bf16(job.chunk);
                const uint32_t d_tmem = tmem_base + slot0 * p.slot_cols, d_tmem1 = tmem_base + slot1 * p.slot_cols;
                const uint32_t b_chunk = static_cast<uint32_t>(job.chunk >> 1) * (kBlockK * 2) >> 4;   // second MMA's B tile, in 16-byte units
                const bool two = job.nchunks == 2;
                for (int kb = 0; kb < job.kblocks; ++kb) {
                    if (!mbar_wait(full_bar + 8u * stage, phase, abort_p)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_lo = smem_desc_lo(tiles + stage * kStageBytes);
                    const uint32_t b_lo = a_lo + (kBytesA >> 4);
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < kBlockK / kMmaK; ++kk) {
                            const uint32_t acc_flag = (kb | kk) != 0 ? 1u : 0u;
                            umma_bf16(d_tmem, a_lo + kk * (kMmaK * 2 >> 4), b_lo + kk * (kMmaK * 2 >> 4), idesc, acc_flag);
                            if (two)
                                umma_bf16(d_tmem1, a_lo + kk * (kMmaK * 2 >> 4), b_lo + b_chunk + kk * (kMmaK * 2 >> 4), idesc, acc_flag);
                        }
                        umma_commit_pair(empty_bar + 8u * stage);      // frees the stage in both CTAs once these MMAs have read it
                    }
                    __syncwarp();
                    if (++stage == kStagesG) { stage = 0; phase ^= 1u; }
                }
                if (ok && elect_one()) umma_commit_pair(acc_full + 8u * (tile_n & 1u));     // tile complete, in both CTAs
                __syncwarp();
            }
            if (!ok && lane == 0) raise_abort(&abort_flag, peer, p.status);
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
        const int quarter = warp & 3;                   // the TMEM lanes this warp may read: 32 * quarter ..
        const int half_id = (warp - 2) >> 2;            // which of the quarter's two warps this is
        const uint32_t leader_slot_empty = cluster_addr(slot_empty, 0);
        float* scratch = stat_scratch + (warp - 2) * (16 * kScratchPitch);
        uint32_t tile_n = 0, epi_phase = 0;
        bool ok = true;
        for (int item = first_item; ok && item >= 0 && item < p.total_items; item += item_step, ++tile_n) {
            int j, vt, nb;
            decode_item(p, item, &j, &vt, &nb);
            const GemmJob& job = p.job[j];
            if (!mbar_wait_relaxed(acc_full + 8u * (tile_n & 1u), (tile_n >> 1) & 1u, abort_p)) { ok = false; break; }
            tc_fence_after();
            const uint32_t pos0 = tile_n * p.slots_per_tile;
            const uint32_t slot0 = pos0 % p.n_slots, slot1 = (pos0 + p.slots_per_tile - 1) % p.n_slots;
            const int v_base = vt * kPairV + static_cast<int>(rank) * kTileV + quarter * 32;     // this warp's 32 vocabulary entries
            const int row0 = nb * job.block_cols;
            const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            // TMEM address of column c of the tile: chunk 0 lives in slot0, chunk 1 (if any) in slot1
            auto t_col = [&](int c) {
                return c < job.chunk ? t_lane + slot0 * p.slot_cols + c : t_lane + slot1 * p.slot_cols + (c - job.chunk);
            };
            bool freed0 = p.slots_per_tile == 1;        // slot0 handed back already (or is the only, last one)
            const bool stats = job.partials != nullptr;
            const int slice = vt * 2 + static_cast<int>(rank);      // this CTA's 128-entry slice of the row
            // the two warps of a quarter take alternate 16-column chunks; a warp's next chunk is already
            // on its way from TMEM while it works on the current one
            uint32_t nxt[16];
            const int c_first = 16 * half_id;
            if (c_first < job.block_cols) tmem_ld16(t_col(c_first), nxt);
            for (int c0 = c_first; c0 < job.block_cols; c0 += 32) {
                uint32_t r[16];
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; ++i) r[i] = nxt[i];
                if (!freed0 && c0 >= job.chunk) {
                    // everything this warp reads from the first slot is in registers: the next tile may overwrite it
                    freed0 = true;
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(leader_slot_empty + 8u * slot0);
                }
                if (c0 + 32 < job.block_cols) tmem_ld16(t_col(c0 + 32), nxt);
                if (row0 + c0 >= job.rows) continue;                       // no such hidden rows (warp-uniform)
                if (v_base >= p.V) {                                       // no such vocabulary entries: an empty share
                    if (stats && lane < 16) stat_merge[quarter * kMaxCols + c0 + lane] = make_float2(kEmptyRef, 0.0f);
                    continue;
                }
                // registers -> staging tile [hidden row][vocabulary entry]; one TMA store writes its 16 rows of
                // 128 bytes, the row statistics are read from the same tile
                if (lane == 0) tma_store_wait_read();           // the previous store has read the tile
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 16; ++i) scratch[i * kScratchPitch + lane] = __uint_as_float(r[i]);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) tma_store_2d(&job.map_out, v_base, row0 + c0, smem_addr(scratch));
                if (stats) {
                    // A lane owns one hidden row (col) and 16 of the 32 entries, visited in an order rotated by
                    // col so that the lanes hit different banks; the two lanes of a row are then combined.
                    // Result: (E, s) with sum_v 2^(z_v c - E) = s, E an integer at or just above the largest z_v c.
                    const int col = lane & 15, e0 = (lane >> 4) * 16;
                    float z[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int e = e0 + ((j + col) & 15);
                        z[j] = (v_base + e < p.V) ? scratch[col * kScratchPitch + e] : -INFINITY;
                    }
                    float m = z[0];
#pragma unroll
                    for (int j = 1; j < 16; ++j) m = fmaxf(m, z[j]);
                    const float E = (m == -INFINITY) ? kEmptyRef : ceilf(m * p.c);
                    float sm = 0.0f;
#pragma unroll
                    for (int j = 0; j < 16; ++j) sm = __fadd_rn(sm, ex2f(__fmaf_rn(z[j], p.c, -E)));
                    const float E2 = __shfl_xor_sync(0xffffffffu, E, 16), s2 = __shfl_xor_sync(0xffffffffu, sm, 16);
                    const float Em = fmaxf(E, E2);
                    const float lo = (lane & 16) ? s2 : sm, hi = (lane & 16) ? sm : s2;       // same order in both lanes
                    const float Elo = (lane & 16) ? E2 : E, Ehi = (lane & 16) ? E : E2;
                    const float tot = __fadd_rn(__fmul_rn(lo, pow2_neg(Elo - Em)), __fmul_rn(hi, pow2_neg(Ehi - Em)));
                    if (lane < 16) stat_merge[quarter * kMaxCols + c0 + col] = make_float2(Em, tot);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (!freed0 && lane == 0) mbar_arrive_cluster(leader_slot_empty + 8u * slot0);     // (a warp without chunks in slot1)
            if (lane == 0) mbar_arrive_cluster(leader_slot_empty + 8u * slot1);     // the accumulator may be overwritten
            if (stats) {
                // all chunks are in: merge the four quarters of every column into the partial of this CTA's slice
                __syncwarp();
                if (lane == 0) mbar_arrive_local(epi_bar);
                if (!mbar_wait(epi_bar, epi_phase, abort_p)) { ok = false; break; }
                epi_phase ^= 1u;
                for (int col = (warp - 2) * 32 + lane; col < job.block_cols; col += 32 * kEpiWarps) {
                    const int row = row0 + col;
                    if (row < job.rows) {
                        float2 q[4];
#pragma unroll
                        for (int w = 0; w < 4; ++w) q[w] = stat_merge[w * kMaxCols + col];
                        const float Em = fmaxf(fmaxf(q[0].x, q[1].x), fmaxf(q[2].x, q[3].x));
                        float tot = 0.0f;
#pragma unroll
                        for (int w = 0; w < 4; ++w) tot = __fadd_rn(tot, __fmul_rn(q[w].y, pow2_neg(q[w].x - Em)));
                        job.partials[static_cast<size_t>(row) * p.parts + slice] = make_float2(Em, tot);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive_local(epi_bar);
                if (!mbar_wait(epi_bar, epi_phase, abort_p)) { ok = false; break; }     // the merge area may be rewritten
                epi_phase ^= 1u;
            }
        }
        if (lane == 0) tma_store_wait_all();        // this thread's stores have landed before the CTA may exit
        if (!ok && lane == 0) raise_abort(&abort_flag, peer, p.status);
    }

    // Neither CTA may leave (or free TMEM) while the other can still signal its barriers or while
    // MMAs of the pair are in flight: in the normal course every MMA has been waited for through
    // the accumulator barriers by the time the epilogues are done.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    if (warp == 1) {
        if (*abort_p) __nanosleep(1000000);      // aborting: give MMAs in flight a bounded moment
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_init_mutex;
EncodeTiledFn g_encode = nullptr;
bool g_attr_set[64] = {false};
int g_pairs[64] = {0};      // CTA pairs the device can hold at once

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
// [n_rows, V] fp32 row-major; box = 32 vocabulary entries (128 bytes) by 16 rows, no swizzle.
bool encode_out_map(CUtensorMap* map, float* base, int n_rows, int V)
{
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(V), static_cast<cuuint64_t>(n_rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(V) * 4};
    const cuuint32_t box[2] = {32, 16};
    const cuuint32_t estr[2] = {1, 1};
    return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

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

cudaError_t launch_lmhead(const LmHeadProblem* probs, int n, int V, float c, int32_t* device_status, cudaStream_t stream)
{
    if (n < 1 || n > 2) return cudaErrorInvalidValue;
    std::lock_guard<std::mutex> lock(g_init_mutex);      // one-time set-up below; host threads may call concurrently
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
        if (sms <= 0) sms = 148;
        // how many 2-CTA clusters fit at once (an odd SM of a GPC cannot host one)
        int clusters = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(sms / 2 * 2));
        cfg.blockDim = dim3(kGemmThreads);
        cfg.dynamicSmemBytes = kGemmSmemBytes;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (cudaOccupancyMaxActiveClusters(&clusters, lmhead_kernel, &cfg) != cudaSuccess || clusters <= 0) {
            (void)cudaGetLastError();
            clusters = sms / 2;
        }
        g_pairs[dev] = clusters < sms / 2 ? clusters : sms / 2;
        g_attr_set[dev] = true;
    }

    GemmParams p;
    p.n_jobs = n;
    p.V = V;
    p.vtiles = (V + kPairV - 1) / kPairV;
    p.parts = 2 * p.vtiles;
    p.c = c;
    p.status = device_status;
    p.total_items = 0;
    bool wide = false;          // some column block needs more than 256 TMEM columns
    for (int i = 0; i < n; ++i) {
        const int c16 = (probs[i].rows + 15) / 16 * 16;
        if (c16 > 256 && c16 <= kMaxCols) wide = true;
    }
    p.n_slots = wide ? 3 : 2;
    p.slots_per_tile = wide ? 2 : 1;
    p.slot_cols = wide ? kMaxCols / 2 : kTmemCols / 2;
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
        if (wide) {                                             // two MMAs per K block, each a multiple of 16 columns
            if (cols > kMaxCols) cols = kMaxCols;
            cols = (cols + 31) / 32 * 32;
        } else if (cols > 256) {
            cols = 256;                                         // many rows: 256-column blocks
        }
        job.block_cols = cols;
        job.nchunks = wide ? 2 : 1;
        job.chunk = cols / job.nchunks;
        job.nblocks = (pr.rows + cols - 1) / cols;
        job.rows = pr.rows;
        job.kblocks = pr.d / kBlockK;
        job.out = pr.out;
        job.partials = pr.partials;
        job.items = p.vtiles * job.nblocks;
        p.total_items += job.items;
        if (!encode_map(&job.map_w, pr.W, V, pr.d, kTileV)) return cudaErrorInvalidValue;
        if (!encode_map(&job.map_h, pr.hidden, pr.rows, pr.d, job.chunk / 2)) return cudaErrorInvalidValue;
        if (!encode_out_map(&job.map_out, pr.out, pr.rows, V)) return cudaErrorInvalidValue;
    }
    const int pairs = p.total_items < g_pairs[dev] ? p.total_items : g_pairs[dev];
    lmhead_kernel<<<2 * pairs, kGemmThreads, kGemmSmemBytes, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace polyspec
