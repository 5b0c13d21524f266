// The tensor-bound vocabulary head on CTA pairs (tcgen05.mma.cta_group::2): levels of more than 128 nodes.
//
// Why pairs.  With one CTA per tile every K block of [128 + block_n] rows x 128 bytes is written into shared
// memory once (TMA) and read from it once (MMA): 2 * (128 + 224) * 128 bytes per 448 tensor-pipe cycles =
// 201 bytes per cycle against the 128 bytes per cycle one SM's shared memory moves, so the tensor pipe cannot be
// busy more than about two thirds of the time (measured: 66 %).  A pair of CTAs on neighbouring SMs computes a
// [256 nodes x block_n vocabulary rows] tile with ONE instruction stream: each CTA holds its own 128 node rows (A)
// and HALF of the weight rows (B); the hardware feeds both tensor cores from both halves.  Per SM that is
// 2 * (128 + block_n / 2) * 128 bytes per K block: 137 bytes per cycle at block_n = 224.
//
// Roles per CTA (224 threads) as in gemm_tc_kernel: warps 0 and 6 issue the TMA copies of this CTA's operand
// halves (their completion bytes go to the barrier of the pair's first CTA), warp 1 of the first CTA issues the
// MMAs for both and releases ring slots and accumulators in both CTAs with commits that arrive in both, warps 2-5 of
// either CTA run the fused top-k / log-sum-exp epilogue on their own 128 rows of the accumulator (tc_gemm.cuh,
// one thread per node row) and then tell the first CTA that the accumulator slot is free.  Every wait on an
// mbarrier is bounded; every thread of both CTAs reaches the cluster barrier at the end whatever happened, TMEM is
// freed behind it.  Every TMA copy here has one destination: the shared memory of the CTA that issued it.
#include <cuda.h>

#include <mutex>

#include "tc_gemm.cuh"

namespace spec {

namespace {

using namespace tc;

constexpr int kPairStagesMax = 8;
constexpr int kPairRows = 2 * kBlockM;      // node rows of one tile of a pair
constexpr int kPairTmemCols = 512;          // two accumulator slots of up to 256 columns

struct __align__(8) PairBars {
    uint64_t full[kPairStagesMax];          // used in the pair's first CTA: both CTAs' copies complete here
    uint64_t empty[kPairStagesMax];         // in each CTA: the MMAs that read the slot have finished
    uint64_t acc_full[2];                   // in each CTA: the tile's MMAs have finished
    uint64_t acc_empty[2];                  // used in the first CTA: 8 arrivals, one per epilogue warp of the pair
    uint32_t tmem_base;
    volatile int abort_flag;
};

struct PairParams {
    GemmJob job;             // M = nodes, N = vocabulary rows, block_n, n_tiles, epi (mode 1); m_tiles = 256-row tiles
    int n_pairs;             // pairs in the grid (gridDim.x / 2)
    int stages;
    uint32_t slot_bytes;     // [128 x 128 B] A box + [block_n / 2 x 128 B] B box
    int32_t *err;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// All threads of both CTAs.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
}

// The shared::cluster address of the same variable in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local_addr), "r"(rank));
    return a;
}

__device__ __forceinline__ void remote_arrive(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// Bounded wait on a barrier of this CTA.
__device__ __forceinline__ bool pair_wait(uint64_t *bar, uint32_t parity, PairBars *bars, int32_t *err) {
    for (uint32_t it = 0; it < kSpinMax; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > kSpinFast) {
            if (bars->abort_flag) return false;
            __nanosleep(64);
        }
    }
    bars->abort_flag = 1;
    report_error(err, SPEC_ERR_TIMEOUT);
    return false;
}

// After a wait that ran out: copies and MMAs already issued still target this CTA's (and its partner's) shared
// memory and TMEM, and their completion barriers live partly in the other CTA.  Rather than chase them across the
// pair, the thread that gave up simply stays for a few hundred microseconds - orders of magnitude longer than any
// copy or MMA in flight takes - before it joins the tear-down.
__device__ __forceinline__ void abort_grace() {
    for (int i = 0; i < 4096; ++i) __nanosleep(128);
}

// This CTA's box of a pair's tile; the completion bytes are counted on `bar_cluster_addr` (a barrier of the pair's
// first CTA).  Every CTA fetches its own box into its own shared memory; nothing is broadcast across the pair.
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, int c0, int c1, uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(bar_cluster_addr)
        : "memory");
}

// Arrives on the barrier at this shared-memory offset in both CTAs once the MMAs issued so far have finished.
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(smem_u32(bar)), "h"((uint16_t)3)
        : "memory");
}

// The four MMAs of one K block, M = 256 over the pair.
__device__ __forceinline__ void umma_k_block_pair(uint32_t tmem_d, uint32_t lo_a, uint32_t lo_b, uint32_t desc_hi,
                                                  uint32_t idesc, uint32_t first_acc) {
    asm volatile(
        "{\n\t"
        ".reg .pred p, t;\n\t"
        ".reg .b64 da, db;\n\t"
        ".reg .b32 la, lb, z;\n\t"
        "mov.b32 z, 0;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "setp.eq.b32 t, 0, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, {z, z, z, z, z, z, z, z}, p;\n\t"
        "add.u32 la, %1, 2;\n\t"
        "add.u32 lb, %2, 2;\n\t"
        "mov.b64 da, {la, %3};\n\t"
        "mov.b64 db, {lb, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, {z, z, z, z, z, z, z, z}, t;\n\t"
        "add.u32 la, %1, 4;\n\t"
        "add.u32 lb, %2, 4;\n\t"
        "mov.b64 da, {la, %3};\n\t"
        "mov.b64 db, {lb, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, {z, z, z, z, z, z, z, z}, t;\n\t"
        "add.u32 la, %1, 6;\n\t"
        "add.u32 lb, %2, 6;\n\t"
        "mov.b64 da, {la, %3};\n\t"
        "mov.b64 db, {lb, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, {z, z, z, z, z, z, z, z}, t;\n\t"
        "}"
        ::"r"(tmem_d), "r"(lo_a), "r"(lo_b), "r"(desc_hi), "r"(idesc), "r"(first_acc)
        : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ PairParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    PairBars *bars = (PairBars *)(tiles + (size_t)p.stages * p.slot_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0: the CTA that issues the MMAs
    const GemmJob &j = p.job;
    const int half_n = j.block_n / 2;
    const int num_kb = (j.Kd + kSlabBytes / 2 - 1) / (kSlabBytes / 2);
    const int num_tiles = j.m_tiles * j.n_tiles;
    const int pair = (int)(blockIdx.x >> 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->acc_full[a], 1);
            mbar_init(&bars->acc_empty[a], 2 * (kEpilogueThreads / 32));
        }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // the same warp in both CTAs, the same destination offset: one allocation for the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)),
                     "r"((uint32_t)kPairTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();      // both CTAs' barriers are initialised before either is signalled from the other side
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    griddep_launch();
    griddep_wait();          // the states are the preceding kernel's output

    if (warp == 0 || warp == kThreads / 32 - 1) {
        if (lane == 0) {
            const int me = warp == 0 ? 0 : 1;
            int stage = 0, seq = 0;
            uint32_t phase = 0;
            const uint32_t tx = 2u * ((uint32_t)kABytes + (uint32_t)half_n * kSlabBytes);   // both CTAs' boxes
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += p.n_pairs) {
                const int m_tile = tile % j.m_tiles, n_tile = tile / j.m_tiles;
                const int a_row = m_tile * kPairRows + (int)rank * kBlockM;
                const int b_row = n_tile * j.block_n + (int)rank * half_n;
                for (int kb = 0; kb < num_kb; ++kb, ++seq) {
                    if (seq % kMaxProducers == me) {
                        if (!pair_wait(&bars->empty[stage], phase ^ 1u, bars, p.err)) { ok = false; break; }
                        uint8_t *sa = tiles + (size_t)stage * p.slot_bytes;
                        if (rank == 0) mbar_arrive_expect_tx(&bars->full[stage], tx);
                        const uint32_t full0 = map_to_rank(smem_u32(&bars->full[stage]), 0);
                        tma_load_2d_pair(sa, &map_a, kb * (kSlabBytes / 2), a_row, full0);
                        tma_load_2d_pair(sa + kABytes, &map_b, kb * (kSlabBytes / 2), b_row, full0);
                    }
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) abort_grace();
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = make_instr_desc(kPairRows, j.block_n, false);
            const uint32_t desc_hi = (uint32_t)(make_smem_desc(0) >> 32);
            const uint32_t lo_base = (smem_u32(tiles) & 0x3ffffu) >> 4, lo_slot = p.slot_bytes >> 4;
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += p.n_pairs) {
                if (!pair_wait(&bars->acc_empty[acc], acc_phase ^ 1u, bars, p.err)) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * j.block_n);
                uint32_t first = 0u;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!pair_wait(&bars->full[stage], phase, bars, p.err)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t lo_a = lo_base + (uint32_t)stage * lo_slot;
                    umma_k_block_pair(tmem_d, lo_a, lo_a + (kABytes >> 4), desc_hi, idesc, first);
                    first = 1u;
                    umma_commit_pair(&bars->empty[stage]);    // frees the slot in both CTAs
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_pair(&bars->acc_full[acc]);       // both CTAs' epilogues may read their rows
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (bars->abort_flag) abort_grace();
        }
    } else {
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        int acc = 0;
        uint32_t acc_phase = 0;
        const uint32_t acc_empty0[2] = {map_to_rank(smem_u32(&bars->acc_empty[0]), 0),
                                        map_to_rank(smem_u32(&bars->acc_empty[1]), 0)};
        for (int tile = pair; tile < num_tiles; tile += p.n_pairs) {
            const int m_tile = tile % j.m_tiles, n_tile = tile / j.m_tiles;
            if (!pair_wait(&bars->acc_full[acc], acc_phase, bars, p.err)) break;
            tc_fence_after();
            const int row = m_tile * kPairRows + (int)rank * kBlockM + row_in_tile;
            const bool row_ok = row < j.M;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * j.block_n);
            const int col0 = n_tile * j.block_n;
            if (j.epi.topk <= 4) epilogue_topk<4, false>(j, taddr, row, row_ok, col0, n_tile);
            else epilogue_topk<SPEC_MAX_TOPK, false>(j, taddr, row, row_ok, col0, n_tile);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) remote_arrive(acc_empty0[acc]);    // (the first CTA's own address for its own warps)
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }
    // Tear-down: nobody leaves while the other CTA may still signal its barriers, read its shared memory or
    // write its TMEM; the accumulators have been read (or given up on) by now.
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kPairTmemCols)
                     : "memory");
    }
}

std::mutex g_pair_mutex;
int g_pair_clusters[64] = {};   // co-resident pairs per device, 0: not asked yet

}  // namespace

// Vocabulary columns per tile of the pair kernel: the width that needs the fewest tile rounds over the pairs of
// the device, a multiple of 32 in [128, 256] (each CTA loads half of it).
int pair_block_n(int rows, int vocab_rows) {
    const int pairs = num_sms() / 2;
    const int m_tiles = (rows + kPairRows - 1) / kPairRows;
    int best = 256;
    long long best_cost = -1;
    for (int bn = 128; bn <= 256; bn += 32) {
        const long long tiles = (long long)m_tiles * ((vocab_rows + bn - 1) / bn);
        const long long rounds = (tiles + pairs - 1) / pairs;
        const long long cost = rounds * (bn + 48);
        if (best_cost < 0 || cost <= best_cost) {
            best_cost = cost;
            best = bn;
        }
    }
    return best;
}

// C = states [rows, Kd] x weights [V, Kd]^T with the mode-1 epilogue (per row and vocabulary tile a partial top-k
// list and (max, sum-exp)), on CTA pairs.  block_n as pair_block_n gives it.
int launch_head_pair(const void *states, const void *W, int rows, int V, int Kd, int block_n, const GemmEpilogue &epi,
                     int32_t *err, cudaStream_t st) {
    if (rows <= 0 || V <= 0 || Kd <= 0 || Kd % 8 != 0 || block_n < 128 || block_n > 256 || block_n % 32 != 0 ||
        epi.mode != 1 || epi.fp8)
        return SPEC_ERR_SHAPE;
    if (((uintptr_t)states & 15) || ((uintptr_t)W & 15)) return SPEC_ERR_INVALID_ARG;
    PairParams p{};
    GemmJob &j = p.job;
    j.M = rows; j.N = V; j.Kd = Kd;
    j.block_n = block_n;
    j.m_tiles = (rows + kPairRows - 1) / kPairRows;
    j.n_tiles = (V + block_n - 1) / block_n;
    j.splits = 1;
    j.kb_per_split = (Kd + 63) / 64;
    j.epi = epi;
    p.err = err;
    p.slot_bytes = (uint32_t)kABytes + (uint32_t)(block_n / 2) * kSlabBytes;
    p.stages = (kSmemLimit - 1024 - (int)sizeof(PairBars) - 64) / (int)p.slot_bytes;
    if (p.stages > kPairStagesMax) p.stages = kPairStagesMax;
    if (p.stages < 2) return SPEC_ERR_SHAPE;
    CUtensorMap map_a, map_b;
    int rc = make_tmap(&map_a, states, (uint64_t)rows, (uint64_t)Kd, kBlockM, false, false);
    if (rc != SPEC_OK) return rc;
    rc = make_tmap(&map_b, W, (uint64_t)V, (uint64_t)Kd, (uint32_t)(block_n / 2), true, false);
    if (rc != SPEC_OK) return rc;
    const size_t smem = 1024 + (size_t)p.stages * p.slot_bytes + sizeof(PairBars);

    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;

    int dev = 0;
    SPEC_CUDA_TRY(cudaGetDevice(&dev));
    int pairs = 0;
    {
        std::lock_guard<std::mutex> lock(g_pair_mutex);
        if (dev < 0 || dev >= 64 || g_pair_clusters[dev] == 0) {
            SPEC_CUDA_TRY(cudaFuncSetAttribute(gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
            cfg.gridDim = dim3(2 * (num_sms() / 2));
            cfg.dynamicSmemBytes = kSmemLimit;
            int n = 0;
            SPEC_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel, &cfg));
            cfg.dynamicSmemBytes = smem;
            if (n < 1) return SPEC_ERR_SHAPE;
            if (n > num_sms() / 2) n = num_sms() / 2;
            if (dev >= 0 && dev < 64) g_pair_clusters[dev] = n;
            pairs = n;
        } else {
            pairs = g_pair_clusters[dev];
        }
    }
    const long long tiles = (long long)j.m_tiles * j.n_tiles;
    if (tiles < pairs) pairs = (int)tiles;
    p.n_pairs = pairs;
    cfg.gridDim = dim3(2 * pairs);
    SPEC_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_pair_kernel, map_a, map_b, p));
    return SPEC_OK;
}

// Co-resident pairs of the current device (0 before the first launch there): what pair_block_n's rounds assume.
int pair_clusters_cached() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    std::lock_guard<std::mutex> lock(g_pair_mutex);
    return g_pair_clusters[dev];
}

}  // namespace spec
