// Device-side building blocks of the sm_100a tensor-core contraction
//     C[M, N] = A[M, Kd] * B[N, Kd]^T,  bf16 operands (row-major = K-major for both), fp32 in TMEM,
// used by the GEMM kernel (gemm_tcgen05.cu).
//
// A CTA has 224 threads in three roles that meet only through mbarriers:
//   warps 0, 6  TMA producers (one lane each, alternating ring slots): 128-byte-swizzled [128 x 64] A boxes
//               and [block_n x 64] B boxes into a ring of shared-memory slots, completion on "full" barriers
//   warp 1      owns the TMEM allocation; one lane issues tcgen05.mma (M 128, N block_n, K 16) and
//               commits to the slot's "empty" barrier and, per tile, to "accumulator full"
//   warps 2-5   epilogue: tcgen05.ld of 32 columns at a time, one thread per accumulator row
// Two accumulator slots in TMEM let the epilogue of tile i overlap the MMAs of tile i + 1.
// Epilogue modes: 0 plain fp32 store; 1 per-row partial top-k + (max, sum-exp) with one thread per accumulator
// row; 2 split-K partials stored transposed (operands swapped: weights on the 128-row side); 3 the vocabulary
// head with the operands swapped (levels of at most 128 nodes: the MMA work then follows the number of nodes
// instead of being padded to 128 rows): the accumulator tile [128 vocabulary rows x nodes] is transposed
// through shared memory and every node's column is scanned by its own threads, which keep one running
// top-k list and (max, sum-exp) pair for all tiles of the CTA.
// A "job" is one contraction; its tiles (m fastest, then n, then the K split) are dealt round-robin to
// the CTAs of the grid, and each role walks the jobs it is given in the same order, carrying its ring
// position from one job to the next.  Every wait is bounded: when one runs out the CTA records
// SPEC_ERR_TIMEOUT, raises its abort flag and every role returns false.
#pragma once

#include <cuda.h>

#include "spec_common.cuh"

namespace spec {
namespace tc {

constexpr int kBlockM = 128;
constexpr int kSlabBytes = 128;        // one K block = one 128-byte swizzle span per row: 64 bf16 or 128 fp8 elements
constexpr int kUmmaBytes = 32;         // K extent of one MMA instruction in bytes: 16 bf16 or 32 fp8 elements
constexpr int kMaxProducers = 2;       // TMA-issuing threads (lane 0 of warp 0 and, optionally, of warp 6, alternating
                                       // the ring slots)
constexpr int kThreads = 224;
constexpr int kEpilogueFirst = 64;     // first epilogue thread
constexpr int kEpilogueThreads = 128;  // warps 2-5
constexpr int kMaxStages = 12;
constexpr int kABytes = kBlockM * kSlabBytes;
constexpr int kSmemLimit = 222 * 1024; // leaves room on the SM for the small kernels that overlap with a GEMM
constexpr uint32_t kSpinFast = 1u << 14;
constexpr uint32_t kSpinMax = 1u << 24;
constexpr int kTPitch = kBlockM + 4;   // floats between the columns of the transposed tile (mode 3): rows of four
                                       // floats stay 16-byte aligned and eight neighbouring columns hit 32 banks
constexpr int kSwapMaxSegs = 8;        // most threads that share one node's column in the mode-3 scan

struct __align__(8) Barriers {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t drained;           // abort path only: completes when every MMA issued so far has finished
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile int epi_ok;        // mode 3: the epilogue leader's verdict on its wait, read by the other epilogue warps
};

// One contraction as the kernels see it.
struct GemmJob {
    int M, N, Kd;
    int block_n, m_tiles, n_tiles;
    int splits, kb_per_split;   // split-K: tile = (m_tile, n_tile, split), split slowest
    int fp8;                    // 0: bf16 operands (kind::f16); 1: e4m3 operands (kind::f8f6f4); fp32 accumulation either way
    int w_is_a;                 // 1: A holds the weights (no kernel writes them), B the states; 0: the reverse
    int first_cta;              // CTA that takes tile 0; tile t goes to CTA (first_cta + t mod deal_ctas) mod grid
    int deal_ctas;              // CTAs the tiles are dealt to, consecutive from first_cta (0: the whole grid)
    int rows_per_cta;           // mode 3: A rows (vocabulary rows) of every CTA of the deal, a multiple of 8: CTA c
                                // of the deal takes rows [c * rows_per_cta, (c + 1) * rows_per_cta) as 128-row tiles
                                // plus one shorter tile, so that every CTA streams the same number of bytes
    GemmEpilogue epi;
};

// Shared-memory ring and accumulator ring of one CTA.
struct Pipe {
    uint8_t *tiles;        // 1024-byte aligned; slot s at tiles + s * slot_bytes: A box, then B box at +kABytes
    Barriers *bars;
    uint32_t tmem_base;
    int stages;
    uint32_t slot_bytes;
    int acc_stride;        // TMEM columns between the two accumulator slots
    float *tbuf;           // mode 3: transposed accumulator tile, [nodes][kTPitch] floats (null when not used)
    int32_t *err;
};

struct RingPos { int stage; uint32_t phase; };
struct AccPos { int acc; uint32_t phase; };

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false when it gave up (or another role already did).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Barriers *bars, int32_t *err) {
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

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
        : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows at a 128-byte
// pitch, groups of 8 rows 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3ffffu) >> 4);        // start address, bits 0-13
    d |= (uint64_t)0 << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024u >> 4) << 32;               // stride byte offset, bits 32-45
    d |= (uint64_t)1 << 46;                          // version, bits 46-47
    d |= (uint64_t)2 << 61;                          // layout type: SWIZZLE_128B
    return d;
}

// Instruction descriptor: D = fp32, A and B of one type (bf16 for kind::f16, e4m3 for kind::f8f6f4), both
// K-major, M x N tile.
__device__ __forceinline__ uint32_t make_instr_desc(int m, int n, bool fp8) {
    uint32_t d = 0;
    d |= 1u << 4;                      // D format: F32
    d |= (fp8 ? 0u : 1u) << 7;         // A format: kind::f16: 1 = BF16; kind::f8f6f4: 0 = E4M3
    d |= (fp8 ? 0u : 1u) << 10;        // B format, same encoding
    d |= (uint32_t)(n >> 3) << 17;     // N / 8
    d |= (uint32_t)(m >> 4) << 24;     // M / 16
    return d;
}

__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- CTA set-up and tear-down ------------------------------------------------------------------------
// Called by all threads.  Initialises the barriers, allocates `tmem_cols` TMEM columns (a power of two,
// at least 32) and returns the pipe description.
__device__ __forceinline__ Pipe pipe_setup(uint8_t *smem_raw, int stages, uint32_t slot_bytes, int tmem_cols,
                                           int acc_stride, uint32_t tbuf_bytes, int32_t *err) {
    Pipe pp;
    pp.tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);   // swizzled tiles: 1024-byte aligned
    pp.tbuf = tbuf_bytes ? (float *)(pp.tiles + (size_t)stages * slot_bytes) : nullptr;
    pp.bars = (Barriers *)(pp.tiles + (size_t)stages * slot_bytes + tbuf_bytes);
    pp.stages = stages;
    pp.slot_bytes = slot_bytes;
    pp.acc_stride = acc_stride;
    pp.err = err;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&pp.bars->full[s], 1);
            mbar_init(&pp.bars->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&pp.bars->acc_full[a], 1);
            mbar_init(&pp.bars->acc_empty[a], 4);   // one arrival per epilogue warp
        }
        mbar_init(&pp.bars->drained, 1);
        pp.bars->abort_flag = 0;
        pp.bars->epi_ok = 1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&pp.bars->tmem_base)),
                     "r"((uint32_t)tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pp.tmem_base = pp.bars->tmem_base;
    return pp;
}

// Called by all threads after every role has left its loops.
__device__ __forceinline__ void pipe_teardown(const Pipe &pp, int tmem_cols) {
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if ((threadIdx.x >> 5) == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(pp.tmem_base), "r"((uint32_t)tmem_cols)
                     : "memory");
    }
}

// Elements of one 128-byte K block, and the number of K blocks of a job.
__device__ __forceinline__ int slab_elems(const GemmJob &j) { return j.fp8 ? kSlabBytes : kSlabBytes / 2; }
__device__ __forceinline__ int num_k_blocks(const GemmJob &j) { return (j.Kd + slab_elems(j) - 1) / slab_elems(j); }

// The tiles of job j that this CTA takes, as a walk  t = first, first + step, ... < end.
// Modes 0-2: tile index = (split, n_tile, m_tile) with m fastest, dealt round-robin over the CTAs of the deal.
// Mode 3: the CTA's own run of A rows cut into 128-row tiles; t counts them from 0.
struct TileWalk { int first, end, step, rel; };
struct TilePos {
    int a_row, b_row;    // first row of the A box and of the B box
    int kb0, kb1;        // K blocks [kb0, kb1)
    int a_rows;          // rows of the A box (mode 3: the last tile of a CTA may be shorter)
    int split, m_tile, n_tile;
};

__device__ __forceinline__ int cta_rel(const GemmJob &j) {
    return (int)((blockIdx.x + gridDim.x - (unsigned)j.first_cta % gridDim.x) % gridDim.x);
}

__device__ __forceinline__ TileWalk walk_of(const GemmJob &j) {
    TileWalk w;
    w.rel = cta_rel(j);
    if (j.epi.mode == 3) {
        int rows = 0;
        if (w.rel < j.deal_ctas) rows = min(j.M - w.rel * j.rows_per_cta, j.rows_per_cta);
        w.first = 0;
        w.end = rows > 0 ? (rows + kBlockM - 1) / kBlockM : 0;
        w.step = 1;
    } else {
        w.step = j.deal_ctas > 0 ? j.deal_ctas : (int)gridDim.x;
        w.end = j.m_tiles * j.n_tiles * j.splits;
        w.first = w.rel < w.step ? w.rel : w.end;
    }
    return w;
}

__device__ __forceinline__ TilePos pos_of(const GemmJob &j, const TileWalk &w, int t) {
    TilePos q;
    const int num_kb = (j.Kd + (j.fp8 ? kSlabBytes : kSlabBytes / 2) - 1) / (j.fp8 ? kSlabBytes : kSlabBytes / 2);
    if (j.epi.mode == 3) {
        q.a_row = w.rel * j.rows_per_cta + t * kBlockM;
        q.b_row = 0;
        q.kb0 = 0; q.kb1 = num_kb;
        q.a_rows = (t + 1) * kBlockM <= j.rows_per_cta ? kBlockM : j.rows_per_cta - t * kBlockM;
        q.split = 0; q.m_tile = t; q.n_tile = 0;
    } else {
        const int mn_tiles = j.m_tiles * j.n_tiles;
        q.split = t / mn_tiles;
        const int mn = t - q.split * mn_tiles;
        q.m_tile = mn % j.m_tiles;
        q.n_tile = mn / j.m_tiles;
        q.a_row = q.m_tile * kBlockM;
        q.b_row = q.n_tile * j.block_n;
        q.kb0 = q.split * j.kb_per_split;
        q.kb1 = min(num_kb, q.kb0 + j.kb_per_split);
        q.a_rows = kBlockM;
    }
    return q;
}

__device__ __forceinline__ void advance(const Pipe &pp, RingPos &rp) {
    if (++rp.stage == pp.stages) { rp.stage = 0; rp.phase ^= 1u; }
}

// ---- producer (one thread) -----------------------------------------------------------------------
// Loads every k block of this CTA's tiles of job `j`.  The first fill of the ring fetches the weight
// operand only; then `dep_wait()` is called once (it must return true once the states are readable:
// the preceding grid has completed, or the grid-wide barrier behind which they are written has
// opened) and the state operand of those slots follows.  A CTA without a tile in the job neither
// loads nor waits.  `issued` counts slots filled since the kernel started (for the abort path).
// Producer `me` of `n_prod` walks every slot like the others and fills the slots whose running number
// `issued` (counted over all jobs of the launch) is congruent to `me`.
template <typename DepWait>
__device__ __forceinline__ bool produce_job(const Pipe &pp, const GemmJob &j, const CUtensorMap *tmap_a,
                                            const CUtensorMap *tmap_a_short, const CUtensorMap *tmap_b, RingPos &rp,
                                            int &issued, int me, int n_prod, DepWait dep_wait) {
    const int ke = slab_elems(j);
    const uint32_t b_bytes = (uint32_t)j.block_n * kSlabBytes;
    const TileWalk w = walk_of(j);
    if (w.first >= w.end) return true;
    Barriers *bars = pp.bars;
    int n_pre = 0;
    {
        const TilePos t0 = pos_of(j, w, w.first);
        const CUtensorMap *ma = t0.a_rows == kBlockM ? tmap_a : tmap_a_short;
        const uint32_t tx = (uint32_t)t0.a_rows * kSlabBytes + b_bytes;
        n_pre = min(pp.stages, t0.kb1 - t0.kb0);
        RingPos q = rp;
        for (int i = 0; i < n_pre; ++i) {
            if ((issued + i) % n_prod == me) {
                if (!mbar_wait(&bars->empty[q.stage], q.phase ^ 1u, bars, pp.err)) return false;
                uint8_t *sa = pp.tiles + (size_t)q.stage * pp.slot_bytes;
                mbar_arrive_expect_tx(&bars->full[q.stage], tx);
                if (j.w_is_a) tma_load_2d(sa, ma, (t0.kb0 + i) * ke, t0.a_row, &bars->full[q.stage]);
                else tma_load_2d(sa + kABytes, tmap_b, (t0.kb0 + i) * ke, t0.b_row, &bars->full[q.stage]);
            }
            advance(pp, q);
        }
    }
    if (!dep_wait()) return false;
    int done = 0;   // k blocks of this job handled so far
    for (int tile = w.first; tile < w.end; tile += w.step) {
        const TilePos t = pos_of(j, w, tile);
        const CUtensorMap *ma = t.a_rows == kBlockM ? tmap_a : tmap_a_short;
        const uint32_t tx = (uint32_t)t.a_rows * kSlabBytes + b_bytes;
        for (int kb = t.kb0; kb < t.kb1; ++kb) {
            uint8_t *sa = pp.tiles + (size_t)rp.stage * pp.slot_bytes;
            uint8_t *sb = sa + kABytes;
            const bool prefetched = done < n_pre;   // the weights of this slot are already on their way
            if (issued % n_prod == me) {
                if (!prefetched) {
                    if (!mbar_wait(&bars->empty[rp.stage], rp.phase ^ 1u, bars, pp.err)) return false;
                    mbar_arrive_expect_tx(&bars->full[rp.stage], tx);
                }
                if (!prefetched || !j.w_is_a) tma_load_2d(sa, ma, kb * ke, t.a_row, &bars->full[rp.stage]);
                if (!prefetched || j.w_is_a) tma_load_2d(sb, tmap_b, kb * ke, t.b_row, &bars->full[rp.stage]);
            }
            ++done;
            ++issued;
            advance(pp, rp);
        }
    }
    return true;
}

// After a failed wait: let the copies already in flight land before the CTA's shared memory is released
// (every producer waits for all recent slots, its own and the others').
__device__ __forceinline__ void producer_drain(const Pipe &pp, RingPos rp, int issued) {
    const int pending = issued < pp.stages ? issued : pp.stages;
    for (int i = 0; i < pending; ++i) {
        if (--rp.stage < 0) { rp.stage = pp.stages - 1; rp.phase ^= 1u; }
        for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(&pp.bars->full[rp.stage], rp.phase); ++it) __nanosleep(32);
    }
}

// ---- MMA issuer (one thread) ----------------------------------------------------------------------
// The four MMAs of one K block in one instruction sequence.  The single issuing thread is on the
// critical path of the tensor pipe, so the loop around this does as little as possible: descriptors are
// (constant high word, start address >> 4 in the low word), and consecutive MMAs advance the low words by
// 32 bytes >> 4 = 2.  `first_acc` = 0 makes the first MMA overwrite the accumulator (start of a tile).
template <bool kFp8>
__device__ __forceinline__ void umma_k_block(uint32_t tmem_d, uint32_t lo_a, uint32_t lo_b, uint32_t desc_hi,
                                             uint32_t idesc, uint32_t first_acc) {
#define SPEC_MMA_SEQ(KIND)                                                                  \
    asm volatile(                                                                           \
        "{\n\t"                                                                             \
        ".reg .pred p, t;\n\t"                                                              \
        ".reg .b64 da, db;\n\t"                                                             \
        ".reg .b32 la, lb;\n\t"                                                             \
        "setp.ne.b32 p, %5, 0;\n\t"                                                         \
        "setp.eq.b32 t, 0, 0;\n\t"                                                          \
        "mov.b64 da, {%1, %3};\n\t"                                                         \
        "mov.b64 db, {%2, %3};\n\t"                                                         \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %4, p;\n\t"                  \
        "add.u32 la, %1, 2;\n\t"                                                            \
        "add.u32 lb, %2, 2;\n\t"                                                            \
        "mov.b64 da, {la, %3};\n\t"                                                         \
        "mov.b64 db, {lb, %3};\n\t"                                                         \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %4, t;\n\t"                  \
        "add.u32 la, %1, 4;\n\t"                                                            \
        "add.u32 lb, %2, 4;\n\t"                                                            \
        "mov.b64 da, {la, %3};\n\t"                                                         \
        "mov.b64 db, {lb, %3};\n\t"                                                         \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %4, t;\n\t"                  \
        "add.u32 la, %1, 6;\n\t"                                                            \
        "add.u32 lb, %2, 6;\n\t"                                                            \
        "mov.b64 da, {la, %3};\n\t"                                                         \
        "mov.b64 db, {lb, %3};\n\t"                                                         \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %4, t;\n\t"                  \
        "}"                                                                                 \
        ::"r"(tmem_d), "r"(lo_a), "r"(lo_b), "r"(desc_hi), "r"(idesc), "r"(first_acc)      \
        : "memory")
    if (kFp8) SPEC_MMA_SEQ("f8f6f4");
    else SPEC_MMA_SEQ("f16");
#undef SPEC_MMA_SEQ
}

template <bool kFp8>
__device__ __forceinline__ bool mma_job_kind(const Pipe &pp, const GemmJob &j, RingPos &rp, AccPos &ap) {
    static_assert(kSlabBytes / kUmmaBytes == 4, "umma_k_block issues four MMAs");
    const uint32_t idesc = make_instr_desc(kBlockM, j.block_n, kFp8);
    const uint32_t desc_hi = (uint32_t)(make_smem_desc(0) >> 32);
    const uint32_t lo_base = (smem_u32(pp.tiles) & 0x3ffffu) >> 4, lo_slot = pp.slot_bytes >> 4;
    Barriers *bars = pp.bars;
    const TileWalk w = walk_of(j);
    for (int tile = w.first; tile < w.end; tile += w.step) {
        if (!mbar_wait(&bars->acc_empty[ap.acc], ap.phase ^ 1u, bars, pp.err)) return false;
        tc_fence_after();
        const uint32_t tmem_d = pp.tmem_base + (uint32_t)(ap.acc * pp.acc_stride);
        const TilePos t = pos_of(j, w, tile);
        uint32_t acc = 0u;
        // (a short A box leaves the rest of the 128 rows as they were: those accumulator lanes are never read)
        for (int kb = t.kb0; kb < t.kb1; ++kb) {
            if (!mbar_wait(&bars->full[rp.stage], rp.phase, bars, pp.err)) return false;
            tc_fence_after();
            const uint32_t lo_a = lo_base + (uint32_t)rp.stage * lo_slot;
            umma_k_block<kFp8>(tmem_d, lo_a, lo_a + (kABytes >> 4), desc_hi, idesc, acc);
            acc = 1u;
            umma_commit(&bars->empty[rp.stage]);   // frees the slot once these MMAs have read it
            advance(pp, rp);
        }
        umma_commit(&bars->acc_full[ap.acc]);
        if (++ap.acc == 2) { ap.acc = 0; ap.phase ^= 1u; }
    }
    return true;
}

// After a failed wait in any role: the MMAs issued so far may still be reading shared memory and writing
// TMEM.  A commit tracks every tcgen05.mma this thread issued before it; its arrival on a barrier of its own
// is waited for (bounded) before the CTA frees TMEM and gives up its shared memory.  Order at tear-down:
// producers wait for their copies (producer_drain), this thread for its MMAs, then all threads meet at the
// barrier in pipe_teardown and only then TMEM is deallocated.
__device__ __forceinline__ void mma_drain(const Pipe &pp) {
    umma_commit(&pp.bars->drained);
    for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(&pp.bars->drained, 0u); ++it) __nanosleep(32);
}

__device__ __forceinline__ bool mma_job(const Pipe &pp, const GemmJob &j, RingPos &rp, AccPos &ap) {
    return j.fp8 ? mma_job_kind<true>(pp, j, rp, ap) : mma_job_kind<false>(pp, j, rp, ap);
}

// ---- epilogue, mode 1 -----------------------------------------------------------------------------
// One thread owns one accumulator row.  Data-dependent insertion into a sorted list diverges in
// every warp (each lane inserts at different columns), so the selection is done branch-free:
//   pass 1  streams the tile once: online (max, sum-exp) and the kCap largest VALUES of the row,
//           kept sorted by a min/max network (new_v[j] = max(v[j], min(v[j-1], x)));
//   pass 2  re-reads the tile from TMEM and emits the columns whose value reaches the topk-th
//           largest; equal values are taken in ascending column order, exactly `topk` entries.
// e4m3 operands: accumulator -> logit, v[i] * row_scale * col_scale[col0 + c + i] (columns past N untouched).
__device__ __forceinline__ void scale_chunk(float (&v)[32], float rs, const float *cs, int valid) {
    if (valid >= 32 && (((uintptr_t)cs) & 15) == 0) {
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            const float4 q = *(const float4 *)(cs + i);
            v[i] *= rs * q.x; v[i + 1] *= rs * q.y; v[i + 2] *= rs * q.z; v[i + 3] *= rs * q.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < valid) v[i] *= rs * cs[i];
    }
}

template <int kCap, bool kFp8>
__device__ __forceinline__ void epilogue_topk(const GemmJob &p, uint32_t taddr, int row, bool row_ok, int col0,
                                              int n_tile) {
    constexpr float kLog2e = 1.4426950408889634f;
    float best[kCap];
#pragma unroll
    for (int j = 0; j < kCap; ++j) best[j] = -INFINITY;
    float run_m = -INFINITY, run_s = 0.0f;
    const float rs = (kFp8 && row_ok) ? p.epi.row_scale[row] : 1.0f;
    for (int c = 0; c < p.block_n; c += 32) {
        float v[32];
        tmem_ld32(taddr + c, v);
        const int valid = p.N - (col0 + c);   // columns of this chunk inside the vocabulary
        if (kFp8) scale_chunk(v, rs, p.epi.col_scale + col0 + c, valid);
        if (valid < 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i >= valid) v[i] = -INFINITY;
        }
        float cm0 = fmaxf(v[0], v[1]), cm1 = fmaxf(v[2], v[3]);
#pragma unroll
        for (int i = 4; i < 32; i += 2) {
            cm0 = fmaxf(cm0, v[i]);
            cm1 = fmaxf(cm1, v[i + 1]);
        }
        const float cm = fmaxf(cm0, cm1);
        if (cm > run_m) {
            run_s *= ex2_approx((run_m - cm) * kLog2e);
            run_m = cm;
        }
        const float ms = run_m * kLog2e;
        float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            s0 += ex2_approx(fmaf(v[i], kLog2e, -ms));
            s1 += ex2_approx(fmaf(v[i + 1], kLog2e, -ms));
            s2 += ex2_approx(fmaf(v[i + 2], kLog2e, -ms));
            s3 += ex2_approx(fmaf(v[i + 3], kLog2e, -ms));
        }
        if (run_m > -INFINITY) run_s += (s0 + s1) + (s2 + s3);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float x = v[i];
#pragma unroll
            for (int j = kCap - 1; j > 0; --j) best[j] = fmaxf(best[j], fminf(best[j - 1], x));
            best[0] = fmaxf(best[0], x);
        }
    }
    // threshold = topk-th largest value of the row in this tile; how many entries lie strictly above it
    const int topk = p.epi.topk;
    float thr = best[0];
#pragma unroll
    for (int j = 1; j < kCap; ++j)
        if (j < topk) thr = best[j];
    int above = 0;
#pragma unroll
    for (int j = 0; j < kCap; ++j)
        if (j < topk && best[j] > thr) ++above;
    int eq_left = topk - above;
    const size_t u = (size_t)row * p.n_tiles + n_tile;
    float *pv = p.epi.part_val + u * SPEC_MAX_TOPK;
    int32_t *pi = p.epi.part_idx + u * SPEC_MAX_TOPK;
    int cnt = 0;
    for (int c = 0; c < p.block_n; c += 32) {
        float v[32];
        tmem_ld32(taddr + c, v);
        const int valid = p.N - (col0 + c);
        if (kFp8) scale_chunk(v, rs, p.epi.col_scale + col0 + c, valid);
        // candidates of this chunk as a bit mask: no per-element branches
        uint32_t mask = 0;
#pragma unroll
        for (int i = 0; i < 32; ++i) mask |= (v[i] >= thr ? 1u : 0u) << i;
        if (valid < 32) mask &= valid > 0 ? ((1u << valid) - 1u) : 0u;
        if (!row_ok) mask = 0;
        while (mask) {   // ascending columns; a handful of iterations per tile
            const int bpos = __ffs(mask) - 1;
            mask &= mask - 1;
            // x = v[bpos] through a select tree (bpos is data dependent, v lives in registers)
            float t16[16], t8[8], t4[4], t2[2];
#pragma unroll
            for (int i = 0; i < 16; ++i) t16[i] = (bpos & 1) ? v[2 * i + 1] : v[2 * i];
#pragma unroll
            for (int i = 0; i < 8; ++i) t8[i] = (bpos & 2) ? t16[2 * i + 1] : t16[2 * i];
#pragma unroll
            for (int i = 0; i < 4; ++i) t4[i] = (bpos & 4) ? t8[2 * i + 1] : t8[2 * i];
#pragma unroll
            for (int i = 0; i < 2; ++i) t2[i] = (bpos & 8) ? t4[2 * i + 1] : t4[2 * i];
            const float x = (bpos & 16) ? t2[1] : t2[0];
            const bool gt = x > thr;
            if (gt || eq_left > 0) {
                if (!gt) --eq_left;
                if (cnt < topk) {
                    pv[cnt] = x;
                    pi[cnt] = col0 + c + bpos + p.epi.idx_offset;
                }
                ++cnt;
            }
        }
    }
    if (row_ok) {
        for (; cnt < topk; ++cnt) {   // fewer than topk comparable values (NaN rows, tiny tiles)
            pv[cnt] = -INFINITY;
            pi[cnt] = 0x7fffffff;
        }
        p.epi.part_ms[2 * u] = run_m;
        p.epi.part_ms[2 * u + 1] = run_s;
    }
}

// ---- epilogue, mode 3 (operands swapped: TMEM lanes are vocabulary rows, columns are nodes) ----------
// What one scan thread carries from tile to tile: the running (max, sum-exp) of its share of a node's
// logits and the best SPEC_MAX_TOPK of them, best first by (value desc, token id asc).
struct SwapRun {
    float m, s;
    float tv[SPEC_MAX_TOPK];
    int ti[SPEC_MAX_TOPK];
};

// (no short-circuit operators: every comparison would be a divergent branch)
__device__ __forceinline__ bool cand_better(float v, int i, float w, int j) { return (v > w) | ((v == w) & (i < j)); }

// Branch-free insertion into the sorted list: slot j takes its left neighbour when the newcomer beats that
// neighbour, the newcomer when it beats only slot j, and keeps its entry otherwise.
__device__ __forceinline__ void list_insert(SwapRun &r, float x, int id) {
    bool beats[SPEC_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < SPEC_MAX_TOPK; ++j) beats[j] = cand_better(x, id, r.tv[j], r.ti[j]);
#pragma unroll
    for (int j = SPEC_MAX_TOPK - 1; j > 0; --j) {
        r.tv[j] = beats[j - 1] ? r.tv[j - 1] : (beats[j] ? x : r.tv[j]);
        r.ti[j] = beats[j - 1] ? r.ti[j - 1] : (beats[j] ? id : r.ti[j]);
    }
    r.tv[0] = beats[0] ? x : r.tv[0];
    r.ti[0] = beats[0] ? id : r.ti[0];
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory"); }

// One thread scans `len` (a multiple of 16) consecutive logits of one node in the transposed tile: `col`
// points at the first, `valid` of them are real vocabulary rows (the rest hold -inf), `idx0` is the token id
// of the first.  Pass 1: online (max, sum-exp) and the kCap largest values (min/max network).  Pass 2: the
// entries that reach the topk-th largest value, ties in ascending token order, exactly topk of them, are
// inserted into the running list.
template <int kCap>
__device__ __forceinline__ void swap_scan_tile(const float *col, int len, int valid, int idx0, int topk, SwapRun &r) {
    constexpr float kLog2e = 1.4426950408889634f;
    float best[kCap];
#pragma unroll
    for (int j = 0; j < kCap; ++j) best[j] = -INFINITY;
    for (int c = 0; c < len; c += 16) {
        float v[16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 f = *(const float4 *)(col + c + 4 * q);
            v[4 * q] = f.x; v[4 * q + 1] = f.y; v[4 * q + 2] = f.z; v[4 * q + 3] = f.w;
        }
        float cm0 = fmaxf(v[0], v[1]), cm1 = fmaxf(v[2], v[3]);
#pragma unroll
        for (int i = 4; i < 16; i += 2) {
            cm0 = fmaxf(cm0, v[i]);
            cm1 = fmaxf(cm1, v[i + 1]);
        }
        const float cm = fmaxf(cm0, cm1);
        if (cm > r.m) {
            r.s *= ex2_approx((r.m - cm) * kLog2e);
            r.m = cm;
        }
        const float ms = r.m * kLog2e;
        float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
#pragma unroll
        for (int i = 0; i < 16; i += 4) {
            s0 += ex2_approx(fmaf(v[i], kLog2e, -ms));
            s1 += ex2_approx(fmaf(v[i + 1], kLog2e, -ms));
            s2 += ex2_approx(fmaf(v[i + 2], kLog2e, -ms));
            s3 += ex2_approx(fmaf(v[i + 3], kLog2e, -ms));
        }
        if (r.m > -INFINITY) r.s += (s0 + s1) + (s2 + s3);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float x = v[i];
#pragma unroll
            for (int j = kCap - 1; j > 0; --j) best[j] = fmaxf(best[j], fminf(best[j - 1], x));
            best[0] = fmaxf(best[0], x);
        }
    }
    float thr = best[0];
#pragma unroll
    for (int j = 1; j < kCap; ++j)
        if (j < topk) thr = best[j];
    int above = 0;
#pragma unroll
    for (int j = 0; j < kCap; ++j)
        if (j < topk && best[j] > thr) ++above;
    int eq_left = topk - above;
    for (int c = 0; c < len; c += 16) {
        uint32_t mask = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 f = *(const float4 *)(col + c + 4 * q);
            mask |= (f.x >= thr ? 1u : 0u) << (4 * q);
            mask |= (f.y >= thr ? 1u : 0u) << (4 * q + 1);
            mask |= (f.z >= thr ? 1u : 0u) << (4 * q + 2);
            mask |= (f.w >= thr ? 1u : 0u) << (4 * q + 3);
        }
        const int left = valid - c;
        if (left < 16) mask &= left > 0 ? ((1u << left) - 1u) : 0u;
        while (mask) {   // ascending token ids; a handful of iterations per tile
            const int bpos = __ffs(mask) - 1;
            mask &= mask - 1;
            const float x = col[c + bpos];
            const bool gt = x > thr;
            if (gt || eq_left > 0) {
                if (!gt) --eq_left;
                list_insert(r, x, idx0 + c + bpos);
            }
        }
    }
}

// The better eight of two lists that are both sorted best first: "the better of a[i] and b[7 - i]" keeps the
// best eight as a bitonic sequence, which three compare-exchange stages sort.
__device__ __forceinline__ void merge_sorted8(SwapRun &r, const float (&ov)[SPEC_MAX_TOPK], const int (&oi)[SPEC_MAX_TOPK]) {
    constexpr int kT = SPEC_MAX_TOPK;
    static_assert(kT == 8, "three stages sort eight entries");
#pragma unroll
    for (int j = 0; j < kT; ++j) {
        const bool take = cand_better(ov[kT - 1 - j], oi[kT - 1 - j], r.tv[j], r.ti[j]);
        r.tv[j] = take ? ov[kT - 1 - j] : r.tv[j];
        r.ti[j] = take ? oi[kT - 1 - j] : r.ti[j];
    }
#pragma unroll
    for (int stride = kT / 2; stride > 0; stride >>= 1) {
#pragma unroll
        for (int j = 0; j < kT; ++j) {
            if ((j & stride) == 0) {   // (compile-time condition: the loops are unrolled)
                const bool sw = cand_better(r.tv[j + stride], r.ti[j + stride], r.tv[j], r.ti[j]);
                const float hv = sw ? r.tv[j + stride] : r.tv[j], lv = sw ? r.tv[j] : r.tv[j + stride];
                const int hi = sw ? r.ti[j + stride] : r.ti[j], li = sw ? r.ti[j] : r.ti[j + stride];
                r.tv[j] = hv; r.tv[j + stride] = lv;
                r.ti[j] = hi; r.ti[j + stride] = li;
            }
        }
    }
}

// Epilogue warps of a mode-3 job.  Per tile: the leader waits for the accumulator and tells the others
// (so that all 128 threads take the same path into the barriers below, also when the wait gives up); every
// thread copies its vocabulary row of the accumulator into the transposed tile in shared memory; after a
// barrier the accumulator slot is released and the scan threads (P per node, each 128 / P rows of the tile)
// fold their segment into their running list.  The barrier at the top of the next tile keeps the transposed
// tile intact until every scan of this one is done.  After the last tile the P threads of a node (neighbouring
// lanes) combine their lists and (max, sum-exp) pairs with shuffles and the first of them writes the node's
// partial slot of this CTA.
__device__ __forceinline__ bool epilogue_job_swapped(const Pipe &pp, const GemmJob &j, AccPos &ap) {
    constexpr float kLog2e = 1.4426950408889634f;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int quarter = warp & 3;                    // TMEM lane quarter this warp may read
    const int vrow = quarter * 32 + lane;            // vocabulary row of the tile held by this thread's TMEM lane
    const int u = (int)threadIdx.x - kEpilogueFirst;
    const int nodes = j.N, P = j.epi.segs, len = kBlockM / P;
    const int node = u / P, seg = u - node * P;
    const bool scans = node < nodes;
    const int topk = j.epi.topk;
    Barriers *bars = pp.bars;
    SwapRun run;
    run.m = -INFINITY;
    run.s = 0.0f;
#pragma unroll
    for (int q = 0; q < SPEC_MAX_TOPK; ++q) {
        run.tv[q] = -INFINITY;
        run.ti[q] = 0x7fffffff;
    }
    const TileWalk w = walk_of(j);
    const int row_end = min(j.M, (w.rel + 1) * j.rows_per_cta);   // the next CTA's rows start here
    for (int tile = w.first; tile < w.end; tile += w.step) {
        if (u == 0) bars->epi_ok = mbar_wait(&bars->acc_full[ap.acc], ap.phase, bars, pp.err) ? 1 : 0;
        epi_bar_sync();
        if (!bars->epi_ok) return false;
        tc_fence_after();
        const uint32_t taddr = pp.tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(ap.acc * pp.acc_stride);
        const int row0 = w.rel * j.rows_per_cta + tile * kBlockM;   // vocabulary row of TMEM lane 0
        const bool v_ok = row0 + vrow < row_end;
        for (int c = 0; c < nodes; c += 16) {
            float v[16];
            tmem_ld16(taddr + c, v);
#pragma unroll
            for (int i = 0; i < 16; ++i)
                if (c + i < nodes) pp.tbuf[(c + i) * kTPitch + vrow] = v_ok ? v[i] : -INFINITY;
        }
        tc_fence_before();
        epi_bar_sync();
        if (lane == 0) mbar_arrive(&bars->acc_empty[ap.acc]);
        if (++ap.acc == 2) { ap.acc = 0; ap.phase ^= 1u; }
        if (scans) {
            const int seg_row = row0 + seg * len;            // first vocabulary row of this thread's segment
            int valid = row_end - seg_row;
            valid = valid < 0 ? 0 : (valid > len ? len : valid);
            const float *col = pp.tbuf + node * kTPitch + seg * len;
            if (topk <= 4) swap_scan_tile<4>(col, len, valid, seg_row + j.epi.idx_offset, topk, run);
            else swap_scan_tile<SPEC_MAX_TOPK>(col, len, valid, seg_row + j.epi.idx_offset, topk, run);
        }
    }
    if (w.first >= w.end) return true;
    // the P neighbouring lanes of a node fold their results (every lane of the warp takes part in the shuffles)
    for (int off = 1; off < P; off <<= 1) {
        float ov[SPEC_MAX_TOPK];
        int oi[SPEC_MAX_TOPK];
#pragma unroll
        for (int q = 0; q < SPEC_MAX_TOPK; ++q) {
            ov[q] = __shfl_xor_sync(0xffffffffu, run.tv[q], off);
            oi[q] = __shfl_xor_sync(0xffffffffu, run.ti[q], off);
        }
        const float om = __shfl_xor_sync(0xffffffffu, run.m, off), os = __shfl_xor_sync(0xffffffffu, run.s, off);
        merge_sorted8(run, ov, oi);
        const float nm = fmaxf(run.m, om);
        if (nm > -INFINITY)
            run.s = run.s * ex2_approx((run.m - nm) * kLog2e) + os * ex2_approx((om - nm) * kLog2e);
        run.m = nm;
    }
    if (scans && seg == 0) {
        const size_t slot = (size_t)node * j.epi.n_parts + (size_t)w.rel;
        float4 *pv = (float4 *)(j.epi.part_val + slot * SPEC_MAX_TOPK);
        int4 *pi = (int4 *)(j.epi.part_idx + slot * SPEC_MAX_TOPK);
        pv[0] = make_float4(run.tv[0], run.tv[1], run.tv[2], run.tv[3]);
        pv[1] = make_float4(run.tv[4], run.tv[5], run.tv[6], run.tv[7]);
        pi[0] = make_int4(run.ti[0], run.ti[1], run.ti[2], run.ti[3]);
        pi[1] = make_int4(run.ti[4], run.ti[5], run.ti[6], run.ti[7]);
        *(float2 *)(j.epi.part_ms + 2 * slot) = make_float2(run.m, run.s);
    }
    return true;
}

// ---- epilogue warps (warps 2-5, all lanes) ----------------------------------------------------------
__device__ __forceinline__ bool epilogue_job(const Pipe &pp, const GemmJob &j, AccPos &ap) {
    if (j.epi.mode == 3) return epilogue_job_swapped(pp, j, ap);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int quarter = warp & 3;               // TMEM lane quarter this warp may read
    const int row_in_tile = quarter * 32 + lane;
    Barriers *bars = pp.bars;
    const TileWalk w = walk_of(j);
    for (int tile = w.first; tile < w.end; tile += w.step) {
        const TilePos t = pos_of(j, w, tile);
        const int split = t.split, m_tile = t.m_tile, n_tile = t.n_tile;
        if (!mbar_wait(&bars->acc_full[ap.acc], ap.phase, bars, pp.err)) return false;
        tc_fence_after();
        const int row = m_tile * kBlockM + row_in_tile;
        const bool row_ok = row < j.M;
        const uint32_t taddr = pp.tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(ap.acc * pp.acc_stride);
        const int col0 = n_tile * j.block_n;
        if (j.epi.mode == 0) {
            for (int c = 0; c < j.block_n; c += 32) {
                float v[32];
                tmem_ld32(taddr + c, v);
                if (row_ok) {
                    float *dst = j.epi.out + (size_t)row * j.epi.ldc + col0 + c;
                    const int valid = j.N - (col0 + c);
                    if (valid >= 32 && (((uintptr_t)dst) & 15) == 0) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            *(float4 *)(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (i < valid) dst[i] = v[i];
                    }
                }
            }
        } else if (j.epi.mode == 2) {
            // transposed store of one split-K partial: out[split][col][row]; a warp's 32 rows are
            // consecutive addresses, so every store instruction is one 128-byte line
            float *dst0 = j.epi.out + (size_t)split * j.epi.split_stride + row;
            for (int c = 0; c < j.block_n; c += 32) {
                float v[32];
                tmem_ld32(taddr + c, v);
                if (row_ok) {
                    const int valid = j.N - (col0 + c);
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < valid) dst0[(size_t)(col0 + c + i) * j.epi.ldc] = v[i];
                }
            }
        } else {
            if (j.fp8) epilogue_topk<SPEC_MAX_TOPK, true>(j, taddr, row, row_ok, col0, n_tile);
            else if (j.epi.topk <= 4) epilogue_topk<4, false>(j, taddr, row, row_ok, col0, n_tile);
            else epilogue_topk<SPEC_MAX_TOPK, false>(j, taddr, row, row_ok, col0, n_tile);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->acc_empty[ap.acc]);
        if (++ap.acc == 2) { ap.acc = 0; ap.phase ^= 1u; }
    }
    return true;
}

}  // namespace tc

// ---- host side (gemm_tcgen05.cu) ---------------------------------------------------------------
// 2-D row-major [rows, cols] tensor of bf16 (or, `fp8`, of bytes), box = [box_rows, 128 bytes], 128-byte
// swizzle; `streamed` marks the operand that is read once from HBM (wider L2 fetches).
int make_tmap(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool streamed,
              bool fp8 = false);
// Fills the tiling fields of a job (m_tiles, n_tiles, splits, kb_per_split, w_is_a) from its shape and epilogue.
int plan_job(tc::GemmJob *j, int M, int N, int Kd, int block_n, const GemmEpilogue &epi);

}  // namespace spec
