// Stand-alone tensor-core GEMM kernel for sm_100a:  C[M, N] = A[M, Kd] * B[N, Kd]^T, bf16 operands
// (row-major, i.e. K-major for both), fp32 accumulation in tensor memory (TMEM).  The roles, the
// shared-memory ring and the epilogues live in tc_gemm.cuh; this file holds the kernel that runs ONE
// contraction per launch, the TMA descriptor set-up and the tile-shape choice.
//
// It serves the two contractions of a speculator stage (Sec. 3.1 of arXiv 2404.19124): the
// projection of the parent states (epilogue mode 0: fp32 store; mode 2: the operands are swapped
// so that the weight matrix fills the 128-row side of the MMA when there are few states, the
// contraction is split over several CTAs and every split stores its partial result transposed)
// and the vocabulary head (epilogue mode 1: the logits tile stays on the SM; each accumulator row
// is reduced to a partial top-k list and a (max, sum-exp) pair, so full logits never reach HBM).
//
// Persistent CTAs, at most one per SM, tiles dealt round-robin with the m index fastest, so the CTAs
// that share a weight tile run at the same time and the second and third readers hit L2.
#include <cuda.h>

#include <mutex>
#include <vector>

#include "tc_gemm.cuh"

namespace spec {

namespace {

using namespace tc;

constexpr int kMaxJobs = 2;

struct GemmParams {
    GemmJob job[kMaxJobs];   // walked in order by every role; both read only what the preceding grid produced
    int n_jobs;
    int stages, tmem_cols, acc_stride;
    uint32_t slot_bytes;
    int producers;           // TMA-issuing threads: 1 or 2
    uint32_t tbuf_bytes;     // transposed accumulator tile of a mode-3 job (0: none in this launch)
    int32_t *clear;          // words that the first kernel of a draft sets to zero (the workspace header) ...
    int clear_words;         // ... by CTA 0, after the preceding grid has completed; 0: nothing
    int32_t *err;
};

struct GemmMaps {
    CUtensorMap a[kMaxJobs], b[kMaxJobs];
    CUtensorMap a_short;   // mode 3 (job 0): the weight box of the last, shorter tile of every CTA
};

__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ GemmMaps maps, const __grid_constant__ GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const Pipe pp = pipe_setup(smem_raw, p.stages, p.slot_bytes, p.tmem_cols, p.acc_stride, p.tbuf_bytes, p.err);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    griddep_launch();   // the next kernel in the stream may start its own set-up now
    if (warp == 0 || warp == kThreads / 32 - 1) {
        const int me = warp == 0 ? 0 : 1;
        if (lane == 0 && me < p.producers) {
            RingPos rp{0, 0u};
            int issued = 0;
            bool ok = true;
            // the weights are fetched before the preceding grid is waited for, the states after
            for (int q = 0; ok && q < p.n_jobs; ++q)
                ok = produce_job(pp, p.job[q], &maps.a[q], &maps.a_short, &maps.b[q], rp, issued, me, p.producers,
                                 [] { griddep_wait(); return true; });
            if (!ok) producer_drain(pp, rp, issued);
        }
        griddep_wait();
    } else if (warp == 1) {
        griddep_wait();
        if (lane == 0) {
            RingPos rp{0, 0u};
            AccPos ap{0, 0u};
            bool ok = true;
            for (int q = 0; ok && q < p.n_jobs; ++q) ok = mma_job(pp, p.job[q], rp, ap);
            if (!ok || pp.bars->abort_flag) mma_drain(pp);
        }
    } else {
        AccPos ap{0, 0u};
        bool ok = true;
        griddep_wait();
        // First kernel of a draft: the header (error word, per-sequence counters) starts at zero.  Nothing of
        // this draft has reported or counted yet: the counters are first touched by the last level's merge,
        // and a wait that runs out does so millions of polls after this point.
        if (p.clear_words > 0 && blockIdx.x == 0)
            for (int i = (int)threadIdx.x - kEpilogueFirst; i < p.clear_words; i += kEpilogueThreads)
                p.clear[i] = 0;
        for (int q = 0; ok && q < p.n_jobs; ++q) ok = epilogue_job(pp, p.job[q], ap);
    }
    pipe_teardown(pp, p.tmem_cols);
}

// ---- host side -------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_host_mutex;   // guards the driver entry point, the tensor-map cache and the per-device attribute flags

EncodeTiledFn get_encode_fn() {   // called with g_host_mutex held
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !ptr) {
        set_last_cuda_error((int)(e != cudaSuccess ? e : cudaErrorUnknown));
        return nullptr;
    }
    fn = (EncodeTiledFn)ptr;
    return fn;
}

// Encoded tensor maps, kept for the life of the process: a map depends only on the address, the shape and
// the box, not on the tensor's contents, and the weights of a handle and the buffers of a workspace come back
// call after call.  A draft therefore encodes nothing after the first call with its workspace.
struct TmapKey {
    const void *base;
    uint64_t rows, cols;
    uint32_t box_rows;
    int streamed, fp8;
    bool operator==(const TmapKey &o) const {
        return base == o.base && rows == o.rows && cols == o.cols && box_rows == o.box_rows && streamed == o.streamed &&
               fp8 == o.fp8;
    }
};
struct TmapEntry {
    TmapKey key;
    CUtensorMap map;
};
constexpr size_t kTmapCacheCap = 1024;   // beyond this the cache starts over
std::vector<TmapEntry> g_tmap_cache;

int encode_tmap(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool streamed,
                bool fp8);

}  // namespace

int make_tmap(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool streamed,
              bool fp8) {
    const TmapKey key{base, rows, cols, box_rows, streamed ? 1 : 0, fp8 ? 1 : 0};
    std::lock_guard<std::mutex> lock(g_host_mutex);
    for (const TmapEntry &e : g_tmap_cache) {
        if (e.key == key) {
            *map = e.map;
            return SPEC_OK;
        }
    }
    const int rc = encode_tmap(map, base, rows, cols, box_rows, streamed, fp8);
    if (rc != SPEC_OK) return rc;
    if (g_tmap_cache.size() >= kTmapCacheCap) g_tmap_cache.clear();
    g_tmap_cache.push_back(TmapEntry{key, *map});
    return SPEC_OK;
}

namespace {

int encode_tmap(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool streamed,
                bool fp8) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return SPEC_ERR_CUDA;
    const uint32_t esz = fp8 ? 1 : 2;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * esz};
    cuuint32_t box[2] = {(cuuint32_t)(kSlabBytes / esz), box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    streamed ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error((int)r);
        return SPEC_ERR_CUDA;
    }
    return SPEC_OK;
}

}  // namespace

// Mode 3: threads per node in the scan (a power of two, at most kSwapMaxSegs, nodes * segs <= 128); the
// vocabulary rows every CTA takes (a multiple of 8, the same for all so that they stream the same number of
// bytes; the last CTA of the deal may get fewer); and the number of partial lists per node = CTAs of the deal.
int swapped_head_segs(int nodes) {
    int segs = 1;
    while (segs < kSwapMaxSegs && nodes * segs * 2 <= kEpilogueThreads) segs *= 2;
    return segs;
}
static int swapped_rows_per_cta(int vocab_rows) {
    const int sms = num_sms();
    const int per = (vocab_rows + sms - 1) / sms;
    return (per + 7) / 8 * 8;
}
int swapped_head_parts(int nodes, int vocab_rows) {
    (void)nodes;
    const int per = swapped_rows_per_cta(vocab_rows);
    return (vocab_rows + per - 1) / per;
}

// Columns per tile: a multiple of 32 in [32, 256].  Scores each candidate by how evenly its
// tiles fill the SMs (tiles / (waves * SMs)); among near-equal fills the widest tile wins
// because it re-reads A least often.
int choose_block_n(int M, int N, int num_sm, bool prefer_wide) {
    // Cost model: the launch takes (tiles per CTA) x (cost of one tile), a tile costing its width plus a fixed
    // part (operand A, commit and epilogue hand-over) worth 96 columns when the MMAs are the bound (more than
    // one 128-row tile) and 32 when the weight stream is.  Ties go to the wider tile.
    const int m_tiles = (M + kBlockM - 1) / kBlockM;
    const int fixed = prefer_wide ? 96 : 32;
    int best = 32;
    long long best_cost = -1;
    for (int bn = 32; bn <= 256; bn += 32) {
        const long long tiles = (long long)m_tiles * ((N + bn - 1) / bn);
        const long long waves = (tiles + num_sm - 1) / num_sm;
        const long long cost = waves * (bn + fixed);
        if (best_cost < 0 || cost <= best_cost) {
            best_cost = cost;
            best = bn;
        }
    }
    return best;
}

int plan_job(tc::GemmJob *j, int M, int N, int Kd, int block_n, const GemmEpilogue &epi) {
    const int fp8 = epi.fp8 ? 1 : 0;
    const int bn_unit = epi.mode == 3 ? 16 : 32;   // mode 3 reads the accumulator 16 columns at a time
    if (M <= 0 || N <= 0 || Kd <= 0 || Kd % (fp8 ? 16 : 8) != 0 || block_n < bn_unit || block_n > 256 ||
        block_n % bn_unit != 0)
        return SPEC_ERR_SHAPE;   // rows are whole 16-byte units
    j->M = M; j->N = N; j->Kd = Kd;
    j->block_n = block_n;
    j->m_tiles = (M + kBlockM - 1) / kBlockM;
    j->n_tiles = (N + block_n - 1) / block_n;
    j->fp8 = fp8;
    const int ke = fp8 ? kSlabBytes : kSlabBytes / 2;
    const int num_kb = (Kd + ke - 1) / ke;
    j->splits = epi.mode == 2 && epi.splits > 1 ? epi.splits : 1;
    j->kb_per_split = (num_kb + j->splits - 1) / j->splits;
    if ((j->splits - 1) * j->kb_per_split >= num_kb) return SPEC_ERR_SHAPE;   // every split must own a K block
    j->w_is_a = (epi.mode == 2 || epi.mode == 3) ? 1 : 0;
    j->first_cta = 0;
    j->deal_ctas = 0;
    j->epi = epi;
    j->rows_per_cta = 0;
    if (epi.mode == 3) {   // all nodes in one tile column; every CTA of the deal leaves one list per node
        if (N > kBlockM || j->n_tiles != 1 || fp8) return SPEC_ERR_SHAPE;
        j->epi.segs = swapped_head_segs(N);
        j->rows_per_cta = swapped_rows_per_cta(M);
        j->deal_ctas = (M + j->rows_per_cta - 1) / j->rows_per_cta;
        j->epi.n_parts = j->deal_ctas;
    }
    return SPEC_OK;
}

// Two by default: one thread issues a 128-row box about every 250 ns, and alternating two threads over the ring
// slots measured 3-6 % faster launches at every row count (16 rows 52.6 -> 50.4 us, 384 rows 98 -> 94 us,
// 768 rows 179 -> 170 us at V = 32000, d = 4096; same process, same GPU).
static int g_gemm_producers = 2;
void set_gemm_producers(int n) { g_gemm_producers = n >= 2 ? 2 : 1; }

// One launch, one or two contractions.  The tiles of the second are dealt to the CTAs starting where
// the first one's stopped, so a CTA that got no tile of the first starts on the second at once.
int launch_gemm_tc_jobs(const GemmCall *calls, int n_calls, int32_t *err, cudaStream_t st, int32_t *clear,
                        int clear_words) {
    if (n_calls < 1 || n_calls > kMaxJobs) return SPEC_ERR_INVALID_ARG;
    GemmParams p{};
    GemmMaps maps{};
    p.n_jobs = n_calls;
    p.producers = g_gemm_producers;
    p.clear = clear;
    p.clear_words = clear ? clear_words : 0;
    int max_block_n = 32;
    long long total_tiles = 0;
    for (int q = 0; q < n_calls; ++q) {
        const GemmCall &c = calls[q];
        int rc = plan_job(&p.job[q], c.M, c.N, c.Kd, c.block_n, c.epi);
        if (rc != SPEC_OK) return rc;
        if (((uintptr_t)c.A & 15) || ((uintptr_t)c.B & 15)) return SPEC_ERR_INVALID_ARG;
        rc = make_tmap(&maps.a[q], c.A, (uint64_t)c.M, (uint64_t)c.Kd, kBlockM, p.job[q].w_is_a != 0, p.job[q].fp8 != 0);
        if (rc != SPEC_OK) return rc;
        rc = make_tmap(&maps.b[q], c.B, (uint64_t)c.N, (uint64_t)c.Kd, (uint32_t)c.block_n, p.job[q].w_is_a == 0,
                       p.job[q].fp8 != 0);
        if (rc != SPEC_OK) return rc;
        if (c.block_n > max_block_n) max_block_n = c.block_n;
        if (c.epi.mode == 3) {
            if (q != 0) return SPEC_ERR_INVALID_ARG;   // its CTAs are the first of the grid
            p.tbuf_bytes = (uint32_t)c.block_n * kTPitch * sizeof(float);
            const int short_rows = p.job[q].rows_per_cta % kBlockM;
            if (short_rows > 0) {
                rc = make_tmap(&maps.a_short, c.A, (uint64_t)c.M, (uint64_t)c.Kd, (uint32_t)short_rows, true, false);
                if (rc != SPEC_OK) return rc;
            }
            total_tiles += p.job[q].deal_ctas;   // what counts for the grid: the CTAs it occupies
        } else {
            total_tiles += (long long)p.job[q].m_tiles * p.job[q].n_tiles * p.job[q].splits;
        }
    }
    const int grid = (int)(total_tiles < num_sms() ? total_tiles : num_sms());
    long long offset = 0;
    for (int q = 0; q < n_calls; ++q) {
        // a job's tiles are dealt to the CTAs starting where the previous job's stopped; behind a mode-3 job
        // that is the first CTA without vocabulary rows
        p.job[q].first_cta = (int)(offset % grid);
        offset += p.job[q].epi.mode == 3 ? (long long)p.job[q].deal_ctas
                                         : (long long)p.job[q].m_tiles * p.job[q].n_tiles * p.job[q].splits;
    }
    p.slot_bytes = (uint32_t)kABytes + (uint32_t)max_block_n * kSlabBytes;
    const int budget = kSmemLimit - 1024 - (int)sizeof(Barriers) - 64 - (int)p.tbuf_bytes;
    p.stages = budget / (int)p.slot_bytes;
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    if (p.stages < 2) return SPEC_ERR_SHAPE;
    int cols = 32;
    while (cols < 2 * max_block_n) cols <<= 1;
    p.tmem_cols = cols;
    p.acc_stride = max_block_n;
    p.err = err;

    const size_t smem = 1024 + (size_t)p.stages * p.slot_bytes + p.tbuf_bytes + sizeof(Barriers);
    int dev = 0;
    SPEC_CUDA_TRY(cudaGetDevice(&dev));
    {
        static bool attr_set[64] = {};
        std::lock_guard<std::mutex> lock(g_host_mutex);
        if (dev < 0 || dev >= 64 || !attr_set[dev]) {
            SPEC_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
            if (dev >= 0 && dev < 64) attr_set[dev] = true;
        }
    }
    SPEC_CUDA_TRY(launch_pdl(gemm_tc_kernel, dim3(grid), dim3(kThreads), smem, st, maps, p));
    return SPEC_OK;
}

int launch_gemm_tc(const void *A, const void *B, int M, int N, int Kd, int block_n, const GemmEpilogue &epi,
                   int32_t *err, cudaStream_t st) {
    GemmCall c{A, B, M, N, Kd, block_n, epi};
    return launch_gemm_tc_jobs(&c, 1, err, st);
}

}  // namespace spec
