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
    int32_t *err;
};

struct GemmMaps {
    CUtensorMap a[kMaxJobs], b[kMaxJobs];
};

__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ GemmMaps maps, const __grid_constant__ GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const Pipe pp = pipe_setup(smem_raw, p.stages, p.slot_bytes, p.tmem_cols, p.acc_stride, p.err);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    griddep_launch();   // the next kernel in the stream may start its own set-up now
    if (warp == 0) {
        if (lane == 0) {
            RingPos rp{0, 0u};
            int issued = 0;
            bool ok = true;
            // the weights are fetched before the preceding grid is waited for, the states after
            for (int q = 0; ok && q < p.n_jobs; ++q)
                ok = produce_job(pp, p.job[q], &maps.a[q], &maps.b[q], rp, issued, [] { griddep_wait(); return true; });
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
        }
    } else {
        AccPos ap{0, 0u};
        bool ok = true;
        griddep_wait();
        for (int q = 0; ok && q < p.n_jobs; ++q) ok = epilogue_job(pp, p.job[q], ap);
    }
    pipe_teardown(pp, p.tmem_cols);
}

// ---- host side -------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
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

}  // namespace

int make_tmap(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool streamed,
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
    if (M <= 0 || N <= 0 || Kd <= 0 || Kd % (fp8 ? 16 : 8) != 0 || block_n < 32 || block_n > 256 || block_n % 32 != 0)
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
    j->w_is_a = epi.mode == 2 ? 1 : 0;
    j->first_cta = 0;
    j->epi = epi;
    return SPEC_OK;
}

// One launch, one or two contractions.  The tiles of the second are dealt to the CTAs starting where
// the first one's stopped, so a CTA that got no tile of the first starts on the second at once.
int launch_gemm_tc_jobs(const GemmCall *calls, int n_calls, int32_t *err, cudaStream_t st) {
    if (n_calls < 1 || n_calls > kMaxJobs) return SPEC_ERR_INVALID_ARG;
    GemmParams p{};
    GemmMaps maps{};
    p.n_jobs = n_calls;
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
        total_tiles += (long long)p.job[q].m_tiles * p.job[q].n_tiles * p.job[q].splits;
    }
    const int grid = (int)(total_tiles < num_sms() ? total_tiles : num_sms());
    long long offset = 0;
    for (int q = 0; q < n_calls; ++q) {
        p.job[q].first_cta = (int)(offset % grid);
        offset += (long long)p.job[q].m_tiles * p.job[q].n_tiles * p.job[q].splits;
    }
    p.slot_bytes = (uint32_t)kABytes + (uint32_t)max_block_n * kSlabBytes;
    const int budget = kSmemLimit - 1024 - (int)sizeof(Barriers) - 64;
    p.stages = budget / (int)p.slot_bytes;
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    if (p.stages < 2) return SPEC_ERR_SHAPE;
    int cols = 32;
    while (cols < 2 * max_block_n) cols <<= 1;
    p.tmem_cols = cols;
    p.acc_stride = max_block_n;
    p.err = err;

    const size_t smem = 1024 + (size_t)p.stages * p.slot_bytes + sizeof(Barriers);
    static bool attr_set[64] = {};
    int dev = 0;
    SPEC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        SPEC_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
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
