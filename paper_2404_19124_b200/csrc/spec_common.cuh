// Internal declarations shared by the translation units of libspec_b200.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "spec_b200.h"

namespace spec {

constexpr int kWsAlign = 256;
constexpr int kNumSMsFallback = 148;

// Device-side error word: the first error wins, later ones do not overwrite it.
__device__ __forceinline__ void report_error(int32_t *err, int code) {
    if (err != nullptr) atomicCAS(err, 0, code);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t lo16) { return __uint_as_float(lo16 << 16); }

// fp32 -> bf16, round to nearest even (NaN stays a quiet NaN).
__device__ __forceinline__ uint32_t float_to_bf16_bits(float f) {
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (u >> 16) | 0x0040u;
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

// Programmatic dependent launch: every kernel of the library is enqueued with the
// "programmatic stream serialization" attribute.  A kernel lets its successor start early
// (griddep_launch, executed by all threads near the top) so the successor's launch latency,
// set-up and loads of data that no kernel writes (the weights) overlap this kernel's tail;
// nothing that an earlier kernel produces is touched before griddep_wait, which returns once
// the preceding grid has completed and its writes are visible.  Every thread of every kernel
// executes griddep_wait, so "grid N complete" implies "grid N-1 complete" along the whole chain.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Host-side bookkeeping ------------------------------------------------------------------
void set_last_cuda_error(int e);
int num_sms();

// cudaLaunchKernelEx with the programmatic-serialization attribute set.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

#define SPEC_CUDA_TRY(expr)                              \
    do {                                                 \
        cudaError_t _e = (expr);                         \
        if (_e != cudaSuccess) {                         \
            spec::set_last_cuda_error((int)_e);          \
            return SPEC_ERR_CUDA;                        \
        }                                                \
    } while (0)

// ---- verify (verify_kernels.cu) ----------------------------------------------------------
struct VerifyPlan {
    int rows;          // B * K * (n + 1)
    int chunk_elems;   // scalar fallback: elements of one (row, chunk) work unit
    int chunks;        // scalar fallback: chunks per row
    int vpr;           // streamed form: 16-byte vectors per row (0 when rows are not whole vectors)
    int vec_per_warp;  // streamed form: vectors in one warp's contiguous range
    int slots;         // partial slots reserved per row
    size_t off_g;      // int32 [rows]
    size_t off_pval;   // fp32 [rows, chunks]
    size_t off_pidx;   // int32 [rows, chunks]
    size_t total;
};
VerifyPlan make_verify_plan(int B, int K, int n, int V, int dtype);
int launch_verify(const int32_t *cand_tok, const void *base_logits, int dtype, int B, int K, int n, int V,
                  int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *ws, const VerifyPlan &plan,
                  cudaStream_t st);

int launch_verify_early(const int32_t *cand_tok, const void *base_logits, int dtype, int B, int K, int n, int V,
                        int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *ws, const VerifyPlan &plan,
                        cudaStream_t st);

// ---- tensor-core GEMM (gemm_tcgen05.cu) -------------------------------------------------
// C[M, N] = A[M, Kd] * B[N, Kd]^T, A and B bf16 row-major (K-major), fp32 accumulation in TMEM.
struct GemmEpilogue {
    int mode;          // 0: store fp32 C; 1: per-row partial top-k + (max, sum-exp) per tile;
                       // 2: split-K partials stored transposed, out[split][n][m];
                       // 3: vocabulary head with the operands swapped (A = head weights [V, Kd], B = states
                       //    [nodes <= 128, Kd]): per node and (CTA, segment) one partial top-k list and
                       //    (max, sum-exp) in the mode-1 arrays, n_parts lists per node
    float *out;        // mode 0: [M, N] row-major; mode 2: [splits][N][ldc]
    int ldc;           // mode 0 / 2: leading dimension of out
    int splits;        // mode 2: number of K ranges, each handled by its own tile
    size_t split_stride; // mode 2: elements between the partial results of consecutive splits
    float *part_val;   // mode 1: [M, n_tiles, SPEC_MAX_TOPK]
    int32_t *part_idx; // mode 1: [M, n_tiles, SPEC_MAX_TOPK]
    float *part_ms;    // mode 1: [M, n_tiles, 2]
    int topk;          // mode 1
    int fp8;           // operands are e4m3 bytes instead of bf16; mode 1 then multiplies every accumulator by
                       // row_scale[m] * col_scale[n] before the selection
    const float *row_scale, *col_scale;
    int idx_offset;    // mode 1 / 3: added to every token id written to part_idx (first vocabulary row of a shard)
    int segs;          // mode 3: threads that share one node's column (swapped_head_segs)
    int n_parts;       // mode 3: partial lists per node = CTAs the tiles are dealt to * segs (swapped_head_parts)
};
// Mode 3 bookkeeping, the same on the host (workspace sizing, merge) and in the launch.
int swapped_head_segs(int nodes);
int swapped_head_parts(int nodes, int vocab_rows);
void set_gemm_producers(int n);   // process-wide: 1 or 2 TMA-issuing threads per CTA
int choose_block_n(int M, int N, int num_sm, bool tensor_bound_pref);
int launch_gemm_tc(const void *A, const void *B, int M, int N, int Kd, int block_n, const GemmEpilogue &epi,
                   int32_t *err, cudaStream_t st);
// Up to two contractions in one launch; neither may read what the other writes.
struct GemmCall {
    const void *A, *B;
    int M, N, Kd, block_n;
    GemmEpilogue epi;
};
// `clear` / `clear_words`: int32 words that CTA 0 zeroes once the preceding grid has completed (the first
// kernel of a draft clears the workspace header this way); null: nothing.
int launch_gemm_tc_jobs(const GemmCall *calls, int n_calls, int32_t *err, cudaStream_t st, int32_t *clear = nullptr,
                        int clear_words = 0);

// ---- the tensor-bound head on CTA pairs (gemm_pair.cu) --------------------------------------------
int pair_block_n(int rows, int vocab_rows);
int launch_head_pair(const void *states, const void *W, int rows, int V, int Kd, int block_n, const GemmEpilogue &epi,
                     int32_t *err, cudaStream_t st);

// ---- debug CUDA-core GEMM (gemm_simt.cu) ------------------------------------------------
int launch_gemm_simt(const void *A, const void *B, int M, int N, int Kd, float *C, int ldc, cudaStream_t st);
// Builds the per-tile partial lists (same format as the fused epilogue) from full logits.
int launch_partials_from_logits(const float *logits, int M, int N, int block_n, int topk, float *part_val,
                                int32_t *part_idx, float *part_ms, cudaStream_t st);

// ---- row-wise steps of the draft (row_ops.cuh, draft_kernels.cu, fp8_kernels.cu) ---------
struct MixArgs {
    const float *P;            // `p_splits` partial projections, `p_split_stride` floats apart: [parent rows, d] each
    int p_splits;
    size_t p_split_stride;
    const uint16_t *emb;       // bf16 [V, d]
    const int32_t *tok;        // [rows]
    const float *gamma, *beta; // fp32 [d]
    int d, V, parent_div;
    float a, b, eps;
    uint16_t *S_out;           // bf16 [rows, d]
    uint8_t *S8_out;           // optional: the same states as e4m3 bytes [rows, d] ...
    float *s8_scale;           // ... with one scale per row [rows] (see fp8.cuh); null: not written
    int32_t *err;
};

struct PruneArgs {
    const int32_t *tok[SPEC_MAX_HEADS]; // tok[l]: tokens of level l+1 nodes
    int32_t topk[SPEC_MAX_HEADS];
    int n;
};

struct MergeArgs {
    const float *part_val;     // [rows, n_tiles, SPEC_MAX_TOPK] (first `topk` of each list valid, any order)
    const int32_t *part_idx;   // same shape
    const float *part_ms;      // [rows, n_tiles, 2] = (max, sum of exp(x - max))
    int n_tiles, topk;
    int list_len;              // valid slots of every partial list; 0: the same as topk
    const float *score_in;     // [rows] or null (score 0)
    int32_t *tok_out;          // [rows, topk]
    float *score_out;          // [rows, topk]
    // Raw form (lse_out != null), for a vocabulary shard: score_out receives the logits themselves and
    // lse_out [rows] the log-sum-exp over this shard's columns; score_in is ignored.
    float *lse_out;
    // Last level only (seq_done != null): the CTA whose row completes a sequence's leaves prunes that
    // sequence in the same launch, so no separate prune kernel waits behind this one.
    int32_t *seq_done;         // [B] rows finished per sequence, zero before the launch
    int rows_per_seq;          // rows of this level per sequence
    int L, Lpad, K;            // leaves per sequence, L padded to a power of two >= 2, candidates kept
    int32_t *cand_tok;         // [B, K, n]
    float *cand_logp;          // [B, K]
    PruneArgs prune;
};

// e4m3 copy of a bf16 matrix: Q [rows, d] bytes and one fp32 scale per row (fp8.cuh).
int launch_quantize_rows(const void *X, int rows, int d, void *Q, float *scale, cudaStream_t st);
// merge of approximate partial lists + exact re-scoring of the short list + expansion (fp8_kernels.cu)
int launch_merge_rescore(const MergeArgs &g, const void *W, const void *S, int rows, int d, int V, cudaStream_t st);

int launch_draft_init(int32_t *hdr, int words, cudaStream_t st);
int launch_mix_ln_gelu(const MixArgs &m, int rows, cudaStream_t st);
int launch_merge_expand(const MergeArgs &g, int rows, cudaStream_t st);
// merge of one level + mix of the next in one kernel; SPEC_ERR_SHAPE: shape not covered, launch them separately
int launch_merge_mix(const MergeArgs &g, const MixArgs &m, int rows, cudaStream_t st);
// Cross-shard merge of a vocabulary-parallel head.  Slot g (g < n_ranks, `slot_bytes` apart, starting at
// `slots`) holds rank g's raw lists: fp32 values [rows, topk], int32 token ids [rows, topk], fp32 lse [rows].
// Children of every row: the topk best of the n_ranks*topk entries (value desc, token id asc) with
// score = score_in + value - log(sum_g exp(lse_g)).
int launch_merge_shards(const void *slots, size_t slot_bytes, int n_ranks, int rows, int topk, const float *score_in,
                        int32_t *tok_out, float *score_out, cudaStream_t st);
int launch_prune(const float *leaf_score, const PruneArgs &pa, int B, int L, int K, int32_t *cand_tok,
                 float *cand_logp, cudaStream_t st);

}  // namespace spec
