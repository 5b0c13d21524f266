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

// Host-side bookkeeping ------------------------------------------------------------------
void set_last_cuda_error(int e);
int num_sms();

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
    int chunk_elems;   // elements of one (row, chunk) work unit
    int chunks;        // chunks per row
    size_t off_g;      // int32 [rows]
    size_t off_pval;   // fp32 [rows, chunks]
    size_t off_pidx;   // int32 [rows, chunks]
    size_t total;
};
VerifyPlan make_verify_plan(int B, int K, int n, int V, int dtype);
int launch_verify(const int32_t *cand_tok, const void *base_logits, int dtype, int B, int K, int n, int V,
                  int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *ws, const VerifyPlan &plan,
                  cudaStream_t st);

// ---- tensor-core GEMM (gemm_tcgen05.cu) -------------------------------------------------
// C[M, N] = A[M, Kd] * B[N, Kd]^T, A and B bf16 row-major (K-major), fp32 accumulation in TMEM.
struct GemmEpilogue {
    int mode;          // 0: store fp32 C; 1: per-row partial top-k + (max, sum-exp) per tile
    float *out;        // mode 0: [M, N] row-major
    int ldc;           // mode 0: leading dimension of out
    float *part_val;   // mode 1: [M, n_tiles, SPEC_MAX_TOPK]
    int32_t *part_idx; // mode 1: [M, n_tiles, SPEC_MAX_TOPK]
    float *part_ms;    // mode 1: [M, n_tiles, 2]
    int topk;          // mode 1
};
int choose_block_n(int M, int N, int num_sm, bool tensor_bound_pref);
int launch_gemm_tc(const void *A, const void *B, int M, int N, int Kd, int block_n, const GemmEpilogue &epi,
                   int32_t *err, cudaStream_t st);

// ---- debug CUDA-core GEMM (gemm_simt.cu) ------------------------------------------------
int launch_gemm_simt(const void *A, const void *B, int M, int N, int Kd, float *C, int ldc, cudaStream_t st);
// Builds the per-tile partial lists (same format as the fused epilogue) from full logits.
int launch_partials_from_logits(const float *logits, int M, int N, int block_n, int topk, float *part_val,
                                int32_t *part_idx, float *part_ms, cudaStream_t st);

// ---- row kernels of the draft (draft_kernels.cu) ----------------------------------------
int launch_mix_ln_gelu(const float *P, const void *emb, const int32_t *tok, const float *gamma, const float *beta,
                       int rows, int d_inner, int V, int parent_div, float a, float b, float eps, void *S_out,
                       int32_t *err, cudaStream_t st);
int launch_merge_expand(const float *part_val, const int32_t *part_idx, const float *part_ms, int rows, int n_tiles,
                        int topk, const float *score_in, int32_t *tok_out, float *score_out, int score_is_logp,
                        cudaStream_t st);
struct PruneArgs {
    const int32_t *tok[SPEC_MAX_HEADS]; // tok[l]: tokens of level l+1 nodes
    int32_t topk[SPEC_MAX_HEADS];
    int n;
};
int launch_prune(const float *leaf_score, const PruneArgs &pa, int B, int L, int K, int32_t *cand_tok,
                 float *cand_logp, cudaStream_t st);

}  // namespace spec
