// Stand-alone row kernels of the draft path (the row-wise steps themselves are in row_ops.cuh):
//   mix_ln_gelu_kernel   one CTA of 256 threads per tree node
//   merge_expand_kernel  one CTA of 128 threads per row of the vocabulary head
//   prune_kernel         one CTA of 256 threads per sequence
// Each is launched with programmatic stream serialization, so its CTAs are usually resident, waiting,
// while the kernel before it still runs.
#include "row_ops.cuh"

namespace spec {

namespace {

using namespace rows;

constexpr int kRowThreads = 256;
constexpr int kMergeThreads = 128;

// Rows of up to 4096 elements: at most 128 registers, so that two CTAs fit beside a resident GEMM CTA.
__global__ void __launch_bounds__(kRowThreads, 2) mix_ln_gelu_kernel(MixArgs m) {
    __shared__ float red[32];
    griddep_launch();
    griddep_wait();
    if (m.d <= 8 * kRowThreads) mix_ln_gelu_row<kRowThreads, 1, 2, BlockSync>(m, blockIdx.x, threadIdx.x, red);
    else mix_ln_gelu_row<kRowThreads, 2, 2, BlockSync>(m, blockIdx.x, threadIdx.x, red);
}

// Rows of 2049 to 4096 elements in levels of at most one CTA per SM: 512 threads, one 8-element group each.  The
// step is a chain of dependent latencies (loads, two reductions, sixteen erf evaluations per thread with 256
// threads), so halving the per-thread work shortens it: 13B-shaped draft 3-5 us faster than with 256 threads.  At
// most 72 registers, so that the CTA fits beside a resident GEMM CTA.
constexpr int kWideRowThreads = 512;
__global__ void __maxnreg__(72) mix_ln_gelu_512_kernel(MixArgs m) {
    __shared__ float red[32];
    griddep_launch();
    griddep_wait();
    mix_ln_gelu_row<kWideRowThreads, 1, 1, BlockSync>(m, blockIdx.x, threadIdx.x, red);
}

// The same for levels with more nodes than one wave of the kernel above holds: one 8-element group in
// flight per thread and at most 80 registers, so three CTAs share an SM and the level stays one wave.
__global__ void __launch_bounds__(kRowThreads, 3) mix_ln_gelu_many_kernel(MixArgs m) {
    __shared__ float red[32];
    griddep_launch();
    griddep_wait();
    if (m.d <= 8 * kRowThreads) mix_ln_gelu_row<kRowThreads, 1, 1, BlockSync>(m, blockIdx.x, threadIdx.x, red);
    else mix_ln_gelu_row<kRowThreads, 2, 1, BlockSync>(m, blockIdx.x, threadIdx.x, red);
}

// Rows of up to 16384 elements.
__global__ void __launch_bounds__(kRowThreads) mix_ln_gelu_mid_kernel(MixArgs m) {
    __shared__ float red[32];
    griddep_launch();
    griddep_wait();
    if (m.d <= 8 * kRowThreads * 4) mix_ln_gelu_row<kRowThreads, 4, 2, BlockSync>(m, blockIdx.x, threadIdx.x, red);
    else mix_ln_gelu_row<kRowThreads, 8, 2, BlockSync>(m, blockIdx.x, threadIdx.x, red);
}

// Rows wider than the register version covers: the mixed row is staged in shared memory.
__global__ void __launch_bounds__(kRowThreads) mix_ln_gelu_wide_kernel(MixArgs m) {
    extern __shared__ float h_s[];   // [d]
    __shared__ float red[32];
    griddep_launch();
    griddep_wait();
    const int r = blockIdx.x, tid = threadIdx.x, d = m.d;
    const int t = m.tok[r];
    const bool tok_ok = (t >= 0) && (t < m.V);
    if (!tok_ok && tid == 0) report_error(m.err, SPEC_ERR_TOKEN_RANGE);
    const float *p = m.P + (size_t)(r / m.parent_div) * d;
    const uint16_t *e = m.emb + (size_t)(tok_ok ? t : 0) * d;
    float sum = 0.0f;
    for (int i = tid; i < d; i += kRowThreads) {
        float pv = 0.0f;
        for (int sp = 0; sp < m.p_splits; ++sp) pv += p[sp * m.p_split_stride + i];
        const float z = tok_ok ? bf16_bits_to_float(e[i]) : 0.0f;
        const float h = m.a * pv + m.b * z;
        h_s[i] = h;
        sum += h;
    }
    const float mean = group_sum<kRowThreads, BlockSync>(sum, red, tid) / (float)d;
    float sq = 0.0f;
    for (int i = tid; i < d; i += kRowThreads) {
        const float c = h_s[i] - mean;
        sq += c * c;
    }
    const float var = group_sum<kRowThreads, BlockSync>(sq, red, tid) / (float)d;
    const float rstd = rsqrtf(var + m.eps);
    for (int i = tid; i < d; i += kRowThreads)
        m.S_out[(size_t)r * d + i] = (uint16_t)float_to_bf16_bits(gelu_erf((h_s[i] - mean) * rstd * m.gamma[i] + m.beta[i]));
}

// First kernel of a draft: clears the workspace header (error word, per-sequence counters).  A kernel
// rather than a memset so that the projection launched behind it may already set itself up and fetch
// weights; like every kernel here it first waits for whatever precedes it in the stream.
__global__ void __launch_bounds__(256) draft_init_kernel(int32_t *hdr, int words) {
    griddep_launch();
    griddep_wait();
    for (int i = threadIdx.x; i < words; i += blockDim.x) hdr[i] = 0;
}

__global__ void __launch_bounds__(kMergeThreads) merge_expand_kernel(MergeArgs g) {
    extern __shared__ LeafKey merge_keys[];   // [Lpad] when the prune is folded in, else nothing
    __shared__ Scratch sc;
    __shared__ int last_of_sequence;
    griddep_launch();
    griddep_wait();
    merge_expand_row<kMergeThreads, BlockSync>(g, blockIdx.x, threadIdx.x, &sc);
    prune_if_last<kMergeThreads, BlockSync>(g, blockIdx.x, threadIdx.x, merge_keys, &last_of_sequence);
}

// Merge of level l and the gather + mix + LayerNorm + GELU of level l + 1 in one launch: one CTA of 256 threads
// per row of level l folds the row's partial lists into its children (tokens, scores) and then computes the
// states of those children, whose tokens it has just found and whose parent projection is this row's.  One
// kernel boundary less between two vocabulary heads.
struct MergeMixArgs {
    MergeArgs merge;   // level l
    MixArgs mix;       // level l + 1 (tok and parent_div unused: the tokens come from the merge)
};

// At most 128 registers: like the other row kernels its CTAs must fit beside a resident GEMM CTA, or they could
// not start (and wait, set up) before that kernel ends.
constexpr int kFusedBatch = 2;
__global__ void __launch_bounds__(kRowThreads, 2) merge_mix_kernel(MergeMixArgs a) {
    __shared__ Scratch sc;
    __shared__ float red_a[kRowThreads / 32 * kFusedBatch], red_b[kRowThreads / 32 * kFusedBatch];
    griddep_launch();
    griddep_wait();
    const int r = blockIdx.x, tid = threadIdx.x;
    merge_expand_row<kRowThreads, BlockSync>(a.merge, r, tid, &sc);
    // sc.out_id[0 .. topk) now hold the children's tokens (valid for the whole CTA after merge_select's last barrier)
    if (a.mix.d <= 8 * kRowThreads)
        mix_children<kRowThreads, 1, kFusedBatch, BlockSync>(a.mix, r, r * a.merge.topk, a.merge.topk, sc.out_id, red_a, red_b, tid);
    else
        mix_children<kRowThreads, 2, kFusedBatch, BlockSync>(a.mix, r, r * a.merge.topk, a.merge.topk, sc.out_id, red_a, red_b, tid);
}

// Rows of 2049 to 4096 elements: 512 threads, one 8-element group each, like mix_ln_gelu_512_kernel (single-
// candidate chain at the 13B widths 210 -> 203 us per draft, at the 34B widths 278 -> 269 us).  72 registers at
// most, so that the CTA fits beside a resident GEMM CTA.
__global__ void __maxnreg__(72) merge_mix_512_kernel(MergeMixArgs a) {
    __shared__ Scratch sc;
    __shared__ float red_a[kWideRowThreads / 32 * kFusedBatch], red_b[kWideRowThreads / 32 * kFusedBatch];
    griddep_launch();
    griddep_wait();
    const int r = blockIdx.x, tid = threadIdx.x;
    merge_expand_row<kWideRowThreads, BlockSync>(a.merge, r, tid, &sc);
    mix_children<kWideRowThreads, 1, kFusedBatch, BlockSync>(a.mix, r, r * a.merge.topk, a.merge.topk, sc.out_id, red_a, red_b, tid);
}

// Vocabulary-parallel head: one warp per row folds the n_ranks raw lists (see launch_merge_shards).
// Lane i owns entries i and i + 32 of the row's n_ranks * topk <= 64 candidates.
constexpr int kShardRowsPerCta = 4;
__global__ void __launch_bounds__(32 * kShardRowsPerCta)
merge_shards_kernel(const char *slots, size_t slot_bytes, int n_ranks, int rows, int topk,
                    const float *__restrict__ score_in, int32_t *__restrict__ tok_out, float *__restrict__ score_out) {
    griddep_launch();
    griddep_wait();
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * kShardRowsPerCta + (threadIdx.x >> 5);
    if (r >= rows) return;
    const int n_cand = n_ranks * topk;
    float v[2];
    int id[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const int c = lane + 32 * q;
        v[q] = -INFINITY;
        id[q] = 0x7fffffff;
        if (c < n_cand) {
            const int g = c / topk, j = c - g * topk;
            const char *slot = slots + (size_t)g * slot_bytes;
            const float *val = reinterpret_cast<const float *>(slot);
            const int32_t *tok = reinterpret_cast<const int32_t *>(slot + sizeof(float) * (size_t)rows * topk);
            v[q] = __ldcg(val + (size_t)r * topk + j);
            id[q] = __ldcg(tok + (size_t)r * topk + j);
        }
    }
    // log-sum-exp over the whole vocabulary from the shards' values, lane g holding shard g
    float l = -INFINITY;
    if (lane < n_ranks) {
        const char *slot = slots + (size_t)lane * slot_bytes;
        l = __ldcg(reinterpret_cast<const float *>(slot + 2 * sizeof(float) * (size_t)rows * topk) + r);
    }
    float m = l;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    float e = (lane < n_ranks && l > -INFINITY) ? expf(l - m) : 0.0f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) e += __shfl_xor_sync(0xffffffffu, e, off);
    const float lse = m + logf(e);
    const float base = score_in ? __ldcg(score_in + r) : 0.0f;
    for (int j = 0; j < topk; ++j) {
        // the lane's better entry, then the warp's best: (value desc, token id asc)
        const int mine = better(v[1], id[1], v[0], id[0]) ? 1 : 0;
        const uint32_t key = float_key(v[mine]);
        const uint32_t bk = __reduce_max_sync(0xffffffffu, key);
        const uint32_t bi = __reduce_min_sync(0xffffffffu, key == bk ? (uint32_t)id[mine] : 0xffffffffu);
        if (lane == 0) {
            tok_out[(size_t)r * topk + j] = (int)bi;
            score_out[(size_t)r * topk + j] = base + (key_float(bk) - lse);
        }
        if (key == bk && (uint32_t)id[mine] == bi) {   // token ids are unique across shards: one owner
            v[mine] = -INFINITY;
            id[mine] = 0x7fffffff;
        }
    }
}

__global__ void __launch_bounds__(kRowThreads)
prune_kernel(const float *leaf_score, PruneArgs pa, int L, int Lpad, int K, int32_t *cand_tok, float *cand_logp) {
    extern __shared__ LeafKey keys[];   // [Lpad]
    griddep_launch();
    griddep_wait();
    prune_sequence<kRowThreads, BlockSync>(leaf_score, pa, L, Lpad, K, cand_tok, cand_logp, blockIdx.x, threadIdx.x,
                                           keys);
}

}  // namespace

int launch_mix_ln_gelu(const MixArgs &m, int rows, cudaStream_t st) {
    const int d_inner = m.d;
    if (d_inner <= 8 * kRowThreads * 2 && rows > num_sms()) {
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_many_kernel, dim3(rows), dim3(kRowThreads), 0, st, m));
    } else if (d_inner <= 8 * kWideRowThreads && d_inner > 8 * kRowThreads) {
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_512_kernel, dim3(rows), dim3(kWideRowThreads), 0, st, m));
    } else if (d_inner <= 8 * kRowThreads * 2) {
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_kernel, dim3(rows), dim3(kRowThreads), 0, st, m));
    } else if (d_inner <= 8 * kRowThreads * 8) {
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_mid_kernel, dim3(rows), dim3(kRowThreads), 0, st, m));
    } else {
        const size_t smem = sizeof(float) * (size_t)d_inner;
        if (smem > 48 * 1024)
            SPEC_CUDA_TRY(cudaFuncSetAttribute(mix_ln_gelu_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               (int)smem));
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_wide_kernel, dim3(rows), dim3(kRowThreads), smem, st, m));
    }
    return SPEC_OK;
}

int launch_draft_init(int32_t *hdr, int words, cudaStream_t st) {
    SPEC_CUDA_TRY(launch_pdl(draft_init_kernel, dim3(1), dim3(256), 0, st, hdr, words));
    return SPEC_OK;
}

int launch_merge_expand(const MergeArgs &g, int rows, cudaStream_t st) {
    const size_t smem = g.seq_done ? sizeof(LeafKey) * (size_t)g.Lpad : 0;
    SPEC_CUDA_TRY(launch_pdl(merge_expand_kernel, dim3(rows), dim3(kMergeThreads), smem, st, g));
    return SPEC_OK;
}

// Returns SPEC_ERR_SHAPE when the fused form does not cover the shape (rows wider than 4096 elements, an e4m3
// copy of the states wanted): the caller then launches the merge and the mix separately.
int launch_merge_mix(const MergeArgs &g, const MixArgs &m, int rows, cudaStream_t st) {
    if (m.d > 8 * kRowThreads * 2 || m.S8_out != nullptr || g.lse_out != nullptr || g.seq_done != nullptr)
        return SPEC_ERR_SHAPE;
    MergeMixArgs a{g, m};
    if (m.d > 8 * kRowThreads && m.d <= 8 * kWideRowThreads) {
        SPEC_CUDA_TRY(launch_pdl(merge_mix_512_kernel, dim3(rows), dim3(kWideRowThreads), 0, st, a));
        return SPEC_OK;
    }
    SPEC_CUDA_TRY(launch_pdl(merge_mix_kernel, dim3(rows), dim3(kRowThreads), 0, st, a));
    return SPEC_OK;
}

int launch_merge_shards(const void *slots, size_t slot_bytes, int n_ranks, int rows, int topk, const float *score_in,
                        int32_t *tok_out, float *score_out, cudaStream_t st) {
    if (n_ranks < 1 || n_ranks > 32 || n_ranks * topk > 64) return SPEC_ERR_SHAPE;
    const int grid = (rows + kShardRowsPerCta - 1) / kShardRowsPerCta;
    SPEC_CUDA_TRY(launch_pdl(merge_shards_kernel, dim3(grid), dim3(32 * kShardRowsPerCta), 0, st, (const char *)slots,
                             slot_bytes, n_ranks, rows, topk, score_in, tok_out, score_out));
    return SPEC_OK;
}

int launch_prune(const float *leaf_score, const PruneArgs &pa, int B, int L, int K, int32_t *cand_tok,
                 float *cand_logp, cudaStream_t st) {
    int Lpad = 2;
    while (Lpad < L) Lpad <<= 1;
    SPEC_CUDA_TRY(launch_pdl(prune_kernel, dim3(B), dim3(kRowThreads), sizeof(LeafKey) * (size_t)Lpad, st, leaf_score, pa,
                             L, Lpad, K, cand_tok, cand_logp));
    return SPEC_OK;
}

}  // namespace spec
