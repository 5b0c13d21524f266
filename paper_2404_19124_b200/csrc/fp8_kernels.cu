// Kernels of the reduced-precision vocabulary head (levels whose head GEMM is bound by reading the
// weights: fewer rows than the roofline ridge).  The head's weights exist a second time as e4m3 bytes
// with one scale per vocabulary row, half the bytes of the bf16 matrix.  Per level:
//   mix step            also writes the states as e4m3 (row_ops.cuh)
//   head GEMM           kind::f8f6f4 on the two e4m3 operands; the epilogue rescales the accumulators
//                       and keeps, per vocabulary tile, 8 candidates by APPROXIMATE logit and the
//                       (max, sum-exp) of the approximate logits
//   merge_rescore       folds the tiles' lists into a short list of 8 to 16 tokens per row and the
//                       row's log-sum-exp, recomputes the short-listed logits EXACTLY from the bf16
//                       weights and states (fp32 accumulation, as the bf16 head does), and takes the
//                       top-k of those
// The tokens and their logits are therefore those of the bf16 path whenever the true top-k are among
// the 16 best approximate logits (the approximation error is a few hundredths of the logits' standard
// deviation; the k-th and the 16th best of tens of thousands of logits are much further apart); only the
// normaliser comes from approximate logits (error of order 1e-3, tolerance 2e-2).
#include "row_ops.cuh"

namespace spec {

namespace {

using namespace rows;

constexpr int kQuantThreads = 256;
constexpr int kRescoreThreads = 512;            // one warp per short-listed token
constexpr int kShortList = kRescoreThreads / 32;
static_assert(kShortList <= kMaxRounds, "scratch arrays");

// One CTA per row of X (bf16 [rows, d], d % 16 == 0): Q = e4m3(X / scale), scale = max|row| / 448.
__global__ void __launch_bounds__(kQuantThreads)
quantize_rows_kernel(const uint16_t *__restrict__ X, int d, uint8_t *__restrict__ Q, float *__restrict__ scale) {
    __shared__ float red[32];
    const size_t r = blockIdx.x;
    const uint16_t *x = X + r * d;
    float amax = 0.0f;
    for (int i = threadIdx.x * 8; i < d; i += kQuantThreads * 8) {
        const uint4 q = *(const uint4 *)(x + i);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
            amax = fmaxf(amax, fmaxf(fabsf(__uint_as_float(w[j] << 16)), fabsf(__uint_as_float(w[j] & 0xffff0000u))));
    }
    const float s = row_scale_of(group_max<kQuantThreads, BlockSync>(amax, red, threadIdx.x));
    const float inv = 1.0f / s;
    for (int i = threadIdx.x * 8; i < d; i += kQuantThreads * 8) {
        const uint4 q = *(const uint4 *)(x + i);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        float v[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            v[2 * j] = __uint_as_float(w[j] << 16);
            v[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
        *(uint2 *)(Q + r * d + i) = e4m3x8(v, inv);
    }
    if (threadIdx.x == 0) scale[r] = s;
}

struct RescoreArgs {
    MergeArgs merge;          // partial lists of approximate logits; tok_out / score_out: the children
    const uint16_t *W;        // bf16 [V, d] head weights
    const uint16_t *S;        // bf16 [rows, d] states of the level
    int d, V;
};

// One CTA per row.
__global__ void __launch_bounds__(kRescoreThreads) merge_rescore_kernel(RescoreArgs a) {
    extern __shared__ LeafKey rescore_keys[];   // [Lpad] when the prune is folded in, else nothing
    __shared__ Scratch sc;
    __shared__ float exact[kShortList];
    __shared__ int last_of_sequence;
    griddep_launch();
    griddep_wait();
    const int r = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float base = (tid == 0 && a.merge.score_in) ? __ldcg(a.merge.score_in + r) : 0.0f;
    // short list: twice the branching factor plus two, at least 8, at most one per warp
    const int n_short = min(kShortList, max(8, 2 * a.merge.topk + 2));
    merge_select<kRescoreThreads, BlockSync>(a.merge, r, tid, &sc, n_short);
    // exact logit of short-listed token `warp`: dot product of two bf16 rows, fp32 accumulation
    const int v = warp < n_short ? sc.out_id[warp] : -1;
    float acc = 0.0f;
    if (v >= 0 && v < a.V) {
        const uint16_t *w = a.W + (size_t)v * a.d, *s = a.S + (size_t)r * a.d;
        constexpr int kBatch = 8;   // 8-element groups per lane whose loads are in flight together
        for (int i0 = lane * 8; i0 < a.d; i0 += 32 * 8 * kBatch) {
            uint4 qw[kBatch], qs[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int i = i0 + u * 32 * 8;
                qw[u] = make_uint4(0u, 0u, 0u, 0u);
                qs[u] = qw[u];
                if (i < a.d) {
                    qw[u] = *(const uint4 *)(w + i);
                    qs[u] = __ldcg((const uint4 *)(s + i));
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const uint32_t ww[4] = {qw[u].x, qw[u].y, qw[u].z, qw[u].w}, ss[4] = {qs[u].x, qs[u].y, qs[u].z, qs[u].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc = fmaf(__uint_as_float(ww[j] << 16), __uint_as_float(ss[j] << 16), acc);
                    acc = fmaf(__uint_as_float(ww[j] & 0xffff0000u), __uint_as_float(ss[j] & 0xffff0000u), acc);
                }
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) exact[warp] = (v >= 0 && v < a.V) ? acc : -INFINITY;
    __syncthreads();
    // warp 0: the top-k of the exact logits, (value desc, token id asc)
    if (warp == 0) {
        float val = lane < n_short ? exact[lane] : -INFINITY;
        int id = lane < n_short ? sc.out_id[lane] : 0x7fffffff;
        const float lse = sc.lse;
        const int topk = a.merge.topk;
        for (int j = 0; j < topk; ++j) {
            const uint32_t key = float_key(val);
            const uint32_t bk = __reduce_max_sync(0xffffffffu, key);
            const uint32_t bi = __reduce_min_sync(0xffffffffu, key == bk ? (uint32_t)id : 0xffffffffu);
            if (lane == 0) {
                a.merge.tok_out[(size_t)r * topk + j] = (int)bi;
                a.merge.score_out[(size_t)r * topk + j] = base + (key_float(bk) - lse);
            }
            if (key == bk && (uint32_t)id == bi) {   // taken
                val = -INFINITY;
                id = 0x7fffffff;
            }
        }
    }
    prune_if_last<kRescoreThreads, BlockSync>(a.merge, r, tid, rescore_keys, &last_of_sequence);
}

}  // namespace

int launch_quantize_rows(const void *X, int rows, int d, void *Q, float *scale, cudaStream_t st) {
    if (rows <= 0 || d <= 0 || d % 16 != 0) return SPEC_ERR_SHAPE;
    quantize_rows_kernel<<<rows, kQuantThreads, 0, st>>>((const uint16_t *)X, d, (uint8_t *)Q, scale);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_merge_rescore(const MergeArgs &g, const void *W, const void *S, int rows, int d, int V, cudaStream_t st) {
    RescoreArgs a{};
    a.merge = g;
    a.W = (const uint16_t *)W;
    a.S = (const uint16_t *)S;
    a.d = d;
    a.V = V;
    const size_t smem = g.seq_done ? sizeof(LeafKey) * (size_t)g.Lpad : 0;
    SPEC_CUDA_TRY(launch_pdl(merge_rescore_kernel, dim3(rows), dim3(kRescoreThreads), smem, st, a));
    return SPEC_OK;
}

}  // namespace spec
