// Row kernels of the draft path (Sec. 3.1 / Sec. 4.1 of arXiv 2404.19124):
//   mix_ln_gelu_kernel   embedding gather + weighted mix with the projected parent state +
//                        LayerNorm + exact GELU, one CTA per tree node, bf16 state out
//   merge_expand_kernel  folds the per-tile partial top-k lists and (max, sum-exp) pairs of
//                        one row into its top-k tokens and log-probabilities and writes the
//                        children (token, cumulative score) of that node
//   prune_kernel         per sequence: order the leaves by (score desc, leaf index asc),
//                        keep K, walk back to the root to emit the K n-grams
#include <math.h>

#include "spec_common.cuh"

namespace spec {

namespace {

constexpr int kRowThreads = 256;

__device__ __forceinline__ float block_sum(float v, float *red) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    __syncthreads();   // red may still be read from a previous call
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = (l < (int)(blockDim.x >> 5)) ? red[l] : 0.0f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    return t;
}

// One CTA per node r of the level.  P holds the projected state of each distinct parent
// (siblings share it): parent(r) = r / parent_div.  h = a * P[parent] + b * E[tok[r]].
__global__ void __launch_bounds__(kRowThreads)
mix_ln_gelu_kernel(const float *__restrict__ P, const uint16_t *__restrict__ emb, const int32_t *__restrict__ tok,
                   const float *__restrict__ gamma, const float *__restrict__ beta, int d, int V, int parent_div,
                   float a, float b, float eps, uint16_t *__restrict__ S_out, int32_t *err) {
    extern __shared__ float h_s[];   // [d]
    __shared__ float red[32];
    const int r = blockIdx.x;
    const int t = tok[r];
    const bool tok_ok = (t >= 0) && (t < V);
    if (!tok_ok && threadIdx.x == 0) report_error(err, SPEC_ERR_TOKEN_RANGE);
    const float *p = P + (size_t)(r / parent_div) * d;
    const uint16_t *e = emb + (size_t)(tok_ok ? t : 0) * d;

    float sum = 0.0f;
    for (int i = threadIdx.x * 8; i < d; i += kRowThreads * 8) {   // d % 8 == 0
        const float4 p0 = *(const float4 *)(p + i), p1 = *(const float4 *)(p + i + 4);
        uint4 ev = make_uint4(0u, 0u, 0u, 0u);
        if (tok_ok) ev = *(const uint4 *)(e + i);
        const float pv[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
        const uint32_t ew[4] = {ev.x, ev.y, ev.z, ev.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float z = (j & 1) ? __uint_as_float(ew[j >> 1] & 0xffff0000u) : __uint_as_float(ew[j >> 1] << 16);
            const float h = a * pv[j] + b * z;
            h_s[i + j] = h;
            sum += h;
        }
    }
    const float mean = block_sum(sum, red) / (float)d;
    float sq = 0.0f;
    for (int i = threadIdx.x; i < d; i += kRowThreads) {
        const float c = h_s[i] - mean;
        sq += c * c;
    }
    const float var = block_sum(sq, red) / (float)d;
    const float rstd = rsqrtf(var + eps);
    for (int i = threadIdx.x * 2; i < d; i += kRowThreads * 2) {
        uint32_t packed = 0;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float y = (h_s[i + j] - mean) * rstd * gamma[i + j] + beta[i + j];
            const float s = 0.5f * y * (1.0f + erff(y * 0.70710678118654752440f));
            packed |= float_to_bf16_bits(s) << (16 * j);
        }
        *(uint32_t *)(S_out + (size_t)r * d + i) = packed;
    }
}

// (value desc, token id asc) ordering of candidates.
__device__ __forceinline__ bool better(float v, int i, float w, int j) { return v > w || (v == w && i < j); }

// One warp per row.  part_val / part_idx: [rows, n_tiles, SPEC_MAX_TOPK] (first `topk` of each
// list valid, sorted), part_ms: [rows, n_tiles, 2] = (max, sum of exp(x - max)).
__global__ void __launch_bounds__(128)
merge_expand_kernel(const float *__restrict__ part_val, const int32_t *__restrict__ part_idx,
                    const float *__restrict__ part_ms, int rows, int n_tiles, int topk,
                    const float *__restrict__ score_in, int32_t *__restrict__ tok_out,
                    float *__restrict__ score_out) {
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= rows) return;
    const float *pv = part_val + (size_t)r * n_tiles * SPEC_MAX_TOPK;
    const int32_t *pi = part_idx + (size_t)r * n_tiles * SPEC_MAX_TOPK;
    const float *pms = part_ms + (size_t)r * n_tiles * 2;

    // log-sum-exp over the whole row from the per-tile (max, sum) pairs
    float m = -INFINITY;
    for (int t = lane; t < n_tiles; t += 32) m = fmaxf(m, pms[2 * t]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    float s = 0.0f;
    for (int t = lane; t < n_tiles; t += 32) s += pms[2 * t + 1] * __expf(pms[2 * t] - m);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    const float lse = m + logf(s);

    // lane-local sorted list of the best `topk` among this lane's share of the partial entries
    float tv[SPEC_MAX_TOPK];
    int ti[SPEC_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < SPEC_MAX_TOPK; ++j) {
        tv[j] = -INFINITY;
        ti[j] = 0x7fffffff;
    }
    const int entries = n_tiles * topk;
    for (int e = lane; e < entries; e += 32) {
        const int t = e / topk, j = e - t * topk;
        const float v = pv[t * SPEC_MAX_TOPK + j];
        const int id = pi[t * SPEC_MAX_TOPK + j];
        if (better(v, id, tv[SPEC_MAX_TOPK - 1], ti[SPEC_MAX_TOPK - 1])) {
            tv[SPEC_MAX_TOPK - 1] = v;
            ti[SPEC_MAX_TOPK - 1] = id;
#pragma unroll
            for (int q = SPEC_MAX_TOPK - 1; q > 0; --q) {
                if (better(tv[q], ti[q], tv[q - 1], ti[q - 1])) {
                    const float fv = tv[q]; tv[q] = tv[q - 1]; tv[q - 1] = fv;
                    const int fi = ti[q]; ti[q] = ti[q - 1]; ti[q - 1] = fi;
                }
            }
        }
    }
    // `topk` rounds: the warp picks the best head among the lanes, the owner pops it
    const float base = score_in ? score_in[r] : 0.0f;
    for (int j = 0; j < topk; ++j) {
        float bv = tv[0];
        int bi = ti[0];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            if (better(ov, oi, bv, bi)) {
                bv = ov;
                bi = oi;
            }
        }
        if (ti[0] == bi && tv[0] == bv) {   // token ids are unique, so exactly one lane owns it
#pragma unroll
            for (int q = 0; q < SPEC_MAX_TOPK - 1; ++q) {
                tv[q] = tv[q + 1];
                ti[q] = ti[q + 1];
            }
            tv[SPEC_MAX_TOPK - 1] = -INFINITY;
            ti[SPEC_MAX_TOPK - 1] = 0x7fffffff;
        }
        if (lane == 0) {
            tok_out[(size_t)r * topk + j] = bi;
            score_out[(size_t)r * topk + j] = base + (bv - lse);
        }
    }
}

struct LeafKey {
    float score;
    int leaf;
};

__device__ __forceinline__ bool leaf_before(const LeafKey &a, const LeafKey &b) {
    return a.score > b.score || (a.score == b.score && a.leaf < b.leaf);
}

// One CTA per sequence; bitonic sort of the (score, leaf) keys in shared memory.
__global__ void __launch_bounds__(256)
prune_kernel(const float *__restrict__ leaf_score, PruneArgs pa, int L, int Lpad, int K,
             int32_t *__restrict__ cand_tok, float *__restrict__ cand_logp) {
    extern __shared__ LeafKey keys[];   // [Lpad]
    const int b = blockIdx.x;
    for (int i = threadIdx.x; i < Lpad; i += blockDim.x) {
        keys[i].score = i < L ? leaf_score[(size_t)b * L + i] : -INFINITY;
        keys[i].leaf = i < L ? i : 0x7fffffff;
    }
    __syncthreads();
    for (int size = 2; size <= Lpad; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = threadIdx.x; i < Lpad / 2; i += blockDim.x) {
                const int lo = 2 * i - (i & (stride - 1));
                const int hi = lo + stride;
                const bool ascending_block = ((lo & size) == 0);   // "ascending" = best first
                const LeafKey x = keys[lo], y = keys[hi];
                const bool swap = ascending_block ? leaf_before(y, x) : leaf_before(x, y);
                if (swap) {
                    keys[lo] = y;
                    keys[hi] = x;
                }
            }
            __syncthreads();
        }
    }
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const LeafKey kk = keys[k];
        cand_logp[(size_t)b * K + k] = kk.score;
        int idx = kk.leaf;         // index among this sequence's nodes of level n
        int per_seq = L;           // nodes of this sequence at level l + 1
        for (int l = pa.n - 1; l >= 0; --l) {
            cand_tok[((size_t)b * K + k) * pa.n + l] = pa.tok[l][(size_t)b * per_seq + idx];
            idx /= pa.topk[l];
            per_seq /= pa.topk[l];
        }
    }
}

}  // namespace

int launch_mix_ln_gelu(const float *P, const void *emb, const int32_t *tok, const float *gamma, const float *beta,
                       int rows, int d_inner, int V, int parent_div, float a, float b, float eps, void *S_out,
                       int32_t *err, cudaStream_t st) {
    const size_t smem = sizeof(float) * (size_t)d_inner;
    if (smem > 48 * 1024)
        SPEC_CUDA_TRY(cudaFuncSetAttribute(mix_ln_gelu_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    mix_ln_gelu_kernel<<<rows, kRowThreads, smem, st>>>(P, (const uint16_t *)emb, tok, gamma, beta, d_inner, V,
                                                        parent_div, a, b, eps, (uint16_t *)S_out, err);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_merge_expand(const float *part_val, const int32_t *part_idx, const float *part_ms, int rows, int n_tiles,
                        int topk, const float *score_in, int32_t *tok_out, float *score_out, int /*unused*/,
                        cudaStream_t st) {
    const int warps = 4;
    merge_expand_kernel<<<(rows + warps - 1) / warps, warps * 32, 0, st>>>(part_val, part_idx, part_ms, rows, n_tiles,
                                                                            topk, score_in, tok_out, score_out);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_prune(const float *leaf_score, const PruneArgs &pa, int B, int L, int K, int32_t *cand_tok,
                 float *cand_logp, cudaStream_t st) {
    int Lpad = 2;
    while (Lpad < L) Lpad <<= 1;
    prune_kernel<<<B, 256, sizeof(LeafKey) * (size_t)Lpad, st>>>(leaf_score, pa, L, Lpad, K, cand_tok, cand_logp);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

}  // namespace spec
