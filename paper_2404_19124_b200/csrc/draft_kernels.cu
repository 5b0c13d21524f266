// Row kernels of the draft path (Sec. 3.1 / Sec. 4.1 of arXiv 2404.19124):
//   mix_ln_gelu_kernel   embedding gather + weighted mix with the projected parent state (sum of
//                        the split-K partials) + LayerNorm + exact GELU, one CTA per tree node,
//                        the row held in registers, bf16 state out
//   merge_expand_kernel  folds the per-tile partial top-k lists and (max, sum-exp) pairs of
//                        one row (one CTA per row) into its top-k tokens and log-probabilities
//                        and writes the children (token, cumulative score) of that node
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

__device__ __forceinline__ float gelu_erf(float y) { return 0.5f * y * (1.0f + erff(y * 0.70710678118654752440f)); }

// One CTA per node r of the level.  P holds the projected state of each distinct parent
// (siblings share it): parent(r) = r / parent_div, as `p_splits` partial sums that are added
// here.  h = a * P[parent] + b * E[tok[r]].  The row lives in registers: thread t owns the
// 8-element groups t, t + 256, ... (kIters of them; d <= 2048 * kIters, d % 8 == 0).
template <int kIters>
__global__ void __launch_bounds__(kRowThreads)
mix_ln_gelu_kernel(const float *__restrict__ P, int p_splits, size_t p_split_stride,
                   const uint16_t *__restrict__ emb, const int32_t *__restrict__ tok,
                   const float *__restrict__ gamma, const float *__restrict__ beta, int d, int V, int parent_div,
                   float a, float b, float eps, uint16_t *__restrict__ S_out, int32_t *err) {
    __shared__ float red[32];
    griddep_launch();
    griddep_wait();
    const int r = blockIdx.x;
    const int t = tok[r];
    const bool tok_ok = (t >= 0) && (t < V);
    if (!tok_ok && threadIdx.x == 0) report_error(err, SPEC_ERR_TOKEN_RANGE);
    const float *p = P + (size_t)(r / parent_div) * d;
    const uint16_t *e = emb + (size_t)(tok_ok ? t : 0) * d;

    float h[kIters][8];
    float sum = 0.0f;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int i = (it * kRowThreads + threadIdx.x) * 8;
#pragma unroll
        for (int j = 0; j < 8; ++j) h[it][j] = 0.0f;
        if (i < d) {
            uint4 ev = make_uint4(0u, 0u, 0u, 0u);
            if (tok_ok) ev = *(const uint4 *)(e + i);
            float pv[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
            for (int sp = 0; sp < p_splits; ++sp) {
                const float4 p0 = *(const float4 *)(p + sp * p_split_stride + i);
                const float4 p1 = *(const float4 *)(p + sp * p_split_stride + i + 4);
                pv[0] += p0.x; pv[1] += p0.y; pv[2] += p0.z; pv[3] += p0.w;
                pv[4] += p1.x; pv[5] += p1.y; pv[6] += p1.z; pv[7] += p1.w;
            }
            const uint32_t ew[4] = {ev.x, ev.y, ev.z, ev.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float z = (j & 1) ? __uint_as_float(ew[j >> 1] & 0xffff0000u) : __uint_as_float(ew[j >> 1] << 16);
                h[it][j] = a * pv[j] + b * z;
                sum += h[it][j];
            }
        }
    }
    const float mean = block_sum(sum, red) / (float)d;
    float sq = 0.0f;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int i = (it * kRowThreads + threadIdx.x) * 8;
        if (i < d) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float c = h[it][j] - mean;
                sq += c * c;
            }
        }
    }
    const float var = block_sum(sq, red) / (float)d;
    const float rstd = rsqrtf(var + eps);
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int i = (it * kRowThreads + threadIdx.x) * 8;
        if (i < d) {
            const float4 g0 = *(const float4 *)(gamma + i), g1 = *(const float4 *)(gamma + i + 4);
            const float4 b0 = *(const float4 *)(beta + i), b1 = *(const float4 *)(beta + i + 4);
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
            uint32_t packed[4];
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const float s0 = gelu_erf((h[it][j] - mean) * rstd * gv[j] + bv[j]);
                const float s1 = gelu_erf((h[it][j + 1] - mean) * rstd * gv[j + 1] + bv[j + 1]);
                packed[j >> 1] = float_to_bf16_bits(s0) | (float_to_bf16_bits(s1) << 16);
            }
            *(uint4 *)(S_out + (size_t)r * d + i) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
    }
}

// The same for rows wider than the register version covers: the mixed row is staged in shared memory.
__global__ void __launch_bounds__(kRowThreads)
mix_ln_gelu_wide_kernel(const float *__restrict__ P, int p_splits, size_t p_split_stride,
                        const uint16_t *__restrict__ emb, const int32_t *__restrict__ tok,
                        const float *__restrict__ gamma, const float *__restrict__ beta, int d, int V,
                        int parent_div, float a, float b, float eps, uint16_t *__restrict__ S_out, int32_t *err) {
    extern __shared__ float h_s[];   // [d]
    __shared__ float red[32];
    griddep_launch();
    griddep_wait();
    const int r = blockIdx.x;
    const int t = tok[r];
    const bool tok_ok = (t >= 0) && (t < V);
    if (!tok_ok && threadIdx.x == 0) report_error(err, SPEC_ERR_TOKEN_RANGE);
    const float *p = P + (size_t)(r / parent_div) * d;
    const uint16_t *e = emb + (size_t)(tok_ok ? t : 0) * d;
    float sum = 0.0f;
    for (int i = threadIdx.x; i < d; i += kRowThreads) {
        float pv = 0.0f;
        for (int sp = 0; sp < p_splits; ++sp) pv += p[sp * p_split_stride + i];
        const float z = tok_ok ? bf16_bits_to_float(e[i]) : 0.0f;
        const float h = a * pv + b * z;
        h_s[i] = h;
        sum += h;
    }
    const float mean = block_sum(sum, red) / (float)d;
    float sq = 0.0f;
    for (int i = threadIdx.x; i < d; i += kRowThreads) {
        const float c = h_s[i] - mean;
        sq += c * c;
    }
    const float var = block_sum(sq, red) / (float)d;
    const float rstd = rsqrtf(var + eps);
    for (int i = threadIdx.x; i < d; i += kRowThreads)
        S_out[(size_t)r * d + i] = (uint16_t)float_to_bf16_bits(gelu_erf((h_s[i] - mean) * rstd * gamma[i] + beta[i]));
}

// (value desc, token id asc) ordering of candidates.
__device__ __forceinline__ bool better(float v, int i, float w, int j) { return v > w || (v == w && i < j); }

constexpr int kMergeThreads = 128;
constexpr int kMergeWarps = kMergeThreads / 32;

// One CTA per row.  part_val / part_idx: [rows, n_tiles, SPEC_MAX_TOPK] (first `topk` of each list
// valid, sorted best first), part_ms: [rows, n_tiles, 2] = (max, sum of exp(x - max)).
// Thread t folds the lists of tiles t, t + 128, ... into a sorted list in registers with all of its
// loads independent of one another; the CTA then extracts the `topk` best in `topk` rounds of
// (warp arg-max by shuffles, one shared-memory exchange between the warps).
__global__ void __launch_bounds__(kMergeThreads)
merge_expand_kernel(const float *__restrict__ part_val, const int32_t *__restrict__ part_idx,
                    const float *__restrict__ part_ms, int rows, int n_tiles, int topk,
                    const float *__restrict__ score_in, int32_t *__restrict__ tok_out,
                    float *__restrict__ score_out) {
    __shared__ float red_m[kMergeWarps], red_s[kMergeWarps];
    __shared__ float cand_v[2][kMergeWarps];
    __shared__ int cand_i[2][kMergeWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = blockIdx.x;
    griddep_launch();
    griddep_wait();
    const float4 *pv4 = (const float4 *)(part_val + (size_t)r * n_tiles * SPEC_MAX_TOPK);
    const int4 *pi4 = (const int4 *)(part_idx + (size_t)r * n_tiles * SPEC_MAX_TOPK);
    const float2 *pms = (const float2 *)(part_ms + (size_t)r * n_tiles * 2);

    float tv[SPEC_MAX_TOPK];
    int ti[SPEC_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < SPEC_MAX_TOPK; ++j) {
        tv[j] = -INFINITY;
        ti[j] = 0x7fffffff;
    }
    float m = -INFINITY, s = 0.0f;
    for (int t = threadIdx.x; t < n_tiles; t += kMergeThreads) {
        const float2 ms = pms[t];
        const float4 v0 = pv4[2 * t], v1 = pv4[2 * t + 1];
        const int4 i0 = pi4[2 * t], i1 = pi4[2 * t + 1];
        if (ms.x > m) {
            s = s * __expf(m - ms.x) + ms.y;   // exp(-inf) = 0 on the first tile
            m = ms.x;
        } else if (ms.x > -INFINITY) {
            s += ms.y * __expf(ms.x - m);
        }
        const float lv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        const int li[8] = {i0.x, i0.y, i0.z, i0.w, i1.x, i1.y, i1.z, i1.w};
#pragma unroll
        for (int j = 0; j < SPEC_MAX_TOPK; ++j) {
            if (j < topk && better(lv[j], li[j], tv[SPEC_MAX_TOPK - 1], ti[SPEC_MAX_TOPK - 1])) {
                tv[SPEC_MAX_TOPK - 1] = lv[j];
                ti[SPEC_MAX_TOPK - 1] = li[j];
#pragma unroll
                for (int q = SPEC_MAX_TOPK - 1; q > 0; --q) {
                    if (better(tv[q], ti[q], tv[q - 1], ti[q - 1])) {
                        const float fv = tv[q]; tv[q] = tv[q - 1]; tv[q - 1] = fv;
                        const int fi = ti[q]; ti[q] = ti[q - 1]; ti[q - 1] = fi;
                    }
                }
            }
        }
    }
    // log-sum-exp of the whole row
    float wm = m;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, off));
    float ws = (m > -INFINITY) ? s * __expf(m - wm) : 0.0f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, off);
    if (lane == 0) {
        red_m[warp] = wm;
        red_s[warp] = ws;
    }
    __syncthreads();
    float bm = red_m[0];
#pragma unroll
    for (int w = 1; w < kMergeWarps; ++w) bm = fmaxf(bm, red_m[w]);
    float bs = 0.0f;
#pragma unroll
    for (int w = 0; w < kMergeWarps; ++w)
        if (red_m[w] > -INFINITY) bs += red_s[w] * __expf(red_m[w] - bm);
    const float lse = bm + logf(bs);

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
        if (lane == 0) {
            cand_v[j & 1][warp] = bv;
            cand_i[j & 1][warp] = bi;
        }
        __syncthreads();   // rounds alternate between two buffers, so one barrier per round is enough
        bv = cand_v[j & 1][0];
        bi = cand_i[j & 1][0];
#pragma unroll
        for (int w = 1; w < kMergeWarps; ++w) {
            const float ov = cand_v[j & 1][w];
            const int oi = cand_i[j & 1][w];
            if (better(ov, oi, bv, bi)) {
                bv = ov;
                bi = oi;
            }
        }
        if (ti[0] == bi && tv[0] == bv) {   // token ids are unique, so exactly one thread owns a real entry
#pragma unroll
            for (int q = 0; q < SPEC_MAX_TOPK - 1; ++q) {
                tv[q] = tv[q + 1];
                ti[q] = ti[q + 1];
            }
            tv[SPEC_MAX_TOPK - 1] = -INFINITY;
            ti[SPEC_MAX_TOPK - 1] = 0x7fffffff;
        }
        if (threadIdx.x == 0) {
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
    griddep_launch();
    griddep_wait();
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

int launch_mix_ln_gelu(const float *P, int p_splits, size_t p_split_stride, const void *emb, const int32_t *tok,
                       const float *gamma, const float *beta, int rows, int d_inner, int V, int parent_div, float a,
                       float b, float eps, void *S_out, int32_t *err, cudaStream_t st) {
    const uint16_t *E = (const uint16_t *)emb;
    uint16_t *S = (uint16_t *)S_out;
    const int groups = (d_inner + 8 * kRowThreads - 1) / (8 * kRowThreads);
#define SPEC_MIX_ARGS P, p_splits, p_split_stride, E, tok, gamma, beta, d_inner, V, parent_div, a, b, eps, S, err
    if (groups <= 1) {
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_kernel<1>, dim3(rows), dim3(kRowThreads), 0, st, SPEC_MIX_ARGS));
    } else if (groups <= 2) {
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_kernel<2>, dim3(rows), dim3(kRowThreads), 0, st, SPEC_MIX_ARGS));
    } else if (groups <= 4) {
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_kernel<4>, dim3(rows), dim3(kRowThreads), 0, st, SPEC_MIX_ARGS));
    } else {
        const size_t smem = sizeof(float) * (size_t)d_inner;
        if (smem > 48 * 1024)
            SPEC_CUDA_TRY(cudaFuncSetAttribute(mix_ln_gelu_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               (int)smem));
        SPEC_CUDA_TRY(launch_pdl(mix_ln_gelu_wide_kernel, dim3(rows), dim3(kRowThreads), smem, st, SPEC_MIX_ARGS));
    }
#undef SPEC_MIX_ARGS
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_merge_expand(const float *part_val, const int32_t *part_idx, const float *part_ms, int rows, int n_tiles,
                        int topk, const float *score_in, int32_t *tok_out, float *score_out, int /*unused*/,
                        cudaStream_t st) {
    SPEC_CUDA_TRY(launch_pdl(merge_expand_kernel, dim3(rows), dim3(kMergeThreads), 0, st, part_val, part_idx, part_ms,
                             rows, n_tiles, topk, score_in, tok_out, score_out));
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_prune(const float *leaf_score, const PruneArgs &pa, int B, int L, int K, int32_t *cand_tok,
                 float *cand_logp, cudaStream_t st) {
    int Lpad = 2;
    while (Lpad < L) Lpad <<= 1;
    SPEC_CUDA_TRY(launch_pdl(prune_kernel, dim3(B), dim3(256), sizeof(LeafKey) * (size_t)Lpad, st, leaf_score, pa, L,
                             Lpad, K, cand_tok, cand_logp));
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

}  // namespace spec
