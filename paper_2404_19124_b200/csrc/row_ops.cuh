// Row-wise steps of the draft path (Sec. 3.1 / Sec. 4.1 of arXiv 2404.19124), written for a group of
// kThreads threads that synchronises through `Sync::sync()`: a whole CTA (__syncthreads) in the
// stand-alone kernels, the four epilogue warps (a named barrier) inside the fused draft kernel.
//   mix_ln_gelu_row   embedding gather + weighted mix with the projected parent state (sum of the
//                     split-K partials) + LayerNorm + exact GELU for one tree node, bf16 state out
//   merge_expand_row  folds the per-tile partial top-k lists and (max, sum-exp) pairs of one row into
//                     its top-k tokens and log-probabilities and writes the node's children
//   prune_sequence    orders one sequence's leaves by (score desc, leaf index asc), keeps K, walks
//                     back to the root to emit the K n-grams
// Buffers that an earlier step of the same launch may have written (projections, tokens, scores,
// partial lists) are read with ld.global.cg, never through the non-coherent path.
#pragma once

#include <math.h>

#include "spec_common.cuh"

namespace spec {
namespace rows {

struct BlockSync {
    static __device__ __forceinline__ void sync() { __syncthreads(); }
};
template <int kId, int kCount>
struct NamedSync {
    static __device__ __forceinline__ void sync() { asm volatile("bar.sync %0, %1;" ::"n"(kId), "n"(kCount) : "memory"); }
};

// Scratch in shared memory for one group.
struct Scratch {
    float red[32];
    float red_m[8], red_s[8];
    float cand_v[2][8];
    int cand_i[2][8];
};

template <int kThreads, typename Sync>
__device__ __forceinline__ float group_sum(float v, float *red, int tid) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    const int w = tid >> 5, l = tid & 31;
    Sync::sync();   // red may still be read from a previous call
    if (l == 0) red[w] = v;
    Sync::sync();
    float t = (l < kThreads / 32) ? red[l] : 0.0f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    return t;
}

__device__ __forceinline__ float gelu_erf(float y) { return 0.5f * y * (1.0f + erff(y * 0.70710678118654752440f)); }

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
    int32_t *err;
};

// Node r of the level.  Siblings share a projected parent state: parent(r) = r / parent_div.
// h = a * P[parent] + b * E[tok[r]].  The row lives in registers: thread t owns the 8-element groups
// t, t + kThreads, ... (kIters of them; d <= 8 * kThreads * kIters, d % 8 == 0).
template <int kThreads, int kIters, typename Sync>
__device__ __forceinline__ void mix_ln_gelu_row(const MixArgs &m, int r, int tid, float *red) {
    const int t = __ldcg(m.tok + r);
    const bool tok_ok = (t >= 0) && (t < m.V);
    if (!tok_ok && tid == 0) report_error(m.err, SPEC_ERR_TOKEN_RANGE);
    const int d = m.d;
    const float *p = m.P + (size_t)(r / m.parent_div) * d;
    const uint16_t *e = m.emb + (size_t)(tok_ok ? t : 0) * d;

    float h[kIters][8];
    float sum = 0.0f;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int i = (it * kThreads + tid) * 8;
#pragma unroll
        for (int j = 0; j < 8; ++j) h[it][j] = 0.0f;
        if (i < d) {
            uint4 ev = make_uint4(0u, 0u, 0u, 0u);
            if (tok_ok) ev = *(const uint4 *)(e + i);
            float pv[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
            for (int sp = 0; sp < m.p_splits; ++sp) {
                const float4 p0 = __ldcg((const float4 *)(p + sp * m.p_split_stride + i));
                const float4 p1 = __ldcg((const float4 *)(p + sp * m.p_split_stride + i + 4));
                pv[0] += p0.x; pv[1] += p0.y; pv[2] += p0.z; pv[3] += p0.w;
                pv[4] += p1.x; pv[5] += p1.y; pv[6] += p1.z; pv[7] += p1.w;
            }
            const uint32_t ew[4] = {ev.x, ev.y, ev.z, ev.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float z = (j & 1) ? __uint_as_float(ew[j >> 1] & 0xffff0000u) : __uint_as_float(ew[j >> 1] << 16);
                h[it][j] = m.a * pv[j] + m.b * z;
                sum += h[it][j];
            }
        }
    }
    const float mean = group_sum<kThreads, Sync>(sum, red, tid) / (float)d;
    float sq = 0.0f;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int i = (it * kThreads + tid) * 8;
        if (i < d) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float c = h[it][j] - mean;
                sq += c * c;
            }
        }
    }
    const float var = group_sum<kThreads, Sync>(sq, red, tid) / (float)d;
    const float rstd = rsqrtf(var + m.eps);
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int i = (it * kThreads + tid) * 8;
        if (i < d) {
            const float4 g0 = *(const float4 *)(m.gamma + i), g1 = *(const float4 *)(m.gamma + i + 4);
            const float4 b0 = *(const float4 *)(m.beta + i), b1 = *(const float4 *)(m.beta + i + 4);
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
            uint32_t packed[4];
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const float s0 = gelu_erf((h[it][j] - mean) * rstd * gv[j] + bv[j]);
                const float s1 = gelu_erf((h[it][j + 1] - mean) * rstd * gv[j + 1] + bv[j + 1]);
                packed[j >> 1] = float_to_bf16_bits(s0) | (float_to_bf16_bits(s1) << 16);
            }
            *(uint4 *)(m.S_out + (size_t)r * d + i) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
    }
}

// Picks the register-array size for the row width; false when the row is too wide for this group size.
template <int kThreads, typename Sync>
__device__ __forceinline__ bool mix_ln_gelu_row_any(const MixArgs &m, int r, int tid, float *red) {
    const int groups = (m.d + 8 * kThreads - 1) / (8 * kThreads);
    if (groups <= 1) mix_ln_gelu_row<kThreads, 1, Sync>(m, r, tid, red);
    else if (groups <= 2) mix_ln_gelu_row<kThreads, 2, Sync>(m, r, tid, red);
    else if (groups <= 4) mix_ln_gelu_row<kThreads, 4, Sync>(m, r, tid, red);
    else if (groups <= 8) mix_ln_gelu_row<kThreads, 8, Sync>(m, r, tid, red);
    else return false;
    return true;
}

// (value desc, token id asc) ordering of candidates.
__device__ __forceinline__ bool better(float v, int i, float w, int j) { return v > w || (v == w && i < j); }

struct MergeArgs {
    const float *part_val;     // [rows, n_tiles, SPEC_MAX_TOPK] (first `topk` of each list valid, best first)
    const int32_t *part_idx;   // same shape
    const float *part_ms;      // [rows, n_tiles, 2] = (max, sum of exp(x - max))
    int n_tiles, topk;
    const float *score_in;     // [rows] or null (score 0)
    int32_t *tok_out;          // [rows, topk]
    float *score_out;          // [rows, topk]
};

// Thread t folds the lists of tiles t, t + kThreads, ... into a sorted list in registers with all of
// its loads independent of one another; the group then extracts the `topk` best in `topk` rounds of
// (warp arg-max by shuffles, one shared-memory exchange between the warps).
template <int kThreads, typename Sync>
__device__ __forceinline__ void merge_expand_row(const MergeArgs &g, int r, int tid, Scratch *sc) {
    constexpr int kWarps = kThreads / 32;
    const int lane = tid & 31, warp = tid >> 5;
    const int n_tiles = g.n_tiles, topk = g.topk;
    const float4 *pv4 = (const float4 *)(g.part_val + (size_t)r * n_tiles * SPEC_MAX_TOPK);
    const int4 *pi4 = (const int4 *)(g.part_idx + (size_t)r * n_tiles * SPEC_MAX_TOPK);
    const float2 *pms = (const float2 *)(g.part_ms + (size_t)r * n_tiles * 2);

    float tv[SPEC_MAX_TOPK];
    int ti[SPEC_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < SPEC_MAX_TOPK; ++j) {
        tv[j] = -INFINITY;
        ti[j] = 0x7fffffff;
    }
    float m = -INFINITY, s = 0.0f;
    for (int t = tid; t < n_tiles; t += kThreads) {
        const float2 ms = __ldcg(pms + t);
        const float4 v0 = __ldcg(pv4 + 2 * t), v1 = __ldcg(pv4 + 2 * t + 1);
        const int4 i0 = __ldcg(pi4 + 2 * t), i1 = __ldcg(pi4 + 2 * t + 1);
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
    Sync::sync();   // the scratch may still be read by the previous row's last round
    if (lane == 0) {
        sc->red_m[warp] = wm;
        sc->red_s[warp] = ws;
    }
    Sync::sync();
    float bm = sc->red_m[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) bm = fmaxf(bm, sc->red_m[w]);
    float bs = 0.0f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w)
        if (sc->red_m[w] > -INFINITY) bs += sc->red_s[w] * __expf(sc->red_m[w] - bm);
    const float lse = bm + logf(bs);

    const float base = g.score_in ? __ldcg(g.score_in + r) : 0.0f;
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
            sc->cand_v[j & 1][warp] = bv;
            sc->cand_i[j & 1][warp] = bi;
        }
        Sync::sync();   // rounds alternate between two buffers, so one barrier per round is enough
        bv = sc->cand_v[j & 1][0];
        bi = sc->cand_i[j & 1][0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) {
            const float ov = sc->cand_v[j & 1][w];
            const int oi = sc->cand_i[j & 1][w];
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
        if (tid == 0) {
            g.tok_out[(size_t)r * topk + j] = bi;
            g.score_out[(size_t)r * topk + j] = base + (bv - lse);
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

// Sequence b: bitonic sort of the (score, leaf) keys in shared memory (`keys`: Lpad entries, Lpad the
// power of two >= max(L, 2)), then the K best leaves are traced back to the root.
template <int kThreads, typename Sync>
__device__ __forceinline__ void prune_sequence(const float *leaf_score, const PruneArgs &pa, int L, int Lpad, int K,
                                               int32_t *cand_tok, float *cand_logp, int b, int tid, LeafKey *keys) {
    Sync::sync();   // the previous sequence's back-trace still reads the keys
    for (int i = tid; i < Lpad; i += kThreads) {
        keys[i].score = i < L ? __ldcg(leaf_score + (size_t)b * L + i) : -INFINITY;
        keys[i].leaf = i < L ? i : 0x7fffffff;
    }
    Sync::sync();
    for (int size = 2; size <= Lpad; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = tid; i < Lpad / 2; i += kThreads) {
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
            Sync::sync();
        }
    }
    for (int k = tid; k < K; k += kThreads) {
        const LeafKey kk = keys[k];
        cand_logp[(size_t)b * K + k] = kk.score;
        int idx = kk.leaf;         // index among this sequence's nodes of level n
        int per_seq = L;           // nodes of this sequence at level l + 1
        for (int l = pa.n - 1; l >= 0; --l) {
            cand_tok[((size_t)b * K + k) * pa.n + l] = __ldcg(pa.tok[l] + (size_t)b * per_seq + idx);
            idx /= pa.topk[l];
            per_seq /= pa.topk[l];
        }
    }
}

}  // namespace rows
}  // namespace spec
