// Row-wise steps of the draft path (Sec. 3.1 / Sec. 4.1 of arXiv 2404.19124), written for a group of
// kThreads threads that synchronises through `Sync::sync()` (a whole CTA in the stand-alone kernels).
//   mix_ln_gelu_row   embedding gather + weighted mix with the projected parent state (sum of the
//                     split-K partials) + LayerNorm + exact GELU for one tree node, bf16 state out
//   merge_expand_row  folds the per-tile partial top-k lists and (max, sum-exp) pairs of one row into
//                     its top-k tokens and log-probabilities and writes the node's children
//   prune_sequence    orders one sequence's leaves by (score desc, leaf index asc), keeps K, walks
//                     back to the root to emit the K n-grams
// These steps run once per launch on a handful of rows, so what they cost is latency: every load of a
// step is issued before the first one is used, and dependent chains are kept short.
// Buffers that a preceding kernel wrote are read with ld.global.cg, never through the non-coherent path.
#pragma once

#include <math.h>

#include "fp8.cuh"
#include "spec_common.cuh"

namespace spec {
namespace rows {

using spec::MergeArgs;
using spec::MixArgs;

struct BlockSync {
    static __device__ __forceinline__ void sync() { __syncthreads(); }
};

// Scratch in shared memory for one group.
constexpr int kMaxGroupWarps = 16;
constexpr int kMaxRounds = 16;        // most entries a selection can return (top-k itself needs at most 8)
struct Scratch {
    float red[32];
    float red_m[kMaxGroupWarps], red_s[kMaxGroupWarps];
    uint32_t cand_k[2][kMaxGroupWarps];
    int cand_i[2][kMaxGroupWarps];
    float out_val[kMaxRounds];        // result of merge_select: values, best first ...
    int out_id[kMaxRounds];           // ... and their token ids
    float lse;
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

template <int kThreads, typename Sync>
__device__ __forceinline__ float group_max(float v, float *red, int tid) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
    const int w = tid >> 5, l = tid & 31;
    Sync::sync();
    if (l == 0) red[w] = v;
    Sync::sync();
    float t = (l < kThreads / 32) ? red[l] : 0.0f;   // used for magnitudes only
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, off));
    return t;
}

// Exact (erf) GELU.  erff is kept out of line: inlined it would be the bulk of the row step's code.
static __device__ __noinline__ float erf_call(float x) { return erff(x); }
__device__ __forceinline__ float gelu_erf(float y) { return 0.5f * y * (1.0f + erf_call(y * 0.70710678118654752440f)); }

// Node r of the level.  Siblings share a projected parent state: parent(r) = r / parent_div.
// h = a * P[parent] + b * E[tok[r]].  The row lives in registers: thread t owns the 8-element groups
// t, t + kThreads, ... (kIters of them; d <= 8 * kThreads * kIters, d % 8 == 0).  kDepth of those
// groups have their loads in flight together (registers against latency).
template <int kThreads, int kIters, int kDepth, typename Sync>
__device__ __forceinline__ void mix_ln_gelu_row(const MixArgs &m, int r, int tid, float *red) {
    constexpr int kSp = 4;                                        // partial projections fetched per batch
    constexpr int kGroup = kIters >= 8 ? 1 : (kIters < kDepth ? kIters : kDepth);
    const int t = __ldcg(m.tok + r);
    const bool tok_ok = (t >= 0) && (t < m.V);
    if (!tok_ok && tid == 0) report_error(m.err, SPEC_ERR_TOKEN_RANGE);
    const int d = m.d;
    const float *p = m.P + (size_t)(r / m.parent_div) * d;
    const uint16_t *e = m.emb + (size_t)(tok_ok ? t : 0) * d;

    float h[kIters][8];
    float sum = 0.0f;
#pragma unroll
    for (int g0 = 0; g0 < kIters; g0 += kGroup) {
        // every load of the group is issued before the first value is used: one round trip per group
        uint4 ev[kGroup];
        float4 pa[kGroup][kSp], pb[kGroup][kSp];
#pragma unroll
        for (int q = 0; q < kGroup; ++q) {
            const int i = ((g0 + q) * kThreads + tid) * 8;
            ev[q] = make_uint4(0u, 0u, 0u, 0u);
            if (i < d && tok_ok) ev[q] = *(const uint4 *)(e + i);
#pragma unroll
            for (int sp = 0; sp < kSp; ++sp) {
                pa[q][sp] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                pb[q][sp] = pa[q][sp];
                if (i < d && sp < m.p_splits) {
                    pa[q][sp] = __ldcg((const float4 *)(p + sp * m.p_split_stride + i));
                    pb[q][sp] = __ldcg((const float4 *)(p + sp * m.p_split_stride + i + 4));
                }
            }
        }
#pragma unroll
        for (int q = 0; q < kGroup; ++q) {
            const int it = g0 + q;
            const int i = (it * kThreads + tid) * 8;
            float pv[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int sp = 0; sp < kSp; ++sp) {      // partials are added in ascending order: reproducible
                pv[0] += pa[q][sp].x; pv[1] += pa[q][sp].y; pv[2] += pa[q][sp].z; pv[3] += pa[q][sp].w;
                pv[4] += pb[q][sp].x; pv[5] += pb[q][sp].y; pv[6] += pb[q][sp].z; pv[7] += pb[q][sp].w;
            }
            if (i < d) {
                for (int sp = kSp; sp < m.p_splits; ++sp) {   // more partials than one batch holds (rare)
                    const float4 p0 = __ldcg((const float4 *)(p + sp * m.p_split_stride + i));
                    const float4 p1 = __ldcg((const float4 *)(p + sp * m.p_split_stride + i + 4));
                    pv[0] += p0.x; pv[1] += p0.y; pv[2] += p0.z; pv[3] += p0.w;
                    pv[4] += p1.x; pv[5] += p1.y; pv[6] += p1.z; pv[7] += p1.w;
                }
            }
            const uint32_t ew[4] = {ev[q].x, ev[q].y, ev[q].z, ev[q].w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float z = (j & 1) ? __uint_as_float(ew[j >> 1] & 0xffff0000u) : __uint_as_float(ew[j >> 1] << 16);
                h[it][j] = i < d ? m.a * pv[j] + m.b * z : 0.0f;
                sum += h[it][j];
            }
        }
    }
    // LayerNorm parameters: requested before the two reductions so that they arrive while those run
    // (for the widest rows they are fetched where they are used, to stay within the register file)
    constexpr bool kHoist = kIters <= 2;
    constexpr int kHeld = kHoist ? kIters : 1;
    float4 gq[kHeld][2], bq[kHeld][2];
    if (kHoist) {
#pragma unroll
        for (int it = 0; it < kHeld; ++it) {
            const int i = (it * kThreads + tid) * 8;
            const int ic = i < d ? i : 0;
            gq[it][0] = *(const float4 *)(m.gamma + ic);
            gq[it][1] = *(const float4 *)(m.gamma + ic + 4);
            bq[it][0] = *(const float4 *)(m.beta + ic);
            bq[it][1] = *(const float4 *)(m.beta + ic + 4);
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
    float amax = 0.0f;   // largest magnitude of the bf16-rounded state (for the e4m3 copy); h is reused for it
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int i = (it * kThreads + tid) * 8;
        const int hq = kHoist ? it : 0;
        if (!kHoist) {
            const int ic = i < d ? i : 0;
            gq[0][0] = *(const float4 *)(m.gamma + ic);
            gq[0][1] = *(const float4 *)(m.gamma + ic + 4);
            bq[0][0] = *(const float4 *)(m.beta + ic);
            bq[0][1] = *(const float4 *)(m.beta + ic + 4);
        }
        const float gv[8] = {gq[hq][0].x, gq[hq][0].y, gq[hq][0].z, gq[hq][0].w, gq[hq][1].x, gq[hq][1].y, gq[hq][1].z, gq[hq][1].w};
        const float bv[8] = {bq[hq][0].x, bq[hq][0].y, bq[hq][0].z, bq[hq][0].w, bq[hq][1].x, bq[hq][1].y, bq[hq][1].z, bq[hq][1].w};
        uint32_t packed[4];
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            const float s0 = gelu_erf((h[it][j] - mean) * rstd * gv[j] + bv[j]);
            const float s1 = gelu_erf((h[it][j + 1] - mean) * rstd * gv[j + 1] + bv[j + 1]);
            packed[j >> 1] = float_to_bf16_bits(s0) | (float_to_bf16_bits(s1) << 16);
            h[it][j] = i < d ? __uint_as_float(packed[j >> 1] << 16) : 0.0f;
            h[it][j + 1] = i < d ? __uint_as_float(packed[j >> 1] & 0xffff0000u) : 0.0f;
            amax = fmaxf(amax, fmaxf(fabsf(h[it][j]), fabsf(h[it][j + 1])));
        }
        if (i < d) *(uint4 *)(m.S_out + (size_t)r * d + i) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    }
    if (m.S8_out != nullptr) {   // uniform over the group
        const float scale = row_scale_of(group_max<kThreads, Sync>(amax, red, tid));
        const float inv = 1.0f / scale;
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int i = (it * kThreads + tid) * 8;
            if (i < d) *(uint2 *)(m.S8_out + (size_t)r * d + i) = e4m3x8(h[it], inv);
        }
        if (tid == 0) m.s8_scale[r] = scale;
    }
}

// (value desc, token id asc) ordering of candidates.
// Written without short-circuit operators and the exchanges below as selects: with "||" / "&&" and an "if"
// around the swap every comparison became a data-dependent branch that diverges inside the warp, and one
// 8-entry list took 2000-6000 cycles to fold instead of a few hundred.
__device__ __forceinline__ bool better(float v, int i, float w, int j) { return (v > w) | ((v == w) & (i < j)); }

// The pair at (va, ia) and the pair at (vb, ib) swap places unless the first is already the better one.
__device__ __forceinline__ void order_pair(float &va, int &ia, float &vb, int &ib) {
    const bool sw = better(vb, ib, va, ia);
    const float hv = sw ? vb : va, lv = sw ? va : vb;
    const int hi = sw ? ib : ia, li = sw ? ia : ib;
    va = hv; vb = lv;
    ia = hi; ib = li;
}

// Order-preserving map of a float (no NaN) onto unsigned integers, and back.
__device__ __forceinline__ uint32_t float_key(float v) {
    const uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Sorts one tile's list (8 slots, any order, slots >= topk ignored) best first with a fixed network and
// folds it into the sorted list (tv, ti): with both lists sorted, "the better of a[i] and b[7 - i]" keeps
// the best 8 of the 16 as a bitonic sequence, which three compare-exchange stages sort (depth 10 in all,
// where an insertion chain has 64).
__device__ __forceinline__ void fold_tile_list(float (&tv)[SPEC_MAX_TOPK], int (&ti)[SPEC_MAX_TOPK], const float4 &v0,
                                               const float4 &v1, const int4 &i0, const int4 &i1, int topk, bool valid) {
    constexpr int kT = SPEC_MAX_TOPK;
    static_assert(kT == 8, "the networks are written for lists of 8");
    float lv[kT] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    int li[kT] = {i0.x, i0.y, i0.z, i0.w, i1.x, i1.y, i1.z, i1.w};
#pragma unroll
    for (int j = 0; j < kT; ++j) {
        const bool none = (j >= topk) | !valid;   // slots past the list's length hold nothing
        lv[j] = none ? -INFINITY : lv[j];
        li[j] = none ? 0x7fffffff : li[j];
    }
    // 19-comparator sorting network for 8 inputs
#define SPEC_CX(a, b) order_pair(lv[a], li[a], lv[b], li[b])
    SPEC_CX(0, 2); SPEC_CX(1, 3); SPEC_CX(4, 6); SPEC_CX(5, 7);
    SPEC_CX(0, 4); SPEC_CX(1, 5); SPEC_CX(2, 6); SPEC_CX(3, 7);
    SPEC_CX(0, 1); SPEC_CX(2, 3); SPEC_CX(4, 5); SPEC_CX(6, 7);
    SPEC_CX(2, 4); SPEC_CX(3, 5);
    SPEC_CX(1, 4); SPEC_CX(3, 6);
    SPEC_CX(1, 2); SPEC_CX(3, 4); SPEC_CX(5, 6);
#undef SPEC_CX
#pragma unroll
    for (int j = 0; j < kT; ++j) {
        const bool take = better(lv[kT - 1 - j], li[kT - 1 - j], tv[j], ti[j]);
        tv[j] = take ? lv[kT - 1 - j] : tv[j];
        ti[j] = take ? li[kT - 1 - j] : ti[j];
    }
#pragma unroll
    for (int stride = kT / 2; stride > 0; stride >>= 1) {
#pragma unroll
        for (int j = 0; j < kT; ++j)
            if ((j & stride) == 0) order_pair(tv[j], ti[j], tv[j + stride], ti[j + stride]);
    }
}

__device__ __forceinline__ void fold_max_sum(float &m, float &s, const float2 &ms) {
    if (ms.x > m) {
        s = s * __expf(m - ms.x) + ms.y;   // exp(-inf) = 0 on the first tile
        m = ms.x;
    } else if (ms.x > -INFINITY) {
        s += ms.y * __expf(ms.x - m);
    }
}

// Thread t folds the lists of tiles t, t + kThreads, ... into one sorted list of 8 in registers, two
// tiles per trip with all ten loads issued before the first is used.  The group then extracts the
// `rounds` best (rounds <= kMaxRounds) in as many rounds; a round is two warp-wide integer reductions
// (redux.sync: maximum of the value keys, then minimum token id among the lanes that hold it) and one
// shared-memory exchange between the warps.  Results: sc->out_val / out_id (best first; exhausted slots
// hold -inf / 0x7fffffff) and sc->lse, valid for the whole group after the function returns.
template <int kThreads, typename Sync>
__device__ __forceinline__ void merge_select(const MergeArgs &g, int r, int tid, Scratch *sc, int rounds) {
    constexpr int kWarps = kThreads / 32;
    constexpr int kT = SPEC_MAX_TOPK;
    static_assert(kWarps <= kMaxGroupWarps, "scratch arrays");
    const int lane = tid & 31, warp = tid >> 5;
    const int n_tiles = g.n_tiles, topk = g.list_len > 0 ? g.list_len : g.topk;   // slots to read per list
    const float4 *pv4 = (const float4 *)(g.part_val + (size_t)r * n_tiles * kT);
    const int4 *pi4 = (const int4 *)(g.part_idx + (size_t)r * n_tiles * kT);
    const float2 *pms = (const float2 *)(g.part_ms + (size_t)r * n_tiles * 2);

    float tv[kT];
    int ti[kT];
#pragma unroll
    for (int j = 0; j < kT; ++j) {
        tv[j] = -INFINITY;
        ti[j] = 0x7fffffff;
    }
    float m = -INFINITY, s = 0.0f;
    for (int t = tid; t < n_tiles; t += 2 * kThreads) {
        const int t2 = t + kThreads;
        const bool has2 = t2 < n_tiles;
        const int tb = has2 ? t2 : t;
        const float2 ms_a = __ldcg(pms + t), ms_b = __ldcg(pms + tb);
        const float4 va0 = __ldcg(pv4 + 2 * t), va1 = __ldcg(pv4 + 2 * t + 1);
        const int4 ia0 = __ldcg(pi4 + 2 * t), ia1 = __ldcg(pi4 + 2 * t + 1);
        const float4 vb0 = __ldcg(pv4 + 2 * tb), vb1 = __ldcg(pv4 + 2 * tb + 1);
        const int4 ib0 = __ldcg(pi4 + 2 * tb), ib1 = __ldcg(pi4 + 2 * tb + 1);
        fold_max_sum(m, s, ms_a);
        if (has2) fold_max_sum(m, s, ms_b);
        fold_tile_list(tv, ti, va0, va1, ia0, ia1, topk, true);
        fold_tile_list(tv, ti, vb0, vb1, ib0, ib1, topk, has2);
    }
    // log-sum-exp of the whole row
    float wm = m;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, off));
    float ws = (m > -INFINITY) ? s * __expf(m - wm) : 0.0f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, off);
    Sync::sync();   // the scratch may still be read by a previous call
    if (lane == 0) {
        sc->red_m[warp] = wm;
        sc->red_s[warp] = ws;
    }
    Sync::sync();
    if (warp == 0) {   // one lane per warp's (max, sum): a second shuffle reduction
        const float pm = lane < kWarps ? sc->red_m[lane] : -INFINITY;
        const float ps = lane < kWarps ? sc->red_s[lane] : 0.0f;
        float bm = pm;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, off));
        float bs = pm > -INFINITY ? ps * __expf(pm - bm) : 0.0f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) bs += __shfl_xor_sync(0xffffffffu, bs, off);
        if (lane == 0) sc->lse = bm + logf(bs);
    }

    for (int j = 0; j < rounds; ++j) {
        const uint32_t my_key = float_key(tv[0]);
        const uint32_t wk = __reduce_max_sync(0xffffffffu, my_key);
        const uint32_t wi = __reduce_min_sync(0xffffffffu, my_key == wk ? (uint32_t)ti[0] : 0xffffffffu);
        if (lane == 0) {
            sc->cand_k[j & 1][warp] = wk;
            sc->cand_i[j & 1][warp] = (int)wi;
        }
        Sync::sync();   // rounds alternate between two buffers, so one barrier per round is enough
        // every warp reduces the warps' candidates again, one per lane: two more redux instead of a scan
        const uint32_t ck = lane < kWarps ? sc->cand_k[j & 1][lane] : 0u;
        const uint32_t ci = lane < kWarps ? (uint32_t)sc->cand_i[j & 1][lane] : 0xffffffffu;
        const uint32_t bk = __reduce_max_sync(0xffffffffu, ck);
        const int bi = (int)__reduce_min_sync(0xffffffffu, (lane < kWarps && ck == bk) ? ci : 0xffffffffu);
        if (ti[0] == bi && my_key == bk) {   // token ids are unique, so exactly one thread owns a real entry
#pragma unroll
            for (int q = 0; q < kT - 1; ++q) {
                tv[q] = tv[q + 1];
                ti[q] = ti[q + 1];
            }
            tv[kT - 1] = -INFINITY;
            ti[kT - 1] = 0x7fffffff;
        }
        if (tid == 0) {
            sc->out_val[j] = key_float(bk);
            sc->out_id[j] = bi;
        }
    }
    Sync::sync();
}

// The row's top-k tokens and log-probabilities become its children.
template <int kThreads, typename Sync>
__device__ __forceinline__ void merge_expand_row(const MergeArgs &g, int r, int tid, Scratch *sc) {
    const float base = (tid < g.topk && g.score_in && !g.lse_out) ? __ldcg(g.score_in + r) : 0.0f;   // in flight during the merge
    merge_select<kThreads, Sync>(g, r, tid, sc, g.topk);
    if (tid < g.topk) {
        g.tok_out[(size_t)r * g.topk + tid] = sc->out_id[tid];
        g.score_out[(size_t)r * g.topk + tid] = g.lse_out ? sc->out_val[tid] : base + (sc->out_val[tid] - sc->lse);
    }
    if (g.lse_out != nullptr && tid == 0) g.lse_out[r] = sc->lse;
}

// The children of one parent row, all at once: gather + mix + LayerNorm + exact GELU of up to kBatch child
// nodes per trip (Sec. 3.1: siblings share the projected parent state and differ in the token embedding).
// `tok` holds the children's tokens (shared memory, written by the merge just before), `first_child` is the
// row of child 0 in the next level.  The projected parent state (sum of the split-K partials, added in
// ascending order) and the LayerNorm parameters are loaded once; per trip the embedding rows of the batch
// are requested together and the two LayerNorm reductions are done for the whole batch with one barrier
// each (red_a / red_b: kThreads / 32 x kBatch floats each; kBatch children per trip).  d <= 8 * kThreads * kIters, d % 8 == 0.
template <int kThreads, int kIters, int kBatch, typename Sync>
__device__ __forceinline__ void mix_children(const MixArgs &m, int parent, int first_child, int n_child, const int *tok,
                                             float *red_a, float *red_b, int tid) {
    constexpr int kWarps = kThreads / 32;
    const int d = m.d, lane = tid & 31, warp = tid >> 5;
    float pv[kIters][8], gv[kIters][8], bv[kIters][8];
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int i = (it * kThreads + tid) * 8;
        const int ic = i < d ? i : 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) pv[it][j] = 0.0f;
        if (i < d) {
            const float *p = m.P + (size_t)parent * d + i;
            for (int sp = 0; sp < m.p_splits; ++sp) {
                const float4 p0 = __ldcg((const float4 *)(p + sp * m.p_split_stride));
                const float4 p1 = __ldcg((const float4 *)(p + sp * m.p_split_stride + 4));
                pv[it][0] += p0.x; pv[it][1] += p0.y; pv[it][2] += p0.z; pv[it][3] += p0.w;
                pv[it][4] += p1.x; pv[it][5] += p1.y; pv[it][6] += p1.z; pv[it][7] += p1.w;
            }
        }
        const float4 g0 = *(const float4 *)(m.gamma + ic), g1 = *(const float4 *)(m.gamma + ic + 4);
        const float4 b0 = *(const float4 *)(m.beta + ic), b1 = *(const float4 *)(m.beta + ic + 4);
        gv[it][0] = g0.x; gv[it][1] = g0.y; gv[it][2] = g0.z; gv[it][3] = g0.w;
        gv[it][4] = g1.x; gv[it][5] = g1.y; gv[it][6] = g1.z; gv[it][7] = g1.w;
        bv[it][0] = b0.x; bv[it][1] = b0.y; bv[it][2] = b0.z; bv[it][3] = b0.w;
        bv[it][4] = b1.x; bv[it][5] = b1.y; bv[it][6] = b1.z; bv[it][7] = b1.w;
    }
    for (int c0 = 0; c0 < n_child; c0 += kBatch) {
        float h[kBatch][kIters][8];
        float part[kBatch];
        uint4 ev[kBatch][kIters];
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            const int t = c0 + q < n_child ? tok[c0 + q] : -1;
            const bool tok_ok = t >= 0 && t < m.V;
            if (c0 + q < n_child && !tok_ok && tid == 0) report_error(m.err, SPEC_ERR_TOKEN_RANGE);
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                const int i = (it * kThreads + tid) * 8;
                ev[q][it] = make_uint4(0u, 0u, 0u, 0u);
                if (tok_ok && i < d) ev[q][it] = *(const uint4 *)(m.emb + (size_t)t * d + i);
            }
        }
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            part[q] = 0.0f;
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                const int i = (it * kThreads + tid) * 8;
                const uint32_t ew[4] = {ev[q][it].x, ev[q][it].y, ev[q][it].z, ev[q][it].w};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float z = (j & 1) ? __uint_as_float(ew[j >> 1] & 0xffff0000u) : __uint_as_float(ew[j >> 1] << 16);
                    h[q][it][j] = i < d ? m.a * pv[it][j] + m.b * z : 0.0f;
                    part[q] += h[q][it][j];
                }
            }
        }
        // batch-wide reductions: warp shuffles, one slot per (warp, child), then every thread adds the warps' slots
        float mean[kBatch], rstd[kBatch];
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
            float *red = pass == 0 ? red_a : red_b;
#pragma unroll
            for (int q = 0; q < kBatch; ++q) {
                float v = part[q];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                if (lane == 0) red[warp * kBatch + q] = v;
            }
            Sync::sync();
#pragma unroll
            for (int q = 0; q < kBatch; ++q) {
                float t = 0.0f;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) t += red[w * kBatch + q];
                if (pass == 0) {
                    mean[q] = t / (float)d;
                    part[q] = 0.0f;
#pragma unroll
                    for (int it = 0; it < kIters; ++it) {
                        const int i = (it * kThreads + tid) * 8;
                        if (i < d) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float c = h[q][it][j] - mean[q];
                                part[q] += c * c;
                            }
                        }
                    }
                } else {
                    rstd[q] = rsqrtf(t / (float)d + m.eps);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            if (c0 + q >= n_child) continue;
            const size_t row = (size_t)first_child + c0 + q;
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                const int i = (it * kThreads + tid) * 8;
                uint32_t packed[4];
#pragma unroll
                for (int j = 0; j < 8; j += 2) {
                    const float s0 = gelu_erf((h[q][it][j] - mean[q]) * rstd[q] * gv[it][j] + bv[it][j]);
                    const float s1 = gelu_erf((h[q][it][j + 1] - mean[q]) * rstd[q] * gv[it][j + 1] + bv[it][j + 1]);
                    packed[j >> 1] = float_to_bf16_bits(s0) | (float_to_bf16_bits(s1) << 16);
                }
                if (i < d) *(uint4 *)(m.S_out + row * d + i) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            }
        }
    }
}

struct LeafKey {
    float score;
    int leaf;
};

__device__ __forceinline__ bool leaf_before(const LeafKey &a, const LeafKey &b) {
    return (a.score > b.score) | ((a.score == b.score) & (a.leaf < b.leaf));
}

// Writes candidate `rank` of sequence b: its score and the tokens on the path from the root to `leaf`.
__device__ __forceinline__ void emit_candidate(const PruneArgs &pa, int L, int K, int32_t *cand_tok, float *cand_logp,
                                               int b, int rank, float score, int leaf) {
    cand_logp[(size_t)b * K + rank] = score;
    int idx = leaf;            // index among this sequence's nodes of level n
    int per_seq = L;           // nodes of this sequence at level l + 1
    for (int l = pa.n - 1; l >= 0; --l) {
        cand_tok[((size_t)b * K + rank) * pa.n + l] = __ldcg(pa.tok[l] + (size_t)b * per_seq + idx);
        idx /= pa.topk[l];
        per_seq /= pa.topk[l];
    }
}

// Tokens on the path from the root to `leaf` of sequence b, requested together (their addresses depend on the
// leaf index only, not on one another).
__device__ __forceinline__ void load_path(const PruneArgs &pa, int L, int b, int leaf, int32_t (&path)[SPEC_MAX_HEADS]) {
    int idx = leaf, per_seq = L;
#pragma unroll
    for (int l = SPEC_MAX_HEADS - 1; l >= 0; --l) {
        if (l < pa.n) {
            path[l] = __ldcg(pa.tok[l] + (size_t)b * per_seq + idx);
            idx /= pa.topk[l];
            per_seq /= pa.topk[l];
        }
    }
}

// Sequence b: the K best leaves by (score desc, leaf index asc), traced back to the root.  `keys`:
// shared memory for Lpad entries, Lpad the power of two >= max(L, 2).  Up to 256 leaves every thread
// counts how many leaves precede its own (that is its rank; no barriers) and has requested the tokens of its
// own leaves' paths together with the scores, so a kept leaf is written out without another trip to memory;
// longer lists are sorted bitonically.
template <int kThreads, typename Sync>
__device__ __forceinline__ void prune_sequence(const float *leaf_score, const PruneArgs &pa, int L, int Lpad, int K,
                                               int32_t *cand_tok, float *cand_logp, int b, int tid, LeafKey *keys) {
    constexpr int kOwn = 256 / kThreads > 0 ? 256 / kThreads : 1;   // leaves per thread in the ranked form
    int32_t path[kOwn][SPEC_MAX_HEADS];
    if (L <= 256) {
#pragma unroll
        for (int q = 0; q < kOwn; ++q)
            if (tid + q * kThreads < L) load_path(pa, L, b, tid + q * kThreads, path[q]);
    }
    Sync::sync();   // a previous call may still be reading the keys
    for (int i = tid; i < Lpad; i += kThreads) {
        keys[i].score = (i < L) ? __ldcg(leaf_score + (size_t)b * L + i) : -INFINITY;
        keys[i].leaf = i < L ? i : 0x7fffffff;
    }
    Sync::sync();
    if (L <= 256) {
#pragma unroll
        for (int q = 0; q < kOwn; ++q) {
            const int i = tid + q * kThreads;
            if (i >= L) continue;
            const LeafKey mine = keys[i];
            int rank = 0;
            for (int j = 0; j < L; ++j) rank += leaf_before(keys[j], mine) ? 1 : 0;
            if (rank < K) {
                cand_logp[(size_t)b * K + rank] = mine.score;
#pragma unroll
                for (int l = 0; l < SPEC_MAX_HEADS; ++l)
                    if (l < pa.n) cand_tok[((size_t)b * K + rank) * pa.n + l] = path[q][l];
            }
        }
        return;
    }
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
    for (int k = tid; k < K; k += kThreads)
        emit_candidate(pa, L, K, cand_tok, cand_logp, b, k, keys[k].score, keys[k].leaf);
}

// Prune folded into the kernel that writes the last level.  Every row's CTA makes its children visible
// (fence), then counts itself in for its sequence; the CTA that brings the count to rows_per_seq sees all
// of the sequence's leaves and prunes it.  No CTA ever waits for another.  `flag`: one shared int.
template <int kThreads, typename Sync>
__device__ __forceinline__ void prune_if_last(const MergeArgs &g, int r, int tid, LeafKey *keys, int *flag) {
    if (g.seq_done == nullptr) return;
    const int b = r / g.rows_per_seq;
    if (g.rows_per_seq > 1) {   // (a sequence of one row is complete with this CTA's own children)
        __threadfence();        // this CTA's children before its count
        Sync::sync();
        if (tid == 0) *flag = (atomicAdd(g.seq_done + b, 1) == g.rows_per_seq - 1) ? 1 : 0;
        Sync::sync();
        if (*flag == 0) return;
        __threadfence();        // the other CTAs' children after the last count
    } else {
        Sync::sync();
    }
    prune_sequence<kThreads, Sync>(g.score_out, g.prune, g.L, g.Lpad, g.K, g.cand_tok, g.cand_logp, b, tid, keys);
}

}  // namespace rows
}  // namespace spec
