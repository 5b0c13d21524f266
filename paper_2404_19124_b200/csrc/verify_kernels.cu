// Greedy multi-candidate verification (Sec. 1, Sec. 3.1, Sec. 5 of arXiv 2404.19124):
// a bandwidth-bound streaming arg-max over every row of the base model's logits followed by
// the longest-matching-prefix / best-candidate reduction.
//
// Kernel 1 (verify_stream_kernel): the whole tensor is one run of 16-byte vectors, cut into equal
//   contiguous ranges, one per warp, sized so that the grid is a single wave of resident CTAs on
//   every SM (no ragged second wave).  A warp walks the row segments inside its range with eight
//   128-bit streaming loads in flight per lane.  For bf16 the running maximum is taken on packed
//   pairs (max.bf16x2) and the element index is only resolved when a vector beats the lane's
//   current best, so the common case costs about one ALU operation per element.  Each (row, warp)
//   intersection writes one (value, index) partial into the row's slot list.
//   (verify_argmax_kernel is the scalar fallback for unaligned tensors or odd row lengths: fixed
//   chunks per row, one warp per chunk.)
// Kernel 2 (verify_accept_kernel): one CTA per sequence folds the partials of its K*(n+1)
//   rows into g[b,k,j], counts the matching prefix of every candidate and picks the best one.
#include <float.h>

#include <mutex>

#include "spec_common.cuh"

namespace spec {

namespace {

constexpr int kArgmaxThreads = 256;
constexpr int kWarpsPerBlock = kArgmaxThreads / 32;
constexpr int kIdxNone = 0x7fffffff;

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));   // a NaN operand is dropped
    return d;
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// best/idx: the lane's running (maximum, first index).  `base` is the index of element 0 of v.
__device__ __forceinline__ void consume_bf16(const uint4 &v, int base, float &best, int &idx) {
    uint32_t m2 = max_bf16x2(max_bf16x2(v.x, v.y), max_bf16x2(v.z, v.w));
    float mx = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xffff0000u));
    if (mx > best) {   // rare after the first few vectors
        best = mx;
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        int pos = 7;
#pragma unroll
        for (int i = 3; i >= 0; --i) {
            if (__uint_as_float(w[i] & 0xffff0000u) == mx) pos = 2 * i + 1;
            if (__uint_as_float(w[i] << 16) == mx) pos = 2 * i;
        }
        idx = base + pos;
    }
}

__device__ __forceinline__ void consume_f32(const uint4 &v, int base, float &best, int &idx) {
    const float f[4] = {__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z), __uint_as_float(v.w)};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (f[i] > best) {
            best = f[i];
            idx = base + i;
        }
    }
}

// (value desc, index asc) combine across the warp.
__device__ __forceinline__ void warp_argmax(float &best, int &idx) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        float ob = __shfl_xor_sync(0xffffffffu, best, off);
        int oi = __shfl_xor_sync(0xffffffffu, idx, off);
        const bool take = (ob > best) | ((ob == best) & (oi < idx));
        best = take ? ob : best;
        idx = take ? oi : idx;
    }
}

constexpr int kStreamUnroll = 8;

// vec_per_warp vectors per warp; row r owns vectors [r * vpr, (r + 1) * vpr); the partial of the
// (row, warp) intersection goes to slot  warp - first_warp(row)  of the row.
template <bool kBf16>
__global__ void __launch_bounds__(kArgmaxThreads, 4)
verify_stream_kernel(const uint4 *__restrict__ logits, long long total_vec, int vpr, int vec_per_warp, int slots,
                     float *pval, int32_t *pidx) {
    griddep_launch();
    griddep_wait();
    constexpr int kEpv = kBf16 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const long long beg = w * vec_per_warp;
    if (beg >= total_vec) return;
    const long long end = min(total_vec, beg + vec_per_warp);
    long long sb = beg;
    int row = (int)(beg / vpr);
    while (sb < end) {
        const long long row0 = (long long)row * vpr;
        const long long se = min(end, row0 + vpr);   // end of this row's segment inside the range
        float best = -INFINITY;
        int idx = kIdxNone;
        for (long long p0 = sb + lane; p0 < se; p0 += 32 * kStreamUnroll) {
            uint4 q[kStreamUnroll];
#pragma unroll
            for (int u = 0; u < kStreamUnroll; ++u)
                if (p0 + 32 * u < se) q[u] = ld_stream(logits + p0 + 32 * u);
#pragma unroll
            for (int u = 0; u < kStreamUnroll; ++u) {
                if (p0 + 32 * u < se) {
                    const int base = (int)(p0 + 32 * u - row0) * kEpv;
                    if (kBf16) consume_bf16(q[u], base, best, idx);
                    else consume_f32(q[u], base, best, idx);
                }
            }
        }
        warp_argmax(best, idx);
        if (lane == 0) {
            const long long first_w = row0 / vec_per_warp;
            const size_t slot = (size_t)row * slots + (size_t)(w - first_w);
            pval[slot] = best;
            pidx[slot] = idx;
        }
        sb = se;
        ++row;
    }
}

// Scalar fallback for tensors whose rows are not whole 16-byte vectors (or an unaligned base): fixed
// chunks per row, one warp per (row, chunk).
template <bool kBf16>
__global__ void __launch_bounds__(kArgmaxThreads)
verify_argmax_kernel(const void *__restrict__ logits, int rows, int V, int chunk_elems, int chunks,
                     float *__restrict__ pval, int32_t *__restrict__ pidx) {
    griddep_launch();
    griddep_wait();
    const int lane = threadIdx.x & 31;
    const long long unit = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (unit >= (long long)rows * chunks) return;
    const int row = (int)(unit / chunks), chunk = (int)(unit - (long long)row * chunks);
    const int begin = chunk * chunk_elems;
    const int count = min(chunk_elems, V - begin);
    constexpr int kEsz = kBf16 ? 2 : 4;
    const char *rp = (const char *)logits + ((size_t)row * V + begin) * kEsz;
    float best = -INFINITY;
    int idx = kIdxNone;
    for (int i = lane; i < count; i += 32) {
        const float x = kBf16 ? bf16_bits_to_float(((const uint16_t *)rp)[i]) : ((const float *)rp)[i];
        if (x > best) {
            best = x;
            idx = begin + i;
        }
    }
    warp_argmax(best, idx);
    if (lane == 0) {
        pval[unit] = best;
        pidx[unit] = idx;
    }
}

// (Everything an earlier kernel of the stream wrote - the partials, the candidates, the match lengths and the
// indices spec_next_ctx consumes - is read with ld.global.cg, never through the non-coherent path: these
// kernels start early under programmatic dependent launch and the same addresses are rewritten call after call.
// base_logits itself is streamed with ld.global.nc: it must be complete before the call is enqueued behind
// its producer on the stream, which stream order guarantees.)
__global__ void __launch_bounds__(128)
verify_accept_kernel(const int32_t *cand_tok, const float *pval, const int32_t *pidx, int K, int n, int slots, int vpr,
                     int vec_per_warp, int32_t *g_out, int g_in_smem, int32_t *accept_len, int32_t *best_cand,
                     int32_t *next_tok, int32_t *err) {
    // The sequence's arg-max table is re-read by other threads for the prefix match: from shared memory
    // when it fits the default 48 KB, otherwise from the copy in g_out this CTA has just written (global
    // writes of a CTA are visible to its own threads after the barrier).
    extern __shared__ int32_t g_s[];   // [K * (n + 1)] if g_in_smem
    __shared__ unsigned int key_s;
    const int b = blockIdx.x, rows_b = K * (n + 1);
    griddep_launch();
    griddep_wait();
    if (threadIdx.x == 0) {
        key_s = 0u;
        if (b == 0 && err != nullptr) *err = 0;
    }
    // The step is a handful of dependent round trips to L2, so every load that does not depend on another is
    // requested before the first one is used: the tokens of this thread's first candidate now, a row's partials
    // (values and indices alike) eight slots at a time.
    constexpr int kBatch = 8;
    int32_t ctok[SPEC_MAX_HEADS];
    {
        const int k0 = threadIdx.x;
#pragma unroll
        for (int j = 0; j < SPEC_MAX_HEADS; ++j)
            ctok[j] = (k0 < K && j < n) ? __ldcg(cand_tok + ((size_t)b * K + k0) * n + j) : -1;
    }
    for (int r = threadIdx.x; r < rows_b; r += blockDim.x) {
        const size_t gr = (size_t)b * rows_b + r;
        const size_t u0 = gr * slots;
        // streamed layout: the row's slots are the warps whose ranges intersect it
        int chunks = slots;
        if (vec_per_warp > 0)
            chunks = (int)(((long long)(gr + 1) * vpr - 1) / vec_per_warp - ((long long)gr * vpr) / vec_per_warp) + 1;
        float best = -INFINITY;
        int arg = 0;   // a row without any value above -inf (all NaN) yields 0
        for (int c0 = 0; c0 < chunks; c0 += kBatch) {
            float v[kBatch];
            int id[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const bool in = c0 + j < chunks;
                v[j] = in ? __ldcg(pval + u0 + c0 + j) : -INFINITY;
                id[j] = in ? __ldcg(pidx + u0 + c0 + j) : 0;
            }
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const bool take = v[j] > best;   // chunks ascend, so the first maximum wins
                best = take ? v[j] : best;
                arg = take ? id[j] : arg;
            }
        }
        if (g_in_smem) g_s[r] = arg;
        g_out[(size_t)b * rows_b + r] = arg;
    }
    __syncthreads();
    const int32_t *gtab = g_in_smem ? g_s : g_out + (size_t)b * rows_b;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const int32_t *gk = gtab + k * (n + 1);
        if (k != (int)threadIdx.x) {   // more candidates than threads: the later ones are fetched here
#pragma unroll
            for (int j = 0; j < SPEC_MAX_HEADS; ++j)
                ctok[j] = j < n ? __ldcg(cand_tok + ((size_t)b * K + k) * n + j) : -1;
        }
        int m = 0;
        bool open = true;
#pragma unroll
        for (int j = 0; j < SPEC_MAX_HEADS; ++j) {
            open = open && j < n && ctok[j] == gk[j];
            m += open ? 1 : 0;
        }
        if (open && n > SPEC_MAX_HEADS) {   // longer candidates than the registers hold: one token at a time
            const int32_t *c = cand_tok + ((size_t)b * K + k) * n;
            while (m < n && __ldcg(c + m) == gk[m]) ++m;
        }
        // longest prefix first, then the lowest candidate index
        atomicMax(&key_s, ((unsigned)m << 16) | (unsigned)(0xffff - k));
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int m = (int)(key_s >> 16), k = 0xffff - (int)(key_s & 0xffffu);
        accept_len[b] = m;
        best_cand[b] = k;
        next_tok[b] = gtab[k * (n + 1) + m];
    }
}

// ---- early-exit form ------------------------------------------------------------------------------
// The rows of a candidate matter only up to its first mismatch (Sec. 1: the tokens after a rejected
// one are discarded), so reading them is optional work: one CTA per candidate walks its rows in order,
// takes the arg-max of a row with the whole CTA (eight 128-bit loads in flight per thread) and stops
// after the first row whose arg-max differs from the speculated token.  Bytes read fall from
// B K (n+1) V to sum over candidates of (m + 1) V elements; rows that were not read get g = -1.
template <bool kBf16>
__global__ void __launch_bounds__(kArgmaxThreads)
verify_early_kernel(const uint4 *__restrict__ logits, const int32_t *cand_tok, int n, int vpr, int32_t *g,
                    int32_t *match_len) {
    __shared__ float s_val[kWarpsPerBlock];
    __shared__ int s_idx[kWarpsPerBlock];
    __shared__ int s_arg;
    griddep_launch();
    griddep_wait();
    constexpr int kEpv = kBf16 ? 8 : 4;
    const int c = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int m = n, j = 0;
    for (; j <= n; ++j) {
        const uint4 *rp = logits + ((size_t)c * (n + 1) + j) * vpr;
        float best = -INFINITY;
        int idx = kIdxNone;
        for (int p0 = tid; p0 < vpr; p0 += kArgmaxThreads * kStreamUnroll) {
            uint4 q[kStreamUnroll];
#pragma unroll
            for (int u = 0; u < kStreamUnroll; ++u)
                if (p0 + kArgmaxThreads * u < vpr) q[u] = ld_stream(rp + p0 + kArgmaxThreads * u);
#pragma unroll
            for (int u = 0; u < kStreamUnroll; ++u) {
                if (p0 + kArgmaxThreads * u < vpr) {
                    const int base = (p0 + kArgmaxThreads * u) * kEpv;
                    if (kBf16) consume_bf16(q[u], base, best, idx);
                    else consume_f32(q[u], base, best, idx);
                }
            }
        }
        warp_argmax(best, idx);
        if (lane == 0) {
            s_val[warp] = best;
            s_idx[warp] = idx;
        }
        __syncthreads();
        if (tid == 0) {
            float bv = -INFINITY;
            int arg = 0;   // a row without any value above -inf (all NaN) yields 0
            int bi = kIdxNone;
            for (int w = 0; w < kWarpsPerBlock; ++w) {
                if (s_val[w] > bv || (s_val[w] == bv && s_idx[w] < bi)) {   // the lowest index among equal maxima
                    bv = s_val[w];
                    bi = s_idx[w];
                }
            }
            if (bi != kIdxNone && bv > -INFINITY) arg = bi;
            s_arg = arg;
            g[(size_t)c * (n + 1) + j] = arg;
        }
        __syncthreads();
        const int arg = s_arg;
        if (j < n && __ldcg(cand_tok + (size_t)c * n + j) != arg) {   // uniform over the CTA
            m = j;
            break;
        }
    }
    for (int jj = j + 1 + tid; jj <= n; jj += kArgmaxThreads) g[(size_t)c * (n + 1) + jj] = -1;
    if (tid == 0) match_len[c] = m;
}

// One CTA per sequence: the candidate with the longest match (lowest index among equals) and its bonus token.
__global__ void __launch_bounds__(128)
verify_accept_early_kernel(const int32_t *g, const int32_t *match_len, int K, int n, int32_t *accept_len,
                           int32_t *best_cand, int32_t *next_tok, int32_t *err) {
    __shared__ unsigned int key_s;
    griddep_launch();
    griddep_wait();
    const int b = blockIdx.x;
    if (threadIdx.x == 0) {
        key_s = 0u;
        if (b == 0 && err != nullptr) *err = 0;
    }
    __syncthreads();
    for (int k = threadIdx.x; k < K; k += blockDim.x)
        atomicMax(&key_s, ((unsigned)__ldcg(match_len + (size_t)b * K + k) << 16) | (unsigned)(0xffff - k));
    __syncthreads();
    if (threadIdx.x == 0) {
        const int m = (int)(key_s >> 16), k = 0xffff - (int)(key_s & 0xffffu);
        accept_len[b] = m;
        best_cand[b] = k;
        next_tok[b] = __ldcg(g + ((size_t)b * K + k) * (n + 1) + m);
    }
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

// Resident CTAs per SM of the streaming kernel (launch bound above) times the SM count gives the
// number of warps of one full wave; every warp gets an equal range of at least one unrolled trip.
VerifyPlan make_verify_plan(int B, int K, int n, int V, int dtype) {
    VerifyPlan p{};
    p.rows = B * K * (n + 1);
    const int esz = dtype == SPEC_BF16 ? 2 : 4;
    const int epv = 16 / esz;
    // scalar fallback layout (also the upper bound used for the workspace when V % epv != 0)
    {
        const int gran = 32 * 4 * epv;
        const long long target_units = (long long)num_sms() * 64 * 2;
        int chunks = (int)((target_units + p.rows - 1) / p.rows);
        const int max_chunks = (V + gran - 1) / gran;
        if (chunks > max_chunks) chunks = max_chunks;
        if (chunks < 1) chunks = 1;
        const int per = (V + chunks - 1) / chunks;
        p.chunk_elems = (per + gran - 1) / gran * gran;
        p.chunks = (V + p.chunk_elems - 1) / p.chunk_elems;
    }
    p.vpr = 0;
    p.vec_per_warp = 0;
    p.slots = p.chunks;
    if (V % epv == 0) {
        p.vpr = V / epv;
        const long long total = (long long)p.rows * p.vpr;
        const long long wave_warps = (long long)num_sms() * 4 * kWarpsPerBlock;
        long long c = (total + wave_warps - 1) / wave_warps;
        const long long min_c = 32 * kStreamUnroll;
        if (c < min_c) c = min_c;
        if (c > (1ll << 30)) c = 1ll << 30;
        p.vec_per_warp = (int)c;
        const int stream_slots = (int)((p.vpr + c - 1) / c) + 1;
        if (stream_slots > p.slots) p.slots = stream_slots;
    }
    p.off_g = kWsAlign;
    p.off_pval = align_up(p.off_g + sizeof(int32_t) * (size_t)p.rows, kWsAlign);
    p.off_pidx = align_up(p.off_pval + sizeof(float) * (size_t)p.rows * p.slots, kWsAlign);
    p.total = align_up(p.off_pidx + sizeof(int32_t) * (size_t)p.rows * p.slots, kWsAlign);
    return p;
}

int launch_verify(const int32_t *cand_tok, const void *base_logits, int dtype, int B, int K, int n, int V,
                  int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *ws, const VerifyPlan &plan,
                  cudaStream_t st) {
    char *w = (char *)ws;
    int32_t *err = (int32_t *)w;
    int32_t *g = (int32_t *)(w + plan.off_g);
    float *pval = (float *)(w + plan.off_pval);
    int32_t *pidx = (int32_t *)(w + plan.off_pidx);
    const bool stream = plan.vec_per_warp > 0 && ((uintptr_t)base_logits % 16 == 0);
    int vec_per_warp = 0;
    if (stream) {
        vec_per_warp = plan.vec_per_warp;
        const long long total = (long long)plan.rows * plan.vpr;
        const long long warps = (total + vec_per_warp - 1) / vec_per_warp;
        const unsigned grid = (unsigned)((warps + kWarpsPerBlock - 1) / kWarpsPerBlock);
        const uint4 *lp = (const uint4 *)base_logits;
        if (dtype == SPEC_BF16)
            SPEC_CUDA_TRY(launch_pdl(verify_stream_kernel<true>, dim3(grid), dim3(kArgmaxThreads), 0, st, lp, total,
                                     plan.vpr, vec_per_warp, plan.slots, pval, pidx));
        else
            SPEC_CUDA_TRY(launch_pdl(verify_stream_kernel<false>, dim3(grid), dim3(kArgmaxThreads), 0, st, lp, total,
                                     plan.vpr, vec_per_warp, plan.slots, pval, pidx));
    } else {
        // scalar fallback; its partials use the first plan.chunks slots of every row, laid out with
        // plan.chunks as the row pitch
        const long long units = (long long)plan.rows * plan.chunks;
        const unsigned grid = (unsigned)((units + kWarpsPerBlock - 1) / kWarpsPerBlock);
        if (dtype == SPEC_BF16)
            SPEC_CUDA_TRY(launch_pdl(verify_argmax_kernel<true>, dim3(grid), dim3(kArgmaxThreads), 0, st,
                                     base_logits, plan.rows, V, plan.chunk_elems, plan.chunks, pval, pidx));
        else
            SPEC_CUDA_TRY(launch_pdl(verify_argmax_kernel<false>, dim3(grid), dim3(kArgmaxThreads), 0, st,
                                     base_logits, plan.rows, V, plan.chunk_elems, plan.chunks, pval, pidx));
    }
    size_t smem = sizeof(int32_t) * (size_t)K * (n + 1);
    const int g_in_smem = smem <= 40 * 1024;
    if (!g_in_smem) smem = 0;
    SPEC_CUDA_TRY(launch_pdl(verify_accept_kernel, dim3(B), dim3(128), smem, st, cand_tok, (const float *)pval,
                             (const int32_t *)pidx, K, n, stream ? plan.slots : plan.chunks, plan.vpr, vec_per_warp,
                             g, g_in_smem, accept_len, best_cand, next_tok, err));
    return SPEC_OK;
}

// Early-exit form; returns SPEC_ERR_SHAPE when the rows are not whole 16-byte vectors (the caller then
// uses the streaming form).
int launch_verify_early(const int32_t *cand_tok, const void *base_logits, int dtype, int B, int K, int n, int V,
                        int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *ws, const VerifyPlan &plan,
                        cudaStream_t st) {
    if (plan.vpr <= 0 || ((uintptr_t)base_logits % 16) != 0) return SPEC_ERR_SHAPE;
    char *w = (char *)ws;
    int32_t *err = (int32_t *)w;
    int32_t *g = (int32_t *)(w + plan.off_g);
    int32_t *match_len = (int32_t *)(w + plan.off_pval);   // B * K words; the partial-maxima area is not used here
    const uint4 *lp = (const uint4 *)base_logits;
    if (dtype == SPEC_BF16)
        SPEC_CUDA_TRY(launch_pdl(verify_early_kernel<true>, dim3(B * K), dim3(kArgmaxThreads), 0, st, lp, cand_tok, n,
                                 plan.vpr, g, match_len));
    else
        SPEC_CUDA_TRY(launch_pdl(verify_early_kernel<false>, dim3(B * K), dim3(kArgmaxThreads), 0, st, lp, cand_tok, n,
                                 plan.vpr, g, match_len));
    SPEC_CUDA_TRY(launch_pdl(verify_accept_early_kernel, dim3(B), dim3(128), 0, st, (const int32_t *)g,
                             (const int32_t *)match_len, K, n, accept_len, best_cand, next_tok, err));
    return SPEC_OK;
}

}  // namespace spec

// ---- spec_next_ctx: the state vector the next draft starts from (Sec. 3.1) ----------------------
namespace spec {
namespace {

// One CTA per sequence copies base_state[b, best_cand[b], accept_len[b], :] to ctx_state[b, :].  The two
// indices come from the verify kernels earlier in the stream, hence the dependency wait before they are read.
__global__ void __launch_bounds__(128)
next_ctx_kernel(const uint16_t *__restrict__ base_state, const int32_t *best_cand, const int32_t *accept_len, int K,
                int n, int d, int vec_ok, uint16_t *__restrict__ ctx_state, int32_t *err) {
    griddep_launch();
    griddep_wait();
    const int b = blockIdx.x;
    const int k = __ldcg(best_cand + b), m = __ldcg(accept_len + b);
    uint16_t *dst = ctx_state + (size_t)b * d;
    if (k < 0 || k >= K || m < 0 || m > n) {   // never read outside the tensor: the row becomes zero
        if (threadIdx.x == 0) report_error(err, SPEC_ERR_INDEX_RANGE);
        for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = 0;
        return;
    }
    const uint16_t *src = base_state + (((size_t)b * K + k) * (n + 1) + m) * d;
    if (vec_ok) {
        const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
        uint4 *d4 = reinterpret_cast<uint4 *>(dst);
        for (int i = threadIdx.x; i < d / 8; i += blockDim.x) d4[i] = s4[i];
    } else {
        for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = src[i];
    }
}

}  // namespace
}  // namespace spec

extern "C" int spec_next_ctx(const void *base_state, const int32_t *best_cand, const int32_t *accept_len, int B, int K,
                             int n, int d_base, void *ctx_state, int32_t *err_word, void *cuda_stream) {
    using namespace spec;
    if (!base_state || !best_cand || !accept_len || !ctx_state) return SPEC_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || n <= 0 || d_base <= 0) return SPEC_ERR_INVALID_ARG;
    if (((uintptr_t)base_state % 2) != 0 || ((uintptr_t)ctx_state % 2) != 0) return SPEC_ERR_INVALID_ARG;
    if (err_word && ((uintptr_t)err_word % 4) != 0) return SPEC_ERR_INVALID_ARG;
    const int vec_ok = (d_base % 8 == 0) && ((uintptr_t)base_state % 16) == 0 && ((uintptr_t)ctx_state % 16) == 0;
    SPEC_CUDA_TRY(launch_pdl(next_ctx_kernel, dim3((unsigned)B), dim3(128), 0, (cudaStream_t)cuda_stream,
                             (const uint16_t *)base_state, best_cand, accept_len, K, n, d_base, vec_ok,
                             (uint16_t *)ctx_state, err_word));
    return SPEC_OK;
}

// ---- spec_verify_static: the verify scratch lives in the library's own device image ------------
// For hosts that cannot give the library a workspace (all device memory already committed to their
// own pools, or no allocation allowed where this runs).  Inside host code the array's name is only a
// handle for the runtime, not a device address: the address each device mapped it to is asked for
// once per device with cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_verify_static_scratch[SPEC_VERIFY_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices] = {};
}  // namespace

extern "C" int spec_verify_static(const int32_t *cand_tok, const void *base_logits, int logits_dtype, int B, int K,
                                  int n, int V, int32_t *accept_len, int32_t *best_cand, int32_t *next_tok,
                                  void *cuda_stream) {
    using namespace spec;
    if (!cand_tok || !base_logits || !accept_len || !best_cand || !next_tok) return SPEC_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || n <= 0 || V <= 0) return SPEC_ERR_INVALID_ARG;
    if (logits_dtype != SPEC_BF16 && logits_dtype != SPEC_F32) return SPEC_ERR_INVALID_ARG;
    if (K > 65535 || (long long)K * (n + 1) > 12288 || n > 32767) return SPEC_ERR_SHAPE;
    if ((long long)B * K * (n + 1) > (1ll << 30)) return SPEC_ERR_SHAPE;
    if (((uintptr_t)base_logits % (logits_dtype == SPEC_BF16 ? 2 : 4)) != 0) return SPEC_ERR_INVALID_ARG;
    const VerifyPlan plan = make_verify_plan(B, K, n, V, logits_dtype);
    if (plan.total > (size_t)SPEC_VERIFY_STATIC_SCRATCH_BYTES) return SPEC_ERR_STATIC_SCRATCH;

    int dev = -1;
    SPEC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SPEC_ERR_NO_DEVICE;
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (g_static_ptr[dev] == nullptr) {
            // first call on this device (which is current): where did this device map the array?
            void *ptr = nullptr;
            SPEC_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_verify_static_scratch));
            if (ptr == nullptr || ((uintptr_t)ptr % kWsAlign) != 0) return SPEC_ERR_WORKSPACE;
            g_static_ptr[dev] = ptr;
        }
        scratch = g_static_ptr[dev];
    }
    return launch_verify(cand_tok, base_logits, logits_dtype, B, K, n, V, accept_len, best_cand, next_tok, scratch, plan,
                         (cudaStream_t)cuda_stream);
}

