// C ABI of libspec_b200: host-side validation, workspace layout and the launch sequences of
// spec_draft / spec_verify (declared and documented in include/spec_b200.h).
#include <atomic>
#include <new>
#include <string.h>

#include "spec_common.cuh"

namespace spec {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }

int num_sms() {
    static std::atomic<int> cached[64];   // zero-initialised; any thread may fill an entry, all write the same value
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return kNumSMsFallback;
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = kNumSMsFallback;
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

}  // namespace spec

using namespace spec;

constexpr int kMaxProfEvents = 4 * SPEC_MAX_HEADS + 2;

struct spec_handle_s {
    spec_weights_t w;
    int gemm_impl;
    int head_block_n;
    int proj_block_n;
    int profile;
    int fp8_max_rows;                      // SPEC_OPT_FP8_MAX_ROWS
    int swap_max_rows;                     // SPEC_OPT_HEAD_SWAP_MAX_ROWS
    int head_pair;                         // SPEC_OPT_HEAD_PAIR
    const void *head8[SPEC_MAX_HEADS];     // e4m3 copies of the heads (caller-owned), null: none
    const float *head8_scale[SPEC_MAX_HEADS];
    int vp_rank, vp_ranks;                 // vocabulary-parallel heads: this handle's shard (vp_ranks 1: none)
    int vocab_offset, head_rows;           // its head matrices hold vocabulary rows [vocab_offset, +head_rows)
    int prof_count;                        // events recorded by the last profiled draft
    cudaEvent_t prof_ev[kMaxProfEvents];   // created when profiling is switched on
};

namespace {

constexpr int kFusedMixMaxChildren = 2;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int d_in_of(const spec_weights_t &w, int l) { return l == 0 ? w.d_base : w.d_inner; }

// Shapes of one draft call and where everything lives in the workspace.
struct DraftPlan {
    int n;
    int N[SPEC_MAX_HEADS + 1];   // nodes per level
    int L;
    spec_draft_layout_t lay;
    int proj_block_n[SPEC_MAX_HEADS];
    int proj_splits[SPEC_MAX_HEADS];   // > 0: swapped split-K projection (few parent rows); 0: plain
    bool use_fp8[SPEC_MAX_HEADS];      // the level's head runs on the e4m3 copy of its weights
    bool swapped[SPEC_MAX_HEADS];      // the level's head runs with the operands swapped (few nodes: weight stream)
    bool paired[SPEC_MAX_HEADS];       // the level's head runs on CTA pairs (more than 128 nodes: tensor-bound)
    size_t seq_done;                   // byte offset of the per-sequence counters of the folded prune
    int header_words;                  // int32 words cleared at the start of a draft
    size_t xchg;                       // vocabulary-parallel heads: byte offset of the rank slots
    size_t slot_bytes[SPEC_MAX_HEADS]; // bytes of one rank's slot at each level
};

int head_block_n_for(const spec_handle_s *h, int rows) {
    if (h->head_block_n > 0) return h->head_block_n;
    return choose_block_n(rows, h->head_rows, num_sms(), rows > 128);
}

// Levels of few nodes run the head with the weights on the 128-row side of the MMA (epilogue mode 3).
// Which levels: set explicitly, or by what measured faster inside whole drafts.  The swapped form costs fewer
// TMA requests and MMA cycles per weight byte but ends every CTA with a longer epilogue (transposition, scan,
// combination of the segment lists), which only a long weight stream pays back: up to 8 nodes at any
// vocabulary, up to 32 nodes when every CTA streams at least four 128-row tiles (V = 128256: 121 against
// 137 us at 16 nodes); at 16 nodes and V = 32000 the one-thread-per-node form is 2-3 us per level faster.
bool head_swapped_for(const spec_handle_s *h, int rows) {
    if (h->gemm_impl != 0 || h->head_block_n != 0 || rows > 128) return false;
    if (h->swap_max_rows >= 0) return rows <= h->swap_max_rows;
    return rows <= 8 || (rows <= 32 && h->head_rows >= 4 * 128 * num_sms());
}

// Levels of more than 128 nodes (several 128-row tiles per weight tile) may run on CTA pairs.
// A pair's tile has 256 node rows, so a level whose row count is not a multiple of 256 pays for the padding:
// 384 rows run as 512 (measured 100 against 88 us, V = 32000), 256 / 512 / 768 / 2048 / 6144 rows gain 4-9 %.
// Automatic: at most a tenth of padding (233-256 rows, 466-512, 699-768, ...).
bool head_paired_for(const spec_handle_s *h, int rows) {
    if (h->gemm_impl != 0 || h->head_block_n != 0 || rows <= 128 || h->head_pair == 0) return false;
    if (h->head_pair == 1) return true;
    const int padded = (rows + 255) / 256 * 256;
    return 10 * padded <= 11 * rows;
}

// Partial lists per row that the head of `rows` nodes leaves for the merge, and its tile width.
int head_parts_for(const spec_handle_s *h, int rows, bool swapped, int *block_n_out) {
    if (head_paired_for(h, rows)) {
        const int bn = pair_block_n(rows, h->head_rows);
        if (block_n_out) *block_n_out = bn;
        return (h->head_rows + bn - 1) / bn;
    }
    if (swapped) {
        if (block_n_out) *block_n_out = 128;
        return swapped_head_parts(rows, h->head_rows);
    }
    const int bn = head_block_n_for(h, rows);
    if (block_n_out) *block_n_out = bn;
    return (h->head_rows + bn - 1) / bn;
}

int proj_block_n_for(const spec_handle_s *h, int rows) {
    if (h->proj_block_n > 0) return h->proj_block_n;
    return choose_block_n(rows, h->w.d_inner, num_sms(), rows > 128);
}

// Projection with at most 128 parent rows: the weight matrix takes the 128-row side of the MMA,
// the states the narrow side, and the contraction is cut into as many K ranges as keep every SM
// busy (each range at least four 64-wide K blocks).  Returns 0 when the plain form is used.
int proj_splits_for(const spec_handle_s *h, int parent_rows, int d_in) {
    if (h->gemm_impl != 0 || parent_rows > 128 || h->proj_block_n > 0) return 0;
    const int m_tiles = (h->w.d_inner + 127) / 128, num_kb = (d_in + 63) / 64;
    int splits = num_sms() / m_tiles;
    if (splits > num_kb / 4) splits = num_kb / 4;
    if (splits > 8) splits = 8;
    if (splits < 1) splits = 1;
    const int per = (num_kb + splits - 1) / splits;
    return (num_kb + per - 1) / per;   // no empty range
}

int make_draft_plan(const spec_handle_s *h, int B, const int32_t *topk, int K, DraftPlan *p) {
    if (!h || !topk || !p) return SPEC_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0) return SPEC_ERR_INVALID_ARG;
    const spec_weights_t &w = h->w;
    memset(p, 0, sizeof(*p));
    p->n = w.n_heads;
    long long nodes = B, leaves = 1;
    p->N[0] = B;
    for (int l = 0; l < p->n; ++l) {
        if (topk[l] < 1 || topk[l] > SPEC_MAX_TOPK || topk[l] > h->head_rows) return SPEC_ERR_SHAPE;
        leaves *= topk[l];
        nodes *= topk[l];
        if (leaves > SPEC_MAX_LEAVES || nodes > (1ll << 24)) return SPEC_ERR_SHAPE;
        p->N[l + 1] = (int)nodes;
    }
    if (K > leaves) return SPEC_ERR_SHAPE;
    p->L = (int)leaves;

    spec_draft_layout_t &y = p->lay;
    // header: the error word at offset 0, one int32 counter per sequence from byte 256 on
    y.error_word = 0;
    p->seq_done = kWsAlign;
    p->header_words = (int)(kWsAlign / sizeof(int32_t)) + B;
    size_t off = align_up(kWsAlign + sizeof(int32_t) * (size_t)B, kWsAlign);
    // vocabulary-parallel heads: one slot per rank for the lists that are exchanged after every level.  It
    // comes first so that its offset is the same on every rank (what follows depends on the shard's size).
    p->xchg = off;
    if (h->vp_ranks > 1) {
        size_t max_slot = 0;
        for (int l = 0; l < p->n; ++l) {
            p->slot_bytes[l] = align_up((size_t)p->N[l] * (8 * (size_t)topk[l] + 4), kWsAlign);
            if (p->slot_bytes[l] > max_slot) max_slot = p->slot_bytes[l];
        }
        off = align_up(off + max_slot * h->vp_ranks, kWsAlign);
    }
    for (int l = 1; l <= p->n; ++l) {
        y.tok[l] = off;
        off = align_up(off + sizeof(int32_t) * (size_t)p->N[l], kWsAlign);
        y.score[l] = off;
        off = align_up(off + sizeof(float) * (size_t)p->N[l], kWsAlign);
    }
    size_t max_proj_floats = 0;
    size_t max_part_units = 0;
    int max_rows = 0;
    int max_fp8_rows = 0;
    for (int l = 0; l < p->n; ++l) {
        // (the mix kernel for rows wider than 16384 elements keeps them in shared memory and has no e4m3 output)
        p->use_fp8[l] = h->gemm_impl == 0 && !h->profile && h->head8[l] != nullptr && p->N[l] <= h->fp8_max_rows &&
                        w.d_inner <= 16384 && h->vp_ranks == 1;
        if (p->use_fp8[l] && p->N[l] > max_fp8_rows) max_fp8_rows = p->N[l];
        p->swapped[l] = !p->use_fp8[l] && head_swapped_for(h, p->N[l]);
        p->paired[l] = !p->use_fp8[l] && !h->profile && head_paired_for(h, p->N[l]);
    }
    for (int l = 0; l < p->n; ++l) {
        y.state[l] = off;
        off = align_up(off + 2 * (size_t)p->N[l] * w.d_inner, kWsAlign);
        const int parent_rows = l == 0 ? B : p->N[l - 1];
        p->proj_splits[l] = proj_splits_for(h, parent_rows, d_in_of(w, l));
        const size_t pf = (size_t)(p->proj_splits[l] > 0 ? p->proj_splits[l] : 1) * parent_rows * w.d_inner;
        if (pf > max_proj_floats) max_proj_floats = pf;
        int bn = 0;
        y.n_tiles[l] = head_parts_for(h, p->N[l], p->swapped[l], &bn);
        y.block_n[l] = bn;
        const size_t units = (size_t)p->N[l] * y.n_tiles[l];
        if (units > max_part_units) max_part_units = units;
        if (p->N[l] > max_rows) max_rows = p->N[l];
        p->proj_block_n[l] = proj_block_n_for(h, parent_rows);
    }
    y.proj = off;
    off = align_up(off + sizeof(float) * max_proj_floats, kWsAlign);
    y.state8 = off;
    off = align_up(off + (size_t)max_fp8_rows * w.d_inner, kWsAlign);
    y.state8_scale = off;
    off = align_up(off + sizeof(float) * (size_t)max_fp8_rows, kWsAlign);
    y.part_val = off;
    off = align_up(off + sizeof(float) * max_part_units * SPEC_MAX_TOPK, kWsAlign);
    y.part_idx = off;
    off = align_up(off + sizeof(int32_t) * max_part_units * SPEC_MAX_TOPK, kWsAlign);
    y.part_ms = off;
    off = align_up(off + sizeof(float) * max_part_units * 2, kWsAlign);
    y.logits = off;
    if (h->gemm_impl == 1) off = align_up(off + sizeof(float) * (size_t)max_rows * w.V, kWsAlign);
    y.total_bytes = off;
    return SPEC_OK;
}

// One contraction through whichever implementation the handle selects.
int run_gemm_store(const spec_handle_s *h, const void *A, const void *Bm, int M, int N, int Kd, int block_n,
                   float *out, int32_t *err, cudaStream_t st) {
    if (h->gemm_impl == 1) return launch_gemm_simt(A, Bm, M, N, Kd, out, N, st);
    GemmEpilogue e{};
    e.mode = 0;
    e.out = out;
    e.ldc = N;
    return launch_gemm_tc(A, Bm, M, N, Kd, block_n, e, err, st);
}

int run_head_partials(const spec_handle_s *h, const void *states, const void *Wout, int rows, int block_n, int topk,
                      float *part_val, int32_t *part_idx, float *part_ms, float *logits_scratch, int32_t *err,
                      cudaStream_t st) {
    const spec_weights_t &w = h->w;
    if (h->gemm_impl == 1) {
        int rc = launch_gemm_simt(states, Wout, rows, w.V, w.d_inner, logits_scratch, w.V, st);
        if (rc != SPEC_OK) return rc;
        return launch_partials_from_logits(logits_scratch, rows, w.V, block_n, topk, part_val, part_idx, part_ms, st);
    }
    GemmEpilogue e{};
    e.mode = 1;
    e.part_val = part_val;
    e.part_idx = part_idx;
    e.part_ms = part_ms;
    e.topk = topk;
    if (head_paired_for(h, rows)) return launch_head_pair(states, Wout, rows, w.V, w.d_inner, block_n, e, err, st);
    if (head_swapped_for(h, rows)) {
        e.mode = 3;
        return launch_gemm_tc(Wout, states, w.V, rows, w.d_inner, (rows + 15) / 16 * 16, e, err, st);
    }
    return launch_gemm_tc(states, Wout, rows, w.V, w.d_inner, block_n, e, err, st);
}

// The head of level l inside a draft: plain form (one thread per node row of a [128 x block_n] tile), the
// swapped form for levels of few nodes, or e4m3 operands.
GemmCall make_head_call(const spec_handle_s *h, const DraftPlan &p, char *ws, int l, int topk_l) {
    const spec_weights_t &w = h->w;
    GemmCall c{};
    c.A = ws + p.lay.state[l]; c.B = w.head[l]; c.M = p.N[l]; c.N = h->head_rows; c.Kd = w.d_inner;
    c.block_n = p.lay.block_n[l];
    c.epi.mode = 1;
    c.epi.part_val = (float *)(ws + p.lay.part_val);
    c.epi.part_idx = (int32_t *)(ws + p.lay.part_idx);
    c.epi.part_ms = (float *)(ws + p.lay.part_ms);
    c.epi.topk = topk_l;
    c.epi.idx_offset = h->vocab_offset;
    if (p.use_fp8[l]) {   // e4m3 operands; every tile keeps SPEC_MAX_TOPK candidates by approximate logit
        c.A = ws + p.lay.state8;
        c.B = h->head8[l];
        c.epi.fp8 = 1;
        c.epi.topk = SPEC_MAX_TOPK;
        c.epi.row_scale = (const float *)(ws + p.lay.state8_scale);
        c.epi.col_scale = h->head8_scale[l];
    } else if (p.swapped[l]) {
        c.A = w.head[l]; c.M = h->head_rows;
        c.B = ws + p.lay.state[l]; c.N = p.N[l];
        c.block_n = (p.N[l] + 15) / 16 * 16;
        c.epi.mode = 3;
    }
    return c;
}

// State projection of level l as a tensor-core contraction: with few parent rows the weights take the
// 128-row side and split-K partials are stored transposed, otherwise the plain form.
GemmCall make_proj_call(const spec_handle_s *h, const DraftPlan &p, char *ws, const void *ctx_state, int B, int l) {
    const spec_weights_t &w = h->w;
    const int parent_rows = l == 0 ? B : p.N[l - 1];
    const void *parent_states = l == 0 ? ctx_state : (const void *)(ws + p.lay.state[l - 1]);
    GemmCall c{};
    c.Kd = d_in_of(w, l);
    c.epi.out = (float *)(ws + p.lay.proj);
    c.epi.ldc = w.d_inner;
    if (p.proj_splits[l] > 0) {
        c.A = w.proj[l]; c.M = w.d_inner;
        c.B = parent_states; c.N = parent_rows;
        c.block_n = (parent_rows + 31) / 32 * 32;
        c.epi.mode = 2;
        c.epi.splits = p.proj_splits[l];
        c.epi.split_stride = (size_t)parent_rows * w.d_inner;
    } else {
        c.A = parent_states; c.M = parent_rows;
        c.B = w.proj[l]; c.N = w.d_inner;
        c.block_n = p.proj_block_n[l];
        c.epi.mode = 0;
    }
    return c;
}

// Arguments of the gather + mix + LayerNorm + GELU step of level l (bf16 states only).
MixArgs make_mix_args(const spec_handle_s *h, const DraftPlan &p, char *ws, const int32_t *last_tok, int B,
                      const int32_t *topk, int l, int32_t *err) {
    const spec_weights_t &w = h->w;
    const int parent_rows = l == 0 ? B : p.N[l - 1];
    MixArgs mx{};
    mx.P = (float *)(ws + p.lay.proj);
    mx.p_splits = p.proj_splits[l] > 0 ? p.proj_splits[l] : 1;
    mx.p_split_stride = (size_t)parent_rows * w.d_inner;
    mx.emb = (const uint16_t *)w.emb[l];
    mx.tok = l == 0 ? last_tok : (const int32_t *)(ws + p.lay.tok[l]);
    mx.gamma = w.ln_gamma[l]; mx.beta = w.ln_beta[l];
    mx.d = w.d_inner; mx.V = w.V; mx.parent_div = l == 0 ? 1 : topk[l - 1];
    mx.a = w.state_weight; mx.b = w.emb_weight; mx.eps = w.ln_eps;
    mx.S_out = (uint16_t *)(ws + p.lay.state[l]);
    mx.err = err;
    return mx;
}

PruneArgs make_prune_args(const DraftPlan &p, char *ws, const int32_t *topk) {
    PruneArgs pa{};
    pa.n = p.n;
    for (int l = 0; l < p.n; ++l) {
        pa.tok[l] = (const int32_t *)(ws + p.lay.tok[l + 1]);
        pa.topk[l] = topk[l];
    }
    return pa;
}

}  // namespace

extern "C" {

int spec_version(void) { return 1; }

const char *spec_status_str(int s) {
    switch (s) {
        case SPEC_OK: return "ok";
        case SPEC_ERR_INVALID_ARG: return "invalid argument";
        case SPEC_ERR_SHAPE: return "unsupported shape";
        case SPEC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SPEC_ERR_CUDA: return "CUDA call failed";
        case SPEC_ERR_TOKEN_RANGE: return "token id outside the vocabulary";
        case SPEC_ERR_TIMEOUT: return "bounded wait inside a kernel ran out";
        case SPEC_ERR_NO_DEVICE: return "no usable CUDA device";
        case SPEC_ERR_STATIC_SCRATCH: return "problem needs more scratch than the library's built-in array holds";
        case SPEC_ERR_INDEX_RANGE: return "device: best_cand or accept_len out of range in spec_next_ctx";
        default: return "unknown status";
    }
}

int spec_last_cuda_error(void) { return g_last_cuda_error; }

int spec_create(spec_handle_t *out, const spec_weights_t *w) {
    if (!out || !w) return SPEC_ERR_INVALID_ARG;
    *out = nullptr;
    if (w->n_heads < 1 || w->n_heads > SPEC_MAX_HEADS || w->V < 1 || w->d_base < 8 || w->d_inner < 8)
        return SPEC_ERR_SHAPE;
    if (w->d_base % 8 != 0 || w->d_inner % 8 != 0) return SPEC_ERR_SHAPE;   // 16-byte rows for TMA and vector loads
    for (int l = 0; l < w->n_heads; ++l) {
        const void *ptrs[5] = {w->emb[l], w->proj[l], w->ln_gamma[l], w->ln_beta[l], w->head[l]};
        for (const void *q : ptrs) {
            if (!q) return SPEC_ERR_INVALID_ARG;
            if ((uintptr_t)q & 15) return SPEC_ERR_INVALID_ARG;
        }
    }
    if (!(w->ln_eps > 0.0f)) return SPEC_ERR_INVALID_ARG;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || count <= 0) {
        (void)cudaGetLastError();
        return SPEC_ERR_NO_DEVICE;
    }
    int dev = 0, major = 0;
    SPEC_CUDA_TRY(cudaGetDevice(&dev));
    SPEC_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) return SPEC_ERR_NO_DEVICE;
    spec_handle_s *h = new (std::nothrow) spec_handle_s();
    if (!h) return SPEC_ERR_INVALID_ARG;
    h->w = *w;
    h->gemm_impl = 0;
    h->head_block_n = 0;
    h->proj_block_n = 0;
    h->profile = 0;
    h->fp8_max_rows = 128;
    h->swap_max_rows = -1;
    h->head_pair = -1;
    h->vp_rank = 0;
    h->vp_ranks = 1;
    h->vocab_offset = 0;
    h->head_rows = w->V;
    for (int l = 0; l < SPEC_MAX_HEADS; ++l) {
        h->head8[l] = nullptr;
        h->head8_scale[l] = nullptr;
    }
    h->prof_count = 0;
    for (cudaEvent_t &e : h->prof_ev) e = nullptr;
    *out = h;
    return SPEC_OK;
}

int spec_destroy(spec_handle_t h) {
    if (h)
        for (cudaEvent_t e : h->prof_ev)
            if (e) cudaEventDestroy(e);
    delete h;
    return SPEC_OK;
}

int spec_set_option(spec_handle_t h, int option, int value) {
    if (!h) return SPEC_ERR_INVALID_ARG;
    switch (option) {
        case SPEC_OPT_GEMM_IMPL:
            if (value != 0 && value != 1) return SPEC_ERR_INVALID_ARG;
            h->gemm_impl = value;
            return SPEC_OK;
        case SPEC_OPT_HEAD_BLOCK_N:
        case SPEC_OPT_PROJ_BLOCK_N:
            if (value != 0 && (value < 32 || value > 256 || value % 32 != 0)) return SPEC_ERR_INVALID_ARG;
            (option == SPEC_OPT_HEAD_BLOCK_N ? h->head_block_n : h->proj_block_n) = value;
            return SPEC_OK;
        case SPEC_OPT_PROFILE:
            if (value != 0 && value != 1) return SPEC_ERR_INVALID_ARG;
            if (value == 1)
                for (cudaEvent_t &e : h->prof_ev)
                    if (!e) SPEC_CUDA_TRY(cudaEventCreate(&e));
            h->profile = value;
            h->prof_count = 0;
            return SPEC_OK;
        case SPEC_OPT_FP8_MAX_ROWS:
            if (value < 0 || value > (1 << 24)) return SPEC_ERR_INVALID_ARG;
            h->fp8_max_rows = value;
            return SPEC_OK;
        case SPEC_OPT_HEAD_PAIR:
            if (value < -1 || value > 1) return SPEC_ERR_INVALID_ARG;
            h->head_pair = value;
            return SPEC_OK;
        case SPEC_OPT_GEMM_PRODUCERS:
            if (value != 1 && value != 2) return SPEC_ERR_INVALID_ARG;
            set_gemm_producers(value);
            return SPEC_OK;
        case SPEC_OPT_HEAD_SWAP_MAX_ROWS:
            if (value < -1 || value > 128) return SPEC_ERR_INVALID_ARG;
            h->swap_max_rows = value;
            return SPEC_OK;
        default:
            return SPEC_ERR_INVALID_ARG;
    }
}

int spec_quantize_head(spec_handle_t h, int level, void *q_out, float *scale_out, void *cuda_stream) {
    if (!h || !q_out || !scale_out || h->vp_ranks > 1) return SPEC_ERR_INVALID_ARG;
    if (level < 0 || level >= h->w.n_heads || h->w.d_inner % 16 != 0) return SPEC_ERR_SHAPE;
    if ((uintptr_t)q_out & 15) return SPEC_ERR_INVALID_ARG;
    return launch_quantize_rows(h->w.head[level], h->w.V, h->w.d_inner, q_out, scale_out, (cudaStream_t)cuda_stream);
}

int spec_set_head_fp8(spec_handle_t h, int level, const void *q, const float *scale) {
    if (!h) return SPEC_ERR_INVALID_ARG;
    if (level < 0 || level >= h->w.n_heads) return SPEC_ERR_SHAPE;
    if (q != nullptr && (scale == nullptr || ((uintptr_t)q & 15) || ((uintptr_t)scale & 15) || h->w.d_inner % 16 != 0))
        return SPEC_ERR_INVALID_ARG;
    h->head8[level] = q;
    h->head8_scale[level] = q ? scale : nullptr;
    return SPEC_OK;
}

int spec_profile_read(spec_handle_t h, float *ms_out, int max_count, int *count_out) {
    if (!h || !ms_out || !count_out || max_count < 0) return SPEC_ERR_INVALID_ARG;
    *count_out = 0;
    if (h->prof_count < 2) return SPEC_OK;
    SPEC_CUDA_TRY(cudaEventSynchronize(h->prof_ev[h->prof_count - 1]));
    for (int i = 0; i + 1 < h->prof_count && i < max_count; ++i) {
        SPEC_CUDA_TRY(cudaEventElapsedTime(&ms_out[i], h->prof_ev[i], h->prof_ev[i + 1]));
        *count_out = i + 1;
    }
    return SPEC_OK;
}

size_t spec_draft_workspace_bytes(spec_handle_t h, int B, const int32_t *topk, int K) {
    DraftPlan p;
    if (make_draft_plan(h, B, topk, K, &p) != SPEC_OK) return 0;
    return (size_t)p.lay.total_bytes;
}

int spec_draft_layout(spec_handle_t h, int B, const int32_t *topk, int K, spec_draft_layout_t *out) {
    if (!out) return SPEC_ERR_INVALID_ARG;
    DraftPlan p;
    int rc = make_draft_plan(h, B, topk, K, &p);
    if (rc != SPEC_OK) return rc;
    *out = p.lay;
    return SPEC_OK;
}

int spec_draft(spec_handle_t h, const void *ctx_state, const int32_t *last_tok, int B, const int32_t *topk, int K,
               int32_t *cand_tok, float *cand_logp, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!h || !ctx_state || !last_tok || !topk || !cand_tok || !cand_logp) return SPEC_ERR_INVALID_ARG;
    if ((uintptr_t)ctx_state & 15) return SPEC_ERR_INVALID_ARG;
    if (h->vp_ranks > 1) return SPEC_ERR_INVALID_ARG;   // a vocabulary shard: spec_draft_vp_local / _merge
    DraftPlan p;
    int rc = make_draft_plan(h, B, topk, K, &p);
    if (rc != SPEC_OK) return rc;
    if (!workspace || ((uintptr_t)workspace % kWsAlign) != 0 || workspace_bytes < p.lay.total_bytes)
        return SPEC_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const spec_weights_t &w = h->w;
    char *ws = (char *)workspace;
    int32_t *err = (int32_t *)(ws + p.lay.error_word);
    // The header (error word, per-sequence counters) is cleared by the first kernel of the call: the level-0
    // projection itself on the tensor-core path, a kernel of its own otherwise.
    const bool clear_in_proj = h->gemm_impl == 0;
    if (!clear_in_proj) {
        rc = launch_draft_init(err, p.header_words, st);
        if (rc != SPEC_OK) return rc;
    }

    int nev = 0;
    h->prof_count = 0;
#define SPEC_PROF_MARK()                                                     \
    do {                                                                     \
        if (h->profile) SPEC_CUDA_TRY(cudaEventRecord(h->prof_ev[nev++], st)); \
    } while (0)
    SPEC_PROF_MARK();

    float *P = (float *)(ws + p.lay.proj);
    float *part_val = (float *)(ws + p.lay.part_val);
    int32_t *part_idx = (int32_t *)(ws + p.lay.part_idx);
    float *part_ms = (float *)(ws + p.lay.part_ms);
    float *logits_scratch = (float *)(ws + p.lay.logits);

    auto proj_call = [&](int l) { return make_proj_call(h, p, ws, ctx_state, B, l); };
    const PruneArgs pa = make_prune_args(p, ws, topk);
    const bool fold_prune = !h->profile;
    bool proj_done = false;   // the projection of the level about to start ran with the previous head
    bool mix_done = false;    // the states of the level about to start were written by the previous level's merge
    for (int l = 0; l < p.n; ++l) {
        const int rows = p.N[l];
        const int parent_rows = l == 0 ? B : p.N[l - 1];
        const void *parent_states = l == 0 ? ctx_state : (const void *)(ws + p.lay.state[l - 1]);
        const float *score_l = l == 0 ? nullptr : (const float *)(ws + p.lay.score[l]);
        void *S = ws + p.lay.state[l];
        // projection of every distinct parent state: P = S_parent * Wp^T (unless it already ran in the
        // same launch as the previous level's head, see below)
        if (!proj_done) {
            if (h->gemm_impl == 0) {
                const GemmCall c = proj_call(l);
                rc = launch_gemm_tc_jobs(&c, 1, err, st, l == 0 ? err : nullptr, p.header_words);
            } else {
                rc = run_gemm_store(h, parent_states, w.proj[l], parent_rows, w.d_inner, d_in_of(w, l),
                                    p.proj_block_n[l], P, err, st);
            }
            if (rc != SPEC_OK) return rc;
        }
        SPEC_PROF_MARK();
        // gather + mix + LayerNorm + GELU -> bf16 state of every node of this level
        const bool fp8 = p.use_fp8[l];
        if (!mix_done) {
            MixArgs mx = make_mix_args(h, p, ws, last_tok, B, topk, l, err);
            if (fp8) {   // the head of this level reads the states as e4m3
                mx.S8_out = (uint8_t *)(ws + p.lay.state8);
                mx.s8_scale = (float *)(ws + p.lay.state8_scale);
            }
            rc = launch_mix_ln_gelu(mx, rows, st);
            if (rc != SPEC_OK) return rc;
        }
        mix_done = false;
        SPEC_PROF_MARK();
        // vocabulary head with the fused per-tile top-k / log-sum-exp epilogue.  The next level's
        // projection needs nothing newer than this level's states either, so it rides in the same
        // launch: its weight tiles follow the head's through the same ring and one kernel boundary less
        // lies on the critical path (with per-kernel profiling it stays a launch of its own).
        proj_done = false;
        if (p.paired[l]) {
            // tensor-bound level: the head on CTA pairs; the next level's projection follows as a launch of its own
            const GemmCall hc = make_head_call(h, p, ws, l, topk[l]);
            rc = launch_head_pair(hc.A, hc.B, hc.M, hc.N, hc.Kd, hc.block_n, hc.epi, err, st);
            if (rc == SPEC_OK && l + 1 < p.n) {
                const GemmCall pc = proj_call(l + 1);
                rc = launch_gemm_tc_jobs(&pc, 1, err, st);
                proj_done = rc == SPEC_OK;
            }
        } else if (h->gemm_impl == 0 && !h->profile) {
            GemmCall c[2];
            c[0] = make_head_call(h, p, ws, l, topk[l]);
            const bool pair = l + 1 < p.n;
            if (pair) c[1] = proj_call(l + 1);
            rc = launch_gemm_tc_jobs(c, pair ? 2 : 1, err, st);
            proj_done = pair;
        } else {
            rc = run_head_partials(h, S, w.head[l], rows, p.lay.block_n[l], topk[l], part_val, part_idx, part_ms,
                                   logits_scratch, err, st);
        }
        if (rc != SPEC_OK) return rc;
        SPEC_PROF_MARK();
        // fold the partials, branch: children (token, cumulative score) of every node.  On the last
        // level the CTA that completes a sequence's leaves also prunes it (one kernel less on the
        // critical path; with per-kernel profiling the prune stays a launch of its own).
        MergeArgs g{};
        g.part_val = part_val; g.part_idx = part_idx; g.part_ms = part_ms;
        g.n_tiles = p.lay.n_tiles[l]; g.topk = topk[l];
        g.score_in = score_l;
        g.tok_out = (int32_t *)(ws + p.lay.tok[l + 1]);
        g.score_out = (float *)(ws + p.lay.score[l + 1]);
        if (l == p.n - 1 && fold_prune) {
            g.seq_done = (int32_t *)(ws + p.seq_done);
            g.rows_per_seq = rows / B;
            g.L = p.L; g.K = K;
            g.Lpad = 2;
            while (g.Lpad < p.L) g.Lpad <<= 1;
            g.cand_tok = cand_tok; g.cand_logp = cand_logp;
            g.prune = pa;
        }
        if (fp8) {
            // short list by approximate logit, exact re-scoring from the bf16 weights, then the children
            g.list_len = SPEC_MAX_TOPK;
            rc = launch_merge_rescore(g, w.head[l], S, rows, w.d_inner, w.V, st);
        } else {
            rc = SPEC_ERR_SHAPE;
            if (proj_done && topk[l] <= kFusedMixMaxChildren && !p.use_fp8[l + 1]) {
                // the children's states in the same launch: their tokens are found here and their parent
                // projection (this level's rows) ran with the head above.  Only for one or two children per
                // row (the single-candidate chain above all): with more, a row's CTA would compute several
                // states one after the other on one SM while a kernel of its own spreads them over the GPU
                // (measured at the 13B shape: a draft 25 us slower with six and four children per CTA)
                rc = launch_merge_mix(g, make_mix_args(h, p, ws, last_tok, B, topk, l + 1, err), rows, st);
                mix_done = rc == SPEC_OK;
            }
            if (rc == SPEC_ERR_SHAPE) rc = launch_merge_expand(g, rows, st);
        }
        if (rc != SPEC_OK) return rc;
        SPEC_PROF_MARK();
    }

    if (!fold_prune) {
        rc = launch_prune((const float *)(ws + p.lay.score[p.n]), pa, B, p.L, K, cand_tok, cand_logp, st);
        if (rc != SPEC_OK) return rc;
        SPEC_PROF_MARK();
    }
#undef SPEC_PROF_MARK
    h->prof_count = nev;
    return SPEC_OK;
}

int spec_choose_k(int B, int n_heads, const spec_k_rule_t *rules, int n_rules, int32_t *K_out, int32_t *topk_out) {
    if (B <= 0 || n_heads < 1 || n_heads > SPEC_MAX_HEADS || !rules || n_rules < 1 || !K_out) return SPEC_ERR_INVALID_ARG;
    for (int i = 0; i < n_rules; ++i) {
        const spec_k_rule_t &r = rules[i];
        if (r.max_batch < 1 || (i > 0 && r.max_batch <= rules[i - 1].max_batch) || r.K < 0) return SPEC_ERR_INVALID_ARG;
        if (r.K > 0) {
            long long leaves = 1;
            for (int l = 0; l < n_heads; ++l) {
                if (r.topk[l] < 1 || r.topk[l] > SPEC_MAX_TOPK) return SPEC_ERR_INVALID_ARG;
                leaves *= r.topk[l];
            }
            if (leaves > SPEC_MAX_LEAVES || r.K > leaves) return SPEC_ERR_INVALID_ARG;
        }
    }
    *K_out = 0;
    if (topk_out)
        for (int l = 0; l < n_heads; ++l) topk_out[l] = 0;
    for (int i = 0; i < n_rules; ++i) {
        if (B <= rules[i].max_batch) {
            *K_out = rules[i].K;
            if (topk_out && rules[i].K > 0)
                for (int l = 0; l < n_heads; ++l) topk_out[l] = rules[i].topk[l];
            break;
        }
    }
    return SPEC_OK;
}

/* ---- vocabulary-parallel heads ------------------------------------------------------------------ */
int spec_set_vocab_shard(spec_handle_t h, int rank, int n_ranks, int vocab_offset, int head_rows) {
    if (!h) return SPEC_ERR_INVALID_ARG;
    if (n_ranks < 1 || n_ranks > 8 || rank < 0 || rank >= n_ranks) return SPEC_ERR_INVALID_ARG;
    if (vocab_offset < 0 || head_rows < 1 || (long long)vocab_offset + head_rows > h->w.V) return SPEC_ERR_SHAPE;
    if (n_ranks == 1 && (vocab_offset != 0 || head_rows != h->w.V)) return SPEC_ERR_SHAPE;
    h->vp_rank = rank;
    h->vp_ranks = n_ranks;
    h->vocab_offset = vocab_offset;
    h->head_rows = head_rows;
    return SPEC_OK;
}

int spec_draft_vp_exchange(spec_handle_t h, int B, const int32_t *topk, int K, int level, uint64_t *offset,
                           uint64_t *slot_bytes) {
    if (!h || !offset || !slot_bytes || h->vp_ranks < 2) return SPEC_ERR_INVALID_ARG;
    DraftPlan p;
    int rc = make_draft_plan(h, B, topk, K, &p);
    if (rc != SPEC_OK) return rc;
    if (level < 0 || level >= p.n) return SPEC_ERR_INVALID_ARG;
    *offset = p.xchg;
    *slot_bytes = p.slot_bytes[level];
    return SPEC_OK;
}

int spec_draft_vp_local(spec_handle_t h, int level, const void *ctx_state, const int32_t *last_tok, int B,
                        const int32_t *topk, int K, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!h || !ctx_state || !last_tok || !topk) return SPEC_ERR_INVALID_ARG;
    if ((uintptr_t)ctx_state & 15) return SPEC_ERR_INVALID_ARG;
    if (h->vp_ranks < 2 || h->gemm_impl != 0) return SPEC_ERR_INVALID_ARG;
    DraftPlan p;
    int rc = make_draft_plan(h, B, topk, K, &p);
    if (rc != SPEC_OK) return rc;
    if (level < 0 || level >= p.n) return SPEC_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace % kWsAlign) != 0 || workspace_bytes < p.lay.total_bytes)
        return SPEC_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char *ws = (char *)workspace;
    int32_t *err = (int32_t *)(ws + p.lay.error_word);
    const int l = level, rows = p.N[l];
    if (l == 0) {   // the first step of a draft clears the header and projects the context states
        const GemmCall c = make_proj_call(h, p, ws, ctx_state, B, 0);
        rc = launch_gemm_tc_jobs(&c, 1, err, st, err, p.header_words);
        if (rc != SPEC_OK) return rc;
    }
    const MixArgs mx = make_mix_args(h, p, ws, last_tok, B, topk, l, err);
    rc = launch_mix_ln_gelu(mx, rows, st);
    if (rc != SPEC_OK) return rc;
    // this rank's vocabulary rows only; token ids leave the epilogue already offset.  The next level's
    // projection (replicated on every rank) rides in the same launch as in spec_draft.
    GemmCall c[2];
    c[0] = make_head_call(h, p, ws, l, topk[l]);
    const bool pair = l + 1 < p.n;
    if (pair) c[1] = make_proj_call(h, p, ws, ctx_state, B, l + 1);
    rc = launch_gemm_tc_jobs(c, pair ? 2 : 1, err, st);
    if (rc != SPEC_OK) return rc;
    // fold the tiles into this rank's slot: the shard's topk logits, their token ids, its log-sum-exp
    char *slot = ws + p.xchg + (size_t)h->vp_rank * p.slot_bytes[l];
    MergeArgs g{};
    g.part_val = c[0].epi.part_val; g.part_idx = c[0].epi.part_idx; g.part_ms = c[0].epi.part_ms;
    g.n_tiles = p.lay.n_tiles[l]; g.topk = topk[l];
    g.score_out = (float *)slot;
    g.tok_out = (int32_t *)(slot + sizeof(float) * (size_t)rows * topk[l]);
    g.lse_out = (float *)(slot + 2 * sizeof(float) * (size_t)rows * topk[l]);
    return launch_merge_expand(g, rows, st);
}

int spec_draft_vp_merge(spec_handle_t h, int level, int B, const int32_t *topk, int K, int32_t *cand_tok,
                        float *cand_logp, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!h || !topk) return SPEC_ERR_INVALID_ARG;
    if (h->vp_ranks < 2) return SPEC_ERR_INVALID_ARG;
    DraftPlan p;
    int rc = make_draft_plan(h, B, topk, K, &p);
    if (rc != SPEC_OK) return rc;
    if (level < 0 || level >= p.n) return SPEC_ERR_INVALID_ARG;
    const bool last = level == p.n - 1;
    if (last && (!cand_tok || !cand_logp)) return SPEC_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace % kWsAlign) != 0 || workspace_bytes < p.lay.total_bytes)
        return SPEC_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char *ws = (char *)workspace;
    const int l = level;
    rc = launch_merge_shards(ws + p.xchg, p.slot_bytes[l], h->vp_ranks, p.N[l], topk[l],
                             l == 0 ? nullptr : (const float *)(ws + p.lay.score[l]),
                             (int32_t *)(ws + p.lay.tok[l + 1]), (float *)(ws + p.lay.score[l + 1]), st);
    if (rc != SPEC_OK || !last) return rc;
    return launch_prune((const float *)(ws + p.lay.score[p.n]), make_prune_args(p, ws, topk), B, p.L, K, cand_tok,
                        cand_logp, st);
}

size_t spec_verify_workspace_bytes(int B, int K, int n, int V, int logits_dtype) {
    if (B <= 0 || K <= 0 || n <= 0 || V <= 0) return 0;
    if (logits_dtype != SPEC_BF16 && logits_dtype != SPEC_F32) return 0;
    if ((long long)B * K * (n + 1) > (1ll << 30)) return 0;
    return make_verify_plan(B, K, n, V, logits_dtype).total;
}

int spec_verify(const int32_t *cand_tok, const void *base_logits, int logits_dtype, int B, int K, int n, int V,
                int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *workspace, size_t workspace_bytes,
                void *cuda_stream) {
    if (!cand_tok || !base_logits || !accept_len || !best_cand || !next_tok) return SPEC_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || n <= 0 || V <= 0) return SPEC_ERR_INVALID_ARG;
    if (logits_dtype != SPEC_BF16 && logits_dtype != SPEC_F32) return SPEC_ERR_INVALID_ARG;
    if (K > 65535 || (long long)K * (n + 1) > 12288 || n > 32767) return SPEC_ERR_SHAPE;
    if ((long long)B * K * (n + 1) > (1ll << 30)) return SPEC_ERR_SHAPE;
    if (((uintptr_t)base_logits % (logits_dtype == SPEC_BF16 ? 2 : 4)) != 0) return SPEC_ERR_INVALID_ARG;
    const VerifyPlan plan = make_verify_plan(B, K, n, V, logits_dtype);
    if (!workspace || ((uintptr_t)workspace % kWsAlign) != 0 || workspace_bytes < plan.total)
        return SPEC_ERR_WORKSPACE;
    return launch_verify(cand_tok, base_logits, logits_dtype, B, K, n, V, accept_len, best_cand, next_tok, workspace,
                         plan, (cudaStream_t)cuda_stream);
}

int spec_verify_early(const int32_t *cand_tok, const void *base_logits, int logits_dtype, int B, int K, int n, int V,
                      int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *workspace,
                      size_t workspace_bytes, void *cuda_stream) {
    if (!cand_tok || !base_logits || !accept_len || !best_cand || !next_tok) return SPEC_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || n <= 0 || V <= 0) return SPEC_ERR_INVALID_ARG;
    if (logits_dtype != SPEC_BF16 && logits_dtype != SPEC_F32) return SPEC_ERR_INVALID_ARG;
    if (K > 65535 || (long long)K * (n + 1) > 12288 || n > 32767) return SPEC_ERR_SHAPE;
    if ((long long)B * K * (n + 1) > (1ll << 30)) return SPEC_ERR_SHAPE;
    if (((uintptr_t)base_logits % (logits_dtype == SPEC_BF16 ? 2 : 4)) != 0) return SPEC_ERR_INVALID_ARG;
    const VerifyPlan plan = make_verify_plan(B, K, n, V, logits_dtype);
    if (!workspace || ((uintptr_t)workspace % kWsAlign) != 0 || workspace_bytes < plan.total)
        return SPEC_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int rc = launch_verify_early(cand_tok, base_logits, logits_dtype, B, K, n, V, accept_len, best_cand, next_tok,
                                       workspace, plan, st);
    if (rc != SPEC_ERR_SHAPE) return rc;
    // rows that are not whole 16-byte vectors: the streaming form reads everything
    return launch_verify(cand_tok, base_logits, logits_dtype, B, K, n, V, accept_len, best_cand, next_tok, workspace,
                         plan, st);
}

int spec_poll_error(void *workspace, void *cuda_stream) {
    if (!workspace) return SPEC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int32_t word = 0;
    SPEC_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st));
    SPEC_CUDA_TRY(cudaStreamSynchronize(st));
    if (word != 0) {
        SPEC_CUDA_TRY(cudaMemsetAsync(workspace, 0, sizeof(word), st));
        SPEC_CUDA_TRY(cudaStreamSynchronize(st));
    }
    return (int)word;
}

size_t spec_head_workspace_bytes(spec_handle_t h, int rows, int topk) {
    if (!h || rows <= 0 || topk < 1 || topk > SPEC_MAX_TOPK || h->vp_ranks > 1) return 0;
    const size_t units = (size_t)rows * head_parts_for(h, rows, head_swapped_for(h, rows), nullptr);
    size_t off = kWsAlign;
    off = align_up(off + sizeof(float) * units * SPEC_MAX_TOPK, kWsAlign);
    off = align_up(off + sizeof(int32_t) * units * SPEC_MAX_TOPK, kWsAlign);
    off = align_up(off + sizeof(float) * units * 2, kWsAlign);
    if (h->gemm_impl == 1) off = align_up(off + sizeof(float) * (size_t)rows * h->w.V, kWsAlign);
    return off;
}

int spec_head_logits(spec_handle_t h, int level, const void *states, int rows, float *logits, void *cuda_stream) {
    if (!h || !states || !logits || rows <= 0 || h->vp_ranks > 1) return SPEC_ERR_INVALID_ARG;
    if (level < 0 || level >= h->w.n_heads) return SPEC_ERR_SHAPE;
    if ((uintptr_t)states & 15) return SPEC_ERR_INVALID_ARG;
    return run_gemm_store(h, states, h->w.head[level], rows, h->w.V, h->w.d_inner, head_block_n_for(h, rows), logits,
                          nullptr, (cudaStream_t)cuda_stream);
}

// The two kernels of the fused head; `tok` / `logp` null: the GEMM with its epilogue only, and no clearing
// of the error word (so that back-to-back calls are kernel launches and nothing else).
static int head_topk_impl(spec_handle_t h, int level, const void *states, int rows, int topk, int32_t *tok, float *logp,
                          void *workspace, size_t workspace_bytes, void *cuda_stream) {
    const bool merge = tok != nullptr;
    if (!h || !states || rows <= 0 || (merge && !logp) || h->vp_ranks > 1) return SPEC_ERR_INVALID_ARG;
    if (level < 0 || level >= h->w.n_heads || topk < 1 || topk > SPEC_MAX_TOPK || topk > h->w.V) return SPEC_ERR_SHAPE;
    if ((uintptr_t)states & 15) return SPEC_ERR_INVALID_ARG;
    const size_t need = spec_head_workspace_bytes(h, rows, topk);
    if (!workspace || ((uintptr_t)workspace % kWsAlign) != 0 || workspace_bytes < need) return SPEC_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int bn = 0;
    const int n_tiles = head_parts_for(h, rows, head_swapped_for(h, rows), &bn);
    const size_t units = (size_t)rows * n_tiles;
    char *ws = (char *)workspace;
    int32_t *err = (int32_t *)ws;
    if (merge) SPEC_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(int32_t), st));
    size_t off = kWsAlign;
    float *part_val = (float *)(ws + off);
    off = align_up(off + sizeof(float) * units * SPEC_MAX_TOPK, kWsAlign);
    int32_t *part_idx = (int32_t *)(ws + off);
    off = align_up(off + sizeof(int32_t) * units * SPEC_MAX_TOPK, kWsAlign);
    float *part_ms = (float *)(ws + off);
    off = align_up(off + sizeof(float) * units * 2, kWsAlign);
    float *logits_scratch = (float *)(ws + off);
    int rc = run_head_partials(h, states, h->w.head[level], rows, bn, topk, part_val, part_idx, part_ms,
                               logits_scratch, err, st);
    if (rc != SPEC_OK || !merge) return rc;
    MergeArgs g{};
    g.part_val = part_val; g.part_idx = part_idx; g.part_ms = part_ms;
    g.n_tiles = n_tiles; g.topk = topk;
    g.tok_out = tok; g.score_out = logp;
    return launch_merge_expand(g, rows, st);
}

int spec_head_topk(spec_handle_t h, int level, const void *states, int rows, int topk, int32_t *tok, float *logp,
                   void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!tok || !logp) return SPEC_ERR_INVALID_ARG;
    return head_topk_impl(h, level, states, rows, topk, tok, logp, workspace, workspace_bytes, cuda_stream);
}

int spec_head_partials(spec_handle_t h, int level, const void *states, int rows, int topk, void *workspace,
                       size_t workspace_bytes, void *cuda_stream) {
    return head_topk_impl(h, level, states, rows, topk, nullptr, nullptr, workspace, workspace_bytes, cuda_stream);
}

}  // extern "C"
