/*
 * spec_b200 - C ABI of the B200 (sm_100a) draft-tree generation and greedy verification
 * library for the combined token/embedding speculator of arXiv 2404.19124.
 *
 * Conventions
 *   - plain C, no exceptions cross the boundary; every call returns a SPEC_* status.
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory.
 *   - the library never allocates or frees device memory: inputs, outputs, weights and
 *     workspaces are owned by the caller and must stay valid until the work queued on
 *     the stream has finished.
 *   - spec_draft / spec_verify only enqueue work on `cuda_stream` (a cudaStream_t passed
 *     as void*; NULL = default stream) and never synchronise.
 *   - errors found on the host (bad pointers, shapes, workspace too small) are returned
 *     at once and nothing is enqueued.  Errors found on the device (token id outside
 *     [0, V), a bounded wait that ran out) are recorded in an error word at the start of
 *     the workspace and reported by spec_poll_error; kernels never trap.
 */
#ifndef SPEC_B200_H_
#define SPEC_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPEC_MAX_HEADS 8     /* stages of the speculator (the paper uses 3, 5 and 7)         */
#define SPEC_MAX_TOPK 8      /* branching factor of one head                                  */
#define SPEC_MAX_LEAVES 4096 /* product of the branching factors, per sequence                */

enum spec_status {
    SPEC_OK = 0,
    SPEC_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, unknown dtype / option      */
    SPEC_ERR_SHAPE = 2,       /* K > leaves, topk > SPEC_MAX_TOPK, widths not multiples of 8  */
    SPEC_ERR_WORKSPACE = 3,   /* workspace missing, misaligned (256 B) or too small           */
    SPEC_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed: see spec_last_cuda_error  */
    SPEC_ERR_TOKEN_RANGE = 5, /* device: a token id was outside [0, V) (its embedding is
                                 treated as zero and the call runs to completion)             */
    SPEC_ERR_TIMEOUT = 6,     /* device: a bounded wait inside a kernel ran out               */
    SPEC_ERR_NO_DEVICE = 7,   /* no CUDA device / not an sm_100 part                          */
    SPEC_ERR_STATIC_SCRATCH = 8, /* spec_verify_static: the problem needs more scratch than the
                                 built-in array holds (SPEC_VERIFY_STATIC_SCRATCH_BYTES)      */
    SPEC_ERR_INDEX_RANGE = 9  /* device: spec_next_ctx met best_cand outside [0, K) or accept_len
                                 outside [0, n] (that sequence's row is written as zeros)     */
};

enum spec_dtype { SPEC_BF16 = 0, SPEC_F32 = 1 };

enum spec_option {
    SPEC_OPT_GEMM_IMPL = 0,    /* 0 (default): tcgen05/TMEM tensor-core kernels; 1: slow CUDA-core
                                  kernels kept for debugging the tensor-core path              */
    SPEC_OPT_HEAD_BLOCK_N = 1, /* vocabulary columns per tile of the head GEMM; 0 = automatic  */
    SPEC_OPT_PROJ_BLOCK_N = 2, /* output columns per tile of the state projection; 0 = auto    */
    SPEC_OPT_PROFILE = 3,      /* 1: spec_draft brackets each of its kernels with CUDA events on
                                  the caller's stream (read them with spec_profile_read); costs a
                                  few microseconds per call, off by default                    */
    SPEC_OPT_FP8_MAX_ROWS = 4, /* levels with at most this many nodes use the e4m3 copy of their head when
                                  one is attached (default 128, the levels bound by the weight
                                  stream; 0 = never).  Larger values put tensor-bound levels on
                                  the e4m3 path too, which pays from about 768 nodes on        */
    SPEC_OPT_HEAD_SWAP_MAX_ROWS = 5, /* levels with at most this many nodes (0 .. 128) run the head GEMM
                                  with the weight matrix on the 128-row side of the MMA and the nodes
                                  as columns, so the tensor work follows the number of nodes; 0 = never;
                                  -1 (default) = automatic: up to 8 nodes, or up to 32 when the
                                  vocabulary gives every CTA at least four 128-row tiles.  Ignored
                                  while SPEC_OPT_HEAD_BLOCK_N forces a tile width.              */
    SPEC_OPT_GEMM_PRODUCERS = 6, /* 1 or 2 (default) threads per CTA issue the TMA copies of the GEMM
                                  kernels; process-wide, not per handle                        */
    SPEC_OPT_HEAD_PAIR = 7       /* 1: levels of more than 128 nodes run the head GEMM on pairs of CTAs
                                  (tcgen05.mma.cta_group::2: 256 node rows per tile, each CTA loads half
                                  of the weight box); 0: one CTA per tile; -1 (default): pairs for
                                  levels whose padding to a multiple of 256 nodes is at most a tenth */
};

typedef struct spec_handle_s *spec_handle_t;

/* Speculator parameters (Sec. 3.1: every stage has its own embedding table, state
 * projection, LayerNorm and vocabulary output matrix; nothing is tied).  All pointers are
 * dev, row-major, 16-byte aligned, read-only, caller-owned. */
typedef struct {
    int32_t n_heads, V, d_base, d_inner;   /* d_base % 8 == 0, d_inner % 8 == 0              */
    const void *emb[SPEC_MAX_HEADS];       /* bf16 [V, d_inner]                               */
    const void *proj[SPEC_MAX_HEADS];      /* bf16 [d_inner, d_in]; d_in = d_base for head 0,
                                              d_inner for the others                          */
    const float *ln_gamma[SPEC_MAX_HEADS]; /* fp32 [d_inner]                                  */
    const float *ln_beta[SPEC_MAX_HEADS];  /* fp32 [d_inner]                                  */
    const void *head[SPEC_MAX_HEADS];      /* bf16 [V, d_inner]                               */
    float state_weight;                    /* a: weight of the projected state in the mix     */
    float emb_weight;                      /* b: weight of the token embedding in the mix     */
    float ln_eps;
} spec_weights_t;

/* Byte offsets into a draft workspace (for tests and debugging; N_l = B * prod_{j<l} topk[j]). */
typedef struct {
    uint64_t total_bytes;
    uint64_t error_word;                  /* int32                                            */
    uint64_t tok[SPEC_MAX_HEADS + 1];     /* int32 [N_l]: token of every node of level l>=1   */
    uint64_t score[SPEC_MAX_HEADS + 1];   /* fp32  [N_l]: cumulative log-prob, level l>=1     */
    uint64_t state[SPEC_MAX_HEADS];       /* bf16  [N_l, d_inner]: post-GELU state of level l */
    uint64_t proj;                        /* fp32  [max rows, d_inner]: projected parent states */
    uint64_t state8, state8_scale;        /* e4m3 [rows, d_inner] + fp32 [rows]: states of an e4m3 level */
    uint64_t part_val, part_idx, part_ms; /* per-tile partial top-k lists and (max, sum-exp)  */
    uint64_t logits;                      /* fp32 [max N_l, V]; only with SPEC_OPT_GEMM_IMPL=1 */
    int32_t block_n[SPEC_MAX_HEADS];      /* vocabulary columns per head-GEMM tile            */
    int32_t n_tiles[SPEC_MAX_HEADS];      /* vocabulary tiles per row of the head GEMM        */
} spec_draft_layout_t;

int spec_version(void);
const char *spec_status_str(int status);
/* cudaError_t / CUresult of the last failing CUDA call made by this library on this thread. */
int spec_last_cuda_error(void);

/* Host-only: validates and copies `w` (host), prepares host-side launch state.  The
 * current CUDA device must be the one that owns the weight pointers. */
int spec_create(spec_handle_t *out, const spec_weights_t *w);
int spec_destroy(spec_handle_t h);
int spec_set_option(spec_handle_t h, int option, int value);

/* ---- draft (Sec. 3.1: multi-stage MLP emitting a tree of candidates; Sec. 4.1: branch
 * topk[l] ways at head l, then prune the product tree to the K most confident) ----------
 * For each sequence b: level 0 is (ctx_state[b], last_tok[b]); head l maps every node
 * (parent state s, token t) to  s' = GELU(LayerNorm(a * Wp_l s + b * E_l[t])) rounded to
 * bf16, logits = Wout_l s', and branches to the topk[l] largest logits (equal values:
 * lower token id first) with score += logit - logsumexp(logits).  The K leaves with the
 * best scores (equal scores: lower leaf index first) are returned in that order.
 *   ctx_state  dev bf16 [B, d_base]   latest base-model state vector of each sequence
 *   last_tok   dev int32 [B]          token just sampled from it
 *   topk       host int32 [n_heads], 1 <= topk[l] <= SPEC_MAX_TOPK, prod <= SPEC_MAX_LEAVES
 *   K          1 <= K <= prod topk
 *   cand_tok   dev int32 [B, K, n_heads] (out), cand_logp dev fp32 [B, K] (out)
 *   workspace  dev, 256-byte aligned, >= spec_draft_workspace_bytes(...).  Need not be zeroed: the
 *              first kernel of the call clears the header (error word at byte 0, one int32
 *              counter per sequence from byte 256 on).
 */
size_t spec_draft_workspace_bytes(spec_handle_t h, int B, const int32_t *topk, int K);
int spec_draft_layout(spec_handle_t h, int B, const int32_t *topk, int K, spec_draft_layout_t *out /*host*/);
int spec_draft(spec_handle_t h, const void *ctx_state, const int32_t *last_tok, int B, const int32_t *topk, int K,
               int32_t *cand_tok, float *cand_logp, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* ---- how many candidates to draft (Sec. 4.2 and Sec. 5: several candidates per sequence pay at batch size 1
 * - the paper quotes k = 5 there - a single candidate, k = 1, is the better setting under load, and beyond some
 * batch size speculation is switched off altogether because the base model's forward over B * k * (n + 1)
 * tokens becomes compute-bound).  The paper gives the shape of that rule, not its numbers, which depend on the
 * base model and the GPU: they are the caller's, as a table sorted by ascending batch size.
 *   rules     host, n_rules entries with strictly ascending max_batch; entry i applies to
 *             B <= rules[i].max_batch (and B > rules[i-1].max_batch).  K = 0 in an entry means "do not
 *             speculate"; otherwise topk[0 .. n_heads) are the branching factors to draft with
 *             (1 <= topk[l] <= SPEC_MAX_TOPK, K <= prod topk <= SPEC_MAX_LEAVES).
 *   K_out     host: receives the K of the first entry that covers B, 0 when B is larger than every max_batch
 *   topk_out  host int32 [n_heads], may be NULL: receives that entry's branching factors (zeros when K = 0)
 * Host-only: touches no device and no stream.  SPEC_ERR_INVALID_ARG for a malformed table.
 * With K = 1 and topk = 1 everywhere spec_draft runs its shortest launch chain: every head has B rows, a
 * level's top-k is an arg-max and its merge also writes the one child's state. */
typedef struct {
    int32_t max_batch;
    int32_t K;
    int32_t topk[SPEC_MAX_HEADS];
} spec_k_rule_t;
int spec_choose_k(int B, int n_heads, const spec_k_rule_t *rules, int n_rules, int32_t *K_out, int32_t *topk_out);

/* ---- verify (Sec. 1: accept the speculated tokens that match the base model's outputs;
 * Sec. 3.1: score all candidates, keep the best; Sec. 5: at most n + 1 tokens per step) --
 *   g[b,k,j]      = first index of the maximum of base_logits[b,k,j,:] (NaN never wins)
 *   m[b,k]        = number of leading j < n with cand_tok[b,k,j] == g[b,k,j]
 *   best_cand[b]  = lowest k attaining max_k m[b,k];  accept_len[b] = m[b,best];
 *   next_tok[b]   = g[b,best,accept_len[b]]
 *   cand_tok      dev int32 [B, K, n];  base_logits dev [B, K, n+1, V] of logits_dtype (read through the
 *                 non-coherent path: whatever produces it must precede this call on the stream)
 *   accept_len, best_cand, next_tok  dev int32 [B] (out)
 *   workspace     dev, 256-byte aligned, >= spec_verify_workspace_bytes(...); on return it
 *                 holds the error word (offset 0) and g as int32 [B,K,n+1] at offset 256.
 * Limits: K <= 65535, K * (n + 1) <= 12288.
 */
size_t spec_verify_workspace_bytes(int B, int K, int n, int V, int logits_dtype);
int spec_verify(const int32_t *cand_tok, const void *base_logits, int logits_dtype, int B, int K, int n, int V,
                int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *workspace,
                size_t workspace_bytes, void *cuda_stream);

/* Early-exit form of spec_verify (Sec. 1: everything after a candidate's first rejected token is
 * discarded, so the base model's logits behind it need not be looked at).  Same arguments, same
 * three results.  One thread block per candidate reads its rows in order and stops after the first
 * row whose arg-max differs from the speculated token: the bytes read fall from B K (n+1) V elements
 * to sum over the candidates of (m[b,k] + 1) V.  In the workspace, g holds -1 for rows that were not
 * read.  Worth it when many candidates fail early or the tensor is large; when nearly all rows are
 * needed the one-pass streaming form is faster.  Rows must be whole 16-byte vectors and base_logits
 * 16-byte aligned, otherwise the call silently runs the streaming form. */
int spec_verify_early(const int32_t *cand_tok, const void *base_logits, int logits_dtype, int B, int K, int n, int V,
                      int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *workspace,
                      size_t workspace_bytes, void *cuda_stream);

/* ---- closing the loop (Sec. 3.1: the speculator starts from the base model's latest state vector;
 * after a verified step that is the state at the last accepted position of the best candidate) ----
 *   base_state  dev bf16 [B, K, n+1, d_base]  the base model's state vectors at the positions whose
 *                                             logits spec_verify looked at
 *   best_cand, accept_len  dev int32 [B]      as written by spec_verify* earlier on the same stream
 *   ctx_state   dev bf16 [B, d_base] (out)    ctx_state[b,:] = base_state[b, best_cand[b], accept_len[b], :]
 *   err_word    dev int32, or NULL            receives SPEC_ERR_INDEX_RANGE if it was 0 and an index is
 *                                             out of range (e.g. the word at offset 0 of the verify
 *                                             workspace, which spec_poll_error reads); never cleared here
 * Only enqueues one copy kernel on `cuda_stream`; nothing is allocated.  Rows are copied 16 bytes at a
 * time when d_base is a multiple of 8 and both tensors are 16-byte aligned, else element by element. */
int spec_next_ctx(const void *base_state, const int32_t *best_cand, const int32_t *accept_len, int B, int K, int n,
                  int d_base, void *ctx_state, int32_t *err_word, void *cuda_stream);

/* ---- verify without a caller-supplied workspace -----------------------------------------
 * (No counterpart in the paper: this is a packaging variant of spec_verify, same results.)
 * Some hosts of this library cannot hand it scratch memory: a serving process that gave all
 * of its device memory to its own pools (KV cache, activations) at start-up and must not
 * grow afterwards, a decode loop that may not take the implicit device-wide stall of an
 * allocation, or an embedding where another component owns allocation and passes this
 * library nothing but input and output pointers.  For them the scratch of the verify
 * kernels (per-row partial maxima and the arg-max table g) lives in an array built into the
 * library's device image, SPEC_VERIFY_STATIC_SCRATCH_BYTES long; every GPU that loads the
 * library holds that much memory until the process exits.
 *   - Arguments and results as spec_verify, minus workspace / workspace_bytes.  No call in
 *     here allocates or frees memory, on the host or on the device.
 *   - A problem whose scratch would exceed the array (spec_verify_workspace_bytes(...) >
 *     SPEC_VERIFY_STATIC_SCRATCH_BYTES) is refused with SPEC_ERR_STATIC_SCRATCH and nothing
 *     is enqueued.  The five shapes in the benchmark need at most 0.4 MiB.
 *   - The first call on each device looks up the array's device address (a driver query,
 *     made with that device current) before it enqueues anything; make that first call
 *     outside of any stream capture.  Later calls on that device only enqueue kernels.
 *   - All calls on a device share the one array and it keeps what the last call left there.
 *     Nothing in it has to be zero beforehand: the kernels overwrite every slot they later
 *     read and reset the error word themselves.  Two calls whose kernels can overlap on the
 *     GPU (different streams without an ordering between them) race on the array: order
 *     them.  The arg-max table g is not reachable by the caller; device-side errors cannot
 *     occur on this path (it reads no token-indexed memory).
 */
#define SPEC_VERIFY_STATIC_SCRATCH_BYTES (1u << 20)
int spec_verify_static(const int32_t *cand_tok, const void *base_logits, int logits_dtype, int B, int K, int n,
                       int V, int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, void *cuda_stream);

/* ---- vocabulary-parallel heads (optional; Sec. 3.1: nearly all of the speculator's parameters sit in
 * the vocabulary-sized matrices, which is what a small batch spends its time reading) ---------------
 * n_ranks processes, one GPU each, split every head matrix by vocabulary rows: rank g holds rows
 * [vocab_offset_g, vocab_offset_g + head_rows_g) of each head (the shards tile [0, V) without overlap),
 * everything else (embeddings with all V rows, projections, LayerNorm) is replicated.  A draft becomes,
 * per level l = 0 .. n_heads-1,
 *     spec_draft_vp_local(level l)   projection, mix, the head on this rank's rows, and this rank's
 *                                    lists written to slot `rank` of the exchange region
 *     all-gather of the slots        done by the CALLER with whatever collective it has (NCCL, peer
 *                                    copies): afterwards every rank holds all n_ranks slots
 *     spec_draft_vp_merge(level l)   folds the slots into the level's children; at the last level also
 *                                    prunes to the K candidates
 * and every rank ends with the same cand_tok / cand_logp as spec_draft on unsplit weights (token sets and
 * order identical; log-probabilities equal up to the rounding of a two-stage log-sum-exp).
 *   spec_set_vocab_shard     declares that the head[] matrices given to spec_create hold `head_rows` rows
 *                            starting at token `vocab_offset` (weights.V stays the full vocabulary).
 *                            n_ranks <= 8, n_ranks * topk[l] <= 64.  On such a handle spec_draft, the
 *                            spec_head_* calls and the e4m3 option are refused / ignored.  n_ranks = 1
 *                            (offset 0, all rows) makes the handle an ordinary one again.
 *   spec_draft_vp_exchange   byte offset of slot 0 in the workspace and the size of one slot at `level`;
 *                            slot g lies at offset + g * slot_bytes.  A slot is fp32 [N_l, topk[l]] logits,
 *                            int32 [N_l, topk[l]] token ids, fp32 [N_l] log-sum-exp over the shard, padded
 *                            to 256 bytes.
 *                            ORDER ACROSS RANKS: all levels use the same region at the same offset, with a slot
 *                            size that changes from level to level.  A rank's region may therefore receive
 *                            level l + 1 slots only after its own spec_draft_vp_merge(level l) has completed.
 *                            A collective enqueued on the draft's stream (NCCL all-gather) orders this by
 *                            itself; with direct peer stores the writer must first learn (an event, a flag, a
 *                            barrier per level) that the peer's merge of the previous level is done.  Peer
 *                            traffic is plain loads / stores or NCCL; every TMA copy the library issues has one destination CTA.
 *   spec_draft_vp_local / _merge  arguments as spec_draft; the same B, topk, K and workspace for every
 *                            step of one draft (workspace size: spec_draft_workspace_bytes on the sharded
 *                            handle).  cand_tok / cand_logp are written by the merge of the last level
 *                            only and may be NULL before.  All calls only enqueue work on `cuda_stream`.
 */
int spec_set_vocab_shard(spec_handle_t h, int rank, int n_ranks, int vocab_offset, int head_rows);
int spec_draft_vp_exchange(spec_handle_t h, int B, const int32_t *topk, int K, int level, uint64_t *offset /*host*/,
                           uint64_t *slot_bytes /*host*/);
int spec_draft_vp_local(spec_handle_t h, int level, const void *ctx_state, const int32_t *last_tok, int B,
                        const int32_t *topk, int K, void *workspace, size_t workspace_bytes, void *cuda_stream);
int spec_draft_vp_merge(spec_handle_t h, int level, int B, const int32_t *topk, int K, int32_t *cand_tok,
                        float *cand_logp, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* ---- e4m3 copy of a vocabulary head (optional) ---------------------------------------------
 * (The paper runs everything in 16 bits; this is an implementation option for the heads whose
 * cost is reading the weights: levels with few nodes.)  A head's bf16 matrix [V, d_inner] can be
 * given a second form, e4m3 bytes [V, d_inner] with one fp32 scale per vocabulary row, half the
 * bytes.  For a level that has it and at most SPEC_OPT_FP8_MAX_ROWS nodes, spec_draft multiplies
 * in e4m3 (tensor cores, fp32 accumulation), keeps the 16 tokens with the best APPROXIMATE logits
 * per node, recomputes those 16 logits exactly from the bf16 weights and states, and branches
 * to the top-k of the exact values; only the softmax normaliser comes from the approximate
 * logits (its error is of order 1e-3 in log-probability).  d_inner must be a multiple of 16;
 * with d_inner > 16384 the attached copies are ignored and every level runs in bf16.
 *   spec_quantize_head  fills q_out (dev, V * d_inner bytes, 16-byte aligned) and scale_out
 *                       (dev fp32 [V]) from head `level`'s bf16 weights on `cuda_stream`
 *   spec_set_head_fp8   attaches such a pair to the handle (caller-owned, must outlive the calls
 *                       that use it); q = NULL detaches
 */
int spec_quantize_head(spec_handle_t h, int level, void *q_out, float *scale_out, void *cuda_stream);
int spec_set_head_fp8(spec_handle_t h, int level, const void *q, const float *scale);

/* Per-kernel device times of the last spec_draft issued with SPEC_OPT_PROFILE = 1, in launch
 * order: for every head (projection GEMM, mix/LayerNorm/GELU, head GEMM, merge/expand), then
 * the prune kernel: 4 * n_heads + 1 values.  Blocks until that draft has finished.
 *   ms_out host fp32 [max_count]; *count_out receives the number of values written. */
int spec_profile_read(spec_handle_t h, float *ms_out, int max_count, int *count_out);

/* Synchronises the stream, reads and clears the error word at the start of `workspace`
 * (a draft or verify workspace) and returns it as a SPEC_* status. */
int spec_poll_error(void *workspace, void *cuda_stream);

/* ---- single steps, exported for parity tests and kernel benchmarks ---------------------
 * spec_head_logits: logits[r, v] = sum_c head_l[v, c] * states[r, c] written in full
 *   (fp32 [rows, V], dev) through the same tensor-core main loop as spec_draft.
 * spec_head_topk: the fused form used inside spec_draft: per row the topk largest logits
 *   (tok, dev int32 [rows, topk]) and their log-probabilities (logp, dev fp32 [rows, topk]);
 *   full logits are never written.  workspace >= spec_head_workspace_bytes(...).
 * spec_head_partials: only the first of spec_head_topk's two kernels, the head GEMM with its fused
 *   epilogue (per vocabulary tile and row: partial top-k list and (max, sum-exp) in the workspace); for
 *   timing that kernel alone.
 */
size_t spec_head_workspace_bytes(spec_handle_t h, int rows, int topk);
int spec_head_partials(spec_handle_t h, int level, const void *states, int rows, int topk, void *workspace,
                       size_t workspace_bytes, void *cuda_stream);
int spec_head_logits(spec_handle_t h, int level, const void *states /*dev bf16 [rows, d_inner]*/, int rows,
                     float *logits, void *cuda_stream);
int spec_head_topk(spec_handle_t h, int level, const void *states, int rows, int topk, int32_t *tok, float *logp,
                   void *workspace, size_t workspace_bytes, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPEC_B200_H_ */
