// Tensor-core GEMM for sm_100a:  C[M, N] = A[M, Kd] * B[N, Kd]^T, bf16 operands (row-major,
// i.e. K-major for both), fp32 accumulation in tensor memory (TMEM).
//
// It serves the two contractions of a speculator stage (Sec. 3.1 of arXiv 2404.19124): the
// projection of the parent states (epilogue mode 0: fp32 store; mode 2: the operands are swapped
// so that the weight matrix fills the 128-row side of the MMA when there are few states, the
// contraction is split over several CTAs and every split stores its partial result transposed)
// and the vocabulary head (epilogue mode 1: the logits tile stays on the SM; each accumulator row
// is reduced to a partial top-k list and a (max, sum-exp) pair, so full logits never reach HBM).
//
// Structure: persistent CTAs, one per SM, static round-robin over (n_tile, m_tile) tiles with
// the m index fastest, so the CTAs that share a weight tile run at the same time and the
// second and third readers hit L2.  192 threads:
//   warp 0      TMA producer: 128-byte-swizzled [128 x 64] A boxes and [block_n x 64] B boxes
//               into a ring of shared-memory stages, completion on "full" mbarriers
//   warp 1      allocates TMEM; one lane issues tcgen05.mma (M = 128, N = block_n, K = 16 per
//               instruction) and commits to the "empty" barrier of the stage and, at the end
//               of a tile, to the "accumulator full" barrier
//   warps 2-5   epilogue: tcgen05.ld of 32 columns at a time, one thread per accumulator row
// Two accumulator stages in TMEM let the epilogue of tile i overlap the MMAs of tile i + 1.
// Every mbarrier wait is bounded; when one runs out the CTA records SPEC_ERR_TIMEOUT in the
// error word, all roles leave their loops, TMEM is released and the kernel returns.
#include <cuda.h>

#include "spec_common.cuh"

namespace spec {

namespace {

constexpr int kBlockM = 128;
constexpr int kBlockK = 64;            // 64 bf16 = 128 bytes = one swizzle span
constexpr int kUmmaK = 16;
constexpr int kThreads = 192;
constexpr int kMaxStages = 12;
constexpr int kSmemLimit = 222 * 1024;   // leaves room on the SM for the small kernels that overlap with this one
constexpr uint32_t kSpinFast = 1u << 14;
constexpr uint32_t kSpinMax = 1u << 24;

struct __align__(8) Barriers {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false when it gave up (or another role already did).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Barriers *bars, int32_t *err) {
    for (uint32_t it = 0; it < kSpinMax; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > kSpinFast) {
            if (bars->abort_flag) return false;
            __nanosleep(64);
        }
    }
    bars->abort_flag = 1;
    report_error(err, SPEC_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
        : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows at a 128-byte
// pitch, groups of 8 rows 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3ffffu) >> 4);        // start address, bits 0-13
    d |= (uint64_t)0 << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024u >> 4) << 32;               // stride byte offset, bits 32-45
    d |= (uint64_t)1 << 46;                          // version, bits 46-47
    d |= (uint64_t)2 << 61;                          // layout type: SWIZZLE_128B
    return d;
}

// Instruction descriptor for kind::f16: D = fp32, A = B = bf16, both K-major, M x N tile.
__device__ __forceinline__ uint32_t make_instr_desc(int m, int n) {
    uint32_t d = 0;
    d |= 1u << 4;                      // D format: F32
    d |= 1u << 7;                      // A format: BF16
    d |= 1u << 10;                     // B format: BF16
    d |= (uint32_t)(n >> 3) << 17;     // N / 8
    d |= (uint32_t)(m >> 4) << 24;     // M / 16
    return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

struct GemmParams {
    int M, N, Kd;
    int block_n, stages, tmem_cols;
    int m_tiles, n_tiles;
    int splits, kb_per_split;   // split-K: tile = (m_tile, n_tile, split), split slowest
    uint32_t stage_bytes, a_bytes;
    GemmEpilogue epi;
    int32_t *err;
};

// ---- epilogue, mode 1 -----------------------------------------------------------------------
// One thread owns one accumulator row.  Data-dependent insertion into a sorted list diverges in
// every warp (each lane inserts at different columns), so the selection is done branch-free:
//   pass 1  streams the tile once: online (max, sum-exp) and the kCap largest VALUES of the row,
//           kept sorted by a min/max network (new_v[j] = max(v[j], min(v[j-1], x)));
//   pass 2  re-reads the tile from TMEM and emits the columns whose value reaches the topk-th
//           largest; equal values are taken in ascending column order, exactly `topk` entries.
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int kCap>
__device__ __forceinline__ void epilogue_topk(const GemmParams &p, uint32_t taddr, int row, bool row_ok, int col0,
                                              int n_tile) {
    constexpr float kLog2e = 1.4426950408889634f;
    float best[kCap];
#pragma unroll
    for (int j = 0; j < kCap; ++j) best[j] = -INFINITY;
    float run_m = -INFINITY, run_s = 0.0f;
    for (int c = 0; c < p.block_n; c += 32) {
        float v[32];
        tmem_ld32(taddr + c, v);
        const int valid = p.N - (col0 + c);   // columns of this chunk inside the vocabulary
        if (valid < 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i >= valid) v[i] = -INFINITY;
        }
        float cm0 = fmaxf(v[0], v[1]), cm1 = fmaxf(v[2], v[3]);
#pragma unroll
        for (int i = 4; i < 32; i += 2) {
            cm0 = fmaxf(cm0, v[i]);
            cm1 = fmaxf(cm1, v[i + 1]);
        }
        const float cm = fmaxf(cm0, cm1);
        if (cm > run_m) {
            run_s *= ex2_approx((run_m - cm) * kLog2e);
            run_m = cm;
        }
        const float ms = run_m * kLog2e;
        float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            s0 += ex2_approx(fmaf(v[i], kLog2e, -ms));
            s1 += ex2_approx(fmaf(v[i + 1], kLog2e, -ms));
            s2 += ex2_approx(fmaf(v[i + 2], kLog2e, -ms));
            s3 += ex2_approx(fmaf(v[i + 3], kLog2e, -ms));
        }
        if (run_m > -INFINITY) run_s += (s0 + s1) + (s2 + s3);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float x = v[i];
#pragma unroll
            for (int j = kCap - 1; j > 0; --j) best[j] = fmaxf(best[j], fminf(best[j - 1], x));
            best[0] = fmaxf(best[0], x);
        }
    }
    // threshold = topk-th largest value of the row in this tile; how many entries lie strictly above it
    const int topk = p.epi.topk;
    float thr = best[0];
#pragma unroll
    for (int j = 1; j < kCap; ++j)
        if (j < topk) thr = best[j];
    int above = 0;
#pragma unroll
    for (int j = 0; j < kCap; ++j)
        if (j < topk && best[j] > thr) ++above;
    int eq_left = topk - above;
    const size_t u = (size_t)row * p.n_tiles + n_tile;
    float *pv = p.epi.part_val + u * SPEC_MAX_TOPK;
    int32_t *pi = p.epi.part_idx + u * SPEC_MAX_TOPK;
    int cnt = 0;
    for (int c = 0; c < p.block_n; c += 32) {
        float v[32];
        tmem_ld32(taddr + c, v);
        const int valid = p.N - (col0 + c);
        // candidates of this chunk as a bit mask: no per-element branches
        uint32_t mask = 0;
#pragma unroll
        for (int i = 0; i < 32; ++i) mask |= (v[i] >= thr ? 1u : 0u) << i;
        if (valid < 32) mask &= valid > 0 ? ((1u << valid) - 1u) : 0u;
        if (!row_ok) mask = 0;
        while (mask) {   // ascending columns; a handful of iterations per tile
            const int bpos = __ffs(mask) - 1;
            mask &= mask - 1;
            // x = v[bpos] through a select tree (bpos is data dependent, v lives in registers)
            float t16[16], t8[8], t4[4], t2[2];
#pragma unroll
            for (int i = 0; i < 16; ++i) t16[i] = (bpos & 1) ? v[2 * i + 1] : v[2 * i];
#pragma unroll
            for (int i = 0; i < 8; ++i) t8[i] = (bpos & 2) ? t16[2 * i + 1] : t16[2 * i];
#pragma unroll
            for (int i = 0; i < 4; ++i) t4[i] = (bpos & 4) ? t8[2 * i + 1] : t8[2 * i];
#pragma unroll
            for (int i = 0; i < 2; ++i) t2[i] = (bpos & 8) ? t4[2 * i + 1] : t4[2 * i];
            const float x = (bpos & 16) ? t2[1] : t2[0];
            const bool gt = x > thr;
            if (gt || eq_left > 0) {
                if (!gt) --eq_left;
                if (cnt < topk) {
                    pv[cnt] = x;
                    pi[cnt] = col0 + c + bpos;
                }
                ++cnt;
            }
        }
    }
    if (row_ok) {
        for (; cnt < topk; ++cnt) {   // fewer than topk comparable values (NaN rows, tiny tiles)
            pv[cnt] = -INFINITY;
            pi[cnt] = 0x7fffffff;
        }
        p.epi.part_ms[2 * u] = run_m;
        p.epi.part_ms[2 * u + 1] = run_s;
    }
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // the swizzled tiles need 1024-byte alignment
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    Barriers *bars = (Barriers *)(tiles + (size_t)p.stages * p.stage_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (p.Kd + kBlockK - 1) / kBlockK;
    const int mn_tiles = p.m_tiles * p.n_tiles;
    const int num_tiles = mn_tiles * p.splits;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->acc_full[a], 1);
            mbar_init(&bars->acc_empty[a], 4);   // one arrival per epilogue warp
        }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    griddep_launch();   // the next kernel in the stream may start its own set-up now
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            // Which operand holds the weights (written by no kernel) and which the states (written by
            // the preceding kernel): the first fill of the ring fetches weights only, then waits for
            // the preceding grid, then adds the states.
            const bool w_is_a = p.epi.mode == 2;
            int n_pre = 0;
            if ((int)blockIdx.x < num_tiles) {
                const int tile = blockIdx.x;
                const int split = tile / mn_tiles, mn = tile - split * mn_tiles;
                const int m_tile = mn % p.m_tiles, n_tile = mn / p.m_tiles;
                const int kb0 = split * p.kb_per_split, kb1 = min(num_kb, kb0 + p.kb_per_split);
                n_pre = min(p.stages, kb1 - kb0);
                for (int i = 0; i < n_pre; ++i) {
                    uint8_t *sa = tiles + (size_t)i * p.stage_bytes;
                    mbar_arrive_expect_tx(&bars->full[i], p.stage_bytes);
                    if (w_is_a) tma_load_2d(sa, &tmap_a, (kb0 + i) * kBlockK, m_tile * kBlockM, &bars->full[i]);
                    else tma_load_2d(sa + p.a_bytes, &tmap_b, (kb0 + i) * kBlockK, n_tile * p.block_n, &bars->full[i]);
                }
            }
            griddep_wait();
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;   // k blocks issued so far; also bounds the abort path's wait for copies in flight
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int split = tile / mn_tiles, mn = tile - split * mn_tiles;
                const int m_tile = mn % p.m_tiles, n_tile = mn / p.m_tiles;
                const int kb0 = split * p.kb_per_split, kb1 = min(num_kb, kb0 + p.kb_per_split);
                for (int kb = kb0; kb < kb1; ++kb) {
                    uint8_t *sa = tiles + (size_t)stage * p.stage_bytes;
                    uint8_t *sb = sa + p.a_bytes;
                    const bool prefetched = issued < n_pre;   // weights of this stage are already on their way
                    if (!prefetched) {
                        if (!mbar_wait(&bars->empty[stage], phase ^ 1u, bars, p.err)) { ok = false; break; }
                        mbar_arrive_expect_tx(&bars->full[stage], p.stage_bytes);
                    }
                    if (!prefetched || !w_is_a) tma_load_2d(sa, &tmap_a, kb * kBlockK, m_tile * kBlockM, &bars->full[stage]);
                    if (!prefetched || w_is_a) tma_load_2d(sb, &tmap_b, kb * kBlockK, n_tile * p.block_n, &bars->full[stage]);
                    ++issued;
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // let the copies already in flight land before this CTA's shared memory is released
                const int pending = issued < p.stages ? issued : p.stages;
                int s = stage;
                uint32_t ph = phase;
                for (int i = 0; i < pending; ++i) {
                    if (--s < 0) { s = p.stages - 1; ph ^= 1u; }
                    for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(&bars->full[s], ph); ++it) __nanosleep(32);
                }
            }
        } else {
            griddep_wait();
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        griddep_wait();
        if (lane == 0) {
            const uint32_t idesc = make_instr_desc(kBlockM, p.block_n);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                if (!mbar_wait(&bars->acc_empty[acc], acc_phase ^ 1u, bars, p.err)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * p.block_n);
                const int split = tile / mn_tiles;
                const int kb0 = split * p.kb_per_split, kb1 = min(num_kb, kb0 + p.kb_per_split);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(&bars->full[stage], phase, bars, p.err)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(tiles + (size_t)stage * p.stage_bytes);
                    const uint32_t sb = sa + p.a_bytes;
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                        const uint64_t adesc = make_smem_desc(sa + k * kUmmaK * 2);
                        const uint64_t bdesc = make_smem_desc(sb + k * kUmmaK * 2);
                        umma_bf16(tmem_d, adesc, bdesc, idesc, ((kb - kb0) | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(&bars->empty[stage]);   // frees the stage once these MMAs have read it
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(&bars->acc_full[acc]);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        griddep_wait();
        const int quarter = warp & 3;               // TMEM lane quarter this warp may read
        const int row_in_tile = quarter * 32 + lane;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            const int split = tile / mn_tiles, mn = tile - split * mn_tiles;
            const int m_tile = mn % p.m_tiles, n_tile = mn / p.m_tiles;
            if (!mbar_wait(&bars->acc_full[acc], acc_phase, bars, p.err)) { ok = false; break; }
            tc_fence_after();
            const int row = m_tile * kBlockM + row_in_tile;
            const bool row_ok = row < p.M;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * p.block_n);
            const int col0 = n_tile * p.block_n;
            if (p.epi.mode == 0) {
                for (int c = 0; c < p.block_n; c += 32) {
                    float v[32];
                    tmem_ld32(taddr + c, v);
                    if (row_ok) {
                        float *dst = p.epi.out + (size_t)row * p.epi.ldc + col0 + c;
                        const int valid = p.N - (col0 + c);
                        if (valid >= 32 && (((uintptr_t)dst) & 15) == 0) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4)
                                *(float4 *)(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (i < valid) dst[i] = v[i];
                        }
                    }
                }
            } else if (p.epi.mode == 2) {
                // transposed store of one split-K partial: out[split][col][row]; a warp's 32 rows are
                // consecutive addresses, so every store instruction is one 128-byte line
                float *dst0 = p.epi.out + (size_t)split * p.epi.split_stride + row;
                for (int c = 0; c < p.block_n; c += 32) {
                    float v[32];
                    tmem_ld32(taddr + c, v);
                    if (row_ok) {
                        const int valid = p.N - (col0 + c);
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (i < valid) dst0[(size_t)(col0 + c + i) * p.epi.ldc] = v[i];
                    }
                }
            } else {
                if (p.epi.topk <= 4) epilogue_topk<4>(p, taddr, row, row_ok, col0, n_tile);
                else epilogue_topk<SPEC_MAX_TOPK>(p, taddr, row, row_ok, col0, n_tile);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc_empty[acc]);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
}

// ---- host side -------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !ptr) {
        set_last_cuda_error((int)(e != cudaSuccess ? e : cudaErrorUnknown));
        return nullptr;
    }
    fn = (EncodeTiledFn)ptr;
    return fn;
}

// 2-D bf16 row-major [rows, cols] tensor, box = [box_rows, 64 columns], 128-byte swizzle.
int make_tmap(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool streamed) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return SPEC_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    streamed ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error((int)r);
        return SPEC_ERR_CUDA;
    }
    return SPEC_OK;
}

}  // namespace

// Columns per tile: a multiple of 32 in [32, 256].  Scores each candidate by how evenly its
// tiles fill the SMs (tiles / (waves * SMs)); among near-equal fills the widest tile wins
// because it re-reads A least often.
int choose_block_n(int M, int N, int num_sm, bool prefer_wide) {
    const int m_tiles = (M + kBlockM - 1) / kBlockM;
    int best = 32;
    double best_score = -1.0;
    for (int bn = 32; bn <= 256; bn += 32) {
        const long long tiles = (long long)m_tiles * ((N + bn - 1) / bn);
        const long long waves = (tiles + num_sm - 1) / num_sm;
        double fill = (double)tiles / (double)(waves * num_sm);
        // wasted columns of the ragged last tile count against the candidate
        fill *= (double)N / (double)(((N + bn - 1) / bn) * (long long)bn);
        const double score = fill + (prefer_wide ? 0.0004 : 0.0001) * bn;
        if (score > best_score + 1e-9) {
            best_score = score;
            best = bn;
        }
    }
    return best;
}

int launch_gemm_tc(const void *A, const void *B, int M, int N, int Kd, int block_n, const GemmEpilogue &epi,
                   int32_t *err, cudaStream_t st) {
    if (M <= 0 || N <= 0 || Kd <= 0 || Kd % 8 != 0 || block_n < 32 || block_n > 256 || block_n % 32 != 0)
        return SPEC_ERR_SHAPE;
    if (((uintptr_t)A & 15) || ((uintptr_t)B & 15)) return SPEC_ERR_INVALID_ARG;
    CUtensorMap ta, tb;
    int rc = make_tmap(&ta, A, (uint64_t)M, (uint64_t)Kd, kBlockM, false);
    if (rc != SPEC_OK) return rc;
    rc = make_tmap(&tb, B, (uint64_t)N, (uint64_t)Kd, (uint32_t)block_n, true);
    if (rc != SPEC_OK) return rc;

    GemmParams p{};
    p.M = M; p.N = N; p.Kd = Kd;
    p.block_n = block_n;
    p.a_bytes = kBlockM * kBlockK * 2;
    p.stage_bytes = p.a_bytes + (uint32_t)block_n * kBlockK * 2;
    const int budget = kSmemLimit - 1024 - (int)sizeof(Barriers) - 64;
    p.stages = budget / (int)p.stage_bytes;
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    if (p.stages < 2) return SPEC_ERR_SHAPE;
    int cols = 32;
    while (cols < 2 * block_n) cols <<= 1;
    p.tmem_cols = cols;
    p.m_tiles = (M + kBlockM - 1) / kBlockM;
    p.n_tiles = (N + block_n - 1) / block_n;
    p.epi = epi;
    p.err = err;
    const int num_kb = (Kd + kBlockK - 1) / kBlockK;
    p.splits = epi.mode == 2 && epi.splits > 1 ? epi.splits : 1;
    p.kb_per_split = (num_kb + p.splits - 1) / p.splits;
    if ((p.splits - 1) * p.kb_per_split >= num_kb) return SPEC_ERR_SHAPE;   // every split must own a K block

    const size_t smem = 1024 + (size_t)p.stages * p.stage_bytes + sizeof(Barriers);
    static bool attr_set[64] = {};
    int dev = 0;
    SPEC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        SPEC_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    const long long tiles = (long long)p.m_tiles * p.n_tiles * p.splits;
    const int grid = (int)(tiles < num_sms() ? tiles : num_sms());
    SPEC_CUDA_TRY(launch_pdl(gemm_tc_kernel, dim3(grid), dim3(kThreads), smem, st, ta, tb, p));
    return SPEC_OK;
}

}  // namespace spec
