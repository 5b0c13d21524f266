// Debug-only CUDA-core kernels: a plain tiled GEMM that writes full fp32 logits and a scan
// that turns full logits into the per-tile partial lists the fused tensor-core epilogue
// produces.  They exist to bisect faults in the tcgen05 path (SPEC_OPT_GEMM_IMPL = 1) and are
// never selected by default.
#include "spec_common.cuh"

namespace spec {

namespace {

constexpr int kTile = 64, kTk = 32;

// C[M, N] = A[M, Kd] * B[N, Kd]^T; 16x16 threads, each a 4x4 block of C.
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const uint16_t *__restrict__ A, const uint16_t *__restrict__ B, int M, int N, int Kd,
                 float *__restrict__ C, int ldc) {
    __shared__ float As[kTk][kTile + 1], Bs[kTk][kTile + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int m0 = blockIdx.y * kTile, n0 = blockIdx.x * kTile;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < Kd; k0 += kTk) {
        for (int i = threadIdx.x; i < kTile * kTk; i += 256) {
            const int r = i / kTk, c = i - r * kTk;
            const int gm = m0 + r, gn = n0 + r, gk = k0 + c;
            As[c][r] = (gm < M && gk < Kd) ? bf16_bits_to_float(A[(size_t)gm * Kd + gk]) : 0.0f;
            Bs[c][r] = (gn < N && gk < Kd) ? bf16_bits_to_float(B[(size_t)gn * Kd + gk]) : 0.0f;
        }
        __syncthreads();
#pragma unroll 8
        for (int c = 0; c < kTk; ++c) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                a[i] = As[c][ty * 4 + i];
                b[i] = Bs[c][tx * 4 + i];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gm = m0 + ty * 4 + i, gn = n0 + tx * 4 + j;
            if (gm < M && gn < N) C[(size_t)gm * ldc + gn] = acc[i][j];
        }
}

// One thread per (row, tile): serial scan of the tile's columns.
__global__ void partials_from_logits_kernel(const float *__restrict__ logits, int M, int N, int block_n, int n_tiles,
                                            int topk, float *__restrict__ part_val, int32_t *__restrict__ part_idx,
                                            float *__restrict__ part_ms) {
    const long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= (long long)M * n_tiles) return;
    const int r = (int)(u / n_tiles), t = (int)(u - (long long)r * n_tiles);
    const float *x = logits + (size_t)r * N;
    const int c0 = t * block_n, c1 = min(N, c0 + block_n);
    float *pv = part_val + (size_t)u * SPEC_MAX_TOPK;
    int32_t *pi = part_idx + (size_t)u * SPEC_MAX_TOPK;
    for (int j = 0; j < topk; ++j) {
        pv[j] = -INFINITY;
        pi[j] = 0x7fffffff;
    }
    float m = -INFINITY;
    for (int c = c0; c < c1; ++c) m = fmaxf(m, x[c]);
    float s = 0.0f;
    for (int c = c0; c < c1; ++c) {
        const float v = x[c];
        s += expf(v - m);
        if (v > pv[topk - 1]) {
            int j = topk - 1;
            while (j > 0 && v > pv[j - 1]) {
                pv[j] = pv[j - 1];
                pi[j] = pi[j - 1];
                --j;
            }
            pv[j] = v;
            pi[j] = c;
        }
    }
    part_ms[2 * u] = m;
    part_ms[2 * u + 1] = s;
}

}  // namespace

int launch_gemm_simt(const void *A, const void *B, int M, int N, int Kd, float *C, int ldc, cudaStream_t st) {
    dim3 grid((N + kTile - 1) / kTile, (M + kTile - 1) / kTile);
    gemm_simt_kernel<<<grid, 256, 0, st>>>((const uint16_t *)A, (const uint16_t *)B, M, N, Kd, C, ldc);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_partials_from_logits(const float *logits, int M, int N, int block_n, int topk, float *part_val,
                                int32_t *part_idx, float *part_ms, cudaStream_t st) {
    const int n_tiles = (N + block_n - 1) / block_n;
    const long long units = (long long)M * n_tiles;
    partials_from_logits_kernel<<<(unsigned)((units + 127) / 128), 128, 0, st>>>(logits, M, N, block_n, n_tiles, topk,
                                                                                 part_val, part_idx, part_ms);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

}  // namespace spec
