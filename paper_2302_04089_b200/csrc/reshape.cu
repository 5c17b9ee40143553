// Model reshaping (Sec. 3.1, "Pruned structures"): once the columns of removed structures are
// zero, they are dropped from this matrix and the matching rows are dropped from the previous
// layer (FC1 rows and bias for neurons; the Q, K, V rows of a head) without any output change.
//
//   k_kept_structures   order[l][0 .. G-level) -> ascending list of the `level` survivors
//   k_gather_columns    out[l][i][k*g + c] = M[l][i][kept[l][k]*g + c]
//   k_gather_rows       out[l][k*g + c][:] = M[l][kept[l][k]*g + c][:]
//
// All three only move data: results are bit-exact.
#include "common.cuh"

namespace ziplm {
namespace {

constexpr int KEEP_THREADS = 1024;

// One CTA per layer.  The removed structures are marked in a bitmap in shared memory; every thread
// then owns a contiguous chunk of structure indices, counts its survivors, an exclusive scan
// over the threads gives the chunk's first output slot, and the chunk is written in order.
// bad[l] becomes ZIPLM_ERR_INVALID_ARG when order[l][0 .. G-level) is not a list of distinct
// indices in [0, G).
__global__ void __launch_bounds__(KEEP_THREADS) k_kept_structures(const int* __restrict__ order, int G,
                                                                  int level, int* __restrict__ kept,
                                                                  int* __restrict__ bad) {
    extern __shared__ unsigned int sm[];
    unsigned int* bits = sm;                                  // ceil(G / 32) words
    const int words = (G + 31) / 32;
    int* sums = reinterpret_cast<int*>(sm + words);           // KEEP_THREADS partial counts
    __shared__ int fail;
    const int l = blockIdx.x, tid = threadIdx.x;
    const int* ord = order + (size_t)l * G;
    if (tid == 0) fail = 0;
    for (int w = tid; w < words; w += KEEP_THREADS) bits[w] = 0u;
    __syncthreads();
    const int n_removed = G - level;
    for (int t = tid; t < n_removed; t += KEEP_THREADS) {
        const int s = ord[t];
        if (s < 0 || s >= G) {
            fail = 1;
        } else {
            const unsigned int m = 1u << (s & 31);
            if (atomicOr(&bits[s >> 5], m) & m) fail = 1;     // listed twice
        }
    }
    __syncthreads();
    const int chunk = (G + KEEP_THREADS - 1) / KEEP_THREADS;
    const int lo = tid * chunk, hi = min(lo + chunk, G);
    int cnt = 0;
    for (int s = lo; s < hi; ++s) cnt += !((bits[s >> 5] >> (s & 31)) & 1u);
    sums[tid] = cnt;
    __syncthreads();
    // inclusive Hillis-Steele scan over the per-thread counts
    for (int off = 1; off < KEEP_THREADS; off <<= 1) {
        const int v = (tid >= off) ? sums[tid - off] : 0;
        __syncthreads();
        sums[tid] += v;
        __syncthreads();
    }
    int pos = sums[tid] - cnt;
    if (tid == KEEP_THREADS - 1 && sums[tid] != level) fail = 1;
    __syncthreads();
    if (fail) {
        if (tid == 0) bad[l] = (int)ZIPLM_ERR_INVALID_ARG;
        return;
    }
    int* out = kept + (size_t)l * level;
    for (int s = lo; s < hi; ++s)
        if (!((bits[s >> 5] >> (s & 31)) & 1u)) out[pos++] = s;
}

// grid (column chunks, row chunks, layers); a thread moves one element (coalesced on both sides
// within a structure's g columns; for g = 1 the reads are a gather inside one row).
__global__ void __launch_bounds__(256) k_gather_columns(const float* __restrict__ M, long long ld,
                                                        long long layer_stride,
                                                        const int* __restrict__ kept, int rows, int G,
                                                        int g, int level, float* __restrict__ out) {
    const int l = blockIdx.z;
    const int n_out = level * g;
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (j >= n_out) return;
    const int s = kept[(size_t)l * level + j / g];
    const bool ok = (unsigned)s < (unsigned)G;                 // an index outside [0, G) gives zeros
    const int src = s * g + j % g;
    const float* Ml = M + (size_t)l * (size_t)layer_stride;
    float* Ol = out + (size_t)l * rows * n_out;
    const int i0 = blockIdx.y * 16;
#pragma unroll 4
    for (int i = i0; i < min(i0 + 16, rows); ++i)
        Ol[(size_t)i * n_out + j] = ok ? Ml[(size_t)i * (size_t)ld + src] : 0.f;
}

// One CTA per output row and layer; the row is copied with coalesced accesses.
__global__ void __launch_bounds__(256) k_gather_rows(const float* __restrict__ M, long long ld,
                                                     long long layer_stride,
                                                     const int* __restrict__ kept, int cols, int G,
                                                     int g, int level, float* __restrict__ out) {
    const int l = blockIdx.y;
    const int k = blockIdx.x;                                  // output row
    const int s = kept[(size_t)l * level + k / g];
    const bool ok = (unsigned)s < (unsigned)G;                 // an index outside [0, G) gives zeros
    const float* row = M + (size_t)l * (size_t)layer_stride + (size_t)(ok ? s * g + k % g : 0) * (size_t)ld;
    float* dst = out + ((size_t)l * level * g + k) * (size_t)cols;
    for (int c = threadIdx.x; c < cols; c += 256) dst[c] = ok ? row[c] : 0.f;
}

}  // namespace

ziplm_status run_kept_structures(const int* order, int L, int G, int level, int* kept, int* bad,
                                 cudaStream_t st) {
    ZIPLM_CHECK_CUDA(cudaMemsetAsync(bad, 0, sizeof(int) * L, st));
    const size_t smem = ((size_t)(G + 31) / 32 + KEEP_THREADS) * 4;
    if (smem > 200 * 1024) return ZIPLM_ERR_UNSUPPORTED;
    if (smem > 48 * 1024)
        ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_kept_structures, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem));
    k_kept_structures<<<L, KEEP_THREADS, smem, st>>>(order, G, level, kept, bad);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

ziplm_status run_gather_columns(const float* M, long long ld, long long layer_stride, const int* kept,
                                int L, int rows, int G, int g, int level, float* out, cudaStream_t st) {
    if (level == 0 || rows == 0) return ZIPLM_OK;
    const int n_out = level * g;
    for (int l0 = 0; l0 < L; l0 += 65535) {
        const int ln = (L - l0 < 65535) ? (L - l0) : 65535;
        const dim3 grid((unsigned)((n_out + 255) / 256), (unsigned)((rows + 15) / 16), (unsigned)ln);
        if (grid.y > 65535) return ZIPLM_ERR_UNSUPPORTED;
        k_gather_columns<<<grid, 256, 0, st>>>(M + (size_t)l0 * (size_t)layer_stride, ld, layer_stride,
                                               kept + (size_t)l0 * level, rows, G, g, level,
                                               out + (size_t)l0 * rows * n_out);
        ZIPLM_CHECK_LAUNCH();
    }
    return ZIPLM_OK;
}

ziplm_status run_gather_rows(const float* M, long long ld, long long layer_stride, const int* kept,
                             int L, int cols, int G, int g, int level, float* out, cudaStream_t st) {
    if (level == 0 || cols == 0) return ZIPLM_OK;
    for (int l0 = 0; l0 < L; l0 += 65535) {
        const int ln = (L - l0 < 65535) ? (L - l0) : 65535;
        k_gather_rows<<<dim3((unsigned)(level * g), (unsigned)ln), 256, 0, st>>>(
            M + (size_t)l0 * (size_t)layer_stride, ld, layer_stride, kept + (size_t)l0 * level, cols, G, g,
            level, out + (size_t)l0 * level * g * (size_t)cols);
        ZIPLM_CHECK_LAUNCH();
    }
    return ZIPLM_OK;
}

}  // namespace ziplm
