// base_loss[l] = ||W X||_F^2 = 1/2 tr(W H W^T) with the undamped H = 2 X X^T: the denominator of
// the relative layer error p_s of Sec. 3.2 ("Structured SPDY search").
#include "common.cuh"

namespace ziplm {
namespace {

constexpr int BK = 16;

// One 64 x 64 tile of T = W H, immediately contracted with the matching tile of W.
__global__ void __launch_bounds__(256) k_base_loss(const float* __restrict__ W,
                                                   const float* __restrict__ H, int r, int d,
                                                   double* __restrict__ acc64) {
    __shared__ float sA[BK][64 + 1], sB[BK][64 + 1];
    __shared__ double red[8];
    const int l = blockIdx.z;
    const int j0 = blockIdx.x * 64, i0 = blockIdx.y * 64;
    const float* Wl = W + (size_t)l * r * d;
    const float* Hl = H + (size_t)l * d * d;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    float acc[4][4];
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[p][q] = 0.f;
    for (int k0 = 0; k0 < d; k0 += BK) {
        {   // W tile: rows i0.., cols k0..k0+15 -> sA[k][i]
            const int i = tid >> 2, kq = (tid & 3) * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int k = k0 + kq + e;
                sA[kq + e][i] = (i0 + i < r && k < d) ? Wl[(size_t)(i0 + i) * d + k] : 0.f;
            }
        }
        {   // H tile: rows k0..k0+15, cols j0.. -> sB[k][j]
            const int kk = tid >> 4, jq = (tid & 15) * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = j0 + jq + e;
                sB[kk][jq + e] = (k0 + kk < d && j < d) ? Hl[(size_t)(k0 + kk) * d + j] : 0.f;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) { a[q] = sA[kk][ty + 16 * q]; b[q] = sB[kk][tx + 16 * q]; }
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(a[p], b[q], acc[p][q]);
        }
        __syncthreads();
    }
    double s = 0.0;
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = i0 + ty + 16 * p, j = j0 + tx + 16 * q;
            if (i < r && j < d) s += (double)acc[p][q] * (double)Wl[(size_t)i * d + j];
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((tid & 31) == 0) red[tid >> 5] = s;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        atomicAdd(acc64 + l, t);
    }
}

__global__ void k_base_loss_finish(int L, const double* __restrict__ acc64,
                                   float* __restrict__ base_loss) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l < L) base_loss[l] = (float)(0.5 * acc64[l]);
}

}  // namespace

ziplm_status run_base_loss(const float* W, const float* H, int L, int r, int d, double* acc64,
                           float* base_loss, cudaStream_t st) {
    ZIPLM_CHECK_CUDA(cudaMemsetAsync(acc64, 0, sizeof(double) * L, st));
    k_base_loss<<<dim3((d + 63) / 64, (r + 63) / 64, L), 256, 0, st>>>(W, H, r, d, acc64);
    ZIPLM_CHECK_LAUNCH();
    k_base_loss_finish<<<(L + 63) / 64, 64, 0, st>>>(L, acc64, base_loss);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

}  // namespace ziplm
