// Calibration Hessian H = beta H + alpha X X^T (caption of Algorithm 1: alpha = 2), batched over
// layers.  X is [d, N] with the token index contiguous, so both operands of the contraction are
// K-major tiles of the same matrix; only tiles on or below the diagonal are computed and the
// result is mirrored (symmetric rank-k update).
//
// This file holds the route choice and the CUDA-core route: fp32 FMA on 64 x 64 tiles with a
// two-level fp32 sum (the running tile sum is folded into a second accumulator every 512 tokens,
// which keeps the rounding error of a 1e4 .. 1e5 term sum near the fp32 unit roundoff).  The
// tensor-core route (hessian_tc.cu) is the default; the CUDA-core route serves token counts
// below one K block and can be forced with ziplm_set_option(ZIPLM_OPT_HESSIAN_ROUTE, 1) for comparison.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace ziplm {
namespace {

constexpr int BK = 16;
constexpr int FOLD = 512;   // tokens between folds of the running sum

template <typename T>
__device__ __forceinline__ void load4(const T* p, float (&v)[4]);

template <>
__device__ __forceinline__ void load4<float>(const float* p, float (&v)[4]) {
    const float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}

template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[4]) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
    v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}

template <>
__device__ __forceinline__ void load4<__half>(const __half* p, float (&v)[4]) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    const __half2 a = *reinterpret_cast<const __half2*>(&t.x), b = *reinterpret_cast<const __half2*>(&t.y);
    v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b);
}

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <>
__device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }

// TOK: the input is token-major, [N, ldx] per layer with the feature index contiguous; element
// (feature i, token k) then sits at k * ldx + i and is fetched with scalar loads.
template <typename T, bool TOK>
__global__ void __launch_bounds__(256) k_syrk_simt(float* __restrict__ H, const T* __restrict__ X,
                                                   int d, long long N, long long ldx, float alpha,
                                                   float beta) {
    __shared__ float sA[BK][64 + 1], sB[BK][64 + 1];
    const int l = blockIdx.y;
    int ti = 0, rem = blockIdx.x;
    while (rem > ti) { rem -= ti + 1; ++ti; }
    const int tj = rem;
    const int i0 = ti * 64, j0 = tj * 64;
    const T* Xl = X + (size_t)l * (TOK ? (size_t)N : (size_t)d) * ldx;
    float* Hl = H + (size_t)l * d * d;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    float acc[4][4], tot[4][4];
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) { acc[p][q] = 0.f; tot[p][q] = 0.f; }

    const int lr = tid >> 2, kq = (tid & 3) * 4;
    for (long long k0 = 0; k0 < N; k0 += BK) {
        float va[4] = {0.f, 0.f, 0.f, 0.f}, vb[4] = {0.f, 0.f, 0.f, 0.f};
        const long long k = k0 + kq;
        if (TOK) {
            for (int e = 0; e < 4; ++e) {
                if (k + e >= N) break;
                const T* pk = Xl + (size_t)(k + e) * ldx;
                if (i0 + lr < d) va[e] = to_f32<T>(pk[i0 + lr]);
                if (j0 + lr < d) vb[e] = to_f32<T>(pk[j0 + lr]);
            }
        } else {
            if (i0 + lr < d) {
                const T* pa = Xl + (size_t)(i0 + lr) * ldx + k;
                if (k + 3 < N) load4<T>(pa, va);
                else
                    for (int e = 0; e < 4; ++e) if (k + e < N) va[e] = to_f32<T>(pa[e]);
            }
            if (j0 + lr < d) {
                const T* pb = Xl + (size_t)(j0 + lr) * ldx + k;
                if (k + 3 < N) load4<T>(pb, vb);
                else
                    for (int e = 0; e < 4; ++e) if (k + e < N) vb[e] = to_f32<T>(pb[e]);
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) { sA[kq + e][lr] = va[e]; sB[kq + e][lr] = vb[e]; }
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
        if (((k0 + BK) % FOLD) == 0) {
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q) { tot[p][q] += acc[p][q]; acc[p][q] = 0.f; }
        }
    }
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = i0 + ty + 16 * p, j = j0 + tx + 16 * q;
            if (i >= d || j >= d || j > i) continue;
            float v = alpha * (tot[p][q] + acc[p][q]);
            if (beta != 0.f) v += Hl[(size_t)i * d + j];
            Hl[(size_t)i * d + j] = v;
            if (i != j) Hl[(size_t)j * d + i] = v;
        }
}

__global__ void k_scale_h(float* __restrict__ H, size_t count, float beta) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) H[i] = (beta == 0.f) ? 0.f : H[i] * beta;
}

bool use_tensor_cores(long long N) {
    if (option_value(ZIPLM_OPT_HESSIAN_ROUTE) == 1) return false;   // CUDA-core kernel
    return N >= 32;
}

}  // namespace

size_t hessian_workspace_bytes(int L, int d, long long n_tokens, ziplm_dtype dt, bool token_major) {
    // the larger of the two routes' needs, whatever route the call will take
    return n_tokens > 0 ? hessian_tc_workspace_bytes(L, d, n_tokens, dt, token_major) : 0;
}

ziplm_status run_hessian(float* H, const void* X, ziplm_dtype dt, bool token_major, int L, int d,
                         long long N, long long ldx, float alpha, float beta, void* ws,
                         size_t ws_bytes, cudaStream_t st) {
    if (N == 0) {
        const size_t count = (size_t)L * d * d;
        if (beta != 1.f) {
            k_scale_h<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(H, count, beta);
            ZIPLM_CHECK_LAUNCH();
        }
        return ZIPLM_OK;
    }
    if (use_tensor_cores(N))
        return run_hessian_tc(H, X, dt, token_major, L, d, N, ldx, alpha, beta, ws, ws_bytes, st);
    const int T = (d + 63) / 64;
    const dim3 grid(T * (T + 1) / 2, L);
    const float* Xf = static_cast<const float*>(X);
    const __nv_bfloat16* Xb = static_cast<const __nv_bfloat16*>(X);
    const __half* Xh = static_cast<const __half*>(X);
    if (dt == ZIPLM_F32 && !token_major)
        k_syrk_simt<float, false><<<grid, 256, 0, st>>>(H, Xf, d, N, ldx, alpha, beta);
    else if (dt == ZIPLM_F32)
        k_syrk_simt<float, true><<<grid, 256, 0, st>>>(H, Xf, d, N, ldx, alpha, beta);
    else if (dt == ZIPLM_BF16 && !token_major)
        k_syrk_simt<__nv_bfloat16, false><<<grid, 256, 0, st>>>(H, Xb, d, N, ldx, alpha, beta);
    else if (dt == ZIPLM_BF16)
        k_syrk_simt<__nv_bfloat16, true><<<grid, 256, 0, st>>>(H, Xb, d, N, ldx, alpha, beta);
    else if (!token_major)
        k_syrk_simt<__half, false><<<grid, 256, 0, st>>>(H, Xh, d, N, ldx, alpha, beta);
    else
        k_syrk_simt<__half, true><<<grid, 256, 0, st>>>(H, Xh, d, N, ldx, alpha, beta);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

}  // namespace ziplm
