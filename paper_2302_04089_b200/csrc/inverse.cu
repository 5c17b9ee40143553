// Damped float64 inverse of the calibration Hessian (caption of Algorithm 1:
// H^-1 = (2 X X^T + lambda I)^-1), batched over layers.
//
// Route: H + lambda I = C C^T by a left-looking blocked Cholesky (64 x 64 tiles), M = C^-1 by
// block forward substitution along tile anti-diagonals, H^-1 = M^T M.  Everything is float64:
// the greedy loop that follows needs the diagonal of H^-1 to roughly 1e-7 relative, which an
// fp32 factorisation of a matrix with condition number 1e3 .. 1e5 does not give.  The matrix is
// padded to a multiple of 64 with an identity block, whose inverse is again the identity.
#include <math.h>

#include <mutex>

#include "common.cuh"

// Built-in scratch of ziplm_damped_inverse_noalloc: lives in every GPU that loads this library
// until the process exits.  In host code this name is only a handle for cudaGetSymbolAddress,
// never a device address.
constexpr size_t kBuiltinScratchBytes = (size_t)8 << 20;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

namespace ziplm {
namespace {

constexpr int KC = 16;          // k-chunk staged in shared memory per iteration
constexpr int LDS = kTile + 2;  // padded shared-memory row length (doubles)

// acc(64x64) += opA(64xK) * opB(Kx64); 256 threads, thread (ty,tx) owns rows ty+16a, cols tx+16b.
//   TA == false: A stored 64 x K row-major (opA(i,k) = A[i*lda + k]); true: stored K x 64.
//   TB == false: B stored K x 64 row-major (opB(k,j) = B[k*ldb + j]); true: stored 64 x K.
// Ends with __syncthreads(), so the caller may overwrite the operands afterwards.  The operand
// pointers are deliberately not __restrict__: some callers read tiles that the same block wrote
// earlier in the kernel, which must not go through the non-coherent load path.
template <bool TA, bool TB>
__device__ __forceinline__ void dgemm_tile(double (&acc)[4][4], const double* A, int lda,
                                           const double* B, int ldb, int K,
                                           double (*sA)[LDS], double (*sB)[LDS]) {
    const int tid = threadIdx.x;
    const int ty = tid >> 4, tx = tid & 15;
    for (int k0 = 0; k0 < K; k0 += KC) {
        if (!TA) {
            const int i = tid >> 2, kq = (tid & 3) * 4;
            const double* src = A + (size_t)i * lda + k0 + kq;
            const double2 v0 = *reinterpret_cast<const double2*>(src);
            const double2 v1 = *reinterpret_cast<const double2*>(src + 2);
            sA[kq][i] = v0.x; sA[kq + 1][i] = v0.y; sA[kq + 2][i] = v1.x; sA[kq + 3][i] = v1.y;
        } else {
            const int kk = tid >> 4, iq = (tid & 15) * 4;
            const double* src = A + (size_t)(k0 + kk) * lda + iq;
            const double2 v0 = *reinterpret_cast<const double2*>(src);
            const double2 v1 = *reinterpret_cast<const double2*>(src + 2);
            sA[kk][iq] = v0.x; sA[kk][iq + 1] = v0.y; sA[kk][iq + 2] = v1.x; sA[kk][iq + 3] = v1.y;
        }
        if (!TB) {
            const int kk = tid >> 4, jq = (tid & 15) * 4;
            const double* src = B + (size_t)(k0 + kk) * ldb + jq;
            const double2 v0 = *reinterpret_cast<const double2*>(src);
            const double2 v1 = *reinterpret_cast<const double2*>(src + 2);
            sB[kk][jq] = v0.x; sB[kk][jq + 1] = v0.y; sB[kk][jq + 2] = v1.x; sB[kk][jq + 3] = v1.y;
        } else {
            const int j = tid >> 2, kq = (tid & 3) * 4;
            const double* src = B + (size_t)j * ldb + k0 + kq;
            const double2 v0 = *reinterpret_cast<const double2*>(src);
            const double2 v1 = *reinterpret_cast<const double2*>(src + 2);
            sB[kq][j] = v0.x; sB[kq + 1][j] = v0.y; sB[kq + 2][j] = v1.x; sB[kq + 3][j] = v1.y;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < KC; ++kk) {
            double a[4], b[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) { a[q] = sA[kk][ty + 16 * q]; b[q] = sB[kk][tx + 16 * q]; }
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[p][q] = fma(a[p], b[q], acc[p][q]);
        }
        __syncthreads();
    }
}

__device__ __forceinline__ void zero_acc(double (&acc)[4][4]) {
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[p][q] = 0.0;
}

// lambda[l] = damp_frac * mean(diag H[l]); flags non-finite diagonals and non-positive means.
__global__ void __launch_bounds__(256) k_mean_diag(const float* __restrict__ H, int d,
                                                   float damp_frac, double* __restrict__ lam,
                                                   int* layer_status) {
    const int l = blockIdx.x;
    const float* Hl = H + (size_t)l * d * d;
    double s = 0.0;
    bool bad = false;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = Hl[(size_t)i * d + i];
        if (!isfinite(v)) bad = true;
        s += (double)v;
    }
    __shared__ double red[256];
    __shared__ int sbad;
    if (threadIdx.x == 0) sbad = 0;
    __syncthreads();
    if (bad) sbad = 1;
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double mean = red[0] / (double)d;
        double lm = (double)damp_frac * mean;
        if (sbad || !isfinite(mean)) {
            set_layer_status(layer_status, l, ZIPLM_ERR_NONFINITE);
            lm = 1.0;
        } else if (damp_frac > 0.f && !(mean > 0.0)) {
            set_layer_status(layer_status, l, ZIPLM_ERR_NOT_PD);
            lm = 1.0;
        }
        lam[l] = lm;
    }
}

// C = H + lambda I on the d x d corner, identity on the padding (dp x dp, float64).
__global__ void __launch_bounds__(256) k_fill_damped(const float* __restrict__ H, int d, int dp,
                                                     const double* __restrict__ lam,
                                                     double* __restrict__ C, int* layer_status) {
    const int l = blockIdx.z;
    const int row = blockIdx.y * 16 + (threadIdx.x >> 4);
    const int col0 = blockIdx.x * 64 + (threadIdx.x & 15) * 4;
    if (row >= dp) return;
    const float* Hl = H + (size_t)l * d * d;
    double* Cl = C + (size_t)l * dp * dp;
    const double lm = lam[l];
    bool bad = false;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int col = col0 + q;
        if (col >= dp) continue;
        double v;
        if (row < d && col < d) {
            const float h = Hl[(size_t)row * d + col];
            if (!isfinite(h)) bad = true;
            v = (double)h + (row == col ? lm : 0.0);
        } else {
            v = (row == col) ? 1.0 : 0.0;
        }
        Cl[(size_t)row * dp + col] = v;
    }
    if (bad) set_layer_status(layer_status, l, ZIPLM_ERR_NONFINITE);
}

// Left-looking update of block column j: C_ij -= sum_{k<j} C_ik C_jk^T for tiles i >= j.
__global__ void __launch_bounds__(256) k_chol_update(double* C, int dp, int j) {
    __shared__ double sA[KC][LDS], sB[KC][LDS];
    const int l = blockIdx.y;
    const int i = j + blockIdx.x;
    double* Cl = C + (size_t)l * dp * dp;
    double acc[4][4];
    zero_acc(acc);
    dgemm_tile<false, true>(acc, Cl + (size_t)i * kTile * dp, dp, Cl + (size_t)j * kTile * dp, dp,
                            j * kTile, sA, sB);
    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
    double* out = Cl + (size_t)i * kTile * dp + (size_t)j * kTile;
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) out[(size_t)(ty + 16 * p) * dp + tx + 16 * q] -= acc[p][q];
}

// Unblocked Cholesky of the diagonal tile C_jj (in place, lower) and the inverse of its factor.
__global__ void __launch_bounds__(256) k_potf2(double* C, int dp, int T, int j, double* Linv,
                                               int* layer_status) {
    __shared__ double s[kTile][kTile + 1];
    __shared__ double dinv[kTile];   // diagonal of the inverse factor
    __shared__ int sflag;
    const int l = blockIdx.x;
    const int tid = threadIdx.x;
    double* tile = C + (size_t)l * dp * dp + (size_t)j * kTile * dp + (size_t)j * kTile;
    if (tid == 0) sflag = 0;
    for (int e = tid; e < kTile * kTile; e += 256)
        s[e >> 6][e & 63] = tile[(size_t)(e >> 6) * dp + (e & 63)];
    __syncthreads();
    for (int c = 0; c < kTile; ++c) {
        if (tid == 0) {
            double p = s[c][c];
            if (!(p > 0.0) || !isfinite(p)) {   // not positive definite (or NaN): flag, keep going
                if (!sflag) sflag = isfinite(p) ? ZIPLM_ERR_NOT_PD : ZIPLM_ERR_NONFINITE;
                p = 1.0;
            }
            s[c][c] = sqrt(p);
        }
        __syncthreads();
        if (tid > c && tid < kTile) s[tid][c] /= s[c][c];
        __syncthreads();
        // trailing update of the lower triangle: (i, jj) with c < jj <= i < 64
        const int m = kTile - 1 - c;
        for (int e = tid; e < m * m; e += 256) {
            const int i = c + 1 + e / m, jj = c + 1 + e % m;
            if (jj <= i) s[i][jj] -= s[i][c] * s[jj][c];
        }
        __syncthreads();
    }
    // inverse of the lower-triangular factor: thread `cidx` builds column cidx by forward
    // substitution.  Entry (i, cidx), i > cidx, is parked transposed in the unused strict upper
    // triangle of s (slot [cidx][i]); the diagonal goes to dinv.
    if (tid < kTile) {
        const int cidx = tid;
        dinv[cidx] = 1.0 / s[cidx][cidx];
        for (int i = cidx + 1; i < kTile; ++i) {
            double acc = -s[i][cidx] * dinv[cidx];
            for (int k = cidx + 1; k < i; ++k) acc -= s[i][k] * s[cidx][k];
            s[cidx][i] = acc / s[i][i];
        }
    }
    __syncthreads();
    double* li = Linv + ((size_t)l * T + j) * kTile * kTile;
    for (int e = tid; e < kTile * kTile; e += 256) {
        const int i = e >> 6, jj = e & 63;
        tile[(size_t)i * dp + jj] = (jj <= i) ? s[i][jj] : 0.0;
        li[e] = (jj < i) ? s[jj][i] : (jj == i ? dinv[i] : 0.0);
    }
    if (tid == 0 && sflag) set_layer_status(layer_status, l, sflag);
}

// Panel below the diagonal tile: C_ij <- C_ij * inv(C_jj)^T for i > j.
__global__ void __launch_bounds__(256) k_chol_panel(double* C, int dp, int T, int j,
                                                    const double* Linv) {
    __shared__ double sA[KC][LDS], sB[KC][LDS];
    const int l = blockIdx.y;
    const int i = j + 1 + blockIdx.x;
    double* tile = C + (size_t)l * dp * dp + (size_t)i * kTile * dp + (size_t)j * kTile;
    const double* li = Linv + ((size_t)l * T + j) * kTile * kTile;
    double acc[4][4];
    zero_acc(acc);
    dgemm_tile<false, true>(acc, tile, dp, li, kTile, kTile, sA, sB);
    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) tile[(size_t)(ty + 16 * p) * dp + tx + 16 * q] = acc[p][q];
}

// M_jj = inv(C_jj) for every diagonal tile.
__global__ void __launch_bounds__(256) k_trtri_diag(double* M, int dp, int T, const double* Linv) {
    const int l = blockIdx.y, j = blockIdx.x;
    double* tile = M + (size_t)l * dp * dp + (size_t)j * kTile * dp + (size_t)j * kTile;
    const double* li = Linv + ((size_t)l * T + j) * kTile * kTile;
    for (int e = threadIdx.x; e < kTile * kTile; e += 256)
        tile[(size_t)(e >> 6) * dp + (e & 63)] = li[e];
}

// Tiles on anti-diagonal s of M = C^-1:  M_ij = -inv(C_ii) * sum_{k=j}^{i-1} C_ik M_kj, i = j + s.
__global__ void __launch_bounds__(256) k_trtri_offdiag(const double* C, double* M, int dp, int T,
                                                       int s, const double* Linv) {
    __shared__ double sA[KC][LDS], sB[KC][LDS];
    const int l = blockIdx.y;
    const int j = blockIdx.x, i = j + s;
    const double* Cl = C + (size_t)l * dp * dp;
    double* Ml = M + (size_t)l * dp * dp;
    double* tile = Ml + (size_t)i * kTile * dp + (size_t)j * kTile;
    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
    double acc[4][4];
    zero_acc(acc);
    dgemm_tile<false, false>(acc, Cl + (size_t)i * kTile * dp + (size_t)j * kTile, dp,
                             Ml + (size_t)j * kTile * dp + (size_t)j * kTile, dp, s * kTile, sA, sB);
    // park the partial sum in the output tile (this block owns it), then multiply by -inv(C_ii)
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) tile[(size_t)(ty + 16 * p) * dp + tx + 16 * q] = acc[p][q];
    __syncthreads();
    zero_acc(acc);
    dgemm_tile<false, false>(acc, Linv + ((size_t)l * T + i) * kTile * kTile, kTile, tile, dp, kTile,
                             sA, sB);
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) tile[(size_t)(ty + 16 * p) * dp + tx + 16 * q] = -acc[p][q];
}

// H^-1 = M^T M on the lower tiles (i >= j): sum over k >= i of M_ki^T M_kj; writes the cropped
// d x d result as float64 (mirrored to the upper triangle) and/or fp32 strict lower + fp64 diag.
__global__ void __launch_bounds__(256) k_lauum(const double* M, int dp, int T, int d,
                                               double* out64, float* tri32, int pitch32,
                                               double* diag64) {
    __shared__ double sA[KC][LDS], sB[KC][LDS];
    const int l = blockIdx.y;
    // linear tile index -> (i, j), rows of the lower triangle in order i = 0, 1, ...
    int i = 0, rem = blockIdx.x;
    while (rem > i) { rem -= i + 1; ++i; }
    const int j = rem;
    const double* Ml = M + (size_t)l * dp * dp;
    double acc[4][4];
    zero_acc(acc);
    dgemm_tile<true, false>(acc, Ml + (size_t)i * kTile * dp + (size_t)i * kTile, dp,
                            Ml + (size_t)i * kTile * dp + (size_t)j * kTile, dp, (T - i) * kTile, sA,
                            sB);
    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int row = i * kTile + ty + 16 * p, col = j * kTile + tx + 16 * q;
            if (row >= d || col >= d) continue;
            const double v = acc[p][q];
            if (out64 && row >= col) {
                double* o = out64 + (size_t)l * d * d;
                o[(size_t)row * d + col] = v;
                o[(size_t)col * d + row] = v;
            }
            if (tri32 && row > col)
                tri32[(size_t)l * d * pitch32 + (size_t)row * pitch32 + col] = (float)v;
            if (diag64 && row == col) diag64[(size_t)l * d + row] = v;
        }
}

}  // namespace

size_t inverse_workspace_bytes(int L, int d) {
    const int dp = round_up_int(d, kTile), T = dp / kTile;
    Carver c(nullptr);
    c.take<double>((size_t)L * dp * dp);               // C: damped Hessian -> Cholesky factor
    c.take<double>((size_t)L * dp * dp);               // M: inverse of the factor
    c.take<double>((size_t)L * T * kTile * kTile);     // inverses of the diagonal tiles
    c.take<double>((size_t)L);                         // lambda
    return c.off;
}

ziplm_status run_damped_inverse(const float* H, int L, int d, float damp_frac, double* out64,
                                float* tri32, int pitch32, double* diag64, double* lam_out,
                                int* layer_status, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (ws_bytes < inverse_workspace_bytes(L, d)) return ZIPLM_ERR_WORKSPACE;
    const int dp = round_up_int(d, kTile), T = dp / kTile;
    Carver c(ws);
    double* C = c.take<double>((size_t)L * dp * dp);
    double* M = c.take<double>((size_t)L * dp * dp);
    double* Linv = c.take<double>((size_t)L * T * kTile * kTile);
    double* lam = c.take<double>((size_t)L);

    k_mean_diag<<<L, 256, 0, st>>>(H, d, damp_frac, lam, layer_status);
    ZIPLM_CHECK_LAUNCH();
    k_fill_damped<<<dim3(T, dp / 16, L), 256, 0, st>>>(H, d, dp, lam, C, layer_status);
    ZIPLM_CHECK_LAUNCH();
    for (int j = 0; j < T; ++j) {
        if (j > 0) {
            k_chol_update<<<dim3(T - j, L), 256, 0, st>>>(C, dp, j);
            ZIPLM_CHECK_LAUNCH();
        }
        k_potf2<<<L, 256, 0, st>>>(C, dp, T, j, Linv, layer_status);
        ZIPLM_CHECK_LAUNCH();
        if (j + 1 < T) {
            k_chol_panel<<<dim3(T - j - 1, L), 256, 0, st>>>(C, dp, T, j, Linv);
            ZIPLM_CHECK_LAUNCH();
        }
    }
    k_trtri_diag<<<dim3(T, L), 256, 0, st>>>(M, dp, T, Linv);
    ZIPLM_CHECK_LAUNCH();
    for (int s = 1; s < T; ++s) {
        k_trtri_offdiag<<<dim3(T - s, L), 256, 0, st>>>(C, M, dp, T, s, Linv);
        ZIPLM_CHECK_LAUNCH();
    }
    k_lauum<<<dim3(T * (T + 1) / 2, L), 256, 0, st>>>(M, dp, T, d, out64, tri32, pitch32, diag64);
    ZIPLM_CHECK_LAUNCH();
    if (lam_out) {
        ZIPLM_CHECK_CUDA(cudaMemcpyAsync(lam_out, lam, sizeof(double) * L, cudaMemcpyDeviceToDevice, st));
    }
    return ZIPLM_OK;
}

}  // namespace ziplm

// ---------------------------------------------------------------------------------------------
// Variant of the damped inverse for callers that cannot allocate device memory.
namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_builtin_scratch, per device
}  // namespace

extern "C" ziplm_status ziplm_damped_inverse_noalloc(const float* H, int L, int d, float damp_frac,
                                                     double* Hinv, int* layer_status,
                                                     void* cuda_stream) {
    using namespace ziplm;
    if (L < 1 || d < 1 || !H || !Hinv || !layer_status) return ZIPLM_ERR_INVALID_ARG;
    if (!(damp_frac >= 0.f) || !isfinite(damp_frac)) return ZIPLM_ERR_INVALID_ARG;
    if (inverse_workspace_bytes(L, d) > kBuiltinScratchBytes) return ZIPLM_ERR_UNSUPPORTED;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ZIPLM_ERR_CUDA;
    void* scratch = nullptr;
    {
        // once per device, with that device current: turn the symbol into its device address
        std::lock_guard<std::mutex> lk(g_scratch_mu);
        if (!g_scratch_addr[dev]) {
            void* addr = nullptr;
            if (cudaGetSymbolAddress(&addr, g_builtin_scratch) != cudaSuccess || !addr)
                return ZIPLM_ERR_CUDA;
            g_scratch_addr[dev] = addr;
        }
        scratch = g_scratch_addr[dev];
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ZIPLM_CHECK_CUDA(cudaMemsetAsync(layer_status, 0, sizeof(int) * L, st));
    // Every part of the scratch that a kernel reads is written earlier in the same call (the
    // damped copy, the factor, the lower tiles of its inverse, lambda), so nothing left behind
    // by the previous call needs clearing.
    return run_damped_inverse(H, L, d, damp_frac, Hinv, nullptr, 0, nullptr, nullptr, layer_status,
                              scratch, kBuiltinScratchBytes, st);
}
