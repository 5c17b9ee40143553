// Greedy structured OBS for structures of g > 1 consecutive columns (attention heads: g = 64).
//
// With B = (H^-1)[S,S] = C_B C_B^T (Cholesky of the g x g block, once per structure and shared
// by all rows -- remark after Algorithm 1):
//     Y_S = C_B^-1 W[:,S]^T  (g x d_row),   rho_S = ||Y_S||_F^2                    (Eq. 2)
//     P   = C_B^-1 (H^-1)[S,:]  (g x d_col)
//     W    <- W    - Y_S^T P                                                       (Eq. 3)
//     H^-1 <- H^-1 - P^T P                                                         (Eq. 4)
// A layer has only d_col / g structures (12 .. 16 heads), so the loop is a handful of steps and
// latency-bound; the whole state (H^-1, W) is therefore kept in float64, which makes the
// saliencies exact to ~1e-12 and costs nothing measurable.  Removed structures stay in place
// and are skipped through a live mask (their entries never feed later steps).
// Four launches per step for all L layers: score every live structure, select, solve for P and
// Y of the selected structure, rank-g update of the stacked matrix [H^-1; W].
#include <math.h>

#include "common.cuh"

namespace ziplm {
namespace {

constexpr int GMAX = 128;     // widest structure; kernels are instantiated for 64 and 128

struct BlockState {
    int chosen;      // structure selected in the current step
    int bad;         // scratch flag
    double sumrho;   // sum of the saliencies of all removed structures
    double dw2;      // scratch: ||W - W_snap||_F^2 of the snapshot being written
};

// In-place lower Cholesky of the g x g matrix in s (row pitch GM + 1), all threads of the block.
// Returns through *flag a ziplm_status if a pivot is not positive / not finite.
template <int GM>
__device__ void chol_smem(double (*s)[GM + 1], int g, int* flag) {
    const int tid = threadIdx.x, nt = blockDim.x;
    for (int c = 0; c < g; ++c) {
        if (tid == 0) {
            double p = s[c][c];
            if (!(p > 0.0) || !isfinite(p)) {
                if (!*flag) *flag = isfinite(p) ? ZIPLM_ERR_NOT_PD : ZIPLM_ERR_NONFINITE;
                p = 1.0;
            }
            s[c][c] = sqrt(p);
        }
        __syncthreads();
        for (int i = c + 1 + tid; i < g; i += nt) s[i][c] /= s[c][c];
        __syncthreads();
        const int m = g - 1 - c;
        for (int e = tid; e < m * m; e += nt) {
            const int i = c + 1 + e / m, jj = c + 1 + e % m;
            if (jj <= i) s[i][jj] -= s[i][c] * s[jj][c];
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256) k_block_init(const float* __restrict__ W, size_t count,
                                                    double* __restrict__ W64) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) W64[i] = (double)W[i];
}

__global__ void k_block_init_state(int L, int G, BlockState* __restrict__ state,
                                   int* __restrict__ alive) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < L) { state[i].chosen = 0; state[i].bad = 0; state[i].sumrho = 0.0; state[i].dw2 = 0.0; }
    if (i < L * G) alive[i] = 1;
}

// rho_S for every live structure: one block per (structure, layer).  The g x g block lives in
// dynamic shared memory ((GM + 1) * g doubles), GM = 64 or 128 bounding g.
template <int GM>
__global__ void __launch_bounds__(256) k_block_score(int r, int d, int g, int G,
                                                     const double* __restrict__ A,
                                                     const double* __restrict__ W64,
                                                     const int* __restrict__ alive,
                                                     double* __restrict__ rho, int* layer_status) {
    extern __shared__ double dyn_block[];
    double (*sB)[GM + 1] = reinterpret_cast<double (*)[GM + 1]>(dyn_block);
    __shared__ double red[8];
    __shared__ int flag;
    const int l = blockIdx.y, s = blockIdx.x;
    if (!alive[(size_t)l * G + s]) return;
    const int tid = threadIdx.x;
    const double* Al = A + (size_t)l * d * d;
    const double* Wl = W64 + (size_t)l * r * d;
    const int c0 = s * g;
    if (tid == 0) flag = 0;
    for (int e = tid; e < g * g; e += 256) sB[e / g][e % g] = Al[(size_t)(c0 + e / g) * d + c0 + e % g];
    __syncthreads();
    chol_smem<GM>(sB, g, &flag);
    double acc = 0.0;
    for (int i = tid; i < r; i += 256) {
        double y[GM];
        const double* w = Wl + (size_t)i * d + c0;
        for (int k = 0; k < g; ++k) {
            double v = w[k];
            for (int m = 0; m < k; ++m) v -= sB[k][m] * y[m];
            v /= sB[k][k];
            y[k] = v;
            acc += v * v;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((tid & 31) == 0) red[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        rho[(size_t)l * G + s] = t;
        if (flag) set_layer_status(layer_status, l, flag);
    }
}

// rho_S for structures of up to 64 columns without a dependent chain per weight row:
//     rho_S = tr(W[:,S] B^-1 W[:,S]^T) = < C_B^-1 G_S , C_B^-1 >_F ,   G_S = W[:,S]^T W[:,S]
// One block per (structure, layer): Cholesky of B, the g x g Gram block of the structure's weight
// columns as a register-tiled product over the d_row rows, the inverse of the factor (one thread
// per column), the g x g product and the reduction -- all in float64.  The inverse of the factor
// is also written to Cinv[l][s] for the solve kernel of the structure that gets selected.
// Dynamic shared memory: three g x 65 matrices and a 32 x 65 staging tile.
constexpr int GS = 64;                         // widest structure of this kernel
constexpr size_t kScoreGramSmem = sizeof(double) * (3 * GS + 32) * (GS + 1);
__global__ void __launch_bounds__(256) k_block_score_gram(int r, int d, int g, int G,
                                                          const double* __restrict__ A,
                                                          const double* __restrict__ W64,
                                                          const int* __restrict__ alive,
                                                          double* __restrict__ rho,
                                                          double* __restrict__ Cinv, int* layer_status) {
    extern __shared__ double dyn_block[];
    double (*sB)[GS + 1] = reinterpret_cast<double (*)[GS + 1]>(dyn_block);                  // B, then C
    double (*sG)[GS + 1] = reinterpret_cast<double (*)[GS + 1]>(dyn_block + GS * (GS + 1));  // Gram block
    double (*sI)[GS + 1] = reinterpret_cast<double (*)[GS + 1]>(dyn_block + 2 * GS * (GS + 1));  // C^-1
    double (*sW)[GS + 1] = reinterpret_cast<double (*)[GS + 1]>(dyn_block + 3 * GS * (GS + 1));  // 32 rows of W
    __shared__ double red[8];
    __shared__ int flag;
    const int l = blockIdx.y, s = blockIdx.x;
    if (!alive[(size_t)l * G + s]) return;
    const int tid = threadIdx.x;
    const double* Al = A + (size_t)l * d * d;
    const double* Wl = W64 + (size_t)l * r * d;
    const int c0 = s * g;
    if (tid == 0) flag = 0;
    for (int e = tid; e < g * g; e += 256) sB[e / g][e % g] = Al[(size_t)(c0 + e / g) * d + c0 + e % g];
    // Gram block: thread (ty, tx) owns entries (4 ty + a, 4 tx + b); rows of W staged 32 at a time
    const int ty = tid >> 4, tx = tid & 15;
    double acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
    for (int i0 = 0; i0 < r; i0 += 32) {
        __syncthreads();
        for (int e = tid; e < 32 * g; e += 256) {
            const int ii = e / g, k = e % g;
            sW[ii][k] = (i0 + ii < r) ? Wl[(size_t)(i0 + ii) * d + c0 + k] : 0.0;
        }
        __syncthreads();
        if (4 * ty < g && 4 * tx < g) {
#pragma unroll 4
            for (int ii = 0; ii < 32; ++ii) {
                double wa[4], wb[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) { wa[a] = sW[ii][4 * ty + a]; wb[a] = sW[ii][4 * tx + a]; }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) acc[a][b] = fma(wa[a], wb[b], acc[a][b]);
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
            if (4 * ty + a < g && 4 * tx + b < g) sG[4 * ty + a][4 * tx + b] = acc[a][b];
    __syncthreads();
    chol_smem<GS>(sB, g, &flag);
    // C^-1, one thread per column j: column j of the inverse of a lower triangular matrix
    if (tid < g) {
        const int j = tid;
        for (int k = 0; k < j; ++k) sI[k][j] = 0.0;
        for (int k = j; k < g; ++k) {
            double v = (k == j) ? 1.0 : 0.0;
            for (int m = j; m < k; ++m) v -= sB[k][m] * sI[m][j];
            sI[k][j] = v / sB[k][k];
        }
    }
    __syncthreads();
    // rho = sum_{k,j} (C^-1 G)[k][j] * C^-1[k][j]; C^-1 is lower triangular
    double part = 0.0;
    for (int e = tid; e < g * g; e += 256) {
        const int k = e / g, j = e % g;
        if (j > k) continue;
        double t = 0.0;
        for (int m = 0; m <= k; ++m) t = fma(sI[k][m], sG[m][j], t);
        part = fma(t, sI[k][j], part);
    }
    double* Ci = Cinv + ((size_t)l * G + s) * g * g;
    for (int e = tid; e < g * g; e += 256) Ci[e] = sI[e / g][e % g];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if ((tid & 31) == 0) red[tid >> 5] = part;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        rho[(size_t)l * G + s] = t;
        if (flag) set_layer_status(layer_status, l, flag);
    }
}

// Q = C_B^-1 [ (H^-1)[S,:] | W[:,S]^T ] for the selected structure from the stored inverse factor:
// a plain product, one column per thread (g <= 64).
__global__ void __launch_bounds__(256) k_block_solve_inv(int r, int d, int g, int gp, int G,
                                                         const double* __restrict__ A,
                                                         const double* __restrict__ W64,
                                                         const double* __restrict__ Cinv,
                                                         const BlockState* __restrict__ state,
                                                         double* __restrict__ Q) {
    __shared__ double sI[GS * (GS + 1) / 2];       // rows of the lower triangle, packed
    const int l = blockIdx.y, tid = threadIdx.x;
    const double* Al = A + (size_t)l * d * d;
    const double* Wl = W64 + (size_t)l * r * d;
    double* Ql = Q + (size_t)l * gp * (d + r);
    const int chosen = state[l].chosen, c0 = chosen * g;
    const double* Ci = Cinv + ((size_t)l * G + chosen) * g * g;
    for (int e = tid; e < g * g; e += 256) {
        const int k = e / g, m = e % g;
        if (m <= k) sI[k * (k + 1) / 2 + m] = Ci[e];
    }
    __syncthreads();
    const int j = blockIdx.x * 256 + tid;
    if (j >= d + r) return;
    double x[GS];
#pragma unroll
    for (int k = 0; k < GS; ++k)
        x[k] = (k < g) ? ((j < d) ? Al[(size_t)(c0 + k) * d + j] : Wl[(size_t)(j - d) * d + c0 + k]) : 0.0;
    for (int k = 0; k < g; ++k) {
        const double* row = sI + k * (k + 1) / 2;
        double v0 = 0.0, v1 = 0.0;
        int m = 0;
        for (; m + 1 <= k; m += 2) { v0 = fma(row[m], x[m], v0); v1 = fma(row[m + 1], x[m + 1], v1); }
        if (m <= k) v0 = fma(row[m], x[m], v0);
        Ql[(size_t)k * (d + r) + j] = v0 + v1;
    }
    for (int k = g; k < gp; ++k) Ql[(size_t)k * (d + r) + j] = 0.0;
}

// argmin over live structures (ties -> lowest index), bookkeeping.  One block per layer.
__global__ void __launch_bounds__(256) k_block_select(int G, int t, const double* __restrict__ rho,
                                                      int* __restrict__ alive,
                                                      BlockState* __restrict__ state,
                                                      int* __restrict__ order,
                                                      float* __restrict__ saliency,
                                                      int* layer_status) {
    __shared__ double sv[256];
    __shared__ int si[256];
    const int l = blockIdx.x, tid = threadIdx.x;
    double bv = INFINITY;
    int bi = 0x7fffffff;
    for (int s = tid; s < G; s += 256) {
        if (!alive[(size_t)l * G + s]) continue;
        double v = rho[(size_t)l * G + s];
        if (!(v == v)) v = INFINITY;
        if (v < bv || (v == bv && s < bi)) { bv = v; bi = s; }
    }
    sv[tid] = bv; si[tid] = bi;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (tid < o) {
            if (sv[tid + o] < sv[tid] || (sv[tid + o] == sv[tid] && si[tid + o] < si[tid])) {
                sv[tid] = sv[tid + o]; si[tid] = si[tid + o];
            }
        }
        __syncthreads();
    }
    if (tid == 0) {
        const int s = si[0];
        if (!isfinite(sv[0])) set_layer_status(layer_status, l, ZIPLM_ERR_NONFINITE);
        state[l].chosen = s;
        state[l].sumrho += isfinite(sv[0]) ? sv[0] : 0.0;
        alive[(size_t)l * G + s] = 0;
        order[(size_t)l * G + t] = s;
        if (saliency) saliency[(size_t)l * G + t] = (float)sv[0];
    }
}

// Q = C_B^-1 [ (H^-1)[S,:] | W[:,S]^T ]  (gp x (d + r), rows >= g zero) for the selected structure.
template <int GM>
__global__ void __launch_bounds__(256) k_block_solve(int r, int d, int g, int gp,
                                                     const double* __restrict__ A,
                                                     const double* __restrict__ W64,
                                                     const BlockState* __restrict__ state,
                                                     double* __restrict__ Q) {
    extern __shared__ double dyn_block[];
    double (*sB)[GM + 1] = reinterpret_cast<double (*)[GM + 1]>(dyn_block);
    __shared__ int flag;
    const int l = blockIdx.y, tid = threadIdx.x;
    const double* Al = A + (size_t)l * d * d;
    const double* Wl = W64 + (size_t)l * r * d;
    double* Ql = Q + (size_t)l * gp * (d + r);
    const int c0 = state[l].chosen * g;
    if (tid == 0) flag = 0;
    for (int e = tid; e < g * g; e += 256) sB[e / g][e % g] = Al[(size_t)(c0 + e / g) * d + c0 + e % g];
    __syncthreads();
    chol_smem<GM>(sB, g, &flag);
    const int j = blockIdx.x * 256 + tid;
    if (j >= d + r) return;
    double y[GM];
    for (int k = 0; k < g; ++k) {
        double v = (j < d) ? Al[(size_t)(c0 + k) * d + j] : Wl[(size_t)(j - d) * d + c0 + k];
        for (int m = 0; m < k; ++m) v -= sB[k][m] * y[m];
        v /= sB[k][k];
        y[k] = v;
        Ql[(size_t)k * (d + r) + j] = v;
    }
    for (int k = g; k < gp; ++k) Ql[(size_t)k * (d + r) + j] = 0.0;
}

// Stacked rank-g update  [H^-1; W] -= Q^T P  with P = Q[:, :d].  64 x 64 tiles, guarded edges.
__global__ void __launch_bounds__(256) k_block_update(int r, int d, int gp, double* __restrict__ A,
                                                      double* __restrict__ W64,
                                                      const double* __restrict__ Q) {
    __shared__ double sQ[16][64 + 2], sP[16][64 + 2];
    const int l = blockIdx.z;
    const int j0 = blockIdx.x * 64, i0 = blockIdx.y * 64;
    const int ld = d + r;
    const double* Ql = Q + (size_t)l * gp * ld;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    double acc[4][4];
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[p][q] = 0.0;
    for (int k0 = 0; k0 < gp; k0 += 16) {
        const int kk = tid >> 4, cq = (tid & 15) * 4;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int i = i0 + cq + e, j = j0 + cq + e;
            sQ[kk][cq + e] = (i < ld) ? Ql[(size_t)(k0 + kk) * ld + i] : 0.0;
            sP[kk][cq + e] = (j < d) ? Ql[(size_t)(k0 + kk) * ld + j] : 0.0;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            double a[4], b[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) { a[q] = sQ[k][ty + 16 * q]; b[q] = sP[k][tx + 16 * q]; }
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[p][q] = fma(a[p], b[q], acc[p][q]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = i0 + ty + 16 * p, j = j0 + tx + 16 * q;
            if (i >= ld || j >= d) continue;
            double* dst = (i < d) ? (A + (size_t)l * d * d + (size_t)i * d + j)
                                  : (W64 + (size_t)l * r * d + (size_t)(i - d) * d + j);
            *dst -= acc[p][q];
        }
}

// W_snap = W (.) M_R in fp32, and ||W - W_snap||_F^2 for the loss identity.
__global__ void __launch_bounds__(256) k_block_snapshot(int r, int d, int g, int G,
                                                        const float* __restrict__ W,
                                                        const double* __restrict__ W64,
                                                        const int* __restrict__ alive,
                                                        float* __restrict__ W_snap, int n_levels,
                                                        int slot, BlockState* __restrict__ state) {
    __shared__ double red[8];
    const int l = blockIdx.y;
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    double acc = 0.0;
    if (e < (size_t)r * d) {
        const int c = (int)(e % d);
        const float v = alive[(size_t)l * G + c / g] ? (float)W64[(size_t)l * r * d + e] : 0.f;
        W_snap[((size_t)l * n_levels + slot) * (size_t)r * d + e] = v;
        const float df = W[(size_t)l * r * d + e] - v;
        acc = (double)df * (double)df;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        if (t != 0.0) atomicAdd(&state[l].dw2, t);
    }
}

__global__ void k_block_loss(int L, int n_levels, int slot, const double* __restrict__ lam,
                             BlockState* __restrict__ state, float* __restrict__ loss) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= L) return;
    const double v = 0.5 * state[l].sumrho - 0.5 * lam[l] * state[l].dw2;
    loss[(size_t)l * n_levels + slot] = (float)(v > 0.0 ? v : 0.0);
    state[l].dw2 = 0.0;
}

struct BlockWs {
    double* A; double* W64; double* Q; double* rho; double* Cinv; int* alive; BlockState* state; double* lam;
    double* base_acc; void* inv_ws; size_t inv_bytes; int gp; size_t total;
};

BlockWs carve_block(void* ws, int L, int r, int d, int g) {
    BlockWs w;
    const int G = d / g;
    w.gp = round_up_int(g, 16);
    Carver c(ws);
    w.A = c.take<double>((size_t)L * d * d);
    w.W64 = c.take<double>((size_t)L * r * d);
    w.Q = c.take<double>((size_t)L * w.gp * (d + r));
    w.rho = c.take<double>((size_t)L * G);
    w.Cinv = c.take<double>(g <= GS ? (size_t)L * G * g * g : 0);      // inverse factors (g <= 64)
    w.alive = c.take<int>((size_t)L * G);
    w.state = c.take<BlockState>((size_t)L);
    w.lam = c.take<double>((size_t)L);
    w.base_acc = c.take<double>((size_t)L);
    w.inv_bytes = inverse_workspace_bytes(L, d);
    w.inv_ws = c.take<char>(w.inv_bytes);
    w.total = c.off;
    return w;
}

}  // namespace

size_t block_workspace_bytes(int L, int r, int d, int g, int n_levels) {
    (void)n_levels;
    return carve_block(nullptr, L, r, d, g).total;
}

ziplm_status run_prune_blocks(const float* W, const float* H, int L, int r, int d, int g,
                              float damp_frac, const int* levels, int n_levels, float* W_snap,
                              float* loss, float* base_loss, int* order, float* saliency,
                              int* layer_status, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (g > GMAX) return ZIPLM_ERR_UNSUPPORTED;
    if (ws_bytes < block_workspace_bytes(L, r, d, g, n_levels)) return ZIPLM_ERR_WORKSPACE;
    BlockWs w = carve_block(ws, L, r, d, g);
    const int G = d / g;
    ziplm_status s;
    {
        PhaseScope ps(PH_INVERSE, st);
        s = run_damped_inverse(H, L, d, damp_frac, w.A, nullptr, 0, nullptr, w.lam, layer_status,
                               w.inv_ws, w.inv_bytes, st);
    }
    if (s != ZIPLM_OK) return s;
    auto init = [&]() -> ziplm_status {
        PhaseScope ps(PH_INIT, st);
        ZIPLM_CHECK_CUDA(cudaMemsetAsync(order, 0xFF, sizeof(int) * (size_t)L * G, st));
        if (saliency)
            ZIPLM_CHECK_CUDA(cudaMemsetAsync(saliency, 0, sizeof(float) * (size_t)L * G, st));
        const size_t count = (size_t)L * r * d;
        k_block_init<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(W, count, w.W64);
        ZIPLM_CHECK_LAUNCH();
        k_block_init_state<<<(L * G + 255) / 256, 256, 0, st>>>(L, G, w.state, w.alive);
        ZIPLM_CHECK_LAUNCH();
        if (base_loss) return run_base_loss(W, H, L, r, d, w.base_acc, base_loss, st);
        return ZIPLM_OK;
    };
    s = init();
    if (s != ZIPLM_OK) return s;

    auto snapshot = [&](int slot) -> ziplm_status {
        PhaseScope ps(PH_SNAPSHOT, st);
        k_block_snapshot<<<dim3((unsigned)(((size_t)r * d + 255) / 256), L), 256, 0, st>>>(
            r, d, g, G, W, w.W64, w.alive, W_snap, n_levels, slot, w.state);
        ZIPLM_CHECK_LAUNCH();
        k_block_loss<<<(L + 63) / 64, 64, 0, st>>>(L, n_levels, slot, w.lam, w.state, loss);
        ZIPLM_CHECK_LAUNCH();
        return ZIPLM_OK;
    };

    // the g x g block of the score and solve kernels: g rows of GM + 1 doubles
    const size_t blk_smem = sizeof(double) * (size_t)g * ((g <= 64 ? 64 : 128) + 1);
    if (g <= GS)
        ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_block_score_gram, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kScoreGramSmem));
    if (g > 64) {
        ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_block_score<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)blk_smem));
        ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_block_solve<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)blk_smem));
    }
    int n = G, slot = 0;
    if (slot < n_levels && levels[slot] == n) {
        s = snapshot(slot++);
        if (s != ZIPLM_OK) return s;
    }
    const int n_min = n_levels > 0 ? levels[n_levels - 1] : G;
    for (int t = 0; n > n_min; ++t) {
        {
            PhaseScope ps(PH_BLOCK_SCORE, st);
            if (g <= GS)
                k_block_score_gram<<<dim3(G, L), 256, kScoreGramSmem, st>>>(r, d, g, G, w.A, w.W64, w.alive,
                                                                            w.rho, w.Cinv, layer_status);
            else
                k_block_score<128><<<dim3(G, L), 256, blk_smem, st>>>(r, d, g, G, w.A, w.W64, w.alive, w.rho,
                                                                      layer_status);
            ZIPLM_CHECK_LAUNCH();
            k_block_select<<<L, 256, 0, st>>>(G, t, w.rho, w.alive, w.state, order, saliency,
                                              layer_status);
            ZIPLM_CHECK_LAUNCH();
        }
        if (n > 1) {
            PhaseScope ps(PH_BLOCK_UPDATE, st);
            if (g <= GS)
                k_block_solve_inv<<<dim3((d + r + 255) / 256, L), 256, 0, st>>>(r, d, g, w.gp, G, w.A, w.W64,
                                                                               w.Cinv, w.state, w.Q);
            else
                k_block_solve<128><<<dim3((d + r + 255) / 256, L), 256, blk_smem, st>>>(r, d, g, w.gp, w.A, w.W64,
                                                                                       w.state, w.Q);
            ZIPLM_CHECK_LAUNCH();
            k_block_update<<<dim3((d + 63) / 64, (d + r + 63) / 64, L), 256, 0, st>>>(r, d, w.gp, w.A,
                                                                                     w.W64, w.Q);
            ZIPLM_CHECK_LAUNCH();
        }
        --n;
        if (slot < n_levels && levels[slot] == n) {
            s = snapshot(slot++);
            if (s != ZIPLM_OK) return s;
        }
    }
    return ZIPLM_OK;
}

}  // namespace ziplm
