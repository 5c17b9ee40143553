// Greedy one-column-at-a-time structured OBS with delayed (blocked) updates.
//
// Same arithmetic as the streaming neuron path (Algorithm 1 with |M_S| = 1; Eq. 2, 3, 4), but
// the rank-1 updates of a block of up to B steps are kept pending and applied together:
//
//   * Only three things are needed exactly at every step: the saliencies, the pivot column of
//     H^-1 and the pivot column of W.  With Q = W^T W (Gram matrix of the weight columns)
//         rho_k = Q[k,k] / H^-1[k,k]                                               (Eq. 2)
//     and one step (pivot p, h = H^-1[p,p], u = H^-1[:,p]/sqrt(h), q = Q[:,p]/sqrt(h),
//     z = q - Q[p,p]/(2h) u) acts as
//         H^-1 <- H^-1 - u u^T                                                     (Eq. 4)
//         Q    <- Q - z u^T - u z^T      (the Gram matrix of W - c u^T, c = W[:,p]/sqrt(h): Eq. 3)
//     so both diagonals are downdated exactly (float64) from the pivot columns alone, and a
//     pivot column of the true matrix is the stale column minus the pending terms evaluated at
//     p -- O(n * pending) work instead of a pass over n^2 entries.
//   * At the end of a block the pending terms are applied to H^-1, Q and W as rank-B updates
//     (one read + write of each matrix per B steps instead of per step), and the removed
//     positions are squeezed out by a stable, out-of-place compaction, so the live problem is
//     again the leading n x n corner in original column order.
//
// Launches per block, for all L layers at once: one "steps" kernel (one CTA per layer runs the
// B greedy steps back to back with block-level barriers only -- layers are independent, so no
// grid-wide synchronisation is needed) and two update kernels.  Block boundaries are placed on
// the requested levels, where W is up to date and can be snapshotted.
//
// Layout per layer: A, Q fp32 [d, d] strict lower triangles (two buffers each, ping-pong),
// Wt = W^T fp32 [d, rp] (two buffers), float64 diagonals, pending U, Z [B, d] and C [B, rp].
#include <math.h>

#include "common.cuh"

namespace ziplm {
namespace {

constexpr int BMAX = 32;         // pending steps per block
constexpr int STEP_THREADS = 1024;
constexpr int KPT = 4;           // positions per thread in the steps kernel: d <= 4096

struct LazyState {
    double sumrho;
    double dw2;
    int n_new;
    int pad;
};

// Wt = W^T (zero padded to rp), float64 column norms, identity index, state reset.
__global__ void __launch_bounds__(256) k_lazy_init(const float* __restrict__ W, int r, int d, int rp,
                                                   float* __restrict__ Wt, double* __restrict__ dQ,
                                                   int* __restrict__ idx,
                                                   LazyState* __restrict__ state) {
    __shared__ float tile[32][33];
    const int l = blockIdx.y;
    const int c0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const float* Wl = W + (size_t)l * r * d;
    float* Wtl = Wt + (size_t)l * d * rp;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    for (int i0 = 0; i0 < rp; i0 += 32) {
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const int rr = ty + 8 * m;
            const int i = i0 + rr, c = c0 + tx;
            tile[rr][tx] = (i < r && c < d) ? Wl[(size_t)i * d + c] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const int cc = ty + 8 * m;
            const int c = c0 + cc, i = i0 + tx;
            const float v = tile[tx][cc];
            if (c < d && i < rp) Wtl[(size_t)c * rp + i] = v;
            acc[m] += (double)v * (double)v;
        }
        __syncthreads();
    }
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        double s = acc[m];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const int c = c0 + ty + 8 * m;
        if (tx == 0 && c < d) {
            dQ[(size_t)l * d + c] = s;
            idx[(size_t)l * d + c] = c;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        state[l].sumrho = 0.0; state[l].dw2 = 0.0; state[l].n_new = d; state[l].pad = 0;
    }
}

struct Cand {
    double rho, a, q;
    int org, pos;
};

__device__ __forceinline__ bool better(const Cand& x, const Cand& y) {   // x strictly before y
    return x.rho < y.rho || (x.rho == y.rho && x.org < y.org);
}

__device__ __forceinline__ Cand shfl_cand(const Cand& c, int off) {
    Cand o;
    o.rho = __shfl_xor_sync(0xffffffffu, c.rho, off);
    o.a = __shfl_xor_sync(0xffffffffu, c.a, off);
    o.q = __shfl_xor_sync(0xffffffffu, c.q, off);
    o.org = __shfl_xor_sync(0xffffffffu, c.org, off);
    o.pos = __shfl_xor_sync(0xffffffffu, c.pos, off);
    return o;
}

// nsteps greedy steps of one layer per CTA, on the stale matrices plus the pending terms of this
// block; then the stable compaction of the per-position vectors.
__global__ void __launch_bounds__(STEP_THREADS, 1)
k_lazy_steps(int n0, int t0, int nsteps, int d, int G, int r, int rp, const float* __restrict__ A,
             const float* __restrict__ Q, const float* __restrict__ Wt,
             const double* __restrict__ dA_in, const double* __restrict__ dQ_in,
             const int* __restrict__ idx_in, double* __restrict__ dA_out,
             double* __restrict__ dQ_out, int* __restrict__ idx_out, int* __restrict__ src,
             float* U, float* Z, float* C, LazyState* __restrict__ state, int* __restrict__ order,
             float* __restrict__ saliency, int* layer_status) {
    __shared__ Cand s_c[32];
    __shared__ float sUp[BMAX], sZp[BMAX];
    __shared__ int s_p, s_scan[32];
    __shared__ double s_rs, s_half;
    const int l = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* Al = A + (size_t)l * d * d;
    const float* Ql = Q + (size_t)l * d * d;
    const float* Wl = Wt + (size_t)l * d * rp;
    float* Ul = U + (size_t)l * BMAX * d;
    float* Zl = Z + (size_t)l * BMAX * d;
    float* Cl = C + (size_t)l * BMAX * rp;

    double da[KPT], dq[KPT];
    int org[KPT];
    bool alive[KPT];
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        const int k = tid + STEP_THREADS * j;
        alive[j] = k < n0;
        da[j] = alive[j] ? dA_in[(size_t)l * d + k] : 1.0;
        dq[j] = alive[j] ? dQ_in[(size_t)l * d + k] : 0.0;
        org[j] = alive[j] ? idx_in[(size_t)l * d + k] : 0x7fffffff;
    }

    for (int m = 0; m < nsteps; ++m) {
        // ---- argmin of rho = Q[k,k] / H^-1[k,k] over live positions (ties: lowest original index)
        Cand best;
        best.rho = INFINITY; best.a = 1.0; best.q = 0.0; best.org = 0x7fffffff; best.pos = -1;
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            if (!alive[j]) continue;
            Cand c;
            c.rho = dq[j] / da[j];
            if (!(c.rho == c.rho)) c.rho = INFINITY;
            c.a = da[j]; c.q = dq[j]; c.org = org[j]; c.pos = tid + STEP_THREADS * j;
            if (best.pos < 0 || better(c, best)) best = c;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const Cand o = shfl_cand(best, off);
            if (o.pos >= 0 && (best.pos < 0 || better(o, best))) best = o;
        }
        if (lane == 0) s_c[warp] = best;
        __syncthreads();
        if (warp == 0) {
            best = s_c[lane];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const Cand o = shfl_cand(best, off);
                if (o.pos >= 0 && (best.pos < 0 || better(o, best))) best = o;
            }
            if (lane == 0) {
                double h = best.a;
                if (best.pos < 0) best.pos = 0;
                if (!isfinite(best.rho) || !isfinite(h)) {
                    set_layer_status(layer_status, l, ZIPLM_ERR_NONFINITE);
                    h = 1.0;
                } else if (!(h > 0.0)) {
                    set_layer_status(layer_status, l, ZIPLM_ERR_NOT_PD);
                    h = 1.0;
                }
                s_p = best.pos;
                s_rs = 1.0 / sqrt(h);
                s_half = best.q / (2.0 * h);
                state[l].sumrho += isfinite(best.rho) ? best.rho : 0.0;
                order[(size_t)l * G + t0 + m] = best.org;
                if (saliency) saliency[(size_t)l * G + t0 + m] = (float)best.rho;
            }
        }
        __syncthreads();
        const int p = s_p;
        const double rs = s_rs, half = s_half;
        // ---- values of the pending vectors at p
        if (tid < m) {
            sUp[tid] = Ul[(size_t)tid * d + p];
            sZp[tid] = Zl[(size_t)tid * d + p];
        }
        __syncthreads();
        // ---- true pivot columns of H^-1 and Q, float64 downdate of both diagonals
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const int k = tid + STEP_THREADS * j;
            if (k >= n0) continue;
            float u32 = 0.f, z32 = 0.f;
            if (alive[j] && k != p) {
                const size_t off = (k < p) ? ((size_t)p * d + k) : ((size_t)k * d + p);
                double a = (double)Al[off], q = (double)Ql[off];
#pragma unroll 4
                for (int s = 0; s < m; ++s) {
                    const double us = (double)Ul[(size_t)s * d + k], zs = (double)Zl[(size_t)s * d + k];
                    a = fma(-us, (double)sUp[s], a);
                    q = fma(-zs, (double)sUp[s], q);
                    q = fma(-us, (double)sZp[s], q);
                }
                const double u = a * rs;
                const double z = q * rs - half * u;
                da[j] -= u * u;
                dq[j] -= 2.0 * z * u;
                u32 = (float)u;
                z32 = (float)z;
            }
            if (k == p) alive[j] = false;
            Ul[(size_t)m * d + k] = u32;
            Zl[(size_t)m * d + k] = z32;
        }
        // ---- true pivot column of W, scaled: c = W[:,p] / sqrt(h)
        if (tid < rp) {
            double w = (tid < r) ? (double)Wl[(size_t)p * rp + tid] : 0.0;
            for (int s = 0; s < m; ++s) w = fma(-(double)Cl[(size_t)s * rp + tid], (double)sUp[s], w);
            Cl[(size_t)m * rp + tid] = (float)(w * rs);
        }
        __syncthreads();
    }

    // ---- stable compaction of the per-position vectors; src[new] = old position
    int base = 0;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        const int k = tid + STEP_THREADS * j;
        const int f = alive[j] ? 1 : 0;
        int incl = f;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) s_scan[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int w = s_scan[lane], wi = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, wi, o);
                if (lane >= o) wi += v;
            }
            s_scan[lane] = wi - w;          // exclusive prefix of the warp totals
            if (lane == 31) s_p = wi;       // chunk total
        }
        __syncthreads();
        if (f) {
            const int np = base + s_scan[warp] + incl - 1;
            src[(size_t)l * d + np] = k;
            dA_out[(size_t)l * d + np] = da[j];
            dQ_out[(size_t)l * d + np] = dq[j];
            idx_out[(size_t)l * d + np] = org[j];
        }
        base += s_p;
        __syncthreads();
    }
    if (tid == 0) state[l].n_new = base;
}

// Rank-m update of the strict lower triangles of H^-1 and Q with compaction (out of place):
//   A'[i,j] = A[si,sj] - sum_s U[s,si] U[s,sj],
//   Q'[i,j] = Q[si,sj] - sum_s (Z[s,si] U[s,sj] + U[s,si] Z[s,sj]),    si = src[i] > sj = src[j].
// 64 x 64 tiles of the new index space, 4 x 4 elements per thread.
__global__ void __launch_bounds__(256) k_lazy_update_aq(int n_new, int m, int d,
                                                        const float* __restrict__ A,
                                                        const float* __restrict__ Q,
                                                        float* __restrict__ A2, float* __restrict__ Q2,
                                                        const int* __restrict__ src,
                                                        const float* __restrict__ U,
                                                        const float* __restrict__ Z) {
    __shared__ float sUr[BMAX][64], sZr[BMAX][64], sUc[BMAX][64], sZc[BMAX][64];
    __shared__ int srow[64], scol[64];
    const int l = blockIdx.y;
    int ti = 0, rem = blockIdx.x;
    while (rem > ti) { rem -= ti + 1; ++ti; }
    const int tj = rem;
    const int i0 = ti * 64, j0 = tj * 64;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int* sl = src + (size_t)l * d;
    if (tid < 64) srow[tid] = (i0 + tid < n_new) ? sl[i0 + tid] : -1;
    else if (tid < 128) scol[tid - 64] = (j0 + tid - 64 < n_new) ? sl[j0 + tid - 64] : -1;
    __syncthreads();
    const float* Ul = U + (size_t)l * BMAX * d;
    const float* Zl = Z + (size_t)l * BMAX * d;
    for (int e = tid; e < m * 64; e += 256) {
        const int s = e >> 6, c = e & 63;
        const int sr = srow[c], sc = scol[c];
        sUr[s][c] = sr >= 0 ? Ul[(size_t)s * d + sr] : 0.f;
        sZr[s][c] = sr >= 0 ? Zl[(size_t)s * d + sr] : 0.f;
        sUc[s][c] = sc >= 0 ? Ul[(size_t)s * d + sc] : 0.f;
        sZc[s][c] = sc >= 0 ? Zl[(size_t)s * d + sc] : 0.f;
    }
    const float* Al = A + (size_t)l * d * d;
    const float* Ql = Q + (size_t)l * d * d;
    float a[4][4], q[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int i = i0 + ty + 16 * x, j = j0 + tx + 16 * y;
            if (i < n_new && j < i) {
                const size_t off = (size_t)srow[ty + 16 * x] * d + scol[tx + 16 * y];
                a[x][y] = __ldcs(Al + off);
                q[x][y] = __ldcs(Ql + off);
            } else {
                a[x][y] = 0.f; q[x][y] = 0.f;
            }
        }
    __syncthreads();
    for (int s = 0; s < m; ++s) {
        float ur[4], zr[4], uc[4], zc[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            ur[x] = sUr[s][ty + 16 * x]; zr[x] = sZr[s][ty + 16 * x];
            uc[x] = sUc[s][tx + 16 * x]; zc[x] = sZc[s][tx + 16 * x];
        }
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                a[x][y] = fmaf(-ur[x], uc[y], a[x][y]);
                q[x][y] = fmaf(-zr[x], uc[y], q[x][y]);
                q[x][y] = fmaf(-ur[x], zc[y], q[x][y]);
            }
    }
    float* Ao = A2 + (size_t)l * d * d;
    float* Qo = Q2 + (size_t)l * d * d;
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int i = i0 + ty + 16 * x, j = j0 + tx + 16 * y;
            if (i < n_new && j < i) {
                Ao[(size_t)i * d + j] = a[x][y];
                Qo[(size_t)i * d + j] = q[x][y];
            }
        }
}

// Rank-m update of W^T with row compaction (out of place): Wt'[i,:] = Wt[si,:] - sum_s U[s,si] C[s,:].
__global__ void __launch_bounds__(256) k_lazy_update_w(int n_new, int m, int d, int rp,
                                                       const float* __restrict__ Wt,
                                                       float* __restrict__ Wt2,
                                                       const int* __restrict__ src,
                                                       const float* __restrict__ U,
                                                       const float* __restrict__ C) {
    const int l = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * 8 + warp;
    if (i >= n_new) return;
    const int si = src[(size_t)l * d + i];
    const float* Ul = U + (size_t)l * BMAX * d;
    const float4* Cl = reinterpret_cast<const float4*>(C + (size_t)l * BMAX * rp);
    const float4* in = reinterpret_cast<const float4*>(Wt + (size_t)l * d * rp + (size_t)si * rp);
    float4* out = reinterpret_cast<float4*>(Wt2 + (size_t)l * d * rp + (size_t)i * rp);
    float us[BMAX];
#pragma unroll
    for (int s = 0; s < BMAX; ++s) us[s] = (s < m) ? Ul[(size_t)s * d + si] : 0.f;
    const int nvec = rp >> 2;
    for (int v = lane; v < nvec; v += 32) {
        float4 w = __ldcs(in + v);
#pragma unroll
        for (int s = 0; s < BMAX; ++s) {
            if (s < m) {
                const float4 c = __ldg(Cl + (size_t)s * nvec + v);
                w.x = fmaf(-us[s], c.x, w.x); w.y = fmaf(-us[s], c.y, w.y);
                w.z = fmaf(-us[s], c.z, w.z); w.w = fmaf(-us[s], c.w, w.w);
            }
        }
        out[v] = w;
    }
}

__global__ void __launch_bounds__(256) k_lazy_pos_of(int n, int d, const int* __restrict__ idx,
                                                     int* __restrict__ pos_of) {
    const int l = blockIdx.x;
    for (int c = threadIdx.x; c < d; c += blockDim.x) pos_of[(size_t)l * d + c] = -1;
    __syncthreads();
    for (int k = threadIdx.x; k < n; k += blockDim.x)
        pos_of[(size_t)l * d + idx[(size_t)l * d + k]] = k;
}

// W_snap = current weights in original column order, removed columns exactly zero; accumulates
// ||W - W_snap||_F^2 for the loss identity.
__global__ void __launch_bounds__(256) k_lazy_snapshot(int r, int d, int rp,
                                                       const float* __restrict__ W,
                                                       const float* __restrict__ Wt,
                                                       const int* __restrict__ pos_of,
                                                       float* __restrict__ W_snap, int n_levels,
                                                       int slot, LazyState* __restrict__ state) {
    __shared__ float tile[32][33];
    __shared__ double red[8];
    const int l = blockIdx.z;
    const int c0 = blockIdx.x * 32, i0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const float* Wtl = Wt + (size_t)l * d * rp;
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int cc = ty + 8 * m, c = c0 + cc, i = i0 + tx;
        const int pos = (c < d) ? pos_of[(size_t)l * d + c] : -1;
        tile[cc][tx] = (pos >= 0 && i < r) ? Wtl[(size_t)pos * rp + i] : 0.f;
    }
    __syncthreads();
    const float* Wl = W + (size_t)l * r * d;
    float* out = W_snap + ((size_t)l * n_levels + slot) * (size_t)r * d;
    double acc = 0.0;
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int rr = ty + 8 * m, i = i0 + rr, c = c0 + tx;
        if (i < r && c < d) {
            const float v = tile[tx][rr];
            out[(size_t)i * d + c] = v;
            const float df = Wl[(size_t)i * d + c] - v;
            acc += (double)df * (double)df;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (tx == 0) red[ty] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += red[w];
        if (s != 0.0) atomicAdd(&state[l].dw2, s);
    }
}

__global__ void k_lazy_loss(int L, int n_levels, int slot, const double* __restrict__ lam,
                            LazyState* __restrict__ state, float* __restrict__ loss) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= L) return;
    const double v = 0.5 * state[l].sumrho - 0.5 * lam[l] * state[l].dw2;
    loss[(size_t)l * n_levels + slot] = (float)(v > 0.0 ? v : 0.0);
    state[l].dw2 = 0.0;
}

// base_loss = ||W X||_F^2 = 1/2 tr(W H W^T) = 1/2 <W^T W, H>: one elementwise pass over the Gram
// matrix (full symmetric right after the product kernel) and the undamped Hessian.
__global__ void __launch_bounds__(256) k_lazy_base_loss(int d, const float* __restrict__ Q,
                                                        const float* __restrict__ H,
                                                        double* __restrict__ acc64) {
    __shared__ double red[8];
    const int l = blockIdx.y;
    const size_t count = (size_t)d * d / 4;
    const float4* q4 = reinterpret_cast<const float4*>(Q + (size_t)l * d * d);
    const float4* h4 = reinterpret_cast<const float4*>(H + (size_t)l * d * d);
    double acc = 0.0;
    for (size_t e = (size_t)blockIdx.x * 256 + threadIdx.x; e < count; e += (size_t)gridDim.x * 256) {
        const float4 a = __ldg(q4 + e), b = __ldg(h4 + e);
        acc += (double)a.x * b.x + (double)a.y * b.y + (double)a.z * b.z + (double)a.w * b.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        atomicAdd(acc64 + l, t);
    }
}

__global__ void k_lazy_base_finish(int L, const double* __restrict__ acc64,
                                   float* __restrict__ base_loss) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l < L) base_loss[l] = (float)(0.5 * acc64[l]);
}

struct LazyWs {
    float* A[2]; float* Q[2]; float* Wt[2];
    double* dA[2]; double* dQ[2]; int* idx[2];
    int* src; int* pos_of; float* U; float* Z; float* C;
    LazyState* state; double* lam; double* base_acc;
    void* aux; size_t aux_bytes;       // shared by the inverse and by the Gram-matrix product
    int rp; size_t total;
};

LazyWs carve_lazy(void* ws, int L, int r, int d) {
    LazyWs w;
    w.rp = round_up_int(r, 4);
    Carver c(ws);
    for (int b = 0; b < 2; ++b) w.A[b] = c.take<float>((size_t)L * d * d);
    for (int b = 0; b < 2; ++b) w.Q[b] = c.take<float>((size_t)L * d * d);
    for (int b = 0; b < 2; ++b) w.Wt[b] = c.take<float>((size_t)L * d * w.rp);
    for (int b = 0; b < 2; ++b) w.dA[b] = c.take<double>((size_t)L * d);
    for (int b = 0; b < 2; ++b) w.dQ[b] = c.take<double>((size_t)L * d);
    for (int b = 0; b < 2; ++b) w.idx[b] = c.take<int>((size_t)L * d);
    w.src = c.take<int>((size_t)L * d);
    w.pos_of = c.take<int>((size_t)L * d);
    w.U = c.take<float>((size_t)L * BMAX * d);
    w.Z = c.take<float>((size_t)L * BMAX * d);
    w.C = c.take<float>((size_t)L * BMAX * w.rp);
    w.state = c.take<LazyState>((size_t)L);
    w.lam = c.take<double>((size_t)L);
    w.base_acc = c.take<double>((size_t)L);
    const size_t inv = inverse_workspace_bytes(L, d);
    const size_t gram = hessian_tc_workspace_bytes(L, d, w.rp, ZIPLM_F32);
    w.aux_bytes = inv > gram ? inv : gram;
    w.aux = c.take<char>(w.aux_bytes);
    w.total = c.off;
    return w;
}

}  // namespace

bool lazy_path_supported(int d) { return d % 4 == 0 && d <= KPT * STEP_THREADS && d >= 4; }

size_t lazy_workspace_bytes(int L, int r, int d, int n_levels) {
    (void)n_levels;
    return carve_lazy(nullptr, L, r, d).total;
}

ziplm_status run_prune_lazy(const float* W, const float* H, int L, int r, int d, float damp_frac,
                            const int* levels, int n_levels, float* W_snap, float* loss,
                            float* base_loss, int* order, float* saliency, int* layer_status,
                            void* ws, size_t ws_bytes, cudaStream_t st) {
    if (!lazy_path_supported(d)) return ZIPLM_ERR_UNSUPPORTED;
    if (ws_bytes < lazy_workspace_bytes(L, r, d, n_levels)) return ZIPLM_ERR_WORKSPACE;
    LazyWs w = carve_lazy(ws, L, r, d);
    const int G = d, rp = w.rp;
    ziplm_status s;
    {
        PhaseScope ps(PH_INVERSE, st);
        s = run_damped_inverse(H, L, d, damp_frac, nullptr, w.A[0], d, w.dA[0], w.lam, layer_status,
                               w.aux, w.aux_bytes, st);
    }
    if (s != ZIPLM_OK) return s;
    auto init = [&]() -> ziplm_status {
        PhaseScope ps(PH_INIT, st);
        ZIPLM_CHECK_CUDA(cudaMemsetAsync(order, 0xFF, sizeof(int) * (size_t)L * G, st));
        if (saliency)
            ZIPLM_CHECK_CUDA(cudaMemsetAsync(saliency, 0, sizeof(float) * (size_t)L * G, st));
        k_lazy_init<<<dim3((d + 31) / 32, L), 256, 0, st>>>(W, r, d, rp, w.Wt[0], w.dQ[0], w.idx[0],
                                                           w.state);
        ZIPLM_CHECK_LAUNCH();
        // Q = W^T W: the symmetric product kernel of the Hessian with X = W^T (K = d_row)
        ziplm_status g = run_hessian_tc(w.Q[0], w.Wt[0], ZIPLM_F32, L, d, rp, rp, 1.0f, 0.0f, w.aux,
                                        w.aux_bytes, st);
        if (g != ZIPLM_OK) return g;
        if (base_loss) {
            ZIPLM_CHECK_CUDA(cudaMemsetAsync(w.base_acc, 0, sizeof(double) * L, st));
            k_lazy_base_loss<<<dim3(148, L), 256, 0, st>>>(d, w.Q[0], H, w.base_acc);
            ZIPLM_CHECK_LAUNCH();
            k_lazy_base_finish<<<(L + 63) / 64, 64, 0, st>>>(L, w.base_acc, base_loss);
            ZIPLM_CHECK_LAUNCH();
        }
        return ZIPLM_OK;
    };
    s = init();
    if (s != ZIPLM_OK) return s;

    int cur = 0;
    auto snapshot = [&](int n, int slot) -> ziplm_status {
        PhaseScope ps(PH_SNAPSHOT, st);
        k_lazy_pos_of<<<L, 256, 0, st>>>(n, d, w.idx[cur], w.pos_of);
        ZIPLM_CHECK_LAUNCH();
        k_lazy_snapshot<<<dim3((d + 31) / 32, (r + 31) / 32, L), 256, 0, st>>>(
            r, d, rp, W, w.Wt[cur], w.pos_of, W_snap, n_levels, slot, w.state);
        ZIPLM_CHECK_LAUNCH();
        k_lazy_loss<<<(L + 63) / 64, 64, 0, st>>>(L, n_levels, slot, w.lam, w.state, loss);
        ZIPLM_CHECK_LAUNCH();
        return ZIPLM_OK;
    };

    int n = G, slot = 0, t = 0;
    if (slot < n_levels && levels[slot] == n) {
        s = snapshot(n, slot++);
        if (s != ZIPLM_OK) return s;
    }
    const int n_min = n_levels > 0 ? levels[n_levels - 1] : G;
    while (n > n_min) {
        const int stop = (slot < n_levels) ? levels[slot] : n_min;   // next block boundary
        const int nsteps = (n - stop < BMAX) ? (n - stop) : BMAX;
        const int nxt = cur ^ 1;
        {
            PhaseScope ps(PH_LAZY_STEPS, st);
            k_lazy_steps<<<L, STEP_THREADS, 0, st>>>(n, t, nsteps, d, G, r, rp, w.A[cur], w.Q[cur],
                                                    w.Wt[cur], w.dA[cur], w.dQ[cur], w.idx[cur],
                                                    w.dA[nxt], w.dQ[nxt], w.idx[nxt], w.src, w.U, w.Z,
                                                    w.C, w.state, order, saliency, layer_status);
            ZIPLM_CHECK_LAUNCH();
        }
        const int n_new = n - nsteps;
        if (n_new > 1) {
            PhaseScope ps(PH_LAZY_UPDATE_AQ, st);
            {
                const int T = (n_new + 63) / 64;
                k_lazy_update_aq<<<dim3(T * (T + 1) / 2, L), 256, 0, st>>>(
                    n_new, nsteps, d, w.A[cur], w.Q[cur], w.A[nxt], w.Q[nxt], w.src, w.U, w.Z);
                ZIPLM_CHECK_LAUNCH();
            }
        }
        if (n_new > 0) {
            PhaseScope ps(PH_LAZY_UPDATE_W, st);
            k_lazy_update_w<<<dim3((n_new + 7) / 8, L), 256, 0, st>>>(n_new, nsteps, d, rp, w.Wt[cur],
                                                                     w.Wt[nxt], w.src, w.U, w.C);
            ZIPLM_CHECK_LAUNCH();
        }
        cur = nxt;
        n = n_new;
        t += nsteps;
        if (slot < n_levels && levels[slot] == n) {
            s = snapshot(n, slot++);
            if (s != ZIPLM_OK) return s;
        }
    }
    return ZIPLM_OK;
}

}  // namespace ziplm
