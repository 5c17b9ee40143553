// Damped float64 inverse of the calibration Hessian (caption of Algorithm 1:
// H^-1 = (2 X X^T + lambda I)^-1), batched over layers.
//
// Route: H + lambda I = F F^T (Cholesky), M = F^-1, H^-1 = M^T M, all on 64 x 64 tiles.  The
// factor and its inverse are built together by recursive halving of the tile range [lo, hi):
//     factor [lo, mid);   F21 = A21 M11^T;   A22 -= F21 F21^T;   factor [mid, hi);
//     M21 = -M22 (F21 M11)
// so that nearly all of the work sits in large, wide products (thousands of independent tiles
// per launch) and only the 64 x 64 leaves are sequential.  Everything is float64: the greedy
// loop that follows needs the diagonal of H^-1 to roughly 1e-7 relative, which an fp32
// factorisation of a matrix with condition number 1e3 .. 1e5 does not give.  The matrix is
// padded to a multiple of 64 with an identity block, whose inverse is again the identity.
#include <math.h>

#include <mutex>

#include "common.cuh"

// Built-in scratch of ziplm_damped_inverse_noalloc: lives in every GPU that loads this library
// until the process exits.  In host code this name is only a handle for cudaGetSymbolAddress,
// never a device address.
constexpr size_t kBuiltinScratchBytes = (size_t)12 << 20;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

namespace ziplm {
namespace {
constexpr int KC = 8;           // k-chunk staged in shared memory per iteration
constexpr int LDS = kTile + 2;  // padded shared-memory row length (doubles), keeps rows 16-byte aligned
constexpr int GT = 64;          // threads of a product CTA: 8 x 8 outputs per thread

// Both operands sit in shared memory k-major (s[k][i]): the inner loop then reads two
// neighbouring rows / columns per 128-bit load, 8 loads for 64 FMAs.
struct TileSmem {
    double a[2][KC][LDS];
    double b[2][KC][LDS];
};

// Fetch one 64 x KC chunk of an operand into registers (8 doubles per thread) and put it into
// shared memory as s[k][i].
//   T == false: stored 64 x K row-major (op(i,k) = P[i*ld + k]): a thread takes one row's 8 k's
//               and writes them down a column of s (consecutive threads -> consecutive i);
//   T == true : stored K x 64 (op(i,k) = P[k*ld + i]): a thread takes pairs along i.
template <bool T>
__device__ __forceinline__ void chunk_load(double (&r)[8], const double* P, int ld, int k0) {
    const int tid = threadIdx.x;
    if (T) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const double2 v = *reinterpret_cast<const double2*>(
                P + (size_t)(k0 + (tid >> 5) + 2 * e) * ld + (tid & 31) * 2);
            r[2 * e] = v.x; r[2 * e + 1] = v.y;
        }
    } else {
        const double* src = P + (size_t)tid * ld + k0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const double2 v = *reinterpret_cast<const double2*>(src + 2 * e);
            r[2 * e] = v.x; r[2 * e + 1] = v.y;
        }
    }
}

template <bool T>
__device__ __forceinline__ void chunk_store(double (*s)[LDS], const double (&r)[8]) {
    const int tid = threadIdx.x;
    if (T) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
            *reinterpret_cast<double2*>(&s[(tid >> 5) + 2 * e][(tid & 31) * 2]) =
                make_double2(r[2 * e], r[2 * e + 1]);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) s[e][tid] = r[e];
    }
}

// Row / column of output element (p, q) of thread (ty, tx): pairs of neighbours, 16 apart.
__device__ __forceinline__ int own_index(int t, int p) { return 2 * t + 16 * (p >> 1) + (p & 1); }

// acc(64x64) += opA(64xK) * opB(Kx64); 64 threads, thread (ty,tx) = (tid/8, tid%8) owns the rows
// own_index(ty, p) and the columns own_index(tx, q), p, q < 8.  The next chunk is fetched into
// registers while the current one is multiplied out of shared memory (two buffers, one barrier
// per chunk).  The operand pointers are deliberately not __restrict__: callers may read tiles
// written earlier in the same launch sequence.  Ends with __syncthreads().
//   TA == false: A stored 64 x K row-major; true: stored K x 64.
//   TB == false: B stored K x 64 row-major; true: stored 64 x K.
template <bool TA, bool TB>
__device__ __forceinline__ void dgemm_tile(double (&acc)[8][8], const double* A, int lda,
                                           const double* B, int ldb, int K, TileSmem& sm) {
    const int tid = threadIdx.x;
    const int ty = tid >> 3, tx = tid & 7;
    if (K <= 0) return;
    constexpr bool LA = TA, LB = !TB;       // loader orientation: true = stored K x 64
    double ra[8], rb[8];
    chunk_load<LA>(ra, A, lda, 0);
    chunk_load<LB>(rb, B, ldb, 0);
    chunk_store<LA>(sm.a[0], ra);
    chunk_store<LB>(sm.b[0], rb);
    __syncthreads();
    int buf = 0;
    for (int k0 = 0; k0 < K; k0 += KC) {
        const bool more = k0 + KC < K;
        if (more) {
            chunk_load<LA>(ra, A, lda, k0 + KC);
            chunk_load<LB>(rb, B, ldb, k0 + KC);
        }
#pragma unroll
        for (int kk = 0; kk < KC; ++kk) {
            double a[8], b[8];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const double2 va = *reinterpret_cast<const double2*>(&sm.a[buf][kk][2 * ty + 16 * q]);
                const double2 vb = *reinterpret_cast<const double2*>(&sm.b[buf][kk][2 * tx + 16 * q]);
                a[2 * q] = va.x; a[2 * q + 1] = va.y;
                b[2 * q] = vb.x; b[2 * q + 1] = vb.y;
            }
#pragma unroll
            for (int p = 0; p < 8; ++p)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc[p][q] = fma(a[p], b[q], acc[p][q]);
        }
        if (more) {
            chunk_store<LA>(sm.a[buf ^ 1], ra);
            chunk_store<LB>(sm.b[buf ^ 1], rb);
        }
        __syncthreads();
        buf ^= 1;
    }
}

__device__ __forceinline__ void zero_acc(double (&acc)[8][8]) {
#pragma unroll
    for (int p = 0; p < 8; ++p)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[p][q] = 0.0;
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

// One launch of the recursion: C_out[tile (ti,tj)] = beta * C_out + alpha * sum_k opA(ti,k) opB(k,tj)
// over a rectangle of mt x nt tiles, with the k range cut to the non-zero tiles of a triangular
// operand.  All matrices are dp x dp float64 per layer; coordinates are in tiles.
struct GemmTask {
    const double* A; int a_r, a_c;      // TA == false: tile (ti,k) at (a_r + ti, a_c + k); true: (a_r + k, a_c + ti)
    const double* B; int b_r, b_c;      // TB == false: tile (k,tj) at (b_r + k, b_c + tj); true: (b_r + tj, b_c + k)
    double* C; int c_r, c_c;
    int mt, nt, kt;
    int kmode;                          // 0: all k; 1: k <= tj; 2: k <= ti; 3: k >= tj
    int lower_only;                     // square region: only tiles ti >= tj
    double alpha; int beta;             // beta in {0, 1}
};

template <bool TA, bool TB>
__global__ void __launch_bounds__(GT) k_dgemm_tiles(GemmTask t, int dp) {
    __shared__ TileSmem sm;
    const int l = blockIdx.y;
    int ti, tj;
    if (t.lower_only) {
        ti = 0; int rem = blockIdx.x;
        while (rem > ti) { rem -= ti + 1; ++ti; }
        tj = rem;
    } else {
        ti = blockIdx.x / t.nt; tj = blockIdx.x % t.nt;
    }
    int klo = 0, khi = t.kt;
    if (t.kmode == 1) khi = min(t.kt, tj + 1);
    else if (t.kmode == 2) khi = min(t.kt, ti + 1);
    else if (t.kmode == 3) klo = tj;
    const size_t lay = (size_t)l * dp * dp;
    const double* A = t.A + lay + (TA ? ((size_t)(t.a_r + klo) * kTile * dp + (size_t)(t.a_c + ti) * kTile)
                                      : ((size_t)(t.a_r + ti) * kTile * dp + (size_t)(t.a_c + klo) * kTile));
    const double* B = t.B + lay + (TB ? ((size_t)(t.b_r + tj) * kTile * dp + (size_t)(t.b_c + klo) * kTile)
                                      : ((size_t)(t.b_r + klo) * kTile * dp + (size_t)(t.b_c + tj) * kTile));
    double acc[8][8];
    zero_acc(acc);
    dgemm_tile<TA, TB>(acc, A, dp, B, dp, (khi - klo) * kTile, sm);
    double* out = t.C + lay + (size_t)(t.c_r + ti) * kTile * dp + (size_t)(t.c_c + tj) * kTile;
    const int ty = threadIdx.x >> 3, tx = threadIdx.x & 7;
#pragma unroll
    for (int p = 0; p < 8; ++p)
#pragma unroll
        for (int q = 0; q < 8; q += 2) {
            double2* o = reinterpret_cast<double2*>(out + (size_t)own_index(ty, p) * dp + own_index(tx, q));
            double2 v = make_double2(t.alpha * acc[p][q], t.alpha * acc[p][q + 1]);
            if (t.beta) { const double2 c = *o; v.x += c.x; v.y += c.y; }
            *o = v;
        }
}

// Leaf of the recursion: unblocked Cholesky of the diagonal tile A_jj -> F_jj (lower, upper part
// zeroed) and the inverse of that factor -> M_jj (lower, upper part zeroed).
__global__ void __launch_bounds__(256) k_potf2(const double* A, double* F, double* M, int dp, int j,
                                               int* layer_status) {
    __shared__ double s[kTile][kTile + 1];
    __shared__ double dinv[kTile];
    __shared__ int sflag;
    const int l = blockIdx.x;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const size_t off = (size_t)l * dp * dp + (size_t)j * kTile * dp + (size_t)j * kTile;
    if (tid == 0) sflag = 0;
    for (int e = tid; e < kTile * kTile; e += 256)
        s[e >> 6][e & 63] = A[off + (size_t)(e >> 6) * dp + (e & 63)];
    __syncthreads();
    for (int c = 0; c < kTile; ++c) {
        // every thread forms 1/sqrt(pivot) itself: no broadcast, two barriers per column
        double p = s[c][c];
        if (!(p > 0.0) || !isfinite(p)) {   // not positive definite (or NaN): flag, keep going
            if (tid == 0 && !sflag) sflag = isfinite(p) ? ZIPLM_ERR_NOT_PD : ZIPLM_ERR_NONFINITE;
            p = 1.0;
        }
        const double rinv = rsqrt(p);
        __syncthreads();                    // all threads have read the pivot
        if (tid == c) s[c][c] = p * rinv;
        else if (tid > c && tid < kTile) s[tid][c] *= rinv;
        __syncthreads();
        // trailing update of the lower triangle: rows ty + 16a, cols tx + 16b
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int i = ty + 16 * a;
            if (i <= c) continue;
            const double lic = s[i][c];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int jj = tx + 16 * b;
                if (jj > c && jj <= i) s[i][jj] -= lic * s[jj][c];
            }
        }
        __syncthreads();
    }
    // inverse of the lower-triangular factor: thread `cidx` builds column cidx by forward
    // substitution.  Entry (i, cidx), i > cidx, is parked transposed in the unused strict upper
    // triangle of s (slot [cidx][i]); the reciprocal diagonal goes to dinv first.
    if (tid < kTile) dinv[tid] = 1.0 / s[tid][tid];
    __syncthreads();
    if (tid < kTile) {
        const int cidx = tid;
        for (int i = cidx + 1; i < kTile; ++i) {
            double a0 = -s[i][cidx] * dinv[cidx], a1 = 0.0, a2 = 0.0, a3 = 0.0;
            int k = cidx + 1;
            for (; k + 3 < i; k += 4) {
                a0 = fma(-s[i][k], s[cidx][k], a0);
                a1 = fma(-s[i][k + 1], s[cidx][k + 1], a1);
                a2 = fma(-s[i][k + 2], s[cidx][k + 2], a2);
                a3 = fma(-s[i][k + 3], s[cidx][k + 3], a3);
            }
            for (; k < i; ++k) a0 = fma(-s[i][k], s[cidx][k], a0);
            s[cidx][i] = ((a0 + a1) + (a2 + a3)) * dinv[i];
        }
    }
    __syncthreads();
    for (int e = tid; e < kTile * kTile; e += 256) {
        const int i = e >> 6, jj = e & 63;
        F[off + (size_t)i * dp + jj] = (jj <= i) ? s[i][jj] : 0.0;
        M[off + (size_t)i * dp + jj] = (jj < i) ? s[jj][i] : (jj == i ? dinv[i] : 0.0);
    }
    if (tid == 0 && sflag) set_layer_status(layer_status, l, sflag);
}

// H^-1 = M^T M on the lower tiles (i >= j): sum over k >= i of M_ki^T M_kj; writes the cropped
// d x d result as float64 (mirrored to the upper triangle) and/or fp32 strict lower + fp64 diag.
__global__ void __launch_bounds__(GT) k_lauum(const double* M, int dp, int T, int d, double* out64,
                                              float* tri32, int pitch32, double* diag64) {
    __shared__ TileSmem sm;
    const int l = blockIdx.y;
    // linear tile index -> (i, j), rows of the lower triangle in order i = 0, 1, ...
    int i = 0, rem = blockIdx.x;
    while (rem > i) { rem -= i + 1; ++i; }
    const int j = rem;
    const double* Ml = M + (size_t)l * dp * dp;
    double acc[8][8];
    zero_acc(acc);
    dgemm_tile<true, false>(acc, Ml + (size_t)i * kTile * dp + (size_t)i * kTile, dp,
                            Ml + (size_t)i * kTile * dp + (size_t)j * kTile, dp, (T - i) * kTile, sm);
    const int ty = threadIdx.x >> 3, tx = threadIdx.x & 7;
#pragma unroll
    for (int p = 0; p < 8; ++p)
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int row = i * kTile + own_index(ty, p), col = j * kTile + own_index(tx, q);
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

struct InvCtx {
    double* A;   // damped Hessian, updated in place (Schur complements); dead blocks serve as scratch
    double* F;   // Cholesky factor
    double* M;   // inverse of the factor
    int dp, L;
    int* layer_status;
    cudaStream_t st;
};

template <bool TA, bool TB>
ziplm_status launch_gemm(const InvCtx& c, const GemmTask& t) {
    const int tiles = t.lower_only ? t.mt * (t.mt + 1) / 2 : t.mt * t.nt;
    if (tiles <= 0 || t.kt <= 0) return ZIPLM_OK;
    PhaseScope ps(PH_INV_PRODUCTS, c.st);
    k_dgemm_tiles<TA, TB><<<dim3(tiles, c.L), GT, 0, c.st>>>(t, c.dp);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

// Factor the tile range [lo, hi): on return F holds the Cholesky factor of the (updated) block
// and M its inverse.
ziplm_status factor_range(const InvCtx& c, int lo, int hi) {
    if (hi - lo == 1) {
        PhaseScope ps(PH_INV_LEAVES, c.st);
        k_potf2<<<c.L, 256, 0, c.st>>>(c.A, c.F, c.M, c.dp, lo, c.layer_status);
        ZIPLM_CHECK_LAUNCH();
        return ZIPLM_OK;
    }
    const int mid = lo + (hi - lo) / 2;
    const int n1 = mid - lo, n2 = hi - mid;
    ziplm_status s = factor_range(c, lo, mid);
    if (s != ZIPLM_OK) return s;
    GemmTask t;
    // F21 = A21 M11^T   (M11 lower triangular: opB(k,j) = M11[j,k] vanishes for k > j)
    t = GemmTask{c.A, mid, lo, c.M, lo, lo, c.F, mid, lo, n2, n1, n1, 1, 0, 1.0, 0};
    if ((s = launch_gemm<false, true>(c, t)) != ZIPLM_OK) return s;
    // A22 -= F21 F21^T  (lower tiles)
    t = GemmTask{c.F, mid, lo, c.F, mid, lo, c.A, mid, mid, n2, n2, n1, 0, 1, -1.0, 1};
    if ((s = launch_gemm<false, true>(c, t)) != ZIPLM_OK) return s;
    if ((s = factor_range(c, mid, hi)) != ZIPLM_OK) return s;
    // scratch (the dead A21 block) = F21 M11   (M11 lower: opB(k,j) vanishes for k < j)
    t = GemmTask{c.F, mid, lo, c.M, lo, lo, c.A, mid, lo, n2, n1, n1, 3, 0, 1.0, 0};
    if ((s = launch_gemm<false, false>(c, t)) != ZIPLM_OK) return s;
    // M21 = -M22 scratch  (M22 lower: opA(i,k) vanishes for k > i)
    t = GemmTask{c.M, mid, mid, c.A, mid, lo, c.M, mid, lo, n2, n1, n2, 2, 0, -1.0, 0};
    return launch_gemm<false, false>(c, t);
}

}  // namespace

size_t inverse_workspace_bytes(int L, int d) {
    const int dp = round_up_int(d, kTile);
    Carver c(nullptr);
    c.take<double>((size_t)L * dp * dp);               // A: damped Hessian / Schur complements
    c.take<double>((size_t)L * dp * dp);               // F: Cholesky factor
    c.take<double>((size_t)L * dp * dp);               // M: inverse of the factor
    c.take<double>((size_t)L);                         // lambda
    return c.off;
}

ziplm_status run_damped_inverse(const float* H, int L, int d, float damp_frac, double* out64,
                                float* tri32, int pitch32, double* diag64, double* lam_out,
                                int* layer_status, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (ws_bytes < inverse_workspace_bytes(L, d)) return ZIPLM_ERR_WORKSPACE;
    const int dp = round_up_int(d, kTile), T = dp / kTile;
    Carver c(ws);
    InvCtx ctx;
    ctx.A = c.take<double>((size_t)L * dp * dp);
    ctx.F = c.take<double>((size_t)L * dp * dp);
    ctx.M = c.take<double>((size_t)L * dp * dp);
    double* lam = c.take<double>((size_t)L);
    ctx.dp = dp; ctx.L = L; ctx.layer_status = layer_status; ctx.st = st;

    k_mean_diag<<<L, 256, 0, st>>>(H, d, damp_frac, lam, layer_status);
    ZIPLM_CHECK_LAUNCH();
    k_fill_damped<<<dim3(T, dp / 16, L), 256, 0, st>>>(H, d, dp, lam, ctx.A, layer_status);
    ZIPLM_CHECK_LAUNCH();
    ziplm_status s = factor_range(ctx, 0, T);
    if (s != ZIPLM_OK) return s;
    {
        PhaseScope ps(PH_INV_LAUUM, st);
        k_lauum<<<dim3(T * (T + 1) / 2, L), GT, 0, st>>>(ctx.M, dp, T, d, out64, tri32, pitch32, diag64);
        ZIPLM_CHECK_LAUNCH();
    }
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
