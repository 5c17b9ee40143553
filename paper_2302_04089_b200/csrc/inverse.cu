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
constexpr int KC = 16;          // k-chunk staged in shared memory per pipeline stage
constexpr int MTM = 128;        // rows of the macro tile one CTA computes (two tiles)
constexpr int MTN = 64;         // columns of the macro tile (one tile)
constexpr int GT = 256;         // threads of a product CTA: 8 warps, 32 x 32 outputs per warp; two CTAs per SM
constexpr int kSmallThreads = 512;   // threads of the base-case kernel
constexpr int kStages = 3;      // cp.async pipeline depth
// Shared-memory pitches (doubles).  All are 4 mod 16, so that the 16 threads of a half-warp
// (4 m-indices x 4 k-indices of an operand fragment) hit 16 different 8-byte banks, and all keep
// rows 16-byte aligned for cp.async.
constexpr int P_MK = KC + 4;    // chunk stored [m][k] (k contiguous in global memory)
__host__ __device__ constexpr int pitch_km(int rows) { return rows + 4; }   // chunk stored [k][m] (m contiguous)
__host__ __device__ constexpr int stage_doubles(int rows) {
    return rows * P_MK > KC * pitch_km(rows) ? rows * P_MK : KC * pitch_km(rows);
}
constexpr int kStageA = stage_doubles(MTM), kStageB = stage_doubles(MTN);
constexpr size_t kProductSmemBytes = sizeof(double) * kStages * (kStageA + kStageB);

__device__ __forceinline__ void cp_async16(double* smem_dst, const double* gmem_src) {
    const unsigned sa = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// D(8x8) += A(8x4) B(4x8) in float64 on the tensor core.  Lane T holds A[T/4][T%4], B[T%4][T/4]
// and D[T/4][2(T%4)], D[T/4][2(T%4)+1].
__device__ __forceinline__ void dmma884(double (&d)[2], double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(d[0]), "+d"(d[1]) : "d"(a), "d"(b));
}

// Start the copy of one ROWS x KC operand chunk into a pipeline stage; rows m >= m_valid (tiles
// beyond the edge of the task) are not touched.
//   KM == false: op(m,k) = P[m*ld + k], kept as s[m][k] (pitch P_MK);
//   KM == true : op(m,k) = P[k*ld + m], kept as s[k][m] (pitch ROWS + 4).
template <bool KM, int ROWS>
__device__ __forceinline__ void chunk_async(double* s, const double* P, int ld, int k0, int m_valid) {
    constexpr int PIECES = ROWS * KC / 2;                 // pieces of 16 bytes
#pragma unroll
    for (int e = 0; e < PIECES / GT; ++e) {
        const int piece = threadIdx.x + e * GT;
        if (KM) {
            const int k = piece / (ROWS / 2), m = (piece % (ROWS / 2)) * 2;
            if (m < m_valid) cp_async16(s + k * pitch_km(ROWS) + m, P + (size_t)(k0 + k) * ld + m);
        } else {
            const int m = piece >> 3, k = (piece & 7) * 2;
            if (m < m_valid) cp_async16(s + m * P_MK + k, P + (size_t)m * ld + k0 + k);
        }
    }
}

// Operand fragment of the k-step kk (4 k's) for the 8 m-indices starting at m0.
template <bool KM, int ROWS>
__device__ __forceinline__ double frag(const double* s, int m0, int kk, int lane) {
    return KM ? s[(kk * 4 + (lane & 3)) * pitch_km(ROWS) + m0 + (lane >> 2)]
              : s[(m0 + (lane >> 2)) * P_MK + kk * 4 + (lane & 3)];
}

// Accumulators of one warp: 4 x 4 fragments of 8 x 8 = a 32 x 32 block of the macro tile.
struct WarpAcc {
    double d[4][4][2];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) d[i][j][0] = d[i][j][1] = 0.0;
    }
};

// acc(128 x 64 macro tile) += opA(128 x K) opB(K x 64) over the tile range [kt_lo, kt_hi) of K (in
// tiles of 64), operands streamed through a three-stage cp.async pipeline with one barrier per
// chunk.  Warp w owns rows 32 (w / 2) .. and columns 32 (w % 2) .. of the macro tile and only
// multiplies the chunks of its own range [my_lo, my_hi) (the triangular operands cut the range
// per 64 x 64 tile; what the other warps' ranges bring into shared memory may be uninitialised
// and is never read by this warp).  rows_valid crops the macro tile at the edge of the task.
// A and B point at k = 0 of the macro tile's rows / columns.
//   TA == false: A stored m x K row-major; true: stored K x m.
//   TB == false: B stored K x n row-major; true: stored n x K.
// The operand pointers are deliberately not __restrict__: callers read tiles written earlier in
// the same launch sequence.
template <bool TA, bool TB>
__device__ __forceinline__ void dgemm_macro(WarpAcc& acc, const double* A, int lda, const double* B,
                                            int ldb, int kt_lo, int kt_hi, int my_lo, int my_hi,
                                            int rows_valid, double* smem) {
    constexpr bool KA = TA, KB = !TB;       // orientation in memory: true = stored K x m
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r0 = 32 * (warp >> 1), c0 = 32 * (warp & 1);
    double* sa = smem;
    double* sb = smem + kStages * kStageA;
    const int nchunks = (kt_hi - kt_lo) * (kTile / KC);
    const int kbase = kt_lo * kTile;
    for (int c = 0; c < kStages - 1; ++c) {
        if (c < nchunks) {
            chunk_async<KA, MTM>(sa + c * kStageA, A, lda, kbase + c * KC, rows_valid);
            chunk_async<KB, MTN>(sb + c * kStageB, B, ldb, kbase + c * KC, MTN);
        }
        cp_async_commit();
    }
    for (int c = 0; c < nchunks; ++c) {
        cp_async_wait<kStages - 2>();       // chunk c has landed (this thread's pieces)
        __syncthreads();                    // ... everyone's; and chunk c - 1 has been consumed
        const int nx = c + kStages - 1;
        if (nx < nchunks) {
            const int st = nx % kStages;
            chunk_async<KA, MTM>(sa + st * kStageA, A, lda, kbase + nx * KC, rows_valid);
            chunk_async<KB, MTN>(sb + st * kStageB, B, ldb, kbase + nx * KC, MTN);
        }
        cp_async_commit();
        const int ktile = kt_lo + c / (kTile / KC);
        if (ktile < my_lo || ktile >= my_hi) continue;
        const double* pa = sa + (c % kStages) * kStageA;
        const double* pb = sb + (c % kStages) * kStageB;
#pragma unroll
        for (int kk = 0; kk < KC / 4; ++kk) {
            double a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                a[i] = frag<KA, MTM>(pa, r0 + 8 * i, kk, lane);
                b[i] = frag<KB, MTN>(pb, c0 + 8 * i, kk, lane);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) dmma884(acc.d[i][j], a[i], b[j]);
        }
    }
    cp_async_wait<0>();
}

// Macro tiles (I, J) of a lower-triangular region of T x T tiles: row block I (tiles 2I, 2I+1)
// meets the column tiles J <= 2I + 1.  Count, and linear index -> (I, J) in row-block order.
__host__ __device__ inline int lower_macro_count(int T) {
    int n = 0;
    for (int I = 0; 2 * I < T; ++I) n += (2 * I + 2 < T) ? 2 * I + 2 : T;
    return n;
}
__device__ __forceinline__ void lower_macro_index(int idx, int T, int& I, int& J) {
    I = 0;
    for (;;) {
        const int w = (2 * I + 2 < T) ? 2 * I + 2 : T;
        if (idx < w) break;
        idx -= w; ++I;
    }
    J = idx;
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

// k range (in tiles) of output tile (ti, tj) under the task's kmode.
__device__ __forceinline__ void task_krange(const GemmTask& t, int ti, int tj, int& klo, int& khi) {
    klo = 0; khi = t.kt;
    if (t.kmode == 1) khi = min(t.kt, tj + 1);
    else if (t.kmode == 2) khi = min(t.kt, ti + 1);
    else if (t.kmode == 3) klo = tj;
}

// One CTA per 128 x 64 macro tile (two tiles high); blockIdx.x runs over the macro tiles of the
// task (those that reach the lower triangle when lower_only), blockIdx.y over the layers.
template <bool TA, bool TB>
__device__ __forceinline__ void dgemm_task(const GemmTask& t, int dp, int bx, int l, double* smem) {
    const int mmt = (t.mt + 1) / 2;
    // macro tiles with the longest k range come first, so that the last wave is the lightest
    int I, J;
    if (t.lower_only) lower_macro_index(bx, t.mt, I, J);
    else if (t.kmode == 1) { J = t.nt - 1 - bx / mmt; I = bx % mmt; }
    else if (t.kmode == 3) { J = bx / mmt; I = bx % mmt; }
    else if (t.kmode == 2) { I = mmt - 1 - bx / t.nt; J = bx % t.nt; }
    else { I = bx / t.nt; J = bx % t.nt; }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ti = 2 * I + (warp >> 2), tj = J;                          // this warp's tile
    const bool mine = ti < t.mt && (!t.lower_only || ti >= tj);
    // CTA range: union over its valid tiles; warp range: its own tile's
    int kt_lo = t.kt, kt_hi = 0;
    for (int a = 0; a < 2; ++a) {
        const int si = 2 * I + a;
        if (si >= t.mt || (t.lower_only && si < tj)) continue;
        int lo, hi;
        task_krange(t, si, tj, lo, hi);
        kt_lo = min(kt_lo, lo); kt_hi = max(kt_hi, hi);
    }
    int my_lo = 0, my_hi = 0;
    if (mine) task_krange(t, ti, tj, my_lo, my_hi);
    const int rows_valid = min(MTM, (t.mt - 2 * I) * kTile);
    const size_t lay = (size_t)l * dp * dp;
    const double* A = t.A + lay + (TA ? ((size_t)t.a_r * kTile * dp + (size_t)(t.a_c + 2 * I) * kTile)
                                      : ((size_t)(t.a_r + 2 * I) * kTile * dp + (size_t)t.a_c * kTile));
    const double* B = t.B + lay + (TB ? ((size_t)(t.b_r + J) * kTile * dp + (size_t)t.b_c * kTile)
                                      : ((size_t)t.b_r * kTile * dp + (size_t)(t.b_c + J) * kTile));
    WarpAcc acc;
    acc.zero();
    dgemm_macro<TA, TB>(acc, A, dp, B, dp, kt_lo, kt_hi, my_lo, my_hi, rows_valid, smem);
    if (!mine) return;
    double* out = t.C + lay + (size_t)((t.c_r + 2 * I) * kTile + 32 * (warp >> 1)) * dp +
                  (size_t)(t.c_c + J) * kTile + 32 * (warp & 1);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            double2* o = reinterpret_cast<double2*>(out + (size_t)(8 * i + (lane >> 2)) * dp + 8 * j + 2 * (lane & 3));
            double2 v = make_double2(t.alpha * acc.d[i][j][0], t.alpha * acc.d[i][j][1]);
            if (t.beta) { const double2 c = *o; v.x += c.x; v.y += c.y; }
            *o = v;
        }
}

template <bool TA, bool TB>
__global__ void __launch_bounds__(GT, 2) k_dgemm_tiles(GemmTask t, int dp) {
    extern __shared__ __align__(16) double smem[];
    dgemm_task<TA, TB>(t, dp, blockIdx.x, blockIdx.y, smem);
}

// Two independent products in one launch: the first n1 CTAs of a layer run t1 (A B^T form), the
// rest t2 (A B form).  Used for A22 -= F21 F21^T and scratch = F21 M11, which both depend on F21
// only: one launch fills the other's last wave.
__global__ void __launch_bounds__(GT, 2) k_dgemm_pair(GemmTask t1, int n1, GemmTask t2, int dp) {
    extern __shared__ __align__(16) double smem[];
    if ((int)blockIdx.x < n1) dgemm_task<false, true>(t1, dp, blockIdx.x, blockIdx.y, smem);
    else dgemm_task<false, false>(t2, dp, blockIdx.x - n1, blockIdx.y, smem);
}

// ---- base case of the recursion: a range of up to kSmallMax tiles, one CTA per layer ----------
constexpr int kSmallMax = 4;
constexpr int PS = kTile + 4;    // pitch of a 64 x 64 operand tile in shared memory (4 mod 16)

struct SmallSmem {
    double ta[kTile * PS];       // operand tiles, as stored (row-major)
    double tb[kTile * PS];
    double td[kTile * PS];       // inverse of the current diagonal factor tile
    double s[kTile][kTile + 1];  // leaf work array: the factor (lower part)
    double col[2][kTile];        // current column of the leaf factorisation (double-buffered)
    double dinv[kTile];          // reciprocal diagonal of the factor
    int flag;                    // first error seen by this CTA
};

// Start the copy of a 64 x 64 tile (row-major, leading dimension ld) into a shared-memory tile.
__device__ __forceinline__ void tile_async(double* dst, const double* src, int ld) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int piece = threadIdx.x + e * kSmallThreads;            // 2048 pieces of 16 bytes
        const int r = piece >> 5, c = (piece & 31) * 2;
        cp_async16(dst + r * PS + c, src + (size_t)r * ld + c);
    }
}

// Fragment of a shared-memory tile: KM == false: op(m,k) = s[m][k]; true: op(m,k) = s[k][m].
template <bool KM>
__device__ __forceinline__ double tile_frag(const double* s, int m0, int kk, int lane) {
    return KM ? s[(kk * 4 + (lane & 3)) * PS + m0 + (lane >> 2)]
              : s[(m0 + (lane >> 2)) * PS + kk * 4 + (lane & 3)];
}

// Accumulators of one warp of the small kernel: 2 x 2 fragments = a 16 x 16 block of a tile;
// warp w owns rows 16 (w / 4) .. and columns 16 (w % 4) ...
struct SmallAcc {
    double d[2][2][2];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j) d[i][j][0] = d[i][j][1] = 0.0;
    }
};

// acc += opA(64 x 64) opB(64 x 64), both operands in shared memory.
//   AKM: opA(m,k) = sa[k][m], else sa[m][k];  BKN: opB(k,n) = sb[k][n], else sb[n][k].
template <bool AKM, bool BKN>
__device__ __forceinline__ void tile_mma(SmallAcc& acc, const double* sa, const double* sb) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r0 = 16 * (warp >> 2), c0 = 16 * (warp & 3);
#pragma unroll 4
    for (int kk = 0; kk < kTile / 4; ++kk) {
        double a[2], b[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            a[i] = tile_frag<AKM>(sa, r0 + 8 * i, kk, lane);
            b[i] = tile_frag<BKN>(sb, c0 + 8 * i, kk, lane);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j) dmma884(acc.d[i][j], a[i], b[j]);
    }
}

// Visit the elements of a warp's accumulators: f(row, col, pair) with col even.
template <typename Fn>
__device__ __forceinline__ void small_epilogue(const SmallAcc& acc, Fn f) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r0 = 16 * (warp >> 2) + (lane >> 2), c0 = 16 * (warp & 3) + 2 * (lane & 3);
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j)
            f(r0 + 8 * i, c0 + 8 * j, make_double2(acc.d[i][j][0], acc.d[i][j][1]));
}

// One warp: acc(16 x 16) += A(16 x K) B(K x 16), operands anywhere in shared memory
// (A[m * lda + k], B[k * ldb + n]); K a multiple of 4.
__device__ __forceinline__ void warp_mma16(double (&acc)[2][2][2], const double* A, int lda,
                                           const double* B, int ldb, int K) {
    const int lane = threadIdx.x & 31;
    for (int k0 = 0; k0 < K; k0 += 4) {
        double a[2], b[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            a[i] = A[(8 * i + (lane >> 2)) * lda + k0 + (lane & 3)];
            b[i] = B[(k0 + (lane & 3)) * ldb + 8 * i + (lane >> 2)];
        }
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j) dmma884(acc[i][j], a[i], b[j]);
    }
}

// One warp: C(16 x 16) = sign * acc, C[m * ldc + n].
__device__ __forceinline__ void warp_store16(const double (&acc)[2][2][2], double* C, int ldc, double sign) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e)
                C[(8 * i + (lane >> 2)) * ldc + 8 * j + 2 * (lane & 3) + e] = sign * acc[i][j][e];
}

// Leaf: Cholesky factor of the 64 x 64 tile at Ag -> Fg (lower, upper part zeroed), the inverse of
// that factor -> Mg and sm.td (lower, upper part zeroed).  Starts and ends with a barrier.
//   Factor: threads 0..255 hold the tile in registers, cyclically (rows ty + 16 a, columns
//   tx + 16 b, tx constant over half a warp), so a column step is one barrier, eight
//   shared-memory reads and 16 FMAs per thread; only the warp that owns the column publishes it.
//   Inverse: the four 16 x 16 diagonal blocks by forward substitution (one thread per column),
//   then the off-diagonal blocks of the 32- and 64-wide levels as products
//   M21 = -M22 (L21 M11) on the tensor core.
__device__ __forceinline__ void leaf_factor(const double* Ag, double* Fg, double* Mg, int dp,
                                            SmallSmem& sm) {
    const int tid = threadIdx.x, warp = tid >> 5;
    const bool worker = tid < 256;
    const int ty = tid & 15, tx = (tid >> 4) & 15;
    __syncthreads();                          // earlier readers of the shared arrays are done
    tile_async(sm.tb, Ag, dp);
    cp_async_commit();
    for (int e = tid; e < kTile * PS; e += kSmallThreads) sm.ta[e] = 0.0;   // the inverse is built in ta
    cp_async_wait<0>();
    __syncthreads();
    double r[4][4];
    if (worker) {
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) r[a][b] = sm.tb[(ty + 16 * a) * PS + tx + 16 * b];
    }
    for (int c = 0; c < kTile; ++c) {
        const int cb = c >> 4, ct = c & 15;
        double* col = sm.col[c & 1];
        if (worker && tx == ct) {
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                double v = r[a][0];
#pragma unroll
                for (int b = 1; b < 4; ++b) v = (b == cb) ? r[a][b] : v;
                col[ty + 16 * a] = v;
            }
        }
        __syncthreads();
        if (worker) {
            double p = col[c];
            if (!(p > 0.0) || !isfinite(p)) {   // not positive definite (or NaN): flag, keep going
                if (tid == 0 && !sm.flag) sm.flag = isfinite(p) ? ZIPLM_ERR_NOT_PD : ZIPLM_ERR_NONFINITE;
                p = 1.0;
            }
            const double rinv = rsqrt(p);
            if (tid == 0) sm.dinv[c] = rinv;    // 1 / L_cc
            double li[4], lj[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                li[a] = col[ty + 16 * a] * rinv;
                lj[a] = col[tx + 16 * a] * rinv;
            }
            // Columns <= c are final.  Rows <= c of the later columns lie above the diagonal:
            // they are never used, so they are updated along with the rest.
#pragma unroll
            for (int b = 0; b < 4; ++b)
                if (tx + 16 * b > c) {
#pragma unroll
                    for (int a = 0; a < 4; ++a) r[a][b] = fma(-li[a], lj[b], r[a][b]);
                }
            if (tx == ct) {
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    const int i = ty + 16 * a;
                    const double v = i > c ? li[a] : p * rinv;
#pragma unroll
                    for (int b = 0; b < 4; ++b)
                        if (b == cb && i >= c) r[a][b] = v;
                }
            }
        }
    }
    if (worker) {
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b)
                if (tx + 16 * b <= ty + 16 * a) sm.s[ty + 16 * a][tx + 16 * b] = r[a][b];
    }
    __syncthreads();
    // ---- inverse of the factor, built in sm.ta (pitch PS, zero above the diagonal) ----
    if (tid < kTile) {
        // column cc of diagonal block q: x_i = (delta_i,cc - sum_{cc <= k < i} L_ik x_k) / L_ii
        const int q0 = tid & ~15, cc = tid & 15;
        double x[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            double acc = (i == cc) ? 1.0 : 0.0;
#pragma unroll
            for (int k = 0; k < i; ++k) acc = fma(-sm.s[q0 + i][q0 + k], x[k], acc);
            x[i] = (i >= cc) ? acc * sm.dinv[q0 + i] : 0.0;
            sm.ta[(q0 + i) * PS + q0 + cc] = x[i];
        }
    }
    __syncthreads();
    double acc[2][2][2];
    auto zero = [&]() {
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;
    };
    // 32-wide level: blocks (1,0) and (3,2) of 16 x 16; warp q does pair q.  tb holds L21 M11.
    if (warp < 2) {
        const int o = 32 * warp;
        zero();
        warp_mma16(acc, &sm.s[o + 16][o], kTile + 1, sm.ta + o * PS + o, PS, 16);
        warp_store16(acc, sm.tb + (o + 16) * PS + o, PS, 1.0);
    }
    __syncthreads();
    if (warp < 2) {
        const int o = 32 * warp;
        zero();
        warp_mma16(acc, sm.ta + (o + 16) * PS + o + 16, PS, sm.tb + (o + 16) * PS + o, PS, 16);
        warp_store16(acc, sm.ta + (o + 16) * PS + o, PS, -1.0);
    }
    __syncthreads();
    // 64-wide level: block (rows 32.., cols 0..31); warp w < 4 does the 16 x 16 part (w / 2, w % 2).
    if (warp < 4) {
        const int rb = 32 + 16 * (warp >> 1), cb = 16 * (warp & 1);
        zero();
        warp_mma16(acc, &sm.s[rb][0], kTile + 1, sm.ta + cb, PS, 32);
        warp_store16(acc, sm.tb + rb * PS + cb, PS, 1.0);
    }
    __syncthreads();
    if (warp < 4) {
        const int rb = 32 + 16 * (warp >> 1), cb = 16 * (warp & 1);
        zero();
        warp_mma16(acc, sm.ta + rb * PS + 32, PS, sm.tb + 32 * PS + cb, PS, 32);
        warp_store16(acc, sm.ta + rb * PS + cb, PS, -1.0);
    }
    __syncthreads();
    for (int e = tid; e < kTile * kTile; e += kSmallThreads) {
        const int i = e >> 6, jj = e & 63;
        const double m = sm.ta[i * PS + jj];
        Fg[(size_t)i * dp + jj] = (jj <= i) ? sm.s[i][jj] : 0.0;
        Mg[(size_t)i * dp + jj] = m;
        sm.td[i * PS + jj] = m;
    }
    __syncthreads();
}

// Factor the tile range [lo, lo + nt), nt <= kSmallMax, of every layer with one CTA per layer:
// right-looking tile Cholesky (A -> F) followed by the block forward substitution for M = F^-1.
// Every product is a 64 x 64 x 64 tile product of the whole CTA on the float64 tensor core, with
// its operands fetched from global memory (the L2) into shared memory.
__global__ void __launch_bounds__(kSmallThreads, 1) k_factor_small(double* A, double* F, double* M, int dp, int lo,
                                                        int nt, int* layer_status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmallSmem& sm = *reinterpret_cast<SmallSmem*>(smem_raw);
    const int l = blockIdx.x;
    const size_t lay = (size_t)l * dp * dp;
    auto tile = [&](double* base, int i, int j) {
        return base + lay + (size_t)(lo + i) * kTile * dp + (size_t)(lo + j) * kTile;
    };
    if (threadIdx.x == 0) sm.flag = 0;
    SmallAcc acc;
    for (int j = 0; j < nt; ++j) {
        leaf_factor(tile(A, j, j), tile(F, j, j), tile(M, j, j), dp, sm);
        // F_ij = A_ij D_j^T
        for (int i = j + 1; i < nt; ++i) {
            tile_async(sm.ta, tile(A, i, j), dp);
            cp_async_commit();
            cp_async_wait<0>();
            __syncthreads();
            acc.zero();
            tile_mma<false, false>(acc, sm.ta, sm.td);
            double* out = tile(F, i, j);
            small_epilogue(acc, [&](int r, int c, double2 v) {
                *reinterpret_cast<double2*>(out + (size_t)r * dp + c) = v;
            });
            __syncthreads();
        }
        // A_ik -= F_ij F_kj^T for j < k <= i
        for (int i = j + 1; i < nt; ++i)
            for (int k = j + 1; k <= i; ++k) {
                tile_async(sm.ta, tile(F, i, j), dp);
                tile_async(sm.tb, tile(F, k, j), dp);
                cp_async_commit();
                cp_async_wait<0>();
                __syncthreads();
                acc.zero();
                tile_mma<false, false>(acc, sm.ta, sm.tb);
                double* out = tile(A, i, k);
                small_epilogue(acc, [&](int r, int c, double2 v) {
                    double2* o = reinterpret_cast<double2*>(out + (size_t)r * dp + c);
                    double2 cur = *o;
                    cur.x -= v.x; cur.y -= v.y;
                    *o = cur;
                });
                __syncthreads();
            }
    }
    // M_ij = -M_ii (sum over j <= k < i of F_ik M_kj), column by column
    for (int j = 0; j < nt; ++j)
        for (int i = j + 1; i < nt; ++i) {
            acc.zero();
            for (int k = j; k < i; ++k) {
                tile_async(sm.ta, tile(F, i, k), dp);
                tile_async(sm.tb, tile(M, k, j), dp);
                cp_async_commit();
                cp_async_wait<0>();
                __syncthreads();
                tile_mma<false, true>(acc, sm.ta, sm.tb);
                __syncthreads();
            }
            tile_async(sm.ta, tile(M, i, i), dp);
            cp_async_commit();
            small_epilogue(acc, [&](int r, int c, double2 v) {
                *reinterpret_cast<double2*>(sm.tb + r * PS + c) = v;
            });
            cp_async_wait<0>();
            __syncthreads();
            acc.zero();
            tile_mma<false, true>(acc, sm.ta, sm.tb);
            double* out = tile(M, i, j);
            small_epilogue(acc, [&](int r, int c, double2 v) {
                *reinterpret_cast<double2*>(out + (size_t)r * dp + c) = make_double2(-v.x, -v.y);
            });
            __syncthreads();
        }
    if (threadIdx.x == 0 && sm.flag) set_layer_status(layer_status, l, sm.flag);
}

// H^-1 = M^T M on the lower tiles (i >= j): sum over k >= i of M_ki^T M_kj; writes the cropped
// d x d result as float64 (mirrored to the upper triangle) and/or fp32 off-diagonal (both
// triangles) + fp64 diag.
// One CTA per 128 x 64 macro tile that reaches the lower triangle.
__global__ void __launch_bounds__(GT, 2) k_lauum(const double* M, int dp, int T, int d, double* out64,
                                                 float* tri32, int pitch32, double* diag64) {
    extern __shared__ __align__(16) double smem[];
    const int l = blockIdx.y;
    int I, J;
    lower_macro_index(blockIdx.x, T, I, J);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ti = 2 * I + (warp >> 2), tj = J;
    const bool mine = ti < T && ti >= tj;
    const double* Ml = M + (size_t)l * dp * dp;
    const int rows_valid = min(MTM, (T - 2 * I) * kTile);
    WarpAcc acc;
    acc.zero();
    // (M^T M)_ij: opA(i,k) = M[k][i] (stored K x m), opB(k,j) = M[k][j]; tile (ti, .) starts at k = ti
    dgemm_macro<true, false>(acc, Ml + (size_t)(2 * I) * kTile, dp, Ml + (size_t)J * kTile, dp,
                             2 * I, T, mine ? ti : 0, mine ? T : 0, rows_valid, smem);
    if (!mine) return;
    const int row0 = 2 * I * kTile + 32 * (warp >> 1) + (lane >> 2);
    const int col0 = J * kTile + 32 * (warp & 1) + 2 * (lane & 3);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int row = row0 + 8 * i, col = col0 + 8 * j + e;
                if (row >= d || col >= d) continue;
                const double v = acc.d[i][j][e];
                if (out64 && row >= col) {
                    double* o = out64 + (size_t)l * d * d;
                    o[(size_t)row * d + col] = v;
                    o[(size_t)col * d + row] = v;
                }
                if (tri32 && row > col) {       // both triangles: a column can then be read as a row
                    float* t = tri32 + (size_t)l * d * pitch32;
                    t[(size_t)row * pitch32 + col] = (float)v;
                    t[(size_t)col * pitch32 + row] = (float)v;
                }
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

int task_ctas(const GemmTask& t) {
    const int mm = (t.mt + 1) / 2;                           // macro tiles: mm x t.nt
    return t.lower_only ? lower_macro_count(t.mt) : mm * t.nt;
}

ziplm_status launch_pair(const InvCtx& c, const GemmTask& t1, const GemmTask& t2) {
    const int n1 = task_ctas(t1), n2 = task_ctas(t2);
    const cudaError_t attr = cudaFuncSetAttribute(
        k_dgemm_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProductSmemBytes);
    if (attr != cudaSuccess) return ZIPLM_ERR_CUDA;
    PhaseScope ps(PH_INV_PRODUCTS, c.st);
    k_dgemm_pair<<<dim3(n1 + n2, c.L), GT, kProductSmemBytes, c.st>>>(t1, n1, t2, c.dp);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

template <bool TA, bool TB>
ziplm_status launch_gemm(const InvCtx& c, const GemmTask& t) {
    const int ctas = task_ctas(t);
    if (ctas <= 0 || t.kt <= 0) return ZIPLM_OK;
    const cudaError_t attr = cudaFuncSetAttribute(
        k_dgemm_tiles<TA, TB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProductSmemBytes);
    if (attr != cudaSuccess) return ZIPLM_ERR_CUDA;
    PhaseScope ps(PH_INV_PRODUCTS, c.st);
    k_dgemm_tiles<TA, TB><<<dim3(ctas, c.L), GT, kProductSmemBytes, c.st>>>(t, c.dp);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

// Factor the tile range [lo, hi): on return F holds the Cholesky factor of the (updated) block
// and M its inverse.
ziplm_status factor_range(const InvCtx& c, int lo, int hi) {
    if (hi - lo <= kSmallMax) {
        const cudaError_t attr = cudaFuncSetAttribute(
            k_factor_small, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SmallSmem));
        if (attr != cudaSuccess) return ZIPLM_ERR_CUDA;
        PhaseScope ps(PH_INV_LEAVES, c.st);
        // One CTA per layer and a long dependent chain: launched at the highest priority, so that
        // it does not queue behind the wide kernels of other layer groups.
        static int prio = [] {
            int least = 0, greatest = 0;
            return cudaDeviceGetStreamPriorityRange(&least, &greatest) == cudaSuccess ? greatest : 0;
        }();
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(c.L);
        cfg.blockDim = dim3(kSmallThreads);
        cfg.dynamicSmemBytes = sizeof(SmallSmem);
        cfg.stream = c.st;
        cudaLaunchAttribute la[1];
        la[0].id = cudaLaunchAttributePriority;
        la[0].val.priority = prio;
        cfg.attrs = la;
        cfg.numAttrs = 1;
        ZIPLM_CHECK_CUDA(cudaLaunchKernelEx(&cfg, k_factor_small, c.A, c.F, c.M, c.dp, lo, hi - lo,
                                            c.layer_status));
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
    // A22 -= F21 F21^T  (lower tiles), and in the same launch
    // scratch (the dead A21 block) = F21 M11   (M11 lower: opB(k,j) vanishes for k < j):
    // its operands are final here and only the M21 product below reads it
    {
        const GemmTask syrk{c.F, mid, lo, c.F, mid, lo, c.A, mid, mid, n2, n2, n1, 0, 1, -1.0, 1};
        const GemmTask scr{c.F, mid, lo, c.M, lo, lo, c.A, mid, lo, n2, n1, n1, 3, 0, 1.0, 0};
        if ((s = launch_pair(c, syrk, scr)) != ZIPLM_OK) return s;
    }
    if ((s = factor_range(c, mid, hi)) != ZIPLM_OK) return s;
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
        const cudaError_t attr = cudaFuncSetAttribute(
            k_lauum, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProductSmemBytes);
        if (attr != cudaSuccess) return ZIPLM_ERR_CUDA;
        k_lauum<<<dim3(lower_macro_count(T), L), GT, kProductSmemBytes, st>>>(ctx.M, dp, T, d, out64, tri32,
                                                                            pitch32, diag64);
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
