// Calibration Hessian H = beta H + alpha X X^T (caption of Algorithm 1) on the 5th-generation
// tensor cores: TMA-fed 128-byte-swizzled K-major tiles, tcgen05.mma issued by one thread,
// fp32 accumulator in tensor memory, read back with tcgen05.ld for the symmetric store.
//
// Both operands of X X^T are row blocks of the same K-major matrix (tokens contiguous), so one
// tensor map serves A and B.  Only the 128 x 128 tiles on or below the diagonal are computed; an
// off-diagonal tile is stored twice (as is, and transposed).
//
//   bf16 / fp16 X : kind::f16 (both operands of the same 16-bit type, exact products, fp32
//            accumulate), K block of 64 tokens.
//   fp32 X : a pre-pass scales every feature row by a power of two s_i (so that its largest
//            entry lies in [2^13, 2^14): the whole fp16 range is used whatever the row's
//            magnitude) and writes two fp16 parts, X_1 = fp16(s x) and X_2 = fp16(s x - X_1);
//            the kernel accumulates X_1 X_1^T + X_1 X_2^T + X_2 X_1^T with kind::f16 (exact
//            products, fp32 accumulate), which keeps ~21 mantissa bits per product, and the
//            epilogue multiplies entry (i, j) by 1 / (s_i s_j) (exact).  K block of 64 tokens:
//            half the operand bytes and half the MMAs of a TF32 hi / lo split of the same
//            accuracy, which matters because the kernel is bound by the L2 -> shared-memory
//            operand traffic.
//
// One CTA per tile: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..9 =
// epilogue (two per TMEM lane quarter; they drain the accumulator every few K blocks, see
// below).  Every mbarrier wait is bounded; if one runs out the kernel raises the error word and
// every role leaves its loop; the issuer then waits (one more commit) for the MMAs it has issued,
// the producer for the copies it has started, and the CTA leaves through the normal exit (TMEM
// freed), so a lost copy can never hang the GPU.  A small kernel after the product launches turns
// a raised error word into NaN in H[l][0][0] of every layer.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace ziplm {
namespace {
using namespace tc;

constexpr int TM = 128;                 // tile rows / cols
constexpr int ROW_BYTES = 128;          // one swizzle row
constexpr int TILE_BYTES = TM * ROW_BYTES;   // 16 KiB per operand tile per K block

template <bool SPLIT> struct Cfg;   // SPLIT: two fp16 parts per operand (fp32 inputs)
template <> struct Cfg<true>  { static constexpr int BK = 64, UK = 16, STAGES = 3, TILES = 4; };
template <> struct Cfg<false> { static constexpr int BK = 64, UK = 16, STAGES = 5, TILES = 2; };

// Tensor-memory accumulators truncate when they add (measured: the error of a chain of S
// accumulating MMAs grows like S * 3e-8, always toward zero), so a chain is kept short: the main
// accumulator is double-buffered, and after every CHUNK K blocks (8 MMAs) the epilogue warps
// drain it into fp32 registers, where the partial sums are added with round-to-nearest in two
// levels (a running sum that is folded into the total every FOLD drains, so that neither level
// adds more than a few dozen terms).  The cross terms X_1 X_2^T + X_2 X_1^T of the split are
// 2^-11 of the main term; they get an accumulator of their own that is only read at the end, so
// their truncation is negligible.
constexpr int CHUNK = 2;
constexpr int FOLD = 32;
constexpr int EPI_WARPS = 8;                  // two warps per TMEM lane quarter, 64 columns each
constexpr int THREADS = 32 * (2 + EPI_WARPS);

// Power-of-two scale of a feature row from the bit pattern of its largest magnitude m: the largest
// scaled entry lies in [2^13, 2^14).  inverse = true gives 1 / scale.  Rows of zeros and
// non-finite rows are left alone; the exponent is clamped so that the scale is a normal number.
__device__ __forceinline__ float row_scale(unsigned amax_bits, bool inverse) {
    const int e = (int)((amax_bits >> 23) & 255u);
    if (amax_bits == 0u || e == 255) return 1.f;
    int k = 140 - e;                       // m in [2^(e-127), 2^(e-126))  ->  m 2^k < 2^14
    k = k > 100 ? 100 : (k < -100 ? -100 : k);
    return __int_as_float((127 + (inverse ? -k : k)) << 23);
}

template <bool TF32>
__global__ void __launch_bounds__(THREADS, 1)
k_syrk_tc(const __grid_constant__ CUtensorMap map_hi, const __grid_constant__ CUtensorMap map_lo,
          float* __restrict__ H, int d, int num_kb, float alpha, float beta, int layer0,
          int* __restrict__ err_word, uint32_t fmt16, uint32_t empty_spin_limit,
          const unsigned* __restrict__ amax) {
    using C = Cfg<TF32>;
    constexpr int STAGE_BYTES = C::TILES * TILE_BYTES;
    constexpr uint32_t TMEM_COLS = TF32 ? 512u : 256u;   // main x2 (+ cross terms), power of two
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[C::STAGES], bar_empty[C::STAGES], bar_acc_full[2], bar_acc_empty[2], bar_final;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;       // swizzled tiles need 1024-byte alignment
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int l = blockIdx.y;                             // layer within the launched chunk
    int ti = 0, rem = blockIdx.x;
    while (rem > ti) { rem -= ti + 1; ++ti; }
    const int tj = rem;
    const int i0 = ti * TM, j0 = tj * TM;
    const bool diag = (ti == tj);
    const int num_chunks = (num_kb + CHUNK - 1) / CHUNK;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), EPI_WARPS);   // one arrival per epilogue warp
        }
        mbar_init(smem_u32(&bar_final), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;            // main[0] = +0, main[1] = +128, cross = +256
    volatile int* abortp = &abort_flag;
    bool failed = false;
    int issued = 0;                                       // K blocks whose copies were started (thread 0)

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer
            const uint32_t bytes = (uint32_t)((diag ? C::TILES / 2 : C::TILES) * TILE_BYTES);
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % C::STAGES;
                const uint32_t ph = (uint32_t)(kb / C::STAGES) & 1u;
                if (!mbar_wait_limit(smem_u32(&bar_empty[s]), ph ^ 1u, abortp, empty_spin_limit)) {
                    failed = true;
                    break;
                }
                const uint32_t full = smem_u32(&bar_full[s]);
                const uint32_t base = tiles + (uint32_t)s * STAGE_BYTES;
                mbar_expect_tx(full, bytes);
                const int x = kb * C::BK;
                tma_load_3d(base, &map_hi, full, x, i0, l);
                if (!diag) tma_load_3d(base + TILE_BYTES, &map_hi, full, x, j0, l);
                if (TF32) {
                    tma_load_3d(base + 2 * TILE_BYTES, &map_lo, full, x, i0, l);
                    if (!diag) tma_load_3d(base + 3 * TILE_BYTES, &map_lo, full, x, j0, l);
                }
                issued = kb + 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer
            // operand format of the instruction: 1 = BF16, 0 = F16 (A and B alike; the split is fp16)
            const uint32_t idesc = make_idesc(TF32 ? 0u : fmt16, TM, TM);
            const uint32_t tmem_cross = tmem_base + 256u;
            int kb = 0;
            for (int c = 0; c < num_chunks && !failed; ++c) {
                const int b = c & 1;
                const uint32_t tmem_main = tmem_base + (uint32_t)b * 128u;
                // the epilogue must have drained this buffer (first use of each buffer passes)
                if (!mbar_wait(smem_u32(&bar_acc_empty[b]), (((uint32_t)c >> 1) & 1u) ^ 1u, abortp)) {
                    failed = true;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int kb_end = (kb + CHUNK < num_kb) ? kb + CHUNK : num_kb;
                const int kb_first = kb;
                for (; kb < kb_end; ++kb) {
                    const int s = kb % C::STAGES;
                    const uint32_t ph = (uint32_t)(kb / C::STAGES) & 1u;
                    if (!mbar_wait(smem_u32(&bar_full[s]), ph, abortp)) { failed = true; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t base = tiles + (uint32_t)s * STAGE_BYTES;
                    const uint64_t a_hi = make_desc(base);
                    const uint64_t b_hi = diag ? a_hi : make_desc(base + TILE_BYTES);
                    const uint64_t a_lo = make_desc(base + 2 * TILE_BYTES);
                    const uint64_t b_lo = diag ? a_lo : make_desc(base + 3 * TILE_BYTES);
#pragma unroll
                    for (int k = 0; k < C::BK / C::UK; ++k) {
                        const uint64_t adv = (uint64_t)(k * 32 / 16);   // 32 bytes per MMA along K
                        const uint32_t acc_main = ((kb - kb_first) | k) ? 1u : 0u;
                        if (TF32) {
                            umma_bf16(tmem_main, a_hi + adv, b_hi + adv, idesc, acc_main);
                            umma_bf16(tmem_cross, a_hi + adv, b_lo + adv, idesc, (kb | k) ? 1u : 0u);
                            umma_bf16(tmem_cross, a_lo + adv, b_hi + adv, idesc, 1u);
                        } else {
                            umma_bf16(tmem_main, a_hi + adv, b_hi + adv, idesc, acc_main);
                        }
                    }
                    umma_commit(smem_u32(&bar_empty[s]));     // stage free once these MMAs have read it
                }
                if (!failed) umma_commit(smem_u32(&bar_acc_full[b]));   // chunk (and all before) done
            }
            // Whatever was issued has completed before tensor memory is given back and the CTA
            // retires, also when a role has given up: one more commit, to a barrier of its own.
            umma_commit(smem_u32(&bar_final));
            mbar_wait_quiet(smem_u32(&bar_final), 0u);
        }
    } else {
        // ---------------- epilogue: warps 2..9; TMEM lane quarter = warp % 4, column half by warp
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        constexpr int NC = TM / 2;                      // columns owned by this thread
        float acc[NC], tot[NC];
#pragma unroll
        for (int e = 0; e < NC; ++e) { acc[e] = 0.f; tot[e] = 0.f; }
        for (int c = 0; c < num_chunks; ++c) {
            const int b = c & 1;
            if (!mbar_wait(smem_u32(&bar_acc_full[b]), ((uint32_t)c >> 1) & 1u, abortp)) failed = true;
            failed = __any_sync(0xffffffffu, failed);
            if (failed) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int cc = 0; cc < NC / 32; ++cc) {
                uint32_t v[32];
                tmem_ld32(tmem_base + lane_base + (uint32_t)(b * 128 + half * NC + cc * 32), v);
#pragma unroll
                for (int e = 0; e < 32; ++e) acc[cc * 32 + e] += __uint_as_float(v[e]);
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[b]));
            if ((c % FOLD) == FOLD - 1) {
#pragma unroll
                for (int e = 0; e < NC; ++e) { tot[e] += acc[e]; acc[e] = 0.f; }
            }
        }
        if (!failed) {
            if (TF32) {
                // the last chunk's commit also covers every cross-term MMA
#pragma unroll
                for (int cc = 0; cc < NC / 32; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + lane_base + (uint32_t)(256 + half * NC + cc * 32), v);
#pragma unroll
                    for (int e = 0; e < 32; ++e) acc[cc * 32 + e] += __uint_as_float(v[e]);
                }
            }
            float* Hl = H + (size_t)(layer0 + l) * d * d;
            const int row = i0 + q * 32 + lane;
            // split route: undo the power-of-two scales of the two feature rows (exact)
            const unsigned* am = TF32 ? amax + (size_t)l * d : nullptr;
            const float inv_row = (TF32 && row < d) ? row_scale(am[row], true) : 1.f;
#pragma unroll
            for (int e = 0; e < NC; ++e) {
                const int col = j0 + half * NC + e;
                float val = alpha * (tot[e] + acc[e]);
                if (TF32 && col < d) val = (val * inv_row) * row_scale(am[col], true);
                if (row < d && col < d && col <= row) {
                    if (beta != 0.f) val += Hl[(size_t)row * d + col];
                    Hl[(size_t)row * d + col] = val;
                    if (col != row) Hl[(size_t)col * d + row] = val;
                }
            }
        }
    }

    if (failed) {
        abort_flag = 1;
        atomicExch(err_word, (int)ZIPLM_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (abort_flag) {
        // Copies that were started land in this CTA's shared memory: wait for them (bounded) before
        // the CTA retires.  The last STAGES K blocks started are the latest phases of their barriers.
        if (threadIdx.x == 0)
            for (int kb = issued > C::STAGES ? issued - C::STAGES : 0; kb < issued; ++kb)
                mbar_wait_quiet(smem_u32(&bar_full[kb % C::STAGES]), (uint32_t)(kb / C::STAGES) & 1u);
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS)
                     : "memory");
    }
}

// A product kernel that gave up on a wait leaves ZIPLM_ERR_TIMEOUT in the error word; the layers'
// first entries then become NaN, after every product launch of the call, so that whichever stage
// reads H next reports ZIPLM_ERR_NONFINITE.
__global__ void k_hessian_flag_timeout(float* __restrict__ H, int L, int d, const int* __restrict__ err_word) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l < L && *err_word != 0) H[(size_t)l * d * d] = __int_as_float(0x7fc00000);
}

// Largest magnitude of every feature row of a token-contiguous X (bit pattern of |x|, which
// orders like the value for non-negative floats; a NaN sorts above everything and switches the
// scaling of its row off).
__global__ void __launch_bounds__(256) k_row_absmax(const float* __restrict__ X, long long ldx, long long N,
                                                    unsigned* __restrict__ amax) {
    __shared__ unsigned red[8];
    const size_t row = blockIdx.x;
    const float* src = X + row * (size_t)ldx;
    unsigned m = 0u;
    for (long long k = threadIdx.x; k < N; k += 256) m = max(m, __float_as_uint(src[k]) & 0x7fffffffu);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) m = max(m, red[w]);
        amax[row] = m;
    }
}

// The same for token-major input A [layers, N, lda] (one token per row): every thread walks one
// feature over a slab of tokens, the slabs meet through atomicMax (amax zeroed beforehand).
__global__ void __launch_bounds__(256) k_tokens_absmax(const float* __restrict__ A, long long lda,
                                                       long long N, int d, long long slab,
                                                       unsigned* __restrict__ amax) {
    const int l = blockIdx.z;
    const int f = blockIdx.x * 256 + threadIdx.x;
    if (f >= d) return;
    const long long t0 = (long long)blockIdx.y * slab, t1 = min(N, t0 + slab);
    const float* Al = A + (size_t)l * (size_t)N * (size_t)lda + f;
    unsigned m = 0u;
    for (long long t = t0; t < t1; ++t) m = max(m, __float_as_uint(Al[(size_t)t * (size_t)lda]) & 0x7fffffffu);
    atomicMax(amax + (size_t)l * d + f, m);
}

// The two fp16 parts of a scaled fp32 value y: y_1 = fp16(y), y_2 = fp16(y - y_1) (the difference
// is exact in fp32).
__device__ __forceinline__ void split_f16x2(float y, __half& p1, __half& p2) {
    p1 = __float2half_rn(y);
    p2 = __float2half_rn(y - __half2float(p1));
}

// X_1, X_2 of a token-contiguous fp32 X, four tokens per thread; np (a multiple of 8) is the row
// pitch of the parts, zero past N.
__global__ void __launch_bounds__(256) k_split_f16(const float* __restrict__ X, long long ldx,
                                                   long long N, long long np, size_t rows,
                                                   const unsigned* __restrict__ amax,
                                                   __half* __restrict__ hi, __half* __restrict__ lo) {
    const size_t row = blockIdx.y;
    const long long k = ((long long)blockIdx.x * 256 + threadIdx.x) * 4;
    if (row >= rows || k >= np) return;
    const float* src = X + row * (size_t)ldx + k;
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (k + 3 < N) {
        const float4 t = *reinterpret_cast<const float4*>(src);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
        for (int e = 0; e < 4; ++e) if (k + e < N) v[e] = src[e];
    }
    const float sc = row_scale(amax[row], false);
    union { uint2 u; __half h[4]; } a, b;
#pragma unroll
    for (int e = 0; e < 4; ++e) split_f16x2(v[e] * sc, a.h[e], b.h[e]);
    *reinterpret_cast<uint2*>(hi + row * (size_t)np + k) = a.u;
    *reinterpret_cast<uint2*>(lo + row * (size_t)np + k) = b.u;
}

// Both pre-passes in one for rows of at most 256 * 4 * VEC tokens: a CTA keeps its feature row in
// registers (VEC 16-byte loads per thread, all in flight together), finds the largest magnitude,
// and writes the two scaled fp16 parts -- X is read once instead of twice.  Values and layout are
// those of k_row_absmax followed by k_split_f16.
template <int VEC>
__global__ void __launch_bounds__(256) k_row_absmax_split(const float* __restrict__ X, long long ldx,
                                                          long long N, long long np,
                                                          unsigned* __restrict__ amax,
                                                          __half* __restrict__ hi, __half* __restrict__ lo) {
    __shared__ unsigned red[8];
    __shared__ unsigned row_max;
    const size_t row = blockIdx.x;
    const float* src = X + row * (size_t)ldx;
    float v[VEC][4];
    unsigned m = 0u;
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        const long long k = ((long long)j * 256 + threadIdx.x) * 4;
        v[j][0] = v[j][1] = v[j][2] = v[j][3] = 0.f;
        if (k + 3 < N) {
            const float4 t = *reinterpret_cast<const float4*>(src + k);
            v[j][0] = t.x; v[j][1] = t.y; v[j][2] = t.z; v[j][3] = t.w;
        } else {
            for (int e = 0; e < 4; ++e) if (k + e < N) v[j][e] = src[k + e];
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) m = max(m, __float_as_uint(v[j][e]) & 0x7fffffffu);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) m = max(m, red[w]);
        amax[row] = m;
        row_max = m;
    }
    __syncthreads();
    const float sc = row_scale(row_max, false);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        const long long k = ((long long)j * 256 + threadIdx.x) * 4;
        if (k >= np) continue;
        union { uint2 u; __half h[4]; } a, b;
#pragma unroll
        for (int e = 0; e < 4; ++e) split_f16x2(v[j][e] * sc, a.h[e], b.h[e]);
        *reinterpret_cast<uint2*>(hi + row * (size_t)np + k) = a.u;
        *reinterpret_cast<uint2*>(lo + row * (size_t)np + k) = b.u;
    }
}

// Token-major input (one calibration token per row, as a forward pass emits activations):
// A is [layers, N, lda] with the feature index contiguous.  A 32 x 32 tile goes through shared
// memory, so the reads run along features and the writes along tokens, both coalesced; the output
// is the K-major [layers * d, np] matrix the product kernel loads.  SPLIT writes the scaled fp16
// parts X_1 / X_2 of an fp32 input directly (same values as k_split_f16; O = __half, amax holds
// the features' largest magnitudes); otherwise the elements are moved as raw bits (T = O =
// uint16_t for bf16 and fp16).
template <typename T, typename O, bool SPLIT>
__global__ void __launch_bounds__(256) k_tokens_to_kmajor(const T* __restrict__ A, long long lda,
                                                          long long N, int d, long long np,
                                                          const unsigned* __restrict__ amax,
                                                          O* __restrict__ hi, O* __restrict__ lo) {
    __shared__ T tile[32][33];
    const int l = blockIdx.z;
    const long long t0 = (long long)blockIdx.x * 32;
    const int f0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const T* Al = A + (size_t)l * (size_t)N * (size_t)lda;
#pragma unroll
    for (int r = ty; r < 32; r += 8) {
        const long long t = t0 + r;
        const int f = f0 + tx;
        tile[r][tx] = (t < N && f < d) ? Al[(size_t)t * (size_t)lda + f] : T(0);
    }
    __syncthreads();
#pragma unroll
    for (int r = ty; r < 32; r += 8) {
        const int f = f0 + r;
        const long long t = t0 + tx;
        if (f >= d || t >= np) continue;
        const size_t o = ((size_t)l * d + f) * (size_t)np + (size_t)t;
        const T v = tile[tx][r];
        if constexpr (SPLIT) {
            split_f16x2(v * row_scale(amax[(size_t)l * d + f], false), hi[o], lo[o]);
        } else {
            hi[o] = v;
        }
    }
}

// The same move for inputs whose rows allow 4-element vector accesses (A aligned to 4 elements,
// lda % 4 == 0): a 64 x 64 tile, four elements per access on both sides, so a row of the output
// leaves in 256-byte (fp32) pieces.  np is a multiple of 4, so a quad that starts below np ends
// below it.
template <typename T, typename V, typename O, bool SPLIT>
__global__ void __launch_bounds__(256) k_tokens_to_kmajor_v4(const T* __restrict__ A, long long lda,
                                                             long long N, int d, long long np,
                                                             const unsigned* __restrict__ amax,
                                                             O* __restrict__ hi, O* __restrict__ lo) {
    __shared__ T tile[64][65];                       // [token][feature]
    union Quad { V v; T e[4]; };
    const int l = blockIdx.z;
    const long long t0 = (long long)blockIdx.x * 64;
    const int f0 = blockIdx.y * 64;
    const int q = threadIdx.x & 15, rr = threadIdx.x >> 4;
    const T* Al = A + (size_t)l * (size_t)N * (size_t)lda;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int tl = rr + 16 * k;
        const long long t = t0 + tl;
        const int f = f0 + 4 * q;
        Quad u;
        if (t < N && f + 3 < d) {
            u.v = *reinterpret_cast<const V*>(Al + (size_t)t * (size_t)lda + f);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                u.e[e] = (t < N && f + e < d) ? Al[(size_t)t * (size_t)lda + f + e] : T(0);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) tile[tl][4 * q + e] = u.e[e];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int fl = rr + 16 * k;
        const int f = f0 + fl;
        const long long t = t0 + 4 * q;
        if (f >= d || t >= np) continue;
        Quad u;
#pragma unroll
        for (int e = 0; e < 4; ++e) u.e[e] = tile[4 * q + e][fl];
        const size_t o = ((size_t)l * d + f) * (size_t)np + (size_t)t;
        if constexpr (SPLIT) {
            union { uint2 v; __half e[4]; } h, w;
            const float sc = row_scale(amax[(size_t)l * d + f], false);
#pragma unroll
            for (int e = 0; e < 4; ++e) split_f16x2(u.e[e] * sc, h.e[e], w.e[e]);
            *reinterpret_cast<uint2*>(hi + o) = h.v;
            *reinterpret_cast<uint2*>(lo + o) = w.v;
        } else {
            *reinterpret_cast<V*>(hi + o) = u.v;
        }
    }
}

bool quad_rows(const void* A, long long lda, size_t esz) {
    return (reinterpret_cast<uintptr_t>(A) % (4 * esz)) == 0 && lda % 4 == 0;
}

// 3-D map over [layers, rows, K] with box {128 bytes of K, 128 rows, 1 layer}, 128-byte swizzle,
// zero fill outside the tensor (ragged d and ragged token counts contribute zeros).
bool make_map(CUtensorMap* m, const void* base, ziplm_dtype dt, long long K, int rows, int layers,
              long long pitch_elems) {
    const bool f32 = (dt == ZIPLM_F32);
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const size_t esz = f32 ? 4 : 2;
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)layers};
    cuuint64_t strides[2] = {(cuuint64_t)pitch_elems * esz, (cuuint64_t)pitch_elems * esz * rows};
    cuuint32_t box[3] = {(cuuint32_t)(ROW_BYTES / esz), (cuuint32_t)TM, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                            : dt == ZIPLM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
                     const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

constexpr size_t kSplitCapBytes = (size_t)8 << 30;   // bound on the hi/lo scratch of one chunk

long long padded_tokens(long long N) { return (N + 3) / 4 * 4; }
long long padded_tokens_bf16(long long N) { return (N + 7) / 8 * 8; }   // 16-byte row pitch

// Layers per chunk of the K-major bf16 copy of a token-major input.
int transpose_chunk_layers(int L, int d, long long N) {
    const size_t per_layer = (size_t)d * (size_t)padded_tokens_bf16(N) * 2;
    size_t lc = kSplitCapBytes / (per_layer ? per_layer : 1);
    if (lc < 1) lc = 1;
    if (lc > 65535) lc = 65535;
    return (int)(lc < (size_t)L ? lc : (size_t)L);
}

int split_chunk_layers(int L, int d, long long N) {
    const size_t per_layer = 2 * (size_t)d * (size_t)padded_tokens_bf16(N) * 2;
    size_t lc = kSplitCapBytes / (per_layer ? per_layer : 1);
    if (lc < 1) lc = 1;
    return (int)(lc < (size_t)L ? lc : (size_t)L);
}

}  // namespace

size_t hessian_tc_workspace_bytes(int L, int d, long long N, ziplm_dtype dt, bool token_major) {
    size_t b = kAlign;   // error word
    if (dt == ZIPLM_F32) {
        const int lc = split_chunk_layers(L, d, N);
        b += align_up((size_t)lc * d * sizeof(unsigned));                            // row magnitudes
        b += 2 * align_up((size_t)lc * d * (size_t)padded_tokens_bf16(N) * 2);       // the two fp16 parts
    } else if (token_major) {
        const int lc = transpose_chunk_layers(L, d, N);
        b += align_up((size_t)lc * d * (size_t)padded_tokens_bf16(N) * 2);
    }
    return b;
}

ziplm_status run_hessian_tc(float* H, const void* X, ziplm_dtype dt, bool token_major, int L, int d,
                            long long N, long long ldx, float alpha, float beta, void* ws,
                            size_t ws_bytes, cudaStream_t st) {
    if (ws_bytes < hessian_tc_workspace_bytes(L, d, N, dt, token_major)) return ZIPLM_ERR_WORKSPACE;
    const bool f32 = (dt == ZIPLM_F32);
    const uint32_t fmt16 = (dt == ZIPLM_F16) ? 0u : 1u;
    Carver c(ws);
    int* err_word = c.take<int>(1);
    ZIPLM_CHECK_CUDA(cudaMemsetAsync(err_word, 0, sizeof(int), st));
    const int spin_opt = option_value(ZIPLM_OPT_SPIN_LIMIT);
    const uint32_t spin = spin_opt > 0 ? (uint32_t)spin_opt : kSpinLimit;
    const int T = (d + TM - 1) / TM;
    const int n_tiles = T * (T + 1) / 2;
    const size_t smem_tf32 = (size_t)Cfg<true>::STAGES * Cfg<true>::TILES * TILE_BYTES + 1024;
    const size_t smem_bf16 = (size_t)Cfg<false>::STAGES * Cfg<false>::TILES * TILE_BYTES + 1024;
    if (f32) {
        ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_syrk_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem_tf32));
    } else {
        ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_syrk_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem_bf16));
    }
    if (f32) {
        const long long np = padded_tokens_bf16(N);
        const int lc = split_chunk_layers(L, d, N);
        unsigned* amax = c.take<unsigned>((size_t)lc * d);
        __half* hi = c.take<__half>((size_t)lc * d * np);
        __half* lo = c.take<__half>((size_t)lc * d * np);
        const int num_kb = (int)((N + Cfg<true>::BK - 1) / Cfg<true>::BK);
        for (int l0 = 0; l0 < L; l0 += lc) {
            const int ln = (L - l0 < lc) ? (L - l0) : lc;
            const size_t rows = (size_t)ln * d;
            if (token_major) {
                const float* Ac = static_cast<const float*>(X) + (size_t)l0 * (size_t)N * ldx;
                ZIPLM_CHECK_CUDA(cudaMemsetAsync(amax, 0, sizeof(unsigned) * rows, st));
                // slabs of at least 256 tokens, at most 65535 of them (grid.y)
                const long long slab = N / 65535 + 1 > 256 ? N / 65535 + 1 : 256;
                // grid.z is limited to 65535 layers per launch
                for (int z0 = 0; z0 < ln; z0 += 65535) {
                    const int zn = ln - z0 < 65535 ? ln - z0 : 65535;
                    k_tokens_absmax<<<dim3((unsigned)((d + 255) / 256), (unsigned)((N + slab - 1) / slab),
                                           (unsigned)zn), 256, 0, st>>>(Ac + (size_t)z0 * N * ldx, ldx, N, d, slab,
                                                                        amax + (size_t)z0 * d);
                    ZIPLM_CHECK_LAUNCH();
                    if (quad_rows(X, ldx, 4))
                        k_tokens_to_kmajor_v4<float, float4, __half, true>
                            <<<dim3((unsigned)((np + 63) / 64), (unsigned)((d + 63) / 64), (unsigned)zn), 256,
                               0, st>>>(Ac + (size_t)z0 * N * ldx, ldx, N, d, np, amax + (size_t)z0 * d,
                                        hi + (size_t)z0 * d * np, lo + (size_t)z0 * d * np);
                    else
                        k_tokens_to_kmajor<float, __half, true>
                            <<<dim3((unsigned)((np + 31) / 32), (unsigned)((d + 31) / 32), (unsigned)zn), 256,
                               0, st>>>(Ac + (size_t)z0 * N * ldx, ldx, N, d, np, amax + (size_t)z0 * d,
                                        hi + (size_t)z0 * d * np, lo + (size_t)z0 * d * np);
                    ZIPLM_CHECK_LAUNCH();
                }
            } else {
                const float* Xc = static_cast<const float*>(X) + (size_t)l0 * d * ldx;
                // rows of up to 16384 tokens stay in registers: 1, 4 or 16 quads per thread
                if (np <= 256ll * 4 * 16) {
                    for (size_t r0 = 0; r0 < rows; r0 += (size_t)1 << 30) {
                        const size_t rn = rows - r0 < ((size_t)1 << 30) ? rows - r0 : ((size_t)1 << 30);
                        const float* xs = Xc + r0 * ldx;
                        if (np <= 256ll * 4)
                            k_row_absmax_split<1><<<(unsigned)rn, 256, 0, st>>>(xs, ldx, N, np, amax + r0,
                                                                                hi + r0 * np, lo + r0 * np);
                        else if (np <= 256ll * 4 * 4)
                            k_row_absmax_split<4><<<(unsigned)rn, 256, 0, st>>>(xs, ldx, N, np, amax + r0,
                                                                                hi + r0 * np, lo + r0 * np);
                        else
                            k_row_absmax_split<16><<<(unsigned)rn, 256, 0, st>>>(xs, ldx, N, np, amax + r0,
                                                                                 hi + r0 * np, lo + r0 * np);
                        ZIPLM_CHECK_LAUNCH();
                    }
                } else {
                    for (size_t r0 = 0; r0 < rows; r0 += (size_t)1 << 30) {
                        const size_t rn = rows - r0 < ((size_t)1 << 30) ? rows - r0 : ((size_t)1 << 30);
                        k_row_absmax<<<(unsigned)rn, 256, 0, st>>>(Xc + r0 * ldx, ldx, N, amax + r0);
                        ZIPLM_CHECK_LAUNCH();
                    }
                    // grid.y is limited to 65535 rows per launch
                    for (size_t r0 = 0; r0 < rows; r0 += 65535) {
                        const size_t rn = rows - r0 < 65535 ? rows - r0 : 65535;
                        k_split_f16<<<dim3((unsigned)((np / 4 + 255) / 256), (unsigned)rn), 256, 0, st>>>(
                            Xc + r0 * ldx, ldx, N, np, rn, amax + r0, hi + r0 * np, lo + r0 * np);
                        ZIPLM_CHECK_LAUNCH();
                    }
                }
            }
            CUtensorMap mh, ml;
            if (!make_map(&mh, hi, ZIPLM_F16, N, d, ln, np) || !make_map(&ml, lo, ZIPLM_F16, N, d, ln, np))
                return ZIPLM_ERR_CUDA;
            k_syrk_tc<true><<<dim3(n_tiles, ln), THREADS, smem_tf32, st>>>(mh, ml, H, d, num_kb, alpha, beta,
                                                                      l0, err_word, 0u, spin, amax);
            ZIPLM_CHECK_LAUNCH();
        }
    } else if (token_major) {
        // K-major bf16 copy of a chunk of layers, then the same product kernel
        const long long np = padded_tokens_bf16(N);
        const int lc = transpose_chunk_layers(L, d, N);
        uint16_t* xt = c.take<uint16_t>((size_t)lc * d * np);
        const int num_kb = (int)((N + Cfg<false>::BK - 1) / Cfg<false>::BK);
        for (int l0 = 0; l0 < L; l0 += lc) {
            const int ln = (L - l0 < lc) ? (L - l0) : lc;
            const uint16_t* Ac = static_cast<const uint16_t*>(X) + (size_t)l0 * (size_t)N * ldx;
            if (quad_rows(X, ldx, 2))
                k_tokens_to_kmajor_v4<uint16_t, uint2, uint16_t, false>
                    <<<dim3((unsigned)((np + 63) / 64), (unsigned)((d + 63) / 64), (unsigned)ln), 256, 0, st>>>(
                        Ac, ldx, N, d, np, nullptr, xt, nullptr);
            else
                k_tokens_to_kmajor<uint16_t, uint16_t, false>
                    <<<dim3((unsigned)((np + 31) / 32), (unsigned)((d + 31) / 32), (unsigned)ln), 256, 0, st>>>(
                        Ac, ldx, N, d, np, nullptr, xt, nullptr);
            ZIPLM_CHECK_LAUNCH();
            CUtensorMap mx;
            if (!make_map(&mx, xt, dt, N, d, ln, np)) return ZIPLM_ERR_CUDA;
            k_syrk_tc<false><<<dim3(n_tiles, ln), THREADS, smem_bf16, st>>>(mx, mx, H, d, num_kb, alpha, beta,
                                                                       l0, err_word, fmt16, spin, nullptr);
            ZIPLM_CHECK_LAUNCH();
        }
    } else {
        const int num_kb = (int)((N + Cfg<false>::BK - 1) / Cfg<false>::BK);
        // tensor-map dimensions are 32-bit boxes over up to 2^32 elements; chunk layers so that the
        // grid stays within limits
        for (int l0 = 0; l0 < L; l0 += 65535) {
            const int ln = (L - l0 < 65535) ? (L - l0) : 65535;
            CUtensorMap mx;
            const __nv_bfloat16* Xc = static_cast<const __nv_bfloat16*>(X) + (size_t)l0 * d * ldx;
            if (!make_map(&mx, Xc, dt, N, d, ln, ldx)) return ZIPLM_ERR_CUDA;
            k_syrk_tc<false><<<dim3(n_tiles, ln), THREADS, smem_bf16, st>>>(mx, mx, H, d, num_kb, alpha, beta,
                                                                       l0, err_word, fmt16, spin, nullptr);
            ZIPLM_CHECK_LAUNCH();
        }
    }
    k_hessian_flag_timeout<<<(L + 127) / 128, 128, 0, st>>>(H, L, d, err_word);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

}  // namespace ziplm
