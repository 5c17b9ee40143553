// Calibration Hessian H = beta H + alpha X X^T (caption of Algorithm 1) on the 5th-generation
// tensor cores: TMA-fed 128-byte-swizzled K-major tiles, tcgen05.mma issued by one thread,
// fp32 accumulator in tensor memory, read back with tcgen05.ld for the symmetric store.
//
// Both operands of X X^T are row blocks of the same K-major matrix (tokens contiguous), so one
// tensor map serves A and B.  Only the 128 x 128 tiles on or below the diagonal are computed; an
// off-diagonal tile is stored twice (as is, and transposed).
//
//   bf16 X : kind::f16 (bf16 x bf16, exact products, fp32 accumulate), K block of 64 tokens.
//   fp32 X : a pre-pass writes X_hi (fp32 with the 13 low mantissa bits cleared = a TF32 value)
//            and X_lo = X - X_hi; the kernel accumulates hi*hi + hi*lo + lo*hi with kind::tf32,
//            which keeps ~21 mantissa bits per product.  K block of 32 tokens.
//
// One CTA per tile: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..9 =
// epilogue (two per TMEM lane quarter; they drain the accumulator every few K blocks, see
// below).  Every mbarrier wait is bounded; if one runs out the
// kernel raises the error word, poisons H[l][0][0] with NaN and leaves through the normal exit
// (TMEM freed), so a lost copy can never hang the GPU.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"

namespace ziplm {
namespace {

constexpr int TM = 128;                 // tile rows / cols
constexpr int ROW_BYTES = 128;          // one swizzle row
constexpr int TILE_BYTES = TM * ROW_BYTES;   // 16 KiB per operand tile per K block
constexpr uint32_t kSpinLimit = 1u << 22;          // polls per wait, and ...
constexpr long long kSpinClocks = 4000000000ll;    // ... about two seconds of SM clocks

template <bool TF32> struct Cfg;
template <> struct Cfg<true>  { static constexpr int BK = 32, UK = 8,  STAGES = 3, TILES = 4; };
template <> struct Cfg<false> { static constexpr int BK = 64, UK = 16, STAGES = 5, TILES = 2; };

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within the spin limit or an abort was raised.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u && (*abort_flag || clock64() - t0 > kSpinClocks)) return false;
    }
    return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
          "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
          "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major, 128-byte-swizzled tile whose rows are 128 bytes:
// start address / 16, leading byte offset 1 (unused for swizzled K-major), stride byte offset
// 1024 / 16 between 8-row groups, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
           (2ull << 61);
}

// Instruction descriptor: fp32 accumulate, A and B K-major, N = 128, M = 128; operand format
// 2 = TF32 or 1 = BF16.
__host__ __device__ constexpr uint32_t make_idesc(uint32_t fmt) {
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(TM >> 3) << 17) |
           ((uint32_t)(TM >> 4) << 24);
}

// Tensor-memory accumulators truncate when they add (measured: the error of a chain of S
// accumulating MMAs grows like S * 3e-8, always toward zero), so a chain is kept short: the main
// accumulator is double-buffered, and after every CHUNK K blocks (8 MMAs) the epilogue warps
// drain it into fp32 registers, where the partial sums are added with round-to-nearest in two
// levels (a running sum that is folded into the total every FOLD drains, so that neither level
// adds more than a few dozen terms).  The TF32 cross terms hi*lo + lo*hi are 2^-11 of the main
// term; they get an accumulator of their own that is only read at the end, so their truncation
// is negligible.
constexpr int CHUNK = 2;
constexpr int FOLD = 32;
constexpr int EPI_WARPS = 8;                  // two warps per TMEM lane quarter, 64 columns each
constexpr int THREADS = 32 * (2 + EPI_WARPS);

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <bool TF32>
__global__ void __launch_bounds__(THREADS, 1)
k_syrk_tc(const __grid_constant__ CUtensorMap map_hi, const __grid_constant__ CUtensorMap map_lo,
          float* __restrict__ H, int d, int num_kb, float alpha, float beta, int layer0,
          int* __restrict__ err_word) {
    using C = Cfg<TF32>;
    constexpr int STAGE_BYTES = C::TILES * TILE_BYTES;
    constexpr uint32_t TMEM_COLS = TF32 ? 512u : 256u;   // main x2 (+ cross terms), power of two
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[C::STAGES], bar_empty[C::STAGES], bar_acc_full[2], bar_acc_empty[2];
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

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer
            const uint32_t bytes = (uint32_t)((diag ? C::TILES / 2 : C::TILES) * TILE_BYTES);
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % C::STAGES;
                const uint32_t ph = (uint32_t)(kb / C::STAGES) & 1u;
                if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, abortp)) { failed = true; break; }
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
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer
            constexpr uint32_t idesc = make_idesc(TF32 ? 2u : 1u);
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
                            umma_tf32(tmem_main, a_hi + adv, b_hi + adv, idesc, acc_main);
                            umma_tf32(tmem_cross, a_hi + adv, b_lo + adv, idesc, (kb | k) ? 1u : 0u);
                            umma_tf32(tmem_cross, a_lo + adv, b_hi + adv, idesc, 1u);
                        } else {
                            umma_bf16(tmem_main, a_hi + adv, b_hi + adv, idesc, acc_main);
                        }
                    }
                    umma_commit(smem_u32(&bar_empty[s]));     // stage free once these MMAs have read it
                }
                if (!failed) umma_commit(smem_u32(&bar_acc_full[b]));   // chunk (and all before) done
            }
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
#pragma unroll
            for (int e = 0; e < NC; ++e) {
                const int col = j0 + half * NC + e;
                float val = alpha * (tot[e] + acc[e]);
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
        // give copies that are still in flight a bounded chance to land before the CTA retires
        if (threadIdx.x == 0) {
            for (int s = 0; s < C::STAGES; ++s)
                for (uint32_t it = 0; it < 4096u; ++it)
                    if (mbar_try_wait(smem_u32(&bar_full[s]), 0u) || mbar_try_wait(smem_u32(&bar_full[s]), 1u))
                        break;
            H[(size_t)(layer0 + l) * d * d] = __int_as_float(0x7fc00000);
        }
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS)
                     : "memory");
    }
}

// X_hi = X with the 13 low mantissa bits cleared (exactly a TF32 value), X_lo = X - X_hi (exact).
__global__ void __launch_bounds__(256) k_split_tf32(const float* __restrict__ X, long long ldx,
                                                    long long N, long long np, size_t rows,
                                                    float* __restrict__ hi, float* __restrict__ lo) {
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
    float h[4], w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        h[e] = __uint_as_float(__float_as_uint(v[e]) & 0xffffe000u);
        w[e] = v[e] - h[e];
    }
    *reinterpret_cast<float4*>(hi + row * (size_t)np + k) = make_float4(h[0], h[1], h[2], h[3]);
    *reinterpret_cast<float4*>(lo + row * (size_t)np + k) = make_float4(w[0], w[1], w[2], w[3]);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !p)
        return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
    return fn;
}

// 3-D map over [layers, rows, K] with box {128 bytes of K, 128 rows, 1 layer}, 128-byte swizzle,
// zero fill outside the tensor (ragged d and ragged token counts contribute zeros).
bool make_map(CUtensorMap* m, const void* base, bool f32, long long K, int rows, int layers,
              long long pitch_elems) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const size_t esz = f32 ? 4 : 2;
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)layers};
    cuuint64_t strides[2] = {(cuuint64_t)pitch_elems * esz, (cuuint64_t)pitch_elems * esz * rows};
    cuuint32_t box[3] = {(cuuint32_t)(ROW_BYTES / esz), (cuuint32_t)TM, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                     const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

constexpr size_t kSplitCapBytes = (size_t)8 << 30;   // bound on the hi/lo scratch of one chunk

long long padded_tokens(long long N) { return (N + 3) / 4 * 4; }

int split_chunk_layers(int L, int d, long long N) {
    const size_t per_layer = 2 * (size_t)d * (size_t)padded_tokens(N) * 4;
    size_t lc = kSplitCapBytes / (per_layer ? per_layer : 1);
    if (lc < 1) lc = 1;
    return (int)(lc < (size_t)L ? lc : (size_t)L);
}

}  // namespace

size_t hessian_tc_workspace_bytes(int L, int d, long long N, ziplm_dtype dt) {
    size_t b = kAlign;   // error word
    if (dt == ZIPLM_F32) {
        const int lc = split_chunk_layers(L, d, N);
        b += 2 * align_up((size_t)lc * d * (size_t)padded_tokens(N) * 4);
    }
    return b;
}

ziplm_status run_hessian_tc(float* H, const void* X, ziplm_dtype dt, int L, int d, long long N,
                            long long ldx, float alpha, float beta, void* ws, size_t ws_bytes,
                            cudaStream_t st) {
    if (ws_bytes < hessian_tc_workspace_bytes(L, d, N, dt)) return ZIPLM_ERR_WORKSPACE;
    const bool f32 = (dt == ZIPLM_F32);
    Carver c(ws);
    int* err_word = c.take<int>(1);
    ZIPLM_CHECK_CUDA(cudaMemsetAsync(err_word, 0, sizeof(int), st));
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
        const long long np = padded_tokens(N);
        const int lc = split_chunk_layers(L, d, N);
        float* hi = c.take<float>((size_t)lc * d * np);
        float* lo = c.take<float>((size_t)lc * d * np);
        const int num_kb = (int)((N + Cfg<true>::BK - 1) / Cfg<true>::BK);
        for (int l0 = 0; l0 < L; l0 += lc) {
            const int ln = (L - l0 < lc) ? (L - l0) : lc;
            const size_t rows = (size_t)ln * d;
            const float* Xc = static_cast<const float*>(X) + (size_t)l0 * d * ldx;
            // grid.y is limited to 65535 rows per launch
            for (size_t r0 = 0; r0 < rows; r0 += 65535) {
                const size_t rn = rows - r0 < 65535 ? rows - r0 : 65535;
                k_split_tf32<<<dim3((unsigned)((np / 4 + 255) / 256), (unsigned)rn), 256, 0, st>>>(
                    Xc + r0 * ldx, ldx, N, np, rn, hi + r0 * np, lo + r0 * np);
                ZIPLM_CHECK_LAUNCH();
            }
            CUtensorMap mh, ml;
            if (!make_map(&mh, hi, true, N, d, ln, np) || !make_map(&ml, lo, true, N, d, ln, np))
                return ZIPLM_ERR_CUDA;
            k_syrk_tc<true><<<dim3(n_tiles, ln), THREADS, smem_tf32, st>>>(mh, ml, H, d, num_kb, alpha, beta,
                                                                      l0, err_word);
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
            if (!make_map(&mx, Xc, false, N, d, ln, ldx)) return ZIPLM_ERR_CUDA;
            k_syrk_tc<false><<<dim3(n_tiles, ln), THREADS, smem_bf16, st>>>(mx, mx, H, d, num_kb, alpha, beta,
                                                                       l0, err_word);
            ZIPLM_CHECK_LAUNCH();
        }
    }
    return ZIPLM_OK;
}

}  // namespace ziplm
