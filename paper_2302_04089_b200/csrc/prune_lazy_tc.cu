// Rank-32 update of H^-1 and of the Gram matrix Q = W^T W (delayed Eq. 4 / Eq. 3) on the
// 5th-generation tensor cores.
//
//   A'[i,j] = A[si,sj] - sum_s U[s,si] U[s,sj]
//   Q'[i,j] = Q[si,sj] - sum_s (Z[s,si] U[s,sj] + U[s,si] Z[s,sj]),   si = src[i] > sj = src[j]
//
// A pre-pass (k_lazy_pack_uz) gathers the pending vectors through src into the new (compacted)
// index space, K-major ([position][step], one 128-byte row per position), split into two TF32
// values x = hi + lo (both rounded to nearest, so |x - hi - lo| <= 2^-24 |x|): U_hi, U_lo, Z_hi,
// Z_lo; all four partial products of a split pair are kept.  The update kernel then needs no gather for its operands:
// TMA brings the 128 rows and 64 columns of a tile into 128-byte-swizzled shared memory, one
// thread issues the 48 tcgen05.mma of the three split products (hi*hi and the cross terms in
// accumulators of their own, all starting from zero), and eight epilogue warps read the
// accumulators back, transpose them through shared memory so that lanes run along a matrix row,
// and subtract them from the gathered old entries with one fp32 operation each; every entry is
// stored at [i][j] and at [j][i].  The kernel is
// left with the streaming of the two triangles; two CTAs per SM overlap each other's phases.
//
// Every mbarrier wait is bounded; a wait that runs out marks the layer ZIPLM_ERR_TIMEOUT and the
// CTA leaves through the normal exit (tensor memory freed).
#include "common.cuh"
#include "tc_common.cuh"

namespace ziplm {
namespace {
using namespace tc;

constexpr int PK = 32;                       // pending steps per block = K of the products
constexpr int RM = 128, CN = 64;             // tile rows, tile columns (new index space)
constexpr int BOX_ROWS = 64;                 // rows per TMA box
constexpr int BOX_BYTES = BOX_ROWS * 128;    // 8 KiB
constexpr int ROW_TILE_BYTES = 2 * BOX_BYTES;
constexpr int OPERAND_BYTES = 4 * ROW_TILE_BYTES + 4 * BOX_BYTES;   // 96 KiB
constexpr int AQ_THREADS = 256;              // 8 epilogue warps; lane 0 of warp 0 also issues TMA and MMA
constexpr uint32_t AQ_TMEM_COLS = 256;       // A main, A cross, Q main, Q cross: 64 columns each
enum { P_UH = 0, P_UL = 1, P_ZH = 2, P_ZL = 3 };

// Nearest TF32 value (10 explicit mantissa bits), as an fp32 number.
__device__ __forceinline__ float round_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// P[l][a][i][s], a in {U_hi, U_lo, Z_hi, Z_lo}: pending vectors of the live positions in the new
// order, zero for steps >= m and for rows n_new .. the next multiple of 128.
__global__ void __launch_bounds__(256) k_lazy_pack_uz(int n_new, int m, int d, int rows_pad,
                                                      const int* __restrict__ src,
                                                      const float* __restrict__ U,
                                                      const float* __restrict__ Z,
                                                      float* __restrict__ P) {
    __shared__ float tu[PK][33], tz[PK][33];
    const int l = blockIdx.y, i0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int pos = i0 + tx;
    const int sp = pos < n_new ? src[(size_t)l * d + pos] : -1;
    const float* Ul = U + (size_t)l * PK * d;
    const float* Zl = Z + (size_t)l * PK * d;
#pragma unroll
    for (int s = ty; s < PK; s += 8) {
        const bool ok = sp >= 0 && s < m;
        tu[s][tx] = ok ? Ul[(size_t)s * d + sp] : 0.f;
        tz[s][tx] = ok ? Zl[(size_t)s * d + sp] : 0.f;
    }
    __syncthreads();
    float* Pl = P + (size_t)l * 4 * rows_pad * PK;
#pragma unroll
    for (int rr = ty; rr < 32; rr += 8) {
        const int i = i0 + rr;
        if (i >= rows_pad) continue;
        const float u = tu[tx][rr], z = tz[tx][rr];
        const float uh = round_tf32(u), zh = round_tf32(z);
        const size_t o = (size_t)i * PK + tx;
        Pl[(size_t)P_UH * rows_pad * PK + o] = uh;
        Pl[(size_t)P_UL * rows_pad * PK + o] = round_tf32(u - uh);
        Pl[(size_t)P_ZH * rows_pad * PK + o] = zh;
        Pl[(size_t)P_ZL * rows_pad * PK + o] = round_tf32(z - zh);
    }
}

// One CTA per tile of 128 rows x 64 columns that reaches below the diagonal; blockIdx.x runs over
// the row blocks I = 0, 1, ... with 2 I + 2 column blocks each, blockIdx.y over the layers.
__global__ void __launch_bounds__(AQ_THREADS, 2)
k_lazy_update_aq_tc(const __grid_constant__ CUtensorMap map, int n_new, int d,
                    const float* __restrict__ A, const float* __restrict__ Q,
                    float* __restrict__ A2, float* __restrict__ Q2, const int* __restrict__ src,
                    int* __restrict__ layer_status) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full, bar_acc;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int srow_off[RM], scol[CN];   // row offsets src[i] * d (0 past the live range)

    int I = 0, rem = blockIdx.x;
    while (rem >= 2 * I + 2) { rem -= 2 * I + 2; ++I; }
    const int J = rem;
    const int i0 = I * RM, j0 = J * CN;
    if (j0 >= n_new) return;                  // column block beyond the live range (ragged last row block)
    const int l = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;       // swizzled tiles need 1024-byte alignment
    uint8_t* tiles_ptr = smem_raw + (tiles - raw);

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar_full), 1);
        mbar_init(smem_u32(&bar_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(AQ_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    {
        const int* sl = src + (size_t)l * d;
        for (int e = threadIdx.x; e < RM + CN; e += AQ_THREADS) {
            if (e < RM) srow_off[e] = (i0 + e < n_new) ? sl[i0 + e] * d : 0;   // d * d < 2^31
            else scol[e - RM] = (j0 + e - RM < n_new) ? sl[j0 + e - RM] : -1;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    bool failed = false;

    // ---------------- epilogue: all 8 warps; TMEM lane quarter q = warp % 4 (rows 32 q ..),
    // column half cc = warp / 4 (columns 32 cc ..); one 32 x 32 block of A and of Q per
    // warp.  All loads are unconditional (clamped to a valid address) so that they pipeline;
    // what lies on or above the diagonal is simply not stored.
    const int q = warp & 3, cc = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const int j = j0 + cc * 32 + lane;
    const int sc = max(scol[cc * 32 + lane], 0);
    const float* Ac = A + (size_t)l * d * d + sc;
    const float* Qc = Q + (size_t)l * d * d + sc;
    const int* roff = srow_off + q * 32;
    float ca[32], cq[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) ca[e] = __ldcs(Ac + roff[e]);   // in flight while the operands load
#pragma unroll
    for (int e = 0; e < 32; ++e) cq[e] = __ldcs(Qc + roff[e]);   // and multiply

    if (warp == 0 && lane == 0) {
        {
            // ---------------- TMA producer: 4 arrays x (two boxes of rows + one box of columns)
            const uint32_t full = smem_u32(&bar_full);
            mbar_expect_tx(full, (uint32_t)OPERAND_BYTES);
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                tma_load_4d(tiles + a * ROW_TILE_BYTES, &map, full, 0, i0, a, l);
                tma_load_4d(tiles + a * ROW_TILE_BYTES + BOX_BYTES, &map, full, 0, i0 + BOX_ROWS, a, l);
                tma_load_4d(tiles + 4 * ROW_TILE_BYTES + a * BOX_BYTES, &map, full, 0, j0, a, l);
            }
            // ---------------- MMA issuer (same thread: the loads above are asynchronous)
            if (!mbar_wait(smem_u32(&bar_full), 0u, abortp)) {
                failed = true;
            } else {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                constexpr uint32_t idesc = make_idesc(2u, RM, CN);
                uint64_t r[4], c[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    r[a] = make_desc(tiles + a * ROW_TILE_BYTES);
                    c[a] = make_desc(tiles + 4 * ROW_TILE_BYTES + a * BOX_BYTES);
                }
                const uint32_t t_am = tmem_base, t_ac = tmem_base + 64u, t_qm = tmem_base + 128u,
                               t_qc = tmem_base + 192u;
#pragma unroll
                for (int k = 0; k < PK / 8; ++k) {
                    const uint64_t adv = (uint64_t)(k * 32 / 16);       // 32 bytes per MMA along K
                    const uint32_t acc = k ? 1u : 0u;
                    umma_tf32(t_am, r[P_UH] + adv, c[P_UH] + adv, idesc, acc);
                    umma_tf32(t_ac, r[P_UH] + adv, c[P_UL] + adv, idesc, acc);
                    umma_tf32(t_ac, r[P_UL] + adv, c[P_UH] + adv, idesc, 1u);
                    umma_tf32(t_ac, r[P_UL] + adv, c[P_UL] + adv, idesc, 1u);
                    umma_tf32(t_qm, r[P_ZH] + adv, c[P_UH] + adv, idesc, acc);
                    umma_tf32(t_qm, r[P_UH] + adv, c[P_ZH] + adv, idesc, 1u);
                    umma_tf32(t_qc, r[P_ZH] + adv, c[P_UL] + adv, idesc, acc);
                    umma_tf32(t_qc, r[P_ZL] + adv, c[P_UH] + adv, idesc, 1u);
                    umma_tf32(t_qc, r[P_UH] + adv, c[P_ZL] + adv, idesc, 1u);
                    umma_tf32(t_qc, r[P_UL] + adv, c[P_ZH] + adv, idesc, 1u);
                    umma_tf32(t_qc, r[P_ZL] + adv, c[P_UL] + adv, idesc, 1u);
                    umma_tf32(t_qc, r[P_UL] + adv, c[P_ZL] + adv, idesc, 1u);
                }
                umma_commit(smem_u32(&bar_acc));
            }
        }
    }
    __syncwarp();
    if (!mbar_wait(smem_u32(&bar_acc), 0u, abortp)) failed = true;
    failed = __any_sync(0xffffffffu, failed);
    if (!failed) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // the operand tiles are dead now: each epilogue warp transposes through a corner of them
        float* tb = reinterpret_cast<float*>(tiles_ptr) + (size_t)warp * 32 * 33;
        const int ibase = i0 + q * 32;
#pragma unroll
        for (int mat = 0; mat < 2; ++mat) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {       // this thread = row `lane` of the warp's block
                uint32_t v[16], w[16];
                tmem_ld16(tmem_base + lane_base + (uint32_t)(mat * 128 + cc * 32 + h * 16), v);
                tmem_ld16(tmem_base + lane_base + (uint32_t)(mat * 128 + 64 + cc * 32 + h * 16), w);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 16; ++e)
                    tb[lane * 33 + h * 16 + e] = __uint_as_float(v[e]) + __uint_as_float(w[e]);
            }
            __syncwarp();
            float* Mo = (mat ? Q2 : A2) + (size_t)l * d * d;
            float* prow = Mo + (size_t)ibase * d + j;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const float val = (mat ? cq[e] : ca[e]) - tb[e * 33 + lane];
                tb[e * 33 + lane] = val;
                if (ibase + e < n_new && j < ibase + e) prow[0] = val;
                prow += d;
            }
            __syncwarp();
            // mirror ([j][i]): back in the row-per-lane view, so that lanes run along i
            float* pcol = Mo + (size_t)(j0 + cc * 32) * d + ibase + lane;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                if (ibase + lane < n_new && j0 + cc * 32 + e < ibase + lane) pcol[0] = tb[lane * 33 + e];
                pcol += d;
            }
            __syncwarp();
        }
    }

    if (failed) {
        abort_flag = 1;
        set_layer_status(layer_status, l, ZIPLM_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (abort_flag && threadIdx.x == 0) {
        // give copies that are still in flight a bounded chance to land before the CTA retires
        for (uint32_t it = 0; it < 4096u; ++it)
            if (mbar_try_wait(smem_u32(&bar_full), 0u)) break;
    }
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(AQ_TMEM_COLS)
                     : "memory");
    }
}

}  // namespace

int lazy_tc_rows_pad(int d) { return round_up_int(d, RM); }

size_t lazy_tc_pack_floats(int L, int d) { return (size_t)L * 4 * lazy_tc_rows_pad(d) * PK; }

// Tensor map over the packed operands P[L][4][rows_pad][32]: box = 64 rows of one array.
bool lazy_tc_make_map(CUtensorMap* m, const float* P, int L, int d) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const int rows_pad = lazy_tc_rows_pad(d);
    cuuint64_t dims[4] = {(cuuint64_t)PK, (cuuint64_t)rows_pad, 4, (cuuint64_t)L};
    cuuint64_t strides[3] = {(cuuint64_t)PK * 4, (cuuint64_t)rows_pad * PK * 4,
                             (cuuint64_t)4 * rows_pad * PK * 4};
    cuuint32_t box[4] = {(cuuint32_t)PK, (cuuint32_t)BOX_ROWS, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(P), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

ziplm_status run_lazy_update_aq_tc(const CUtensorMap& map, int L, int n_new, int m, int d,
                                   const float* A, const float* Q, float* A2, float* Q2,
                                   const int* src, const float* U, const float* Z, float* P,
                                   int* layer_status, cudaStream_t st) {
    static const cudaError_t attr = cudaFuncSetAttribute(
        k_lazy_update_aq_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, OPERAND_BYTES + 1024);
    if (attr != cudaSuccess) return ZIPLM_ERR_CUDA;
    const int rows_pad = lazy_tc_rows_pad(d);
    const int rows_used = round_up_int(n_new, RM);
    k_lazy_pack_uz<<<dim3(rows_used / 32, L), 256, 0, st>>>(n_new, m, d, rows_pad, src, U, Z, P);
    ZIPLM_CHECK_LAUNCH();
    const int TI = rows_used / RM;
    k_lazy_update_aq_tc<<<dim3(TI * (TI + 1), L), AQ_THREADS, OPERAND_BYTES + 1024, st>>>(
        map, n_new, d, A, Q, A2, Q2, src, layer_status);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

}  // namespace ziplm
