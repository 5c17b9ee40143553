// Rank-32 update of H^-1, of the Gram matrix Q = W^T W and of W^T itself (delayed Eq. 4 / Eq. 3)
// for the blocks that leave the removed positions in place, on the 5th-generation tensor cores,
// as one persistent kernel:
//
//   A'[i,j] = A[i,j] - sum_s U[s,i] U[s,j]
//   Q'[i,j] = Q[i,j] - sum_s (Z[s,i] U[s,j] + U[s,i] Z[s,j]),       i > j positions of the arrays
//   Wt'[i,c] = Wt[i,c] - sum_s U[s,i] C[s,c],                         c row indices of W
//
// (the tiles of W^T follow the tiles of their row strip: the same packed rows of U, the packed C
// in the place of the column operand, one accumulator, no mirrored store)
// (the pending vectors are zero at removed positions, whose rows and columns are carried along
// unchanged).  Nothing is gathered: tiles are plain rectangles, read by TMA and written densely.
// A pre-pass (k_lazy_pack_uz) transposes the pending vectors to K-major ([position][step]), each
// value split into three bfloat16 parts x = x1 + x2 + x3 (every part the nearest bfloat16 of what
// the earlier ones left, so |x - x1 - x2 - x3| <= 2^-27 |x|).  Products of two bfloat16 values are
// exact in the fp32 accumulator, and the six partial products x_a y_b with a + b <= 4 are kept
// (the others are below 2^-26 of the product), so a product is as good as an fp32 one.
//
// The update kernel runs one CTA per SM.  Work is cut into tiles of 128 x 128 entries on or
// below the diagonal; runs of consecutive tiles of one row strip ("segments") are handed out
// through an atomic counter, so a CTA that starts late (another kernel holds its SM) simply finds
// less left to do.  Inside a CTA three kinds of warps work as a pipeline, linked by mbarriers only:
//   warp 0      fetches segments, publishes one descriptor per tile (layer, tile origin) and
//               loads the tile's packed operands by TMA (the 128 rows once per segment, the 128
//               columns per tile);
//   warp 1      one thread issues the 36 tcgen05.mma (kind::f16, bfloat16, M = N = 128, K = 16)
//               of a tile (12 for a tile of W^T), the smallest partial products first, so that the truncating
//               accumulation meets them while the accumulator is small, into one of two
//               accumulator stages in tensor memory;
//   warps 2-17  each owns 32 rows x 64 columns of one matrix (H^-1 or Q) in every tile, worked
//               on as four slices of 16 columns: one lane brings the old entries of a slice in
//               by TMA (64-byte swizzle) into a ring of three slices of the warp's own (two in
//               flight while one is worked on), the warp reads the accumulator with tcgen05.ld
//               (one row per lane), subtracts, stores the mirrored entries [j][i] straight from
//               registers (lanes run along i: 128-byte pieces) and the entries [i][j] after a
//               pass through its slice (lanes run along j, 128-bit stores).
// No CTA-wide barrier exists between set-up and exit.  Every mbarrier wait is bounded; a wait that
// runs out raises an abort flag that all roles poll, the issuer still commits and waits for the
// MMAs it has issued, every lane that started copies waits for them, and the CTA leaves through
// the normal exit (tensor memory freed) with ZIPLM_ERR_TIMEOUT in the layers' status.
#include <cuda_bf16.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace ziplm {
namespace {
using namespace tc;

constexpr int PK = 32;                       // pending steps per block = K of the products
constexpr int RM = 128, CN = 128;            // tile rows, tile columns (new index space)
constexpr int NARR = 3;                      // packed arrays: [U1|U2], [U3|Z3], [Z1|Z2], 128-byte rows
constexpr int BOX_ROWS = 64;                 // rows per TMA box
constexpr int BOX_BYTES = BOX_ROWS * 128;    // 8 KiB
constexpr int ARR_BYTES = 2 * BOX_BYTES;     // one packed array, 128 positions
constexpr int ROWS_BYTES = NARR * ARR_BYTES; // 48 KiB
constexpr int COLS_BYTES = NARR * ARR_BYTES; // 48 KiB
constexpr int ACC_STAGES = 2;
constexpr int N_EPI = 16;                    // epilogue warps: 4 lane quarters x 2 matrices x 2 column halves
constexpr int SUBS = 4;                      // slices of 16 columns per warp and tile
constexpr int RING = 3;                      // slices per epilogue warp
constexpr int SLICE_FLOATS = 32 * 16;        // 32 rows x 16 columns
constexpr int RING_BYTES = N_EPI * RING * SLICE_FLOATS * 4;   // 96 KiB
constexpr int AQ_SMEM = ROWS_BYTES + COLS_BYTES + RING_BYTES + 1024;
constexpr int AQ_THREADS = 32 * (2 + N_EPI);
constexpr uint32_t AQ_TMEM_COLS = 512;       // two stages of (H^-1: 128 columns, Q: 128 columns)
constexpr int DESC_RING = 4;
constexpr int MAX_STRIPS = 48;               // d <= 6144
enum { TILE_STOP = 1, TILE_NEW_ROWS = 2, TILE_W = 4 };

// Work list of one launch: the row strips from the longest to the shortest; prefix[k] = number
// of segments (over all layers) of the k longest strips.
struct AqSched {
    int n_strips, seg, n_segments, L;
    int n_wt;                 // tiles of 128 columns of W^T that follow the tiles of a row strip
    int rows_pad;             // first row of the packed C in P
    int prefix[MAX_STRIPS + 1];
};

struct __align__(16) TileSlot {
    int l, i0, j0, flags;
};

// The three bfloat16 parts of x, each the nearest bfloat16 of what the earlier ones left.
__device__ __forceinline__ void split_bf16x3(float x, __nv_bfloat16 (&p)[3]) {
    p[0] = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(p[0]);        // exact
    p[1] = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(p[1]);       // exact
    p[2] = __float2bfloat16_rn(r2);
}

// P[l][a][i][64] (bfloat16), a = 0: [U1 | U2], 1: [U3 | Z3], 2: [Z1 | Z2], each half the 32 steps
// of one part: pending vectors by position, zero for steps >= m and for rows n_pos .. the next
// multiple of 128.
__global__ void __launch_bounds__(256) k_lazy_pack_uz(int n_pos, int m, int d, int rows_pad, int rows_tot,
                                                      int pos_blocks, int rp,
                                                      const float* __restrict__ U,
                                                      const float* __restrict__ Z,
                                                      const float* __restrict__ C,
                                                      __nv_bfloat16* __restrict__ P) {
    __shared__ float tu[PK][33], tz[PK][33];
    const int l = blockIdx.y;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const size_t arr = (size_t)rows_tot * 2 * PK;
    __nv_bfloat16* Pl = P + (size_t)l * NARR * arr;
    if ((int)blockIdx.x >= pos_blocks) {
        // rows rows_pad + c: the scaled pivot columns C[s][c] of W (the column operand of the
        // tiles of W^T) in the place of U, zeros in the place of Z
        const int c0 = ((int)blockIdx.x - pos_blocks) * 32;
        const float* Cl = C + (size_t)l * PK * rp;
#pragma unroll
        for (int s = ty; s < PK; s += 8) {
            const int c = c0 + tx;
            tu[s][tx] = (c < rp && s < m) ? Cl[(size_t)s * rp + c] : 0.f;
        }
        __syncthreads();
        const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
#pragma unroll
        for (int rr = ty; rr < 32; rr += 8) {
            const int i = rows_pad + c0 + rr;
            if (i >= rows_tot) continue;
            __nv_bfloat16 u[3];
            split_bf16x3(tu[tx][rr], u);
            const size_t o = (size_t)i * 2 * PK + tx;
            Pl[o] = u[0];            Pl[o + PK] = u[1];
            Pl[arr + o] = u[2];      Pl[arr + o + PK] = zero;
            Pl[2 * arr + o] = zero;  Pl[2 * arr + o + PK] = zero;
        }
        return;
    }
    const int i0 = blockIdx.x * 32;
    const int pos = i0 + tx;
    const int sp = pos < n_pos ? pos : -1;
    const float* Ul = U + (size_t)l * PK * d;
    const float* Zl = Z + (size_t)l * PK * d;
#pragma unroll
    for (int s = ty; s < PK; s += 8) {
        const bool ok = sp >= 0 && s < m;
        tu[s][tx] = ok ? Ul[(size_t)s * d + sp] : 0.f;
        tz[s][tx] = ok ? Zl[(size_t)s * d + sp] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int rr = ty; rr < 32; rr += 8) {
        const int i = i0 + rr;
        if (i >= rows_pad) continue;
        __nv_bfloat16 u[3], z[3];
        split_bf16x3(tu[tx][rr], u);
        split_bf16x3(tz[tx][rr], z);
        const size_t o = (size_t)i * 2 * PK + tx;
        Pl[o] = u[0];            Pl[o + PK] = u[1];
        Pl[arr + o] = u[2];      Pl[arr + o + PK] = z[2];
        Pl[2 * arr + o] = z[0];  Pl[2 * arr + o + PK] = z[1];
    }
}

__global__ void __launch_bounds__(AQ_THREADS, 1)
k_lazy_update_aq_tc(const __grid_constant__ CUtensorMap map, const __grid_constant__ CUtensorMap map_a,
                    const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_w,
                    const __grid_constant__ AqSched sch, int n_pos, int d, int rp,
                    float* __restrict__ A2, float* __restrict__ Q2, float* __restrict__ W2,
                    int* __restrict__ counter, int* __restrict__ layer_status, uint32_t slot_spin_limit) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_tile_full[DESC_RING], bar_tile_empty[DESC_RING];
    __shared__ uint64_t bar_ops_full, bar_acc_full[ACC_STAGES], bar_acc_empty[ACC_STAGES], bar_final;
    __shared__ uint64_t bar_slice[N_EPI][RING];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ TileSlot slots[DESC_RING];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ops = (raw + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
    const uint32_t rows_smem = ops, cols_smem = ops + ROWS_BYTES;
    const uint32_t rings_smem = cols_smem + COLS_BYTES;
    float* rings_ptr = reinterpret_cast<float*>(smem_raw + (rings_smem - raw));

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < DESC_RING; ++i) {
            mbar_init(smem_u32(&bar_tile_full[i]), 1);
            mbar_init(smem_u32(&bar_tile_empty[i]), 1 + N_EPI);
        }
        mbar_init(smem_u32(&bar_ops_full), 1);
        for (int i = 0; i < ACC_STAGES; ++i) {
            mbar_init(smem_u32(&bar_acc_full[i]), 1);
            mbar_init(smem_u32(&bar_acc_empty[i]), N_EPI);
        }
        mbar_init(smem_u32(&bar_final), 1);
        for (int i = 0; i < N_EPI * RING; ++i) mbar_init(smem_u32(&bar_slice[0][0]) + 8u * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(AQ_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    bool failed = false;

    if (warp == 0) {
        // ---------------- scheduler and TMA producer ----------------
        int t = 0;                       // tiles published so far by this CTA
        int issued = 0;                  // tiles whose operand copies were issued
        int s = 0;
        if (lane == 0) s = atomicAdd(counter, 1);
        s = __shfl_sync(0xffffffffu, s, 0);
        while (s < sch.n_segments && !failed) {
            int s_next = 0;
            if (lane == 0) s_next = atomicAdd(counter, 1);      // in flight while this segment is set up
            int k = 0;
            while (k + 1 < sch.n_strips && sch.prefix[k + 1] <= s) ++k;
            const int I = sch.n_strips - 1 - k;
            const int within = s - sch.prefix[k];
            const int segs_strip = (sch.prefix[k + 1] - sch.prefix[k]) / sch.L;
            const int l = within / segs_strip, sidx = within - l * segs_strip;
            const int nJ = I + 1 + sch.n_wt;      // tiles J = 0 .. I (the last one holds the diagonal), then W^T
            const int Jb = sidx * sch.seg, Je = min(Jb + sch.seg, nJ);
            const int i0 = I * RM;
            for (int J = Jb; J < Je; ++J, ++t) {
                const int slot = t & (DESC_RING - 1);
                if (t >= DESC_RING)
                    failed = !__all_sync(0xffffffffu,
                                         mbar_wait_limit(smem_u32(&bar_tile_empty[slot]),
                                                         (uint32_t)(((t >> 2) - 1) & 1), abortp, slot_spin_limit));
                if (failed) break;
                // a tile of W^T takes its column operand from the rows of P that hold C
                const bool wtile = J > I;
                const int j0 = wtile ? sch.rows_pad + (J - I - 1) * CN : J * CN;
                if (lane == 0) {
                    TileSlot& ts = slots[slot];
                    ts.l = l; ts.i0 = i0; ts.j0 = j0;
                    ts.flags = ((J == Jb) ? TILE_NEW_ROWS : 0) | (wtile ? TILE_W : 0);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_tile_full[slot]));
                // the operand tiles are free once the MMAs of the previous tile have completed
                if (t > 0)
                    failed = !__all_sync(0xffffffffu,
                                         mbar_wait(smem_u32(&bar_acc_full[(t - 1) & 1]),
                                                   (uint32_t)(((t - 1) >> 1) & 1), abortp));
                if (failed) break;
                if (lane == 0) {
                    const uint32_t full = smem_u32(&bar_ops_full);
                    mbar_expect_tx(full, (uint32_t)((J == Jb ? ROWS_BYTES : 0) + COLS_BYTES));
#pragma unroll
                    for (int a = 0; a < NARR; ++a)
#pragma unroll
                        for (int b = 0; b < 2; ++b) {
                            if (J == Jb)
                                tma_load_4d(rows_smem + a * ARR_BYTES + b * BOX_BYTES, &map, full, 0,
                                            i0 + b * BOX_ROWS, a, l);
                            tma_load_4d(cols_smem + a * ARR_BYTES + b * BOX_BYTES, &map, full, 0,
                                        j0 + b * BOX_ROWS, a, l);
                        }
                }
                issued = t + 1;
            }
            s = __shfl_sync(0xffffffffu, s_next, 0);
        }
        if (!failed) {                   // stop descriptor
            const int slot = t & (DESC_RING - 1);
            if (t >= DESC_RING)
                failed = !__all_sync(0xffffffffu,
                                     mbar_wait_limit(smem_u32(&bar_tile_empty[slot]),
                                                     (uint32_t)(((t >> 2) - 1) & 1), abortp, slot_spin_limit));
            if (!failed && lane == 0) {
                slots[slot].flags = TILE_STOP;
                mbar_arrive(smem_u32(&bar_tile_full[slot]));
            }
        }
        if (failed) {
            abort_flag = 1;
            // copies already issued land in this CTA's shared memory: give them a bounded chance
            if (lane == 0 && issued > 0) mbar_wait_quiet(smem_u32(&bar_ops_full), (uint32_t)((issued - 1) & 1));
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (one thread) ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(1u, RM, CN);     // bfloat16 operands, fp32 accumulate
            // descriptor of part p of the rows (r) and of the columns (c): U1 U2 U3 Z1 Z2 Z3
            const uint32_t part_off[6] = {0u, 64u, (uint32_t)ARR_BYTES, 2u * ARR_BYTES, 2u * ARR_BYTES + 64u,
                                          (uint32_t)ARR_BYTES + 64u};
            uint64_t r[6], c[6];
#pragma unroll
            for (int p = 0; p < 6; ++p) {
                r[p] = make_desc(rows_smem + (part_off[p] & ~127u)) + (uint64_t)((part_off[p] & 127u) >> 4);
                c[p] = make_desc(cols_smem + (part_off[p] & ~127u)) + (uint64_t)((part_off[p] & 127u) >> 4);
            }
            enum { U1 = 0, U2 = 1, U3 = 2, Z1 = 3, Z2 = 4, Z3 = 5 };
            for (int t = 0;; ++t) {
                const int slot = t & (DESC_RING - 1);
                if (!mbar_wait(smem_u32(&bar_tile_full[slot]), (uint32_t)((t >> 2) & 1), abortp)) { failed = true; break; }
                const int flags = *reinterpret_cast<volatile int*>(&slots[slot].flags);
                mbar_arrive(smem_u32(&bar_tile_empty[slot]));
                if (flags & TILE_STOP) break;
                const int st = t & 1;
                if (!mbar_wait(smem_u32(&bar_ops_full), (uint32_t)(t & 1), abortp)) { failed = true; break; }
                if (t >= ACC_STAGES &&
                    !mbar_wait(smem_u32(&bar_acc_empty[st]), (uint32_t)(((t >> 1) - 1) & 1), abortp)) {
                    failed = true;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t t_a = tmem_base + (uint32_t)(st * 2 * CN), t_q = t_a + (uint32_t)CN;
                // one partial product x_a y_b over the 32 steps: two MMAs of K = 16 (32 bytes each)
                auto prod = [&](uint32_t acc, int pr, int pc2, bool first) {
                    umma_bf16(acc, r[pr], c[pc2], idesc, first ? 0u : 1u);
                    umma_bf16(acc, r[pr] + 2u, c[pc2] + 2u, idesc, 1u);
                };
                // H^-1: U U^T; smallest terms first
                prod(t_a, U1, U3, true);  prod(t_a, U3, U1, false); prod(t_a, U2, U2, false);
                prod(t_a, U1, U2, false); prod(t_a, U2, U1, false); prod(t_a, U1, U1, false);
                // Q: Z U^T + U Z^T (a tile of W^T has no second matrix: its column operand is C
                // in the place of U, and the products above are the whole update U^T C)
                if (!(flags & TILE_W)) {
                    prod(t_q, Z1, U3, true);  prod(t_q, Z3, U1, false); prod(t_q, Z2, U2, false);
                    prod(t_q, U1, Z3, false); prod(t_q, U3, Z1, false); prod(t_q, U2, Z2, false);
                    prod(t_q, Z1, U2, false); prod(t_q, Z2, U1, false); prod(t_q, U1, Z2, false);
                    prod(t_q, U2, Z1, false); prod(t_q, Z1, U1, false); prod(t_q, U1, Z1, false);
                }
                umma_commit(smem_u32(&bar_acc_full[st]));
            }
            if (failed) abort_flag = 1;
            // whatever was issued has completed before tensor memory is given back
            umma_commit(smem_u32(&bar_final));
            mbar_wait_quiet(smem_u32(&bar_final), 0u);
        }
        __syncwarp();
    } else {
        // ---------------- epilogue warps ----------------
        // warp -> TMEM lane quarter q (rows 32 q ..), matrix, column half h (columns 64 h ..)
        const int ew = warp - 2, q = warp & 3, mat = ew >> 3, h = (ew >> 2) & 1;
        const CUtensorMap* min_map = mat ? &map_q : &map_a;
        float* Mout = mat ? Q2 : A2;
        float* ring = rings_ptr + (size_t)ew * RING * SLICE_FLOATS;
        const uint32_t ring_u32 = rings_smem + (uint32_t)(ew * RING * SLICE_FLOATS * 4);
        const uint32_t bar0 = smem_u32(&bar_slice[ew][0]);
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(mat * CN + 64 * h);
        const size_t dd = (size_t)d * d;
        // A slice is [32 rows][16 columns] as TMA writes it with the 64-byte swizzle: 64-byte rows,
        // the 16-byte unit index of row r XORed with (r >> 1) & 3: a lane per row and four lanes
        // per row both reach it without bank conflicts.

        // Copy cursor: tile pt (descriptor in its ring slot), next slice psub.  One call starts
        // the copy of one slice (lane 0: expect_tx + TMA; the slice's earlier readers and writers,
        // this warp, are done and have fenced their accesses against the asynchronous proxy);
        // after the last slice of a tile the slot is given back and the next descriptor awaited.
        int pt = 0, psub = 0, pflags = TILE_STOP;
        int nl = 0, ni0 = 0, nj0 = 0;                        // tile pt
        int issued = 0;                                      // slices whose copies were started
        auto open_tile = [&]() -> bool {
            const int slot = pt & (DESC_RING - 1);
            const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_tile_full[slot]),
                                                              (uint32_t)((pt >> 2) & 1), abortp));
            if (!ok) { pflags = TILE_STOP; return false; }
            const TileSlot& ts = slots[slot];
            nl = ts.l; ni0 = ts.i0; nj0 = ts.j0;
            pflags = *reinterpret_cast<volatile const int*>(&ts.flags);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_tile_empty[slot]));      // the descriptor is in registers
            return true;
        };
        auto copy_next = [&]() -> bool {
            bool ok = true;
            if (!(pflags & TILE_STOP)) {
                const int c = SUBS * pt + psub;
                if (lane == 0) {
                    const uint32_t bar = bar0 + 8u * (uint32_t)(c % RING);
                    mbar_expect_tx(bar, (uint32_t)(SLICE_FLOATS * 4));
                    // a tile of W^T: both matrices' warps bring the same slices in (the second
                    // copy is served by L2) and work on two of the four each
                    if (pflags & TILE_W)
                        tma_load_3d(ring_u32 + (uint32_t)((c % RING) * SLICE_FLOATS * 4), &map_w, bar,
                                    nj0 - sch.rows_pad + 64 * h + 16 * psub, ni0 + 32 * q, nl);
                    else
                        tma_load_3d(ring_u32 + (uint32_t)((c % RING) * SLICE_FLOATS * 4), min_map, bar,
                                    nj0 + 64 * h + 16 * psub, ni0 + 32 * q, nl);
                }
                issued = c + 1;
                if (++psub == SUBS) {
                    psub = 0;
                    ++pt;
                    ok = open_tile();
                }
            }
            return ok;
        };

        failed = !open_tile();
        int cl = nl, ci0 = ni0, cj0 = nj0, cflags = pflags;   // tile being worked on
        copy_next();
        copy_next();
        for (int t = 0; !(cflags & TILE_STOP) && !failed; ++t) {
            const int stage = t & 1;
#pragma unroll 1
            for (int sub = 0; sub < SUBS; ++sub) {
                const int c = SUBS * t + sub;
                // ---- start the copy of the slice two ahead, then wait for slice c
                if (!copy_next()) { failed = true; break; }
                if (!mbar_wait(bar0 + 8u * (uint32_t)(c % RING), (uint32_t)((c / RING) & 1), abortp)) failed = true;
                if (sub == 0 && !failed &&
                    !mbar_wait(smem_u32(&bar_acc_full[stage]), (uint32_t)((t >> 1) & 1), abortp))
                    failed = true;
                failed = __any_sync(0xffffffffu, failed);
                if (failed) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                uint32_t v[16];
                // (a tile of W^T has one accumulator, which both matrices' warps read)
                tmem_ld16(lane_taddr - ((cflags & TILE_W) ? (uint32_t)(mat * CN) : 0u) +
                              (uint32_t)(stage * 2 * CN + 16 * sub), v);
                tmem_ld_wait();
                if (sub == SUBS - 1) {
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[stage]));
                }
                float* buf = ring + (size_t)(c % RING) * SLICE_FLOATS;
                if (cflags & TILE_W) {
                    // ---- tile of W^T: rows = positions, columns = row indices of W; no mirror.
                    //      The two warps that share a quarter of the rows and a half of the columns
                    //      take two of its four slices each.
                    if ((sub >> 1) == mat) {
                        float4* b4 = reinterpret_cast<float4*>(buf) + lane * 4;
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const int pg = g ^ ((lane >> 1) & 3);
                            const float4 o = b4[pg];
                            b4[pg] = make_float4(o.x - __uint_as_float(v[4 * g]), o.y - __uint_as_float(v[4 * g + 1]),
                                                 o.z - __uint_as_float(v[4 * g + 2]), o.w - __uint_as_float(v[4 * g + 3]));
                        }
                        __syncwarp();
                        float* Wo = W2 + (size_t)cl * d * rp;
                        const int jc = cj0 - sch.rows_pad + 64 * h + 16 * sub, ib = ci0 + 32 * q;
#pragma unroll
                        for (int it = 0; it < 4; ++it) {
                            const int row = 8 * it + (lane >> 2), u = lane & 3;
                            const float4 x = reinterpret_cast<const float4*>(buf)[row * 4 + (u ^ ((row >> 1) & 3))];
                            const int gi = ib + row, gj = jc + 4 * u;
                            if (gi < n_pos && gj < rp) *reinterpret_cast<float4*>(Wo + (size_t)gi * rp + gj) = x;
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (sub == SUBS - 1) { cl = nl; ci0 = ni0; cj0 = nj0; cflags = pflags; }
                    continue;
                }
                // ---- new entries: old - update, one matrix row per lane
                float4* b4 = reinterpret_cast<float4*>(buf) + lane * 4;
                float rr[16];
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int pg = g ^ ((lane >> 1) & 3);
                    const float4 o = b4[pg];
                    rr[4 * g] = o.x - __uint_as_float(v[4 * g]);
                    rr[4 * g + 1] = o.y - __uint_as_float(v[4 * g + 1]);
                    rr[4 * g + 2] = o.z - __uint_as_float(v[4 * g + 2]);
                    rr[4 * g + 3] = o.w - __uint_as_float(v[4 * g + 3]);
                    b4[pg] = make_float4(rr[4 * g], rr[4 * g + 1], rr[4 * g + 2], rr[4 * g + 3]);
                }
                float* Mo = Mout + (size_t)cl * dd;
                const int jc = cj0 + 64 * h + 16 * sub;  // first column of the slice
                const int ib = ci0 + 32 * q;             // first row of the slice
                // ---- mirror [j][i]: lanes run along i
                {
                    const int i = ib + lane;
                    const int jlim = (i < n_pos) ? i - jc : 0;     // entries e < jlim lie below the diagonal
                    float* mp = Mo + (size_t)jc * d + i;
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        if (e < jlim) *mp = rr[e];
                        mp += d;
                    }
                }
                __syncwarp();
                // ---- [i][j]: eight rows per instruction, four lanes along a row
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const int row = 8 * it + (lane >> 2), u = lane & 3;
                    const float4 x = reinterpret_cast<const float4*>(buf)[row * 4 + (u ^ ((row >> 1) & 3))];
                    const int gi = ib + row, gj = jc + 4 * u;
                    if (gi < n_pos) {
                        float* p = Mo + (size_t)gi * d + gj;
                        if (gj + 3 < gi) {
                            *reinterpret_cast<float4*>(p) = x;
                        } else {
                            if (gj < gi) p[0] = x.x;
                            if (gj + 1 < gi) p[1] = x.y;
                            if (gj + 2 < gi) p[2] = x.z;
                        }
                    }
                }
                // the slice may be refilled by a copy: fence this lane's accesses, then the warp
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                // the copy cursor has moved on to the next tile by now: take its origin over
                // before the cursor can replace it (it opens tile t + 2 during slice 1 of tile t + 1)
                if (sub == SUBS - 1) { cl = nl; ci0 = ni0; cj0 = nj0; cflags = pflags; }
            }
        }
        // every copy this warp started has landed before the CTA leaves (the last RING slices
        // started are the latest phases of their barriers)
        if (lane == 0)
            for (int c = max(issued - RING, 0); c < issued; ++c)
                mbar_wait_quiet(bar0 + 8u * (uint32_t)(c % RING), (uint32_t)((c / RING) & 1));
        __syncwarp();
        if (failed) abort_flag = 1;
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (abort_flag)
        for (int l = threadIdx.x; l < sch.L; l += AQ_THREADS) set_layer_status(layer_status, l, ZIPLM_ERR_TIMEOUT);
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(AQ_TMEM_COLS)
                     : "memory");
    }
    // the last CTA to leave puts the work counter back to zero for the next launch
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(counter + 1, 1) == (int)gridDim.x - 1) {
            counter[0] = 0;
            counter[1] = 0;
            __threadfence();
        }
    }
}

int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace

int lazy_tc_rows_pad(int d) { return round_up_int(d, RM); }
// rows of P: the positions, then the row indices of W (the packed C), both padded to whole tiles
static int lazy_tc_rows_tot(int d, int rp) { return lazy_tc_rows_pad(d) + round_up_int(rp, CN); }

// size of the packed operands in floats (NARR arrays of 2 * PK bfloat16 per row of P)
size_t lazy_tc_pack_floats(int L, int d, int rp) { return (size_t)L * NARR * lazy_tc_rows_tot(d, rp) * PK; }

// Tensor map over the packed operands P[L][3][rows_tot][64] (bfloat16): box = 64 rows of one array.
bool lazy_tc_make_map(CUtensorMap* m, const float* P, int L, int d, int rp) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const int rows_pad = lazy_tc_rows_tot(d, rp);
    cuuint64_t dims[4] = {(cuuint64_t)2 * PK, (cuuint64_t)rows_pad, NARR, (cuuint64_t)L};
    cuuint64_t strides[3] = {(cuuint64_t)128, (cuuint64_t)rows_pad * 128,
                             (cuuint64_t)NARR * rows_pad * 128};
    cuuint32_t box[4] = {(cuuint32_t)2 * PK, (cuuint32_t)BOX_ROWS, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<float*>(P), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map over one of the fp32 matrices M[L][d][cols] (cols a multiple of 4; d for H^-1 and Q,
// the padded row count of W for W^T): box = 32 rows x 16 columns, 64-byte swizzle; what lies
// outside the matrix reads as zero.
bool lazy_tc_make_matrix_map(CUtensorMap* m, const float* M, int L, int d, int cols) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)d, (cuuint64_t)L};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 4, (cuuint64_t)d * cols * 4};
    cuuint32_t box[3] = {16, 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(M), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// One block of pending steps applied to H^-1 and Q with every position left in place: map_a /
// map_q cover the matrices as they stand (n_pos positions), A2 / Q2 receive the result.
// `counter` points at two ints (work counter, CTAs that have left) that are zero before the first
// launch; every launch leaves them zero again.  slot_spin_limit = 0 selects the default poll
// limit of the producer's wait for a free descriptor slot.
ziplm_status run_lazy_update_aq_tc(const CUtensorMap& map, const CUtensorMap& map_a,
                                   const CUtensorMap& map_q, const CUtensorMap& map_w, int L, int n_pos,
                                   int m, int d, int rp, float* A2, float* Q2, float* W2, const float* U,
                                   const float* Z, const float* C, float* P, int* counter,
                                   int* layer_status, unsigned slot_spin_limit, cudaStream_t st) {
    ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_lazy_update_aq_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          AQ_SMEM));
    const int sms = sm_count();
    if (sms <= 0) return ZIPLM_ERR_CUDA;
    const int rows_pad = lazy_tc_rows_pad(d), rows_tot = lazy_tc_rows_tot(d, rp);
    const int rows_used = round_up_int(n_pos, RM);
    if (rows_used / RM > MAX_STRIPS) return ZIPLM_ERR_UNSUPPORTED;
    const int pos_blocks = rows_used / 32, c_blocks = (rows_tot - rows_pad) / 32;
    k_lazy_pack_uz<<<dim3(pos_blocks + c_blocks, L), 256, 0, st>>>(n_pos, m, d, rows_pad, rows_tot, pos_blocks,
                                                                  rp, U, Z, C, reinterpret_cast<__nv_bfloat16*>(P));
    ZIPLM_CHECK_LAUNCH();
    // The kernel is bound by memory bandwidth, which two thirds of the SMs saturate (measured: the
    // same time with 96 as with 148 CTAs, 12 % more with 74); the others are left to the kernels
    // of other layer groups and batches that run beside it.
    const int ctas = (2 * sms + 2) / 3;
    AqSched sch;
    sch.n_strips = rows_used / RM;
    sch.L = L;
    sch.n_wt = (rp + CN - 1) / CN;
    sch.rows_pad = rows_pad;
    const long long tiles = (long long)L * sch.n_strips * ((sch.n_strips + 1) / 2 + sch.n_wt);   // about
    // about six segments per CTA, so that the last ones to finish differ by a fraction of the run
    long long seg = tiles / ((long long)ctas * 6);
    sch.seg = (int)(seg < 1 ? 1 : (seg > 8 ? 8 : seg));
    sch.prefix[0] = 0;
    for (int k = 0; k < sch.n_strips; ++k) {
        const int nJ = sch.n_strips - k + sch.n_wt;   // strip I = n_strips - 1 - k: I + 1 tiles, then W^T
        sch.prefix[k + 1] = sch.prefix[k] + L * ((nJ + sch.seg - 1) / sch.seg);
    }
    for (int k = sch.n_strips + 1; k <= MAX_STRIPS; ++k) sch.prefix[k] = sch.prefix[sch.n_strips];
    sch.n_segments = sch.prefix[sch.n_strips];
    const int grid = sch.n_segments < ctas ? sch.n_segments : ctas;
    k_lazy_update_aq_tc<<<grid, AQ_THREADS, AQ_SMEM, st>>>(map, map_a, map_q, map_w, sch, n_pos, d, rp, A2, Q2,
                                                          W2, counter, layer_status,
                                                          slot_spin_limit ? slot_spin_limit : kSpinLimit);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

}  // namespace ziplm
