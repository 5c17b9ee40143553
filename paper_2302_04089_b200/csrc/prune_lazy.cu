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
// Launches per block, for all L layers at once: one "steps" kernel (one thread-block cluster per
// layer runs the B greedy steps back to back with one cluster barrier per step -- layers are
// independent, so no grid-wide synchronisation is needed) and two update kernels.  Block boundaries are placed on
// the requested levels, where W is up to date and can be snapshotted.
//
// Layout per layer: A, Q fp32 [d, d], off-diagonal entries in both triangles (two buffers each, ping-pong),
// Wt = W^T fp32 [d, rp] (two buffers), float64 diagonals, pending U, Z [B, d] and C [B, rp].
#include <cooperative_groups.h>
#include <math.h>


#include <cuda.h>

#include "common.cuh"

namespace ziplm {

// Tensor-core rank-32 update of H^-1, Q and W^T for blocks that leave every position in place
// (prune_lazy_tc.cu).
size_t lazy_tc_pack_floats(int L, int d, int rp);
bool lazy_tc_make_map(CUtensorMap* m, const float* P, int L, int d, int rp);
bool lazy_tc_make_matrix_map(CUtensorMap* m, const float* M, int L, int d, int cols);
ziplm_status run_lazy_update_aq_tc(const CUtensorMap& map, const CUtensorMap& map_a,
                                   const CUtensorMap& map_q, const CUtensorMap& map_w, int L, int n_pos,
                                   int m, int d, int rp, float* A2, float* Q2, float* W2, const float* U,
                                   const float* Z, const float* C, float* P, int* counter,
                                   int* layer_status, unsigned slot_spin_limit, cudaStream_t st);

namespace {

constexpr int BMAX = 32;         // pending steps per block
constexpr int STEP_THREADS = 256; // threads per CTA of the steps kernel, four positions each
constexpr int SLICE_MAX = 768;   // positions per CTA: 2 * BMAX * SLICE_MAX * 4 B = 192 KiB of smem
constexpr int CLUSTER_MAX = 8;   // portable cluster size
constexpr int kDeadMax = 128;    // removed positions tolerated in the arrays before they are squeezed out
constexpr int kDeadFraction = 16; // ... or this fraction of all positions, whichever comes first

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

// Candidate of the argmin of rho = q / a (q = Q[k,k], a = H^-1[k,k]).  Candidates are compared by
// cross-multiplication (q_x a_y < q_y a_x), which needs no float64 division on the critical path;
// the quotient is formed once, for the winner.  An entry whose a is not positive or whose values
// are not finite sorts first, so that it is picked -- and its layer flagged -- at once.
struct Cand {
    double a, q;
    int org, pos;
};

__device__ __forceinline__ bool cand_valid(const Cand& x) {
    return x.a > 0.0 && isfinite(x.a) && isfinite(x.q);
}

__device__ __forceinline__ bool better(const Cand& x, const Cand& y) {   // x strictly before y
    const bool vx = cand_valid(x), vy = cand_valid(y);
    if (vx != vy) return !vx;
    if (!vx) return x.org < y.org;
    const double lhs = x.q * y.a, rhs = y.q * x.a;
    return lhs < rhs || (lhs == rhs && x.org < y.org);
}

__device__ __forceinline__ void merge_cand(Cand& best, const Cand& o) {
    if (o.pos >= 0 && (best.pos < 0 || better(o, best))) best = o;
}

__device__ __forceinline__ Cand bcast_cand(const Cand& c, int src_lane) {
    Cand o;
    o.a = __shfl_sync(0xffffffffu, c.a, src_lane);
    o.q = __shfl_sync(0xffffffffu, c.q, src_lane);
    o.org = __shfl_sync(0xffffffffu, c.org, src_lane);
    o.pos = __shfl_sync(0xffffffffu, c.pos, src_lane);
    return o;
}

// fp32 quotient that orders candidates coarsely: +inf for "none", -inf for an invalid entry.
__device__ __forceinline__ float cand_quotient(const Cand& c) {
    if (c.pos < 0) return INFINITY;
    return cand_valid(c) ? __fdividef((float)c.q, (float)c.a) : -INFINITY;
}

// Best candidate of a warp (every lane returns it).  The cheap fp32 quotient r orders the lanes;
// only the lanes within 1e-5 of the fp32 minimum (almost always a single one) go through the exact
// float64 comparison, so the common case costs one reduction and six 32-bit shuffles instead of
// five rounds of 64-bit exchanges.
__device__ __forceinline__ Cand warp_best(const Cand& mine, float r, float* warp_min = nullptr) {
    // warp minimum in one reduction instruction, on keys that order like the floats they encode
    const unsigned bits = __float_as_uint(r);
    const unsigned key = bits ^ ((bits >> 31) ? 0xffffffffu : 0x80000000u);
    const unsigned kmin = __reduce_min_sync(0xffffffffu, key);
    const float rmin = __uint_as_float(kmin ^ ((kmin >> 31) ? 0x80000000u : 0xffffffffu));
    if (warp_min) *warp_min = rmin;
    const bool near_min = mine.pos >= 0 && (r == rmin || r <= rmin + fabsf(rmin) * 1e-5f);
    unsigned mask = __ballot_sync(0xffffffffu, near_min);
    Cand best;
    best.a = 1.0; best.q = 0.0; best.org = 0x7fffffff; best.pos = -1;
    while (mask) {
        const int b = __ffs(mask) - 1;
        mask &= mask - 1;
        merge_cand(best, bcast_cand(mine, b));
    }
    return best;
}

__device__ __forceinline__ Cand warp_best(const Cand& mine) { return warp_best(mine, cand_quotient(mine)); }

// nsteps greedy steps of one layer, run by a thread-block cluster of CS CTAs (CS = 1, 2, 4 or 8,
// chosen so that a CTA's slice of positions fits its shared memory).  CTA `rank` owns the
// positions [rank * S, rank * S + S); each of its 256 threads owns four consecutive ones and
// keeps their float64 diagonal entries of H^-1 and Q in registers for the whole block.  The
// pending vectors u_s, z_s of the block live in shared memory, sliced the same way, so the
// correction of a pivot column touches no global memory; copies go to global memory only for
// the update kernels that follow.  Per step there is one cluster barrier: every warp publishes
// its best candidate, after the barrier warp 0 of every CTA reads all of them through
// distributed shared memory and reaches the same pick, then fetches the pending vectors'
// entries at the pivot from the CTA that owns it.
// The scaled pivot columns of W (c_s) do not feed the selection; they are solved for at the end
// of the block by forward substitution with the 32 x 32 triangle T[m][s] = u_s[p_m].
// Finally the per-position vectors are compacted (stable) across the cluster.
__global__ void __launch_bounds__(STEP_THREADS, 1)
k_lazy_steps(int n0, int S, int t0, int nsteps, int compact, int d, int G, int r, int rp,
             const float* __restrict__ A, const float* __restrict__ Q, const float* __restrict__ Wt,
             const double* __restrict__ dA_in, const double* __restrict__ dQ_in,
             const int* __restrict__ idx_in, double* __restrict__ dA_out,
             double* __restrict__ dQ_out, int* __restrict__ idx_out, int* __restrict__ src,
             float* __restrict__ U, float* __restrict__ Z, float* __restrict__ C,
             LazyState* __restrict__ state, int* __restrict__ order, float* __restrict__ saliency,
             int* layer_status) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int l = blockIdx.x / CS;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = STEP_THREADS / 32;

    extern __shared__ float4 dyn_smem4[];
    float* sU = reinterpret_cast<float*>(dyn_smem4);       // [BMAX][S]
    float* sZ = sU + (size_t)BMAX * S;                     // [BMAX][S]
    __shared__ Cand s_cand[2][CLUSTER_MAX * NW];           // all warps of the cluster, by step parity
    __shared__ float s_key[2][CLUSTER_MAX * NW];           // ... and their smallest fp32 quotients
    __shared__ float sT[BMAX][BMAX];                       // T[m][s] = u_s[p_m]
    __shared__ double sTd[BMAX][BMAX];                     // ... in float64, for the solve of c_m
    __shared__ float sUp[BMAX], sZp[BMAX];
    __shared__ int s_pm[BMAX];
    __shared__ double s_rsm[BMAX];
    __shared__ int s_p, s_count, s_wsum[NW];
    __shared__ double s_rs, s_half;

    const float* Al = A + (size_t)l * d * d;
    const float* Ql = Q + (size_t)l * d * d;
    const float* Wl = Wt + (size_t)l * d * rp;
    float* Ul = U + (size_t)l * BMAX * d;
    float* Zl = Z + (size_t)l * BMAX * d;
    float* Cl = C + (size_t)l * BMAX * rp;

    const int kloc = 4 * tid;                  // first owned position within the slice
    const int k0 = rank * S + kloc;            // ... and globally
    const bool owner_thread = (kloc < S) && (k0 < n0);
    double da[4], dq[4];
    int org[4];
    bool alive[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int k = k0 + e;
        // a position removed in an earlier block that has not been squeezed out yet carries
        // index -1: it stays dead
        const int o = (owner_thread && k < n0) ? idx_in[(size_t)l * d + k] : -1;
        alive[e] = o >= 0;
        da[e] = alive[e] ? dA_in[(size_t)l * d + k] : 1.0;
        dq[e] = alive[e] ? dQ_in[(size_t)l * d + k] : 0.0;
        org[e] = alive[e] ? o : 0x7fffffff;
    }
    double sumrho = 0.0;                       // meaningful in thread 0 of rank 0

    for (int m = 0; m < nsteps; ++m) {
        const int par = m & 1;
        // ---- per-warp best of rho = Q[k,k] / H^-1[k,k] (ties: lowest original index).  The four
        //      owned positions are ordered by an fp32 quotient; only those within 1e-5 of the
        //      smallest (almost always one) go through the exact float64 comparison.
        Cand best;
        best.a = 1.0; best.q = 0.0; best.org = 0x7fffffff; best.pos = -1;
        float rq[4], rbest = INFINITY;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            rq[e] = INFINITY;
            if (alive[e]) {
                const bool ok = da[e] > 0.0 && isfinite(da[e]) && isfinite(dq[e]);
                rq[e] = ok ? __fdividef((float)dq[e], (float)da[e]) : -INFINITY;
            }
            rbest = fminf(rbest, rq[e]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (!alive[e] || !(rq[e] == rbest || rq[e] <= rbest + fabsf(rbest) * 1e-5f)) continue;
            Cand c;
            c.a = da[e]; c.q = dq[e]; c.org = org[e]; c.pos = k0 + e;
            merge_cand(best, c);
        }
        float wmin;
        best = warp_best(best, best.pos >= 0 ? rbest : INFINITY, &wmin);
        // push: lane c < CS hands the warp's candidate to CTA c, so that after the barrier every
        // CTA finds all candidates in its own shared memory -- together with the warp's smallest
        // fp32 quotient (within 1e-5 of the candidate's own), the key of the coarse ordering below
        if (lane < CS) {
            *cluster.map_shared_rank(&s_cand[par][rank * NW + warp], lane) = best;
            *cluster.map_shared_rank(&s_key[par][rank * NW + warp], lane) = wmin;
        }
        cluster.sync();
        // ---- warp 0 of every CTA: global pick from all warps of all CTAs, then the pending
        //      vectors' entries at the pivot (from the CTA that owns it)
        if (warp == 0) {
            // Coarse ordering by the pushed keys: when exactly one of them lies within 4e-5 of the
            // smallest (the keys are good to 1e-5), its candidate is the pick and is read directly;
            // otherwise -- near ties, an invalid entry, nothing left -- all candidates go through
            // the exact comparison.
            Cand g;
            {
                const float k0v = (lane < CS * NW) ? s_key[par][lane] : INFINITY;
                const float k1v = (lane + 32 < CS * NW) ? s_key[par][lane + 32] : INFINITY;
                const float kl = fminf(k0v, k1v);
                const unsigned bits = __float_as_uint(kl);
                const unsigned key = bits ^ ((bits >> 31) ? 0xffffffffu : 0x80000000u);
                const unsigned kmin = __reduce_min_sync(0xffffffffu, key);
                const float rmin = __uint_as_float(kmin ^ ((kmin >> 31) ? 0x80000000u : 0xffffffffu));
                const float thr = rmin + fabsf(rmin) * 4e-5f;
                const unsigned n0 = __ballot_sync(0xffffffffu, k0v <= thr);
                const unsigned n1 = __ballot_sync(0xffffffffu, k1v <= thr);
                if (fabsf(rmin) < INFINITY && __popc(n0) + __popc(n1) == 1) {
                    g = s_cand[par][n0 ? __ffs(n0) - 1 : 32 + __ffs(n1) - 1];
                } else {
                    g.a = 1.0; g.q = 0.0; g.org = 0x7fffffff; g.pos = -1;
                    for (int e = lane; e < CS * NW; e += 32) merge_cand(g, s_cand[par][e]);
                    g = warp_best(g);
                }
            }
            int p = g.pos;
            if (p < 0) p = 0;
            double h = g.a;
            int bad = 0;
            if (!isfinite(g.q) || !isfinite(h)) { bad = ZIPLM_ERR_NONFINITE; h = 1.0; }
            else if (!(h > 0.0)) { bad = ZIPLM_ERR_NOT_PD; h = 1.0; }
            const double rs = rsqrt(h);
            const int prow = p / S, pl = p - prow * S;
            float up = 0.f, zp = 0.f;
            if (lane < m) {
                up = *cluster.map_shared_rank(sU + (size_t)lane * S + pl, prow);
                zp = *cluster.map_shared_rank(sZ + (size_t)lane * S + pl, prow);
            }
            sUp[lane] = up;
            sZp[lane] = zp;
            sT[m][lane] = up;
            if (lane == 0) {
                s_p = p;
                s_rs = rs;
                s_half = 0.5 * g.q * rs * rs;
                s_pm[m] = p;
                s_rsm[m] = rs;
                if (rank == 0) {
                    const double rho = bad ? 0.0 : g.q * rs * rs;
                    if (bad) set_layer_status(layer_status, l, bad);
                    sumrho += rho;
                    order[(size_t)l * G + t0 + m] = g.org;
                    if (saliency) saliency[(size_t)l * G + t0 + m] = (float)rho;
                }
            }
        }
        __syncthreads();
        const int p = s_p;
        const double rs = s_rs, half = s_half;
        // ---- true pivot columns of H^-1 and Q on the owned positions; float64 diagonal downdate
        if (owner_thread) {
            // both triangles of H^-1 and Q are kept, so the pivot column is the contiguous row p
            const float4 a4 = *reinterpret_cast<const float4*>(Al + (size_t)p * d + k0);
            const float4 q4 = *reinterpret_cast<const float4*>(Ql + (size_t)p * d + k0);
            float a[4] = {a4.x, a4.y, a4.z, a4.w}, q[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (!alive[e] || k0 + e == p) { a[e] = 0.f; q[e] = 0.f; }
            // pending terms at the pivot, summed while the gathered entries are still in flight
            float ca[4] = {0.f, 0.f, 0.f, 0.f}, cq[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
            for (int s = 0; s < m; ++s) {
                const float4 u4 = *reinterpret_cast<const float4*>(sU + (size_t)s * S + kloc);
                const float4 z4 = *reinterpret_cast<const float4*>(sZ + (size_t)s * S + kloc);
                const float up = sUp[s], zp = sZp[s];
                const float uu[4] = {u4.x, u4.y, u4.z, u4.w}, zz[4] = {z4.x, z4.y, z4.z, z4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    ca[e] = fmaf(uu[e], up, ca[e]);
                    cq[e] = fmaf(zz[e], up, cq[e]);
                    cq[e] = fmaf(uu[e], zp, cq[e]);
                }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) { a[e] -= ca[e]; q[e] -= cq[e]; }
            float u32[4], z32[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int k = k0 + e;
                u32[e] = 0.f; z32[e] = 0.f;
                if (alive[e] && k != p) {
                    const double u = (double)a[e] * rs;
                    const double z = (double)q[e] * rs - half * u;
                    da[e] -= u * u;
                    dq[e] -= 2.0 * z * u;
                    u32[e] = (float)u;
                    z32[e] = (float)z;
                }
                if (k == p) alive[e] = false;
            }
            const float4 uo = make_float4(u32[0], u32[1], u32[2], u32[3]);
            const float4 zo = make_float4(z32[0], z32[1], z32[2], z32[3]);
            *reinterpret_cast<float4*>(sU + (size_t)m * S + kloc) = uo;
            *reinterpret_cast<float4*>(sZ + (size_t)m * S + kloc) = zo;
            *reinterpret_cast<float4*>(Ul + (size_t)m * d + k0) = uo;
            *reinterpret_cast<float4*>(Zl + (size_t)m * d + k0) = zo;
        }
        // no barrier here: the next step's cluster barrier orders these writes before any read
    }
    cluster.sync();

    // ---- c_m = (W[:,p_m] - sum_{s<m} c_s T[m][s]) / sqrt(h_m): forward substitution per row
    //      index i of W, each CTA takes a slice of the d_row indices.  The triangle is widened to
    //      float64 once, so that the inner loop is loads and FMAs only.  The solve reads this
    //      CTA's own shared memory only and runs last, when the per-position state is dead.
    auto solve_c = [&]() {
        for (int e = tid; e < BMAX * BMAX; e += STEP_THREADS)
            sTd[e / BMAX][e % BMAX] = (double)sT[e / BMAX][e % BMAX];
        __syncthreads();
        const int per = (rp + CS - 1) / CS;
        for (int i = rank * per + tid; i < min(rp, (rank + 1) * per); i += STEP_THREADS) {
            float w[BMAX];
            double c[BMAX];          // the fp32 values that are stored, widened
#pragma unroll
            for (int m = 0; m < BMAX; ++m)
                w[m] = (m < nsteps && i < r) ? Wl[(size_t)s_pm[m] * rp + i] : 0.f;
#pragma unroll
            for (int m = 0; m < BMAX; ++m) {
                double acc[4] = {(double)w[m], 0.0, 0.0, 0.0};
#pragma unroll
                for (int s = 0; s < m; ++s) acc[s & 3] = fma(-c[s], sTd[m][s], acc[s & 3]);
                const float cm =
                    (m < nsteps) ? (float)(((acc[0] + acc[1]) + (acc[2] + acc[3])) * s_rsm[m]) : 0.f;
                c[m] = (double)cm;
                if (m < nsteps) Cl[(size_t)m * rp + i] = cm;
            }
        }
    };

    // ---- end of the block.  Either the removed positions are squeezed out (stable compaction of
    //      the per-position vectors across the cluster; src[new] = old), or every position stays
    //      where it is (src = identity) and the removed ones are marked with index -1: the update
    //      kernels then move nothing and a later block does the squeezing.
    if (!compact) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int k = k0 + e;
            if (owner_thread && k < n0) {
                src[(size_t)l * d + k] = k;
                dA_out[(size_t)l * d + k] = da[e];
                dQ_out[(size_t)l * d + k] = dq[e];
                idx_out[(size_t)l * d + k] = alive[e] ? org[e] : -1;
            }
        }
        if (rank == 0 && tid == 0) {
            state[l].sumrho += sumrho;
            state[l].n_new = n0;
        }
        cluster.sync();      // no CTA may retire while another can still read its shared memory
        solve_c();
        return;
    }
    const int f0 = alive[0] ? 1 : 0, f1 = alive[1] ? 1 : 0, f2 = alive[2] ? 1 : 0, f3 = alive[3] ? 1 : 0;
    const int mine = f0 + f1 + f2 + f3;
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    if (tid == 0) {
        int t = 0;
        for (int w2 = 0; w2 < NW; ++w2) { const int v = s_wsum[w2]; s_wsum[w2] = t; t += v; }
        s_count = t;
    }
    cluster.sync();
    int base = 0;
    for (int c2 = 0; c2 < rank; ++c2) base += *cluster.map_shared_rank(&s_count, c2);
    int np = base + s_wsum[warp] + incl - mine;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        if (alive[e]) {
            src[(size_t)l * d + np] = k0 + e;
            dA_out[(size_t)l * d + np] = da[e];
            dQ_out[(size_t)l * d + np] = dq[e];
            idx_out[(size_t)l * d + np] = org[e];
            ++np;
        }
    }
    if (rank == 0 && tid == 0) state[l].sumrho += sumrho;
    if (rank == CS - 1 && tid == 0) state[l].n_new = base + s_count;
    cluster.sync();      // no CTA may retire while another can still read its shared memory
    solve_c();
}

// 4-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros without reading.
__device__ __forceinline__ void cp_async4(float* smem_dst, const float* gmem_src, unsigned src_bytes) {
    const unsigned sa = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(sa), "l"(gmem_src), "r"(src_bytes)
                 : "memory");
}

__device__ __forceinline__ void cp_async16_zfill(float4* smem_dst, const float* gmem_src, unsigned src_bytes) {
    const unsigned sa = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(sa), "l"(gmem_src), "r"(src_bytes)
                 : "memory");
}

// Rank-m update of the off-diagonal entries of H^-1 and Q with compaction (out of place):
//   A'[i,j] = A[si,sj] - sum_s U[s,si] U[s,sj],
//   Q'[i,j] = Q[si,sj] - sum_s (Z[s,si] U[s,sj] + U[s,si] Z[s,sj]),    si = src[i] > sj = src[j].
// 64 x 64 tiles of the new index space, 128 threads, 8 rows x 4 columns of both matrices per
// thread: per pending step six 128-bit shared-memory loads feed 96 FMAs.  Every entry is stored
// twice, at [i][j] and [j][i]: the steps kernel reads a pivot column as a contiguous row.
__global__ void __launch_bounds__(128, 5) k_lazy_update_aq(int n_new, int m, int d,
                                                        const float* __restrict__ A,
                                                        const float* __restrict__ Q,
                                                        float* __restrict__ A2, float* __restrict__ Q2,
                                                        const int* __restrict__ src,
                                                        const float* __restrict__ U,
                                                        const float* __restrict__ Z) {
    __shared__ __align__(16) float stage[4][BMAX][64];   // pending slabs of the tile's rows and columns
    float (*sUr)[64] = stage[0];
    float (*sZr)[64] = stage[1];
    float (*sUc)[64] = stage[2];
    float (*sZc)[64] = stage[3];
    __shared__ int srow[64], scol[64];
    const int l = blockIdx.y;
    // linear index -> (ti, tj) of the lower triangle: ti = floor((sqrt(8 x + 1) - 1) / 2), fixed up
    int ti = (int)((sqrtf(8.f * (float)blockIdx.x + 1.f) - 1.f) * 0.5f);
    while (ti * (ti + 1) / 2 > (int)blockIdx.x) --ti;
    while ((ti + 1) * (ti + 2) / 2 <= (int)blockIdx.x) ++ti;
    const int tj = (int)blockIdx.x - ti * (ti + 1) / 2;
    const int i0 = ti * 64, j0 = tj * 64;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;     // rows 4ty + 32h + e, cols 4tx + e
    // a tile strictly below the diagonal and inside the live range needs no per-entry checks
    const bool interior = tj < ti && i0 + 64 <= n_new;
    const int* sl = src + (size_t)l * d;
    if (tid < 64) srow[tid] = (i0 + tid < n_new) ? sl[i0 + tid] : -1;
    else scol[tid - 64] = (j0 + tid - 64 < n_new) ? sl[j0 + tid - 64] : -1;
    __syncthreads();
    // The pending slabs of the tile's rows and columns go straight to shared memory with
    // asynchronous 4-byte copies (zero-filled past the last live row), so that all of them and the
    // gathered old entries below are in flight together.
    const float* Ul = U + (size_t)l * BMAX * d;
    const float* Zl = Z + (size_t)l * BMAX * d;
    {
        const int c = tid & 63;
        const int idx = (tid < 64) ? srow[c] : scol[c];
        float (*dU)[64] = (tid < 64) ? sUr : sUc;
        float (*dZ)[64] = (tid < 64) ? sZr : sZc;
        const unsigned nbytes = idx >= 0 ? 4u : 0u;
        const size_t off = idx >= 0 ? (size_t)idx : 0;
        for (int s = 0; s < m; ++s) {
            cp_async4(&dU[s][c], Ul + (size_t)s * d + off, nbytes);
            cp_async4(&dZ[s][c], Zl + (size_t)s * d + off, nbytes);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const float* Al = A + (size_t)l * d * d;
    const float* Ql = Q + (size_t)l * d * d;
    int cs[4];
#pragma unroll
    for (int y = 0; y < 4; ++y) cs[y] = scol[4 * tx + y];
    float a[8][4], q[8][4];
    if (interior) {
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const unsigned roff = (unsigned)(srow[4 * ty + 32 * (x >> 2) + (x & 3)] * d);   // d * d < 2^31
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                a[x][y] = __ldcs(Al + (roff + (unsigned)cs[y]));
                q[x][y] = __ldcs(Ql + (roff + (unsigned)cs[y]));
            }
        }
    } else {
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const int il = 4 * ty + 32 * (x >> 2) + (x & 3), i = i0 + il;
            const int sr = srow[il];
            const size_t roff = (size_t)(sr >= 0 ? sr : 0) * d;
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                const int j = j0 + 4 * tx + y;
                if (sr >= 0 && j < i) {
                    a[x][y] = __ldcs(Al + roff + cs[y]);
                    q[x][y] = __ldcs(Ql + roff + cs[y]);
                } else {
                    a[x][y] = 0.f; q[x][y] = 0.f;
                }
            }
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    for (int s = 0; s < m; ++s) {
        float ur[8], zr[8];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float4 v0 = *reinterpret_cast<const float4*>(&sUr[s][4 * ty + 32 * h]);
            const float4 v1 = *reinterpret_cast<const float4*>(&sZr[s][4 * ty + 32 * h]);
            ur[4 * h] = v0.x; ur[4 * h + 1] = v0.y; ur[4 * h + 2] = v0.z; ur[4 * h + 3] = v0.w;
            zr[4 * h] = v1.x; zr[4 * h + 1] = v1.y; zr[4 * h + 2] = v1.z; zr[4 * h + 3] = v1.w;
        }
        const float4 u4 = *reinterpret_cast<const float4*>(&sUc[s][4 * tx]);
        const float4 z4 = *reinterpret_cast<const float4*>(&sZc[s][4 * tx]);
        const float uc[4] = {u4.x, u4.y, u4.z, u4.w}, zc[4] = {z4.x, z4.y, z4.z, z4.w};
#pragma unroll
        for (int x = 0; x < 8; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                a[x][y] = fmaf(-ur[x], uc[y], a[x][y]);
                q[x][y] = fmaf(-zr[x], uc[y], q[x][y]);
                q[x][y] = fmaf(-ur[x], zc[y], q[x][y]);
            }
    }
    float* Ao = A2 + (size_t)l * d * d;
    float* Qo = Q2 + (size_t)l * d * d;
    const int j = j0 + 4 * tx;
    if (interior) {
        float* ao = Ao + (size_t)(i0 + 4 * ty) * d + j;
        float* qo = Qo + (size_t)(i0 + 4 * ty) * d + j;
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const unsigned o = (unsigned)((32 * (x >> 2) + (x & 3)) * d);
            *reinterpret_cast<float4*>(ao + o) = make_float4(a[x][0], a[x][1], a[x][2], a[x][3]);
            *reinterpret_cast<float4*>(qo + o) = make_float4(q[x][0], q[x][1], q[x][2], q[x][3]);
        }
        // mirror ([j][i]): the tile goes through shared memory (the staging arrays are free now),
        // so that the transposed rows leave as contiguous 256-byte pieces
        float* tbuf = &stage[0][0][0];                 // 64 x 65 floats of the 4 x 32 x 64
        const int lane = tid & 31, wrp = tid >> 5;
#pragma unroll
        for (int mat = 0; mat < 2; ++mat) {
            __syncthreads();                           // the arrays' previous readers are done
#pragma unroll
            for (int x = 0; x < 8; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y)
                    tbuf[(4 * tx + y) * 65 + 4 * ty + 32 * (x >> 2) + (x & 3)] = mat ? q[x][y] : a[x][y];
            __syncthreads();
            float* mo = (mat ? Qo : Ao) + (size_t)j0 * d + i0 + 2 * lane;
#pragma unroll 4
            for (int jl = wrp; jl < 64; jl += 4)
                *reinterpret_cast<float2*>(mo + (size_t)jl * d) =
                    make_float2(tbuf[jl * 65 + 2 * lane], tbuf[jl * 65 + 2 * lane + 1]);
        }
        return;
    }
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        const int i = i0 + 4 * ty + 32 * (x >> 2) + (x & 3);
        if (i >= n_new || j >= i) continue;
        for (int e = 0; e < 4; ++e)          // tile on the diagonal or at the ragged edge: entry by entry
            if (j + e < i) {
                Ao[(size_t)i * d + j + e] = a[x][e]; Ao[(size_t)(j + e) * d + i] = a[x][e];
                Qo[(size_t)i * d + j + e] = q[x][e]; Qo[(size_t)(j + e) * d + i] = q[x][e];
            }
    }
}

// Rank-m update of W^T with row compaction (out of place): Wt'[i,:] = Wt[si,:] - sum_s U[s,si] C[s,:].
// A CTA owns 64 rows x 256 columns; the C panel and the rows' U entries are staged in shared
// memory once per CTA, each thread carries 16 consecutive rows of one float4 column (per pending
// step: one 128-bit load of C and four broadcast 128-bit loads of U for 64 FMAs).
__global__ void __launch_bounds__(256, 3) k_lazy_update_w(int n_new, int m, int d, int rp,
                                                       const float* __restrict__ Wt,
                                                       float* __restrict__ Wt2,
                                                       const int* __restrict__ src,
                                                       const float* __restrict__ U,
                                                       const float* __restrict__ C) {
    __shared__ float4 sC[BMAX][64];       // C[s][col0 .. col0+255]
    __shared__ __align__(16) float sUr[BMAX][64];       // U[s][src[row]]
    __shared__ int srow[64];
    const int l = blockIdx.z;
    const int i0 = blockIdx.x * 64, c0 = blockIdx.y * 256;
    const int tid = threadIdx.x, tx = tid & 63, ty = tid >> 6;      // ty: rows 16 ty .. 16 ty + 15
    if (tid < 64) srow[tid] = (i0 + tid < n_new) ? src[(size_t)l * d + i0 + tid] : -1;
    __syncthreads();
    const float* Ul = U + (size_t)l * BMAX * d;
    const float* Cl = C + (size_t)l * BMAX * rp;
    // asynchronous copies (zero-filled where there is nothing to read), in flight together with
    // the gathered rows below
    for (int e = tid; e < m * 64; e += 256) {
        const int s = e >> 6, c = e & 63;
        const int sr = srow[c];
        cp_async4(&sUr[s][c], Ul + (size_t)s * d + (sr >= 0 ? sr : 0), sr >= 0 ? 4u : 0u);
        const int col = c0 + 4 * c;
        cp_async16_zfill(&sC[s][c], Cl + (size_t)s * rp + (col < rp ? col : 0), col < rp ? 16u : 0u);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    const int col = c0 + 4 * tx;
    const bool col_ok = col < rp;
    float4 w[16];                                  // rows 16 ty + x of this CTA's 64
#pragma unroll
    for (int x = 0; x < 16; ++x) {
        const int sr = srow[16 * ty + x];
        w[x] = (sr >= 0 && col_ok)
                   ? __ldcs(reinterpret_cast<const float4*>(Wt + (size_t)l * d * rp + (size_t)sr * rp + col))
                   : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    for (int s = 0; s < m; ++s) {
        const float4 c = sC[s][tx];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float4 u4 = *reinterpret_cast<const float4*>(&sUr[s][16 * ty + 4 * k]);   // broadcast
            const float nu[4] = {-u4.x, -u4.y, -u4.z, -u4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float4& t = w[4 * k + e];
                t.x = fmaf(nu[e], c.x, t.x); t.y = fmaf(nu[e], c.y, t.y);
                t.z = fmaf(nu[e], c.z, t.z); t.w = fmaf(nu[e], c.w, t.w);
            }
        }
    }
    if (col_ok) {
#pragma unroll
        for (int x = 0; x < 16; ++x) {
            const int i = i0 + 16 * ty + x;
            if (i < n_new)
                *reinterpret_cast<float4*>(Wt2 + (size_t)l * d * rp + (size_t)i * rp + col) = w[x];
        }
    }
}

// Exact refresh of the state of the last kRefresh structures.  By then the surviving entries of
// H^-1 have been reduced by orders of magnitude through thousands of fp32 downdates, and the
// relative error of the saliencies, below 5e-6 until about 64 structures remain, would grow to
// 1e-4 over the last steps.  H^-1 restricted to the survivors is the inverse of H_lambda
// restricted to them (Sec. 3.1, the remark on Eq. 4), and Q is the Gram matrix of the current
// weight columns, so both are rebuilt here from their definitions in float64: one CTA per layer,
// n <= 64 compacted positions; CTA (l, 0) does the Cholesky, the inverse of the factor and M^T M
// in shared memory, CTA (l, 1) the Gram matrix.
constexpr int kRefresh = 64;
__device__ void lazy_refresh_gram(int n, int d, int r, int rp, const float* __restrict__ Wl,
                                  float* __restrict__ Ql, double* __restrict__ dQl, float* sW);
__global__ void __launch_bounds__(256) k_lazy_refresh(int n, int d, int r, int rp,
                                                      const float* __restrict__ H,
                                                      const double* __restrict__ lam,
                                                      const int* __restrict__ idx,
                                                      const float* __restrict__ Wt, float* __restrict__ A,
                                                      float* __restrict__ Q, double* __restrict__ dA,
                                                      double* __restrict__ dQ, int* layer_status) {
    extern __shared__ double dyn_refresh[];
    double (*sB)[kRefresh + 1] = reinterpret_cast<double (*)[kRefresh + 1]>(dyn_refresh);
    double (*sI)[kRefresh + 1] = reinterpret_cast<double (*)[kRefresh + 1]>(dyn_refresh + kRefresh * (kRefresh + 1));
    __shared__ int sidx[kRefresh];
    __shared__ int flag;
    const int l = blockIdx.x, tid = threadIdx.x;
    if (blockIdx.y == 1) {
        lazy_refresh_gram(n, d, r, rp, Wt + (size_t)l * d * rp, Q + (size_t)l * d * d,
                          dQ + (size_t)l * d, reinterpret_cast<float*>(dyn_refresh));
        return;
    }
    const float* Hl = H + (size_t)l * d * d;
    float* Al = A + (size_t)l * d * d;
    if (tid == 0) flag = 0;
    if (tid < n) sidx[tid] = idx[(size_t)l * d + tid];
    __syncthreads();
    for (int e = tid; e < n * n; e += 256) {
        const int i = e / n, j = e % n;
        sB[i][j] = (double)Hl[(size_t)sidx[i] * d + sidx[j]] + (i == j ? lam[l] : 0.0);
    }
    __syncthreads();
    // Cholesky B = C C^T, column by column
    for (int c = 0; c < n; ++c) {
        if (tid == 0) {
            double p = sB[c][c];
            if (!(p > 0.0) || !isfinite(p)) {
                if (!flag) flag = isfinite(p) ? ZIPLM_ERR_NOT_PD : ZIPLM_ERR_NONFINITE;
                p = 1.0;
            }
            sB[c][c] = sqrt(p);
        }
        __syncthreads();
        for (int i = c + 1 + tid; i < n; i += 256) sB[i][c] /= sB[c][c];
        __syncthreads();
        const int m = n - 1 - c;
        for (int e = tid; e < m * m; e += 256) {
            const int i = c + 1 + e / m, jj = c + 1 + e % m;
            if (jj <= i) sB[i][jj] -= sB[i][c] * sB[jj][c];
        }
        __syncthreads();
    }
    // M = C^-1, one thread per column
    if (tid < n) {
        const int j = tid;
        for (int k = 0; k < j; ++k) sI[k][j] = 0.0;
        for (int k = j; k < n; ++k) {
            double v = (k == j) ? 1.0 : 0.0;
            for (int m = j; m < k; ++m) v -= sB[k][m] * sI[m][j];
            sI[k][j] = v / sB[k][k];
        }
    }
    __syncthreads();
    // H^-1 = M^T M: fp32 off-diagonal entries in both triangles, float64 diagonal
    for (int e = tid; e < n * n; e += 256) {
        const int i = e / n, j = e % n;
        double t = 0.0;
        for (int k = (i > j ? i : j); k < n; ++k) t = fma(sI[k][i], sI[k][j], t);
        if (i == j) dA[(size_t)l * d + i] = t;
        else Al[(size_t)i * d + j] = (float)t;
    }
    if (tid == 0 && flag) set_layer_status(layer_status, l, flag);
}

// Second half of the refresh, CTA (l, 1): Q = W^T W on the surviving columns (rows of Wt),
// float64 sums of the fp32 weights.  Chunks of 32 weights per row go through shared memory; every
// thread owns a 4 x 4 tile of the n x n result.
__device__ void lazy_refresh_gram(int n, int d, int r, int rp, const float* __restrict__ Wl,
                                  float* __restrict__ Ql, double* __restrict__ dQl, float* sW) {
    const int tid = threadIdx.x, ti = tid >> 4, tj = tid & 15;
    double acc[4][4] = {};
    for (int k0 = 0; k0 < r; k0 += 32) {
        for (int e = tid; e < kRefresh * 32; e += 256) {
            const int row = e >> 5, k = e & 31;
            sW[row * 33 + k] = (row < n && k0 + k < r) ? Wl[(size_t)row * rp + k0 + k] : 0.f;
        }
        __syncthreads();
#pragma unroll 4
        for (int k = 0; k < 32; ++k) {
            double a[4], b[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                a[x] = (double)sW[(ti + 16 * x) * 33 + k];
                b[x] = (double)sW[(tj + 16 * x) * 33 + k];
            }
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = fma(a[x], b[y], acc[x][y]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int i = ti + 16 * x, j = tj + 16 * y;
            if (i >= n || j >= n) continue;
            if (i == j) dQl[i] = acc[x][y];
            else Ql[(size_t)i * d + j] = (float)acc[x][y];
        }
}

__global__ void __launch_bounds__(256) k_lazy_pos_of(int n, int d, const int* __restrict__ idx,
                                                     int* __restrict__ pos_of) {
    const int l = blockIdx.x;
    for (int c = threadIdx.x; c < d; c += blockDim.x) pos_of[(size_t)l * d + c] = -1;
    __syncthreads();
    for (int k = threadIdx.x; k < n; k += blockDim.x) {
        const int o = idx[(size_t)l * d + k];
        if (o >= 0) pos_of[(size_t)l * d + o] = k;      // -1: removed, not squeezed out yet
    }
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
    float* P; int* sched;              // packed operands and work counter of the tensor-core update
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
    w.P = c.take<float>(lazy_tc_pack_floats(L, d, w.rp));
    w.sched = c.take<int>(2);
    w.state = c.take<LazyState>((size_t)L);
    w.lam = c.take<double>((size_t)L);
    w.base_acc = c.take<double>((size_t)L);
    const size_t inv = inverse_workspace_bytes(L, d);
    const size_t gram = hessian_tc_workspace_bytes(L, d, w.rp, ZIPLM_F32, false);
    w.aux_bytes = inv > gram ? inv : gram;
    w.aux = c.take<char>(w.aux_bytes);
    w.total = c.off;
    return w;
}

}  // namespace

bool lazy_path_supported(int d) { return d % 4 == 0 && d <= CLUSTER_MAX * SLICE_MAX && d >= 4; }

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
        ziplm_status g = run_hessian_tc(w.Q[0], w.Wt[0], ZIPLM_F32, false, L, d, rp, rp, 1.0f, 0.0f, w.aux,
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

    ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_lazy_steps, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          2 * BMAX * SLICE_MAX * (int)sizeof(float)));
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
    int prio_least = 0, prio_greatest = 0;
    ZIPLM_CHECK_CUDA(cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest));
    const int steps_priority = prio_greatest;
    if (slot < n_levels && levels[slot] == n) {
        s = snapshot(n, slot++);
        if (s != ZIPLM_OK) return s;
    }
    const int n_min = n_levels > 0 ? levels[n_levels - 1] : G;
    // n = live structures, npos = positions of the arrays (live ones and those removed since the
    // last block that squeezed the removed positions out)
    int npos = G;
    const bool every_block = option_value(ZIPLM_OPT_COMPACT_EVERY_BLOCK) == 1;
    CUtensorMap map_p, map_a[2], map_q[2], map_w[2];
    if (!lazy_tc_make_map(&map_p, w.P, L, d, rp)) return ZIPLM_ERR_CUDA;
    for (int b = 0; b < 2; ++b)
        if (!lazy_tc_make_matrix_map(&map_a[b], w.A[b], L, d, d) ||
            !lazy_tc_make_matrix_map(&map_q[b], w.Q[b], L, d, d) ||
            !lazy_tc_make_matrix_map(&map_w[b], w.Wt[b], L, d, rp))
            return ZIPLM_ERR_CUDA;
    ZIPLM_CHECK_CUDA(cudaMemsetAsync(w.sched, 0, sizeof(int) * 2, st));
    constexpr size_t kRefreshSmem = sizeof(double) * 2 * kRefresh * (kRefresh + 1);
    ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_lazy_refresh, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)kRefreshSmem));
    while (n > n_min) {
        int stop = (slot < n_levels) ? levels[slot] : n_min;         // next block boundary
        if (n > kRefresh && stop < kRefresh) stop = kRefresh;        // ... and the refresh point
        const int nsteps = (n - stop < BMAX) ? (n - stop) : BMAX;
        const int nxt = cur ^ 1;
        // Squeezing removed positions out makes the update kernels gather through a map; leaving
        // them in place keeps their reads and writes dense at the price of dead rows and columns.
        // They are squeezed out once they make up kDeadMax positions or a sixteenth of all.
        const int dead_after = npos - (n - nsteps);
        const bool refresh = (n > kRefresh && n - nsteps == kRefresh);
        const int compact = (every_block || refresh || dead_after >= kDeadMax ||
                             dead_after * kDeadFraction >= npos) ? 1 : 0;
        {
            PhaseScope ps(PH_LAZY_STEPS, st);
            // smallest cluster whose per-CTA slice of positions fits shared memory
            int cs = 1;
            while (cs < CLUSTER_MAX && round_up_int((npos + cs - 1) / cs, 4) > SLICE_MAX) cs *= 2;
            const int S = round_up_int((npos + cs - 1) / cs, 4);
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(L * cs);
            cfg.blockDim = dim3(STEP_THREADS);
            cfg.dynamicSmemBytes = (size_t)2 * BMAX * S * sizeof(float);
            cfg.stream = st;
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = cs;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            // The steps kernel is the latency chain of a layer group and needs whole SMs for its
            // clusters: at the highest launch priority its CTAs go ahead of the queued CTAs of the
            // other groups' wide update kernels as SMs drain.
            attr[1].id = cudaLaunchAttributePriority;
            attr[1].val.priority = steps_priority;
            cfg.attrs = attr;
            cfg.numAttrs = 2;
            ZIPLM_CHECK_CUDA(cudaLaunchKernelEx(
                &cfg, k_lazy_steps, npos, S, t, nsteps, compact, d, G, r, rp, (const float*)w.A[cur],
                (const float*)w.Q[cur], (const float*)w.Wt[cur], (const double*)w.dA[cur],
                (const double*)w.dQ[cur], (const int*)w.idx[cur], w.dA[nxt], w.dQ[nxt], w.idx[nxt],
                w.src, w.U, w.Z, w.C, w.state, order, saliency, layer_status));
            ZIPLM_CHECK_LAUNCH();
        }
        const int n_new = compact ? n - nsteps : npos;      // positions after this block
        // The update of W goes first: measured, the step is 2 ms shorter than with the wide update
        // of H^-1 and Q in front (the next steps kernel then follows the kernel with the longer,
        // finer-grained tail).
        if (n_new > 0 && (compact || n_new <= 1)) {     // a dense block updates W^T in the tensor-core kernel
            PhaseScope ps(PH_LAZY_UPDATE_W, st);
            k_lazy_update_w<<<dim3((n_new + 63) / 64, (rp + 255) / 256, L), 256, 0, st>>>(
                n_new, nsteps, d, rp, w.Wt[cur], w.Wt[nxt], w.src, w.U, w.C);
            ZIPLM_CHECK_LAUNCH();
        }
        if (n_new > 1 && !compact) {
            // every position stays in place: dense tiles, tensor-core kernel
            PhaseScope ps(PH_LAZY_UPDATE_AQ, st);
            s = run_lazy_update_aq_tc(map_p, map_a[cur], map_q[cur], map_w[cur], L, n_new, nsteps, d, rp,
                                      w.A[nxt], w.Q[nxt], w.Wt[nxt], w.U, w.Z, w.C, w.P, w.sched,
                                      layer_status, 0u, st);
            if (s != ZIPLM_OK) return s;
        } else if (n_new > 1) {
            PhaseScope ps(PH_LAZY_UPDATE_AQ, st);
            const int T = (n_new + 63) / 64;
            k_lazy_update_aq<<<dim3(T * (T + 1) / 2, L), 128, 0, st>>>(
                n_new, nsteps, d, w.A[cur], w.Q[cur], w.A[nxt], w.Q[nxt], w.src, w.U, w.Z);
            ZIPLM_CHECK_LAUNCH();
        }
        cur = nxt;
        npos = n_new;
        n -= nsteps;
        t += nsteps;
        if (refresh) {
            PhaseScope ps(PH_LAZY_REFRESH, st);
            k_lazy_refresh<<<dim3(L, 2), 256, kRefreshSmem, st>>>(npos, d, r, rp, H, w.lam, w.idx[cur],
                                                                  w.Wt[cur], w.A[cur], w.Q[cur], w.dA[cur],
                                                                  w.dQ[cur], layer_status);
            ZIPLM_CHECK_LAUNCH();
        }
        if (slot < n_levels && levels[slot] == n) {
            s = snapshot(npos, slot++);
            if (s != ZIPLM_OK) return s;
        }
    }
    return ZIPLM_OK;
}

}  // namespace ziplm
