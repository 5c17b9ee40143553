// Greedy one-column-at-a-time structured OBS (Algorithm 1 with |M_S| = 1: FFN neurons).
//
// With a single column j the block ((H^-1)_SS)^-1 is the scalar 1 / H^-1[j,j] = 1/h, so with
// u = H^-1[:,j] / sqrt(h) and c = W[:,j] / sqrt(h):
//     rho_j = ||W[:,j]||^2 / H^-1[j,j]         (Eq. 2)
//     W    <- W    - c u^T                     (Eq. 3)
//     H^-1 <- H^-1 - u u^T                     (Eq. 4)
// One greedy step is two launches for all L layers at once: a small "prep" kernel (argmin, pivot
// column, float64 diagonal downdate, bookkeeping) and a streaming "update" kernel that makes one
// read-modify-write pass over the live part of H^-1 and W and produces the next saliencies.
//
// Data layout per layer
//   A    fp32 [d, pitch]  strictly lower triangle of the live H^-1 (symmetry: 4 n^2 bytes per
//                         step instead of 8 n^2); slot (k, j), j < k, holds H^-1 between the
//                         structures at positions k and j.
//   diag fp64 [d]         diagonal of H^-1.  Kept in float64 so that rho stays within ~1e-6 of
//                         exact arithmetic over thousands of downdates.
//   Wt   fp32 [d, rp]     W transposed: row k is column k of W, so a column norm is a
//                         contiguous, coalesced reduction done by one warp.
//   idx  int  [d]         original column index of the structure at each position.
// Removed structures are compacted away by swap-remove: when position p is removed the last live
// position takes its place (values of removed entries never feed later steps -- remark after
// Algorithm 1 -- so they are simply dropped).  The live problem is therefore always the leading
// n x n corner, and every step streams exactly the live bytes.
#include <math.h>

#include <mutex>
#include <vector>

#include "common.cuh"

namespace ziplm {
namespace {

struct StepState {
    int p;          // position removed in the current step
    int last;       // last live position (n - 1), which moves into p
    double sumrho;  // sum of the saliencies of all removed structures
    double dw2;     // scratch: ||W - W_snap||_F^2 of the snapshot being written
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void axpy4(float4& a, float s, const float4& v) {
    a.x = fmaf(s, v.x, a.x); a.y = fmaf(s, v.y, a.y);
    a.z = fmaf(s, v.z, a.z); a.w = fmaf(s, v.w, a.w);
}

__device__ __forceinline__ void set_comp(float4& a, int c, float v) {
    if (c == 0) a.x = v; else if (c == 1) a.y = v; else if (c == 2) a.z = v; else a.w = v;
}

__device__ __forceinline__ float sq4(const float4& w, float acc) {
    acc = fmaf(w.x, w.x, acc); acc = fmaf(w.y, w.y, acc);
    acc = fmaf(w.z, w.z, acc); acc = fmaf(w.w, w.w, acc);
    return acc;
}

// Wt = W^T, idx = identity, rho = ||W[:,k]||^2 / diag[k].  One block per 32 columns.
__global__ void __launch_bounds__(256) k_neuron_init(const float* __restrict__ W, int r, int d,
                                                     int rp, float* __restrict__ Wt,
                                                     const double* __restrict__ diag,
                                                     double* __restrict__ rho, int* __restrict__ idx,
                                                     StepState* __restrict__ state) {
    __shared__ float tile[32][33];
    const int l = blockIdx.y;
    const int c0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const float* Wl = W + (size_t)l * r * d;
    float* Wtl = Wt + (size_t)l * d * rp;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
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
            acc[m] += v * v;
        }
        __syncthreads();
    }
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const float s = warp_sum(acc[m]);
        const int c = c0 + ty + 8 * m;
        if (tx == 0 && c < d) {
            rho[(size_t)l * d + c] = (double)s / diag[(size_t)l * d + c];
            idx[(size_t)l * d + c] = c;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        state[l].p = 0; state[l].last = 0; state[l].sumrho = 0.0; state[l].dw2 = 0.0;
    }
}

// Step prologue for n live structures: argmin of rho (ties -> lowest original index), pivot
// column u = H^-1[:,p] / sqrt(h), c = W[:,p] / sqrt(h), float64 diagonal downdate, swap-remove of
// the per-position vectors, log of (order, saliency).  One block per layer.
__global__ void __launch_bounds__(512) k_neuron_prep(int n, int t, int d, int G, int pitch, int r,
                                                     int rp, const float* __restrict__ A,
                                                     const float* __restrict__ Wt,
                                                     double* __restrict__ diag,
                                                     const double* __restrict__ rho,
                                                     int* __restrict__ idx, float* __restrict__ ubuf,
                                                     float* __restrict__ cbuf,
                                                     StepState* __restrict__ state,
                                                     int* __restrict__ order,
                                                     float* __restrict__ saliency,
                                                     int* layer_status) {
    const int l = blockIdx.x;
    const int tid = threadIdx.x;
    const float* Al = A + (size_t)l * d * pitch;
    double* dg = diag + (size_t)l * d;
    const double* rh = rho + (size_t)l * d;
    int* ix = idx + (size_t)l * d;

    // ---- argmin over live positions, key (rho, original index)
    double bv = INFINITY;
    int bo = 0x7fffffff, bp = -1;
    for (int k = tid; k < n; k += blockDim.x) {
        double v = rh[k];
        if (!(v == v)) v = INFINITY;          // NaN never wins
        const int o = ix[k];
        if (v < bv || (v == bv && o < bo)) { bv = v; bo = o; bp = k; }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int oo = __shfl_xor_sync(0xffffffffu, bo, off);
        const int op = __shfl_xor_sync(0xffffffffu, bp, off);
        if (ov < bv || (ov == bv && oo < bo)) { bv = ov; bo = oo; bp = op; }
    }
    __shared__ double sv[16];
    __shared__ int so[16], sp[16];
    __shared__ int s_p;
    __shared__ double s_rs;
    const int warp = tid >> 5, lane = tid & 31;
    if (lane == 0) { sv[warp] = bv; so[warp] = bo; sp[warp] = bp; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
            if (sv[w] < bv || (sv[w] == bv && so[w] < bo)) { bv = sv[w]; bo = so[w]; bp = sp[w]; }
        if (bp < 0) bp = 0;
        const int p = bp;
        double h = dg[p];
        if (!isfinite(bv) || !isfinite(h)) {
            set_layer_status(layer_status, l, ZIPLM_ERR_NONFINITE);
            h = 1.0;
        } else if (!(h > 0.0)) {
            set_layer_status(layer_status, l, ZIPLM_ERR_NOT_PD);
            h = 1.0;
        }
        s_p = p;
        s_rs = 1.0 / sqrt(h);
        state[l].p = p;
        state[l].last = n - 1;
        state[l].sumrho += rh[p];
        order[(size_t)l * G + t] = ix[p];
        if (saliency) saliency[(size_t)l * G + t] = (float)rh[p];
    }
    __syncthreads();
    const int p = s_p, last = n - 1;
    const double rs = s_rs;
    // ---- pivot column (row prefix + column suffix of the stored triangle) and diagonal downdate
    float* ub = ubuf + (size_t)l * pitch;
    for (int k = tid; k < n; k += blockDim.x) {
        if (k == p) { ub[k] = 0.f; continue; }
        const float v = (k < p) ? Al[(size_t)p * pitch + k] : Al[(size_t)k * pitch + p];
        const double u = (double)v * rs;
        ub[k] = (float)u;
        dg[k] -= u * u;
    }
    const float* wp = Wt + (size_t)l * d * rp + (size_t)p * rp;
    float* cb = cbuf + (size_t)l * rp;
    for (int i = tid; i < rp; i += blockDim.x) cb[i] = (i < r) ? (float)((double)wp[i] * rs) : 0.f;
    __syncthreads();
    // ---- swap-remove on the per-position vectors (the matrices move in the update kernel)
    if (tid == 0 && p != last) {
        dg[p] = dg[last];
        ix[p] = ix[last];
    }
}

// One streaming pass over the live triangle of H^-1 and the live rows of Wt (Eq. 3, Eq. 4),
// fused with the column norms / saliencies of the next step (Eq. 2) and with the swap-remove
// move of the last live position into the removed one.  One warp per row.
//   row k (k != p, k != last): A[k, j] -= u_k u_j for j < k; the slot of the removed column p
//       (if p < k) receives the moved entry  A[last, k] - u_last u_k.
//   row last: its entries j < p are written, updated, to row p; nothing else of it is written,
//       so every other row can still read its old values.
__global__ void __launch_bounds__(256) k_neuron_update(int n, int d, int pitch, int rp,
                                                       float* A, float* Wt,
                                                       const double* __restrict__ diag,
                                                       double* __restrict__ rho,
                                                       const float* __restrict__ ubuf,
                                                       const float* __restrict__ cbuf,
                                                       const StepState* __restrict__ state) {
    const int l = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rb = (gridDim.x - 1 - blockIdx.x);          // longest rows first
    const int p = state[l].p, last = state[l].last;
    float* Al = A + (size_t)l * d * pitch;
    float* Wl = Wt + (size_t)l * d * rp;
    const float* ub = ubuf + (size_t)l * pitch;
    const float4* u4 = reinterpret_cast<const float4*>(ub);
    const float4* c4 = reinterpret_cast<const float4*>(cbuf + (size_t)l * rp);

    const int k = rb * 8 + warp;
    if (k >= n || k == p) return;
    const float uk = ub[k];
    const float nuk = -uk;
    const bool is_last = (k == last);
    const int dest = is_last ? p : k;
    const int len = is_last ? p : k;
    // ---- H^-1 row
    {
        const float4* src = reinterpret_cast<const float4*>(Al + (size_t)k * pitch);
        float4* dst = reinterpret_cast<float4*>(Al + (size_t)dest * pitch);
        const int nvec = (len + 3) >> 2;
        const bool pull = (!is_last) && (p < k);
        float pulled = 0.f;
        if (pull) pulled = fmaf(-ub[last], uk, Al[(size_t)last * pitch + k]);
        const int pq = pull ? (p >> 2) : -1, pc = p & 3;
        int q = lane;
        for (; q + 96 < nvec; q += 128) {
            float4 a0 = __ldcs(src + q), a1 = __ldcs(src + q + 32);
            float4 a2 = __ldcs(src + q + 64), a3 = __ldcs(src + q + 96);
            const float4 v0 = __ldg(u4 + q), v1 = __ldg(u4 + q + 32);
            const float4 v2 = __ldg(u4 + q + 64), v3 = __ldg(u4 + q + 96);
            axpy4(a0, nuk, v0); axpy4(a1, nuk, v1); axpy4(a2, nuk, v2); axpy4(a3, nuk, v3);
            if (q == pq) set_comp(a0, pc, pulled);
            if (q + 32 == pq) set_comp(a1, pc, pulled);
            if (q + 64 == pq) set_comp(a2, pc, pulled);
            if (q + 96 == pq) set_comp(a3, pc, pulled);
            dst[q] = a0; dst[q + 32] = a1; dst[q + 64] = a2; dst[q + 96] = a3;
        }
        for (; q < nvec; q += 32) {
            float4 a0 = __ldcs(src + q);
            const float4 v0 = __ldg(u4 + q);
            axpy4(a0, nuk, v0);
            if (q == pq) set_comp(a0, pc, pulled);
            dst[q] = a0;
        }
    }
    // ---- W column (row of Wt) and its squared norm
    {
        const float4* src = reinterpret_cast<const float4*>(Wl + (size_t)k * rp);
        float4* dst = reinterpret_cast<float4*>(Wl + (size_t)dest * rp);
        const int nvec = rp >> 2;
        float nrm = 0.f;
        int q = lane;
        for (; q + 32 < nvec; q += 64) {
            float4 w0 = __ldcs(src + q), w1 = __ldcs(src + q + 32);
            const float4 v0 = __ldg(c4 + q), v1 = __ldg(c4 + q + 32);
            axpy4(w0, nuk, v0); axpy4(w1, nuk, v1);
            nrm = sq4(w0, nrm); nrm = sq4(w1, nrm);
            dst[q] = w0; dst[q + 32] = w1;
        }
        for (; q < nvec; q += 32) {
            float4 w0 = __ldcs(src + q);
            const float4 v0 = __ldg(c4 + q);
            axpy4(w0, nuk, v0);
            nrm = sq4(w0, nrm);
            dst[q] = w0;
        }
        nrm = warp_sum(nrm);
        if (lane == 0) rho[(size_t)l * d + dest] = (double)nrm / diag[(size_t)l * d + dest];
    }
}

// pos_of[c] = live position of original column c, or -1 if it was removed.  One block per layer.
__global__ void __launch_bounds__(256) k_neuron_pos_of(int n, int d, const int* __restrict__ idx,
                                                       int* __restrict__ pos_of) {
    const int l = blockIdx.x;
    for (int c = threadIdx.x; c < d; c += blockDim.x) pos_of[(size_t)l * d + c] = -1;
    __syncthreads();
    for (int k = threadIdx.x; k < n; k += blockDim.x)
        pos_of[(size_t)l * d + idx[(size_t)l * d + k]] = k;
}

// W_snap[l, slot] = current weights in original column order with removed columns exactly zero
// (last line of Algorithm 1); accumulates ||W - W_snap||_F^2 for the loss identity.
__global__ void __launch_bounds__(256) k_neuron_snapshot(int r, int d, int rp,
                                                         const float* __restrict__ W,
                                                         const float* __restrict__ Wt,
                                                         const int* __restrict__ pos_of,
                                                         float* __restrict__ W_snap, int n_levels,
                                                         int slot, StepState* __restrict__ state) {
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

// loss = 1/2 sum(rho of removed) - lambda/2 ||W - W_snap||_F^2   (each rho is twice the increase
// of the damped objective 1/2 tr(dW (H + lambda I) dW^T); the loss of Eq. 1 is its H part).
__global__ void k_neuron_loss(int L, int n_levels, int slot, const double* __restrict__ lam,
                              StepState* __restrict__ state, float* __restrict__ loss) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= L) return;
    const double v = 0.5 * state[l].sumrho - 0.5 * lam[l] * state[l].dw2;
    loss[(size_t)l * n_levels + slot] = (float)(v > 0.0 ? v : 0.0);
    state[l].dw2 = 0.0;
}

struct NeuronWs {
    float* A; float* Wt; double* diag; double* rho; int* idx; int* pos_of; float* ubuf; float* cbuf;
    StepState* state; double* lam; double* base_acc; void* inv_ws; size_t inv_bytes;
    int pitch, rp;
    size_t total;
};

NeuronWs carve_neuron(void* ws, int L, int r, int d) {
    NeuronWs w;
    w.pitch = round_up_int(d, 4);
    w.rp = round_up_int(r, 4);
    Carver c(ws);
    w.A = c.take<float>((size_t)L * d * w.pitch);
    w.Wt = c.take<float>((size_t)L * d * w.rp);
    w.diag = c.take<double>((size_t)L * d);
    w.rho = c.take<double>((size_t)L * d);
    w.idx = c.take<int>((size_t)L * d);
    w.pos_of = c.take<int>((size_t)L * d);
    w.ubuf = c.take<float>((size_t)L * w.pitch);
    w.cbuf = c.take<float>((size_t)L * w.rp);
    w.state = c.take<StepState>((size_t)L);
    w.lam = c.take<double>((size_t)L);
    w.base_acc = c.take<double>((size_t)L);
    w.inv_bytes = inverse_workspace_bytes(L, d);
    w.inv_ws = c.take<char>(w.inv_bytes);
    w.total = c.off;
    return w;
}

}  // namespace

// The delayed-update variant (prune_lazy.cu) is the default where it applies; the streaming
// variant in this file serves the other shapes and ziplm_set_option(ZIPLM_OPT_NEURON_PATH, 1) selects it always.
static bool use_lazy_path(int d) {
    if (option_value(ZIPLM_OPT_NEURON_PATH) == 1) return false;
    return lazy_path_supported(d);
}

// The delayed-update variant has latency-bound phases (the per-step cluster kernel occupies a
// few dozen SMs, the panel steps of the factorisation even fewer).  Layers are independent, so
// they are split into groups that run the whole pipeline on streams of their own: one group's
// latency-bound kernels then overlap the other groups' bandwidth- and ALU-bound ones.
constexpr int kMaxGroups = 8;
constexpr int kDefaultGroups = 6;

static int layer_groups(int L) {
    int g = option_value(ZIPLM_OPT_LAYER_GROUPS);
    if (g < 1) g = kDefaultGroups;
    if (g > kMaxGroups) g = kMaxGroups;
    if (g > L) g = L;
    return g;
}

static int group_begin(int L, int groups, int g) { return (int)((long long)L * g / groups); }

static size_t grouped_lazy_bytes(int L, int r, int d, int n_levels, int groups) {
    size_t b = 0;
    for (int g = 0; g < groups; ++g)
        b += lazy_workspace_bytes(group_begin(L, groups, g + 1) - group_begin(L, groups, g), r, d,
                                  n_levels);
    return b;
}

// Internal streams and the fork / join events of a call, created once per device and kept for
// the life of the process.  Several host threads may call at the same time: the pool is built
// under a mutex, and every call takes an event set of its own from a free list (a set can be
// used again as soon as the call that held it has enqueued its work, since a stream wait refers
// to the record that precedes it).
struct EventSet {
    cudaEvent_t fork;
    cudaEvent_t join[kMaxGroups];
};
struct DevicePool {
    bool ready = false;
    cudaStream_t streams[kMaxGroups] = {};
    std::vector<EventSet*> free_sets;
};
static std::mutex g_pool_mu;
static DevicePool g_pools[64];

static DevicePool* device_pool() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lk(g_pool_mu);
    DevicePool& p = g_pools[dev];
    if (!p.ready) {
        for (int g = 0; g < kMaxGroups; ++g)
            if (cudaStreamCreateWithFlags(&p.streams[g], cudaStreamNonBlocking) != cudaSuccess) {
                for (int h = 0; h < g; ++h) cudaStreamDestroy(p.streams[h]);
                return nullptr;
            }
        p.ready = true;
    }
    return &p;
}

static EventSet* take_events(DevicePool* p) {
    {
        std::lock_guard<std::mutex> lk(g_pool_mu);
        if (!p->free_sets.empty()) {
            EventSet* e = p->free_sets.back();
            p->free_sets.pop_back();
            return e;
        }
    }
    EventSet* e = new EventSet();
    const bool fork_ok = cudaEventCreateWithFlags(&e->fork, cudaEventDisableTiming) == cudaSuccess;
    int made = 0;
    while (fork_ok && made < kMaxGroups &&
           cudaEventCreateWithFlags(&e->join[made], cudaEventDisableTiming) == cudaSuccess)
        ++made;
    if (made < kMaxGroups) {             // give back what was created
        for (int g = 0; g < made; ++g) cudaEventDestroy(e->join[g]);
        if (fork_ok) cudaEventDestroy(e->fork);
        delete e;
        return nullptr;
    }
    return e;
}

static void give_events(DevicePool* p, EventSet* e) {
    std::lock_guard<std::mutex> lk(g_pool_mu);
    p->free_sets.push_back(e);
}

size_t neuron_workspace_bytes(int L, int r, int d, int n_levels) {
    const size_t a = carve_neuron(nullptr, L, r, d).total;
    size_t b = 0;
    if (lazy_path_supported(d))   // every group count up to the maximum must fit
        for (int g = 1; g <= kMaxGroups && g <= L; ++g) {
            const size_t t = grouped_lazy_bytes(L, r, d, n_levels, g);
            if (t > b) b = t;
        }
    return a > b ? a : b;
}

static ziplm_status run_prune_lazy_grouped(const float* W, const float* H, int L, int r, int d,
                                           float damp_frac, const int* levels, int n_levels,
                                           float* W_snap, float* loss, float* base_loss, int* order,
                                           float* saliency, int* layer_status, void* ws,
                                           cudaStream_t st) {
    const int groups = layer_groups(L);
    DevicePool* pool = groups > 1 ? device_pool() : nullptr;
    EventSet* ev = pool ? take_events(pool) : nullptr;
    if (groups <= 1 || !ev)
        return run_prune_lazy(W, H, L, r, d, damp_frac, levels, n_levels, W_snap, loss, base_loss,
                              order, saliency, layer_status, ws,
                              lazy_workspace_bytes(L, r, d, n_levels), st);
    // Calls take consecutive streams of the pool in turn, so that two calls that the caller runs
    // concurrently (different layers on different streams) do not queue behind each other.
    static std::atomic<unsigned> next_stream{0};
    const unsigned first = next_stream.fetch_add((unsigned)groups);
    if (cudaEventRecord(ev->fork, st) != cudaSuccess) {
        give_events(pool, ev);
        return ZIPLM_ERR_CUDA;
    }
    ziplm_status rc = ZIPLM_OK;
    char* wsp = static_cast<char*>(ws);
    for (int g = 0; g < groups; ++g) {
        const int l0 = group_begin(L, groups, g), Lg = group_begin(L, groups, g + 1) - l0;
        const size_t bytes = lazy_workspace_bytes(Lg, r, d, n_levels);
        cudaStream_t sg = pool->streams[(first + (unsigned)g) % kMaxGroups];
        bool ok = cudaStreamWaitEvent(sg, ev->fork, 0) == cudaSuccess;
        if (ok && rc == ZIPLM_OK)
            rc = run_prune_lazy(W + (size_t)l0 * r * d, H + (size_t)l0 * d * d, Lg, r, d, damp_frac,
                                levels, n_levels, W_snap + (size_t)l0 * n_levels * r * d,
                                loss + (size_t)l0 * n_levels, base_loss ? base_loss + l0 : nullptr,
                                order + (size_t)l0 * d, saliency ? saliency + (size_t)l0 * d : nullptr,
                                layer_status + l0, wsp, bytes, sg);
        // always join, so that the caller's stream stays ordered after whatever was enqueued
        ok = ok && cudaEventRecord(ev->join[g], sg) == cudaSuccess &&
             cudaStreamWaitEvent(st, ev->join[g], 0) == cudaSuccess;
        if (!ok && rc == ZIPLM_OK) rc = ZIPLM_ERR_CUDA;
        wsp += bytes;
    }
    give_events(pool, ev);
    return rc;
}

ziplm_status run_prune_neurons(const float* W, const float* H, int L, int r, int d,
                               float damp_frac, const int* levels, int n_levels, float* W_snap,
                               float* loss, float* base_loss, int* order, float* saliency,
                               int* layer_status, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (ws_bytes < neuron_workspace_bytes(L, r, d, n_levels)) return ZIPLM_ERR_WORKSPACE;
    if (use_lazy_path(d))
        return run_prune_lazy_grouped(W, H, L, r, d, damp_frac, levels, n_levels, W_snap, loss,
                                      base_loss, order, saliency, layer_status, ws, st);
    NeuronWs w = carve_neuron(ws, L, r, d);
    const int G = d;

    ziplm_status s;
    {
        PhaseScope ps(PH_INVERSE, st);
        s = run_damped_inverse(H, L, d, damp_frac, nullptr, w.A, w.pitch, w.diag, w.lam, layer_status,
                               w.inv_ws, w.inv_bytes, st);
    }
    if (s != ZIPLM_OK) return s;
    auto init = [&]() -> ziplm_status {
        PhaseScope ps(PH_INIT, st);
        ZIPLM_CHECK_CUDA(cudaMemsetAsync(order, 0xFF, sizeof(int) * (size_t)L * G, st));
        if (saliency)
            ZIPLM_CHECK_CUDA(cudaMemsetAsync(saliency, 0, sizeof(float) * (size_t)L * G, st));
        k_neuron_init<<<dim3((d + 31) / 32, L), 256, 0, st>>>(W, r, d, w.rp, w.Wt, w.diag, w.rho,
                                                             w.idx, w.state);
        ZIPLM_CHECK_LAUNCH();
        if (base_loss) return run_base_loss(W, H, L, r, d, w.base_acc, base_loss, st);
        return ZIPLM_OK;
    };
    s = init();
    if (s != ZIPLM_OK) return s;

    auto snapshot = [&](int n, int slot) -> ziplm_status {
        PhaseScope ps(PH_SNAPSHOT, st);
        k_neuron_pos_of<<<L, 256, 0, st>>>(n, d, w.idx, w.pos_of);
        ZIPLM_CHECK_LAUNCH();
        k_neuron_snapshot<<<dim3((d + 31) / 32, (r + 31) / 32, L), 256, 0, st>>>(
            r, d, w.rp, W, w.Wt, w.pos_of, W_snap, n_levels, slot, w.state);
        ZIPLM_CHECK_LAUNCH();
        k_neuron_loss<<<(L + 63) / 64, 64, 0, st>>>(L, n_levels, slot, w.lam, w.state, loss);
        ZIPLM_CHECK_LAUNCH();
        return ZIPLM_OK;
    };

    int n = G, slot = 0;
    if (slot < n_levels && levels[slot] == n) {
        s = snapshot(n, slot++);
        if (s != ZIPLM_OK) return s;
    }
    const int n_min = n_levels > 0 ? levels[n_levels - 1] : G;
    for (int t = 0; n > n_min; ++t) {
        {
            PhaseScope ps(PH_PREP, st);
            k_neuron_prep<<<L, 512, 0, st>>>(n, t, d, G, w.pitch, r, w.rp, w.A, w.Wt, w.diag, w.rho,
                                             w.idx, w.ubuf, w.cbuf, w.state, order, saliency,
                                             layer_status);
            ZIPLM_CHECK_LAUNCH();
        }
        if (n > 1) {
            PhaseScope ps(PH_UPDATE, st);
            k_neuron_update<<<dim3((n + 7) / 8, L), 256, 0, st>>>(n, d, w.pitch, w.rp, w.A, w.Wt,
                                                                 w.diag, w.rho, w.ubuf, w.cbuf, w.state);
            ZIPLM_CHECK_LAUNCH();
        }
        --n;
        if (slot < n_levels && levels[slot] == n) {
            s = snapshot(n, slot++);
            if (s != ZIPLM_OK) return s;
        }
    }
    return ZIPLM_OK;
}

}  // namespace ziplm
