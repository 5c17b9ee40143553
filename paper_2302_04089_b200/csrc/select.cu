// Budgeted choice of one database level per module (Sec. 3.2, "Finding the optimal sparsity
// configuration" and "Structured SPDY search"): given, for every module m and every level s of its
// database, the run time t[m][s] from the latency table and the prior p[m][s] = loss[m][s] /
// base_loss[m] (relative layer-wise squared error, 1 for a dropped module), and sensitivity
// coefficients c[m], find the levels that minimise sum_m c[m] p[m][s_m] subject to
// sum_m t[m][s_m] <= budget.  The search of the paper solves this problem once per candidate
// coefficient vector (1000 mutation steps), so the kernel solves K candidates per launch.
//
// Time is discretised into n_buckets units of budget / n_buckets, every option rounded UP, so a
// selection that fits in units also fits in real time.  One CTA per candidate runs the dynamic
// programme over modules with the two value rows f[0 .. n_buckets] in shared memory (float64):
//     f_{m+1}[b] = min over options s with u[m][s] <= b of  f_m[b - u[m][s]] + c[m] p[m][s]
// (ties: lowest s), stores the argmin per (module, b) in global scratch and walks it back from
// b = n_buckets.  All comparisons are on float64 sums formed in module order, which is what makes
// the chosen levels reproducible bit for bit.
#include <math.h>

#include "common.cuh"

namespace ziplm {
namespace {

constexpr int SEL_THREADS = 512;
constexpr int SEL_MAX_OPT = 255;          // options per module (argmin stored in a byte)
constexpr int SEL_MAX_BUCKETS = 12000;    // two float64 rows of n_buckets + 1 fit shared memory

__global__ void __launch_bounds__(SEL_THREADS)
k_select_levels(const float* __restrict__ loss, const float* __restrict__ base_loss,
                const float* __restrict__ time, const int* __restrict__ n_opt, int n_mod, int max_opt,
                const float* __restrict__ coef, double budget, int n_buckets,
                unsigned char* __restrict__ choice, int* __restrict__ selected,
                double* __restrict__ cost_out, double* __restrict__ time_out, int* __restrict__ status) {
    extern __shared__ double sel_smem[];
    double* f0 = sel_smem;
    double* f1 = sel_smem + (n_buckets + 1);
    __shared__ double s_cost[SEL_MAX_OPT];
    __shared__ int s_units[SEL_MAX_OPT];
    __shared__ int s_nonfinite;
    const int k = blockIdx.x, tid = threadIdx.x;
    const double inf = __longlong_as_double(0x7ff0000000000000LL);
    const double per_unit = (double)n_buckets / budget;
    unsigned char* ch = choice + (size_t)k * n_mod * (size_t)(n_buckets + 1);

    if (tid == 0) s_nonfinite = 0;
    for (int b = tid; b <= n_buckets; b += SEL_THREADS) f0[b] = 0.0;
    for (int m = 0; m < n_mod; ++m) {
        const int no = min(max(n_opt[m], 0), max_opt);
        __syncthreads();
        for (int s = tid; s < no; s += SEL_THREADS) {
            const double p = (double)loss[(size_t)m * max_opt + s] / (double)base_loss[m];
            s_cost[s] = (double)coef[(size_t)k * n_mod + m] * p;
            const double u = ceil((double)time[(size_t)m * max_opt + s] * per_unit);
            // an option that cannot fit (or has a negative time) is never taken
            s_units[s] = (u >= 0.0 && u <= (double)n_buckets) ? (int)u : n_buckets + 1;
            if (s_cost[s] != s_cost[s] || u != u) s_nonfinite = 1;
        }
        __syncthreads();
        for (int b = tid; b <= n_buckets; b += SEL_THREADS) {
            double best = inf;
            int arg = 0;
            for (int s = 0; s < no; ++s) {
                const int u = s_units[s];
                if (u > b) continue;
                const double v = f0[b - u] + s_cost[s];
                if (v < best) { best = v; arg = s; }
            }
            f1[b] = best;
            ch[(size_t)m * (n_buckets + 1) + b] = (unsigned char)arg;
        }
        double* t = f0; f0 = f1; f1 = t;
    }
    __syncthreads();
    if (tid == 0) {
        const double total = f0[n_buckets];
        if (s_nonfinite || !(total < inf)) {        // a NaN came in, or nothing fits the budget
            status[k] = s_nonfinite ? (int)ZIPLM_ERR_NONFINITE : (int)ZIPLM_ERR_INVALID_ARG;
            cost_out[k] = inf;
            time_out[k] = 0.0;
            for (int m = 0; m < n_mod; ++m) selected[(size_t)k * n_mod + m] = -1;
        } else {
            int b = n_buckets;
            double tsum = 0.0;
            for (int m = n_mod - 1; m >= 0; --m) {
                const int s = ch[(size_t)m * (n_buckets + 1) + b];
                selected[(size_t)k * n_mod + m] = s;
                const double tm = (double)time[(size_t)m * max_opt + s];
                tsum += tm;
                const double u = ceil(tm * per_unit);
                b -= (int)u;
            }
            status[k] = (int)ZIPLM_OK;
            cost_out[k] = total;
            time_out[k] = tsum;
        }
    }
}

}  // namespace

size_t select_workspace_bytes(int K, int n_mod, int n_buckets) {
    return align_up((size_t)K * n_mod * (size_t)(n_buckets + 1));
}

ziplm_status run_select_levels(const float* loss, const float* base_loss, const float* time,
                               const int* n_opt, int n_mod, int max_opt, const float* coef, int K,
                               double budget, int n_buckets, int* selected, double* cost, double* time_sum,
                               int* status, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (max_opt > SEL_MAX_OPT || n_buckets > SEL_MAX_BUCKETS) return ZIPLM_ERR_UNSUPPORTED;
    if (ws_bytes < select_workspace_bytes(K, n_mod, n_buckets)) return ZIPLM_ERR_WORKSPACE;
    const size_t smem = 2 * (size_t)(n_buckets + 1) * sizeof(double);
    ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_select_levels, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)smem));
    k_select_levels<<<K, SEL_THREADS, smem, st>>>(loss, base_loss, time, n_opt, n_mod, max_opt, coef, budget,
                                                  n_buckets, static_cast<unsigned char*>(ws), selected,
                                                  cost, time_sum, status);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

}  // namespace ziplm
