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

constexpr int SEL_THREADS = 1024;
constexpr int SEL_MAX_OPT = 255;          // options per module (argmin stored in a byte)
constexpr int SEL_MAX_BUCKETS = 12000;    // two float64 rows of n_buckets + 1 fit shared memory
constexpr int SEL_MAX_MOD = 512;          // modules per search (coefficient vectors in shared memory)

// The dynamic programme and its walk back for one coefficient vector `coef` [n_mod] (global or
// shared memory), run by the whole CTA.  f0 / f1 are the two value rows in shared memory, `ch`
// this CTA's [n_mod][n_buckets + 1] argmin scratch.  On return thread 0 holds the result in
// *total / *tsum (total = inf: nothing fits) and has written sel[0 .. n_mod); *nonfinite is a
// shared flag that is raised when a cost or a time is NaN.  Ends with a barrier.
__device__ void dp_solve(const float* __restrict__ loss, const float* __restrict__ base_loss,
                         const float* __restrict__ time, const int* __restrict__ n_opt, int n_mod,
                         int max_opt, const float* coef, double per_unit, int n_buckets, double* f0,
                         double* f1, double* s_cost, int* s_units, int* nonfinite, unsigned char* ch,
                         int* sel, double* total, double* tsum) {
    const int tid = threadIdx.x;
    const double inf = __longlong_as_double(0x7ff0000000000000LL);
    for (int b = tid; b <= n_buckets; b += SEL_THREADS) f0[b] = 0.0;
    for (int m = 0; m < n_mod; ++m) {
        const int no = min(max(n_opt[m], 0), max_opt);
        __syncthreads();
        for (int s = tid; s < no; s += SEL_THREADS) {
            const double p = (double)loss[(size_t)m * max_opt + s] / (double)base_loss[m];
            s_cost[s] = (double)coef[m] * p;
            const double u = ceil((double)time[(size_t)m * max_opt + s] * per_unit);
            // an option that cannot fit (or has a negative time) is never taken
            s_units[s] = (u >= 0.0 && u <= (double)n_buckets) ? (int)u : n_buckets + 1;
            if (s_cost[s] != s_cost[s] || u != u) *nonfinite = 1;
        }
        __syncthreads();
        // four buckets per thread and pass, so that an option's units and cost are fetched once
        // for four evaluations
        for (int b0 = tid; b0 <= n_buckets; b0 += 4 * SEL_THREADS) {
            double best[4] = {inf, inf, inf, inf};
            int arg[4] = {0, 0, 0, 0};
            for (int s = 0; s < no; ++s) {
                const int u = s_units[s];
                const double c = s_cost[s];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int b = b0 + j * SEL_THREADS;
                    if (b <= n_buckets && u <= b) {
                        const double v = f0[b - u] + c;
                        if (v < best[j]) { best[j] = v; arg[j] = s; }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int b = b0 + j * SEL_THREADS;
                if (b <= n_buckets) {
                    f1[b] = best[j];
                    ch[(size_t)m * (n_buckets + 1) + b] = (unsigned char)arg[j];
                }
            }
        }
        double* t = f0; f0 = f1; f1 = t;
    }
    __syncthreads();
    if (tid == 0) {
        *total = f0[n_buckets];
        *tsum = 0.0;
        if (*total < inf) {
            int b = n_buckets;
            double acc = 0.0;
            for (int m = n_mod - 1; m >= 0; --m) {
                const int s = ch[(size_t)m * (n_buckets + 1) + b];
                sel[m] = s;
                const double tm = (double)time[(size_t)m * max_opt + s];
                acc += tm;
                b -= (int)ceil(tm * per_unit);
            }
            *tsum = acc;
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(SEL_THREADS)
k_select_levels(const float* __restrict__ loss, const float* __restrict__ base_loss,
                const float* __restrict__ time, const int* __restrict__ n_opt, int n_mod, int max_opt,
                const float* __restrict__ coef, double budget, int n_buckets,
                unsigned char* __restrict__ choice, int* __restrict__ selected,
                double* __restrict__ cost_out, double* __restrict__ time_out, int* __restrict__ status) {
    extern __shared__ double sel_smem[];
    __shared__ double s_cost[SEL_MAX_OPT];
    __shared__ int s_units[SEL_MAX_OPT];
    __shared__ int s_nonfinite;
    __shared__ double s_total, s_tsum;
    const int k = blockIdx.x, tid = threadIdx.x;
    const double inf = __longlong_as_double(0x7ff0000000000000LL);
    if (tid == 0) s_nonfinite = 0;
    __syncthreads();
    dp_solve(loss, base_loss, time, n_opt, n_mod, max_opt, coef + (size_t)k * n_mod,
             (double)n_buckets / budget, n_buckets, sel_smem, sel_smem + (n_buckets + 1), s_cost, s_units,
             &s_nonfinite, choice + (size_t)k * n_mod * (size_t)(n_buckets + 1),
             selected + (size_t)k * n_mod, &s_total, &s_tsum);
    if (tid == 0) {
        if (s_nonfinite || !(s_total < inf)) {      // a NaN came in, or nothing fits the budget
            status[k] = s_nonfinite ? (int)ZIPLM_ERR_NONFINITE : (int)ZIPLM_ERR_INVALID_ARG;
            cost_out[k] = inf;
            time_out[k] = 0.0;
            for (int m = 0; m < n_mod; ++m) selected[(size_t)k * n_mod + m] = -1;
        } else {
            status[k] = (int)ZIPLM_OK;
            cost_out[k] = s_total;
            time_out[k] = s_tsum;
        }
    }
}

// The mutation search of "Structured SPDY search": starting from coef0, every step replaces the
// coefficients marked in mask[step] by values[step] (the caller draws both: a mark with
// probability 0.1 per coefficient gives the paper's "10 % in expectation"), solves the dynamic
// programme, scores the selection and keeps the mutated vector when the score is strictly lower.
// The score of a selection is sum_m objective[m][s_m]: a separable stand-in for the calibration
// loss of the stitched model, which only the caller's model can give.  One CTA runs one whole
// search (its own budget), so many speedup targets are searched at once.
__global__ void __launch_bounds__(SEL_THREADS)
k_search_levels(const float* __restrict__ loss, const float* __restrict__ base_loss,
                const float* __restrict__ time, const int* __restrict__ n_opt, int n_mod, int max_opt,
                const float* __restrict__ objective, const float* __restrict__ coef0,
                const double* __restrict__ budgets, int n_buckets, const unsigned char* __restrict__ mask,
                const float* __restrict__ values, int n_steps, unsigned char* __restrict__ choice,
                int* __restrict__ trial_sel, int* __restrict__ best_sel, float* __restrict__ best_coef,
                double* __restrict__ best_obj, int* __restrict__ n_accepted, int* __restrict__ status) {
    extern __shared__ double sel_smem[];
    __shared__ double s_cost[SEL_MAX_OPT];
    __shared__ int s_units[SEL_MAX_OPT];
    __shared__ float c_best[SEL_MAX_MOD], c_try[SEL_MAX_MOD];
    __shared__ int s_nonfinite, s_accept;
    __shared__ double s_total, s_tsum, s_best;
    const int k = blockIdx.x, tid = threadIdx.x;
    const double inf = __longlong_as_double(0x7ff0000000000000LL);
    const double per_unit = (double)n_buckets / budgets[k];
    int* trial = trial_sel + (size_t)k * n_mod;
    int* best = best_sel + (size_t)k * n_mod;
    unsigned char* ch = choice + (size_t)k * n_mod * (size_t)(n_buckets + 1);
    if (tid == 0) { s_nonfinite = 0; s_best = inf; }
    for (int m = tid; m < n_mod; m += SEL_THREADS) c_best[m] = coef0[(size_t)k * n_mod + m];
    int accepted = 0;
    for (int step = 0; step <= n_steps; ++step) {          // step 0 scores coef0 itself
        __syncthreads();
        for (int m = tid; m < n_mod; m += SEL_THREADS) {
            float c = c_best[m];
            if (step > 0 && mask[((size_t)k * n_steps + (step - 1)) * n_mod + m])
                c = values[((size_t)k * n_steps + (step - 1)) * n_mod + m];
            c_try[m] = c;
        }
        __syncthreads();
        dp_solve(loss, base_loss, time, n_opt, n_mod, max_opt, c_try, per_unit, n_buckets, sel_smem,
                 sel_smem + (n_buckets + 1), s_cost, s_units, &s_nonfinite, ch, trial, &s_total, &s_tsum);
        if (tid == 0) {
            s_accept = 0;
            if (s_total < inf && !s_nonfinite) {
                double score = 0.0;
                for (int m = 0; m < n_mod; ++m) score += (double)objective[(size_t)m * max_opt + trial[m]];
                if (score < s_best) { s_best = score; s_accept = 1; }
            }
        }
        __syncthreads();
        if (s_accept) {
            for (int m = tid; m < n_mod; m += SEL_THREADS) { c_best[m] = c_try[m]; best[m] = trial[m]; }
            if (step > 0) ++accepted;
        }
    }
    __syncthreads();
    const bool ok = s_best < inf;
    for (int m = tid; m < n_mod; m += SEL_THREADS) {
        best_coef[(size_t)k * n_mod + m] = c_best[m];
        if (!ok) best[m] = -1;
    }
    if (tid == 0) {
        best_obj[k] = s_best;
        n_accepted[k] = accepted;
        status[k] = s_nonfinite ? (int)ZIPLM_ERR_NONFINITE : ok ? (int)ZIPLM_OK : (int)ZIPLM_ERR_INVALID_ARG;
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

size_t search_workspace_bytes(int S, int n_mod, int n_buckets) {
    return align_up((size_t)S * n_mod * (size_t)(n_buckets + 1)) + align_up((size_t)S * n_mod * sizeof(int));
}

ziplm_status run_search_levels(const float* loss, const float* base_loss, const float* time,
                               const int* n_opt, int n_mod, int max_opt, const float* objective,
                               const float* coef0, const double* budgets, int S, int n_buckets,
                               const unsigned char* mask, const float* values, int n_steps, int* best_sel,
                               float* best_coef, double* best_obj, int* n_accepted, int* status, void* ws,
                               size_t ws_bytes, cudaStream_t st) {
    if (max_opt > SEL_MAX_OPT || n_buckets > SEL_MAX_BUCKETS || n_mod > SEL_MAX_MOD) return ZIPLM_ERR_UNSUPPORTED;
    if (ws_bytes < search_workspace_bytes(S, n_mod, n_buckets)) return ZIPLM_ERR_WORKSPACE;
    Carver c(ws);
    unsigned char* choice = c.take<unsigned char>((size_t)S * n_mod * (size_t)(n_buckets + 1));
    int* trial = c.take<int>((size_t)S * n_mod);
    const size_t smem = 2 * (size_t)(n_buckets + 1) * sizeof(double);
    ZIPLM_CHECK_CUDA(cudaFuncSetAttribute(k_search_levels, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)smem));
    k_search_levels<<<S, SEL_THREADS, smem, st>>>(loss, base_loss, time, n_opt, n_mod, max_opt, objective,
                                                  coef0, budgets, n_buckets, mask, values, n_steps, choice,
                                                  trial, best_sel, best_coef, best_obj, n_accepted, status);
    ZIPLM_CHECK_LAUNCH();
    return ZIPLM_OK;
}

}  // namespace ziplm
