// extern "C" boundary: argument validation and dispatch.  No device memory is allocated here and
// nothing synchronises; every stage is enqueued on the caller's stream.
#include <math.h>

#include "common.cuh"

using namespace ziplm;

namespace {

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Diagnostic option: group_size 1 goes through the general block path (float64 state, g x g
// Cholesky per structure) instead of the neuron path.
bool force_block_path() { return option_value(ZIPLM_OPT_FORCE_BLOCK_PATH) == 1; }

bool have_device() {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev >= 0;
}

}  // namespace

extern "C" {

const char* ziplm_status_string(ziplm_status s) {
    switch (s) {
        case ZIPLM_OK: return "ZIPLM_OK";
        case ZIPLM_ERR_INVALID_ARG: return "ZIPLM_ERR_INVALID_ARG";
        case ZIPLM_ERR_WORKSPACE: return "ZIPLM_ERR_WORKSPACE";
        case ZIPLM_ERR_NOT_PD: return "ZIPLM_ERR_NOT_PD";
        case ZIPLM_ERR_NONFINITE: return "ZIPLM_ERR_NONFINITE";
        case ZIPLM_ERR_TIMEOUT: return "ZIPLM_ERR_TIMEOUT";
        case ZIPLM_ERR_CUDA: return "ZIPLM_ERR_CUDA";
        case ZIPLM_ERR_UNSUPPORTED: return "ZIPLM_ERR_UNSUPPORTED";
    }
    return "ZIPLM_ERR_UNKNOWN";
}

size_t ziplm_hessian_workspace_bytes(int L, int d, long long n_tokens, ziplm_dtype x_dtype) {
    if (L < 1 || d < 1 || n_tokens < 0) return 0;
    return hessian_workspace_bytes(L, d, n_tokens, x_dtype, false);
}

ziplm_status ziplm_hessian_accumulate(float* H, const void* X, ziplm_dtype x_dtype, int L, int d,
                                      long long n_tokens, long long ldx, float alpha, float beta,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (L < 1 || d < 1 || n_tokens < 0 || ldx < n_tokens || !H) return ZIPLM_ERR_INVALID_ARG;
    if (x_dtype != ZIPLM_F32 && x_dtype != ZIPLM_BF16 && x_dtype != ZIPLM_F16) return ZIPLM_ERR_INVALID_ARG;
    if (!(beta == 0.f || beta == 1.f) || !isfinite(alpha)) return ZIPLM_ERR_INVALID_ARG;
    const size_t esz = (x_dtype == ZIPLM_F32) ? 4 : 2;
    if (n_tokens > 0) {
        if (!X || !aligned(X, 16) || ((size_t)ldx * esz) % 16 != 0) return ZIPLM_ERR_INVALID_ARG;
    }
    const size_t need = hessian_workspace_bytes(L, d, n_tokens, x_dtype, false);
    if (need > 0 && (!workspace || !aligned(workspace, kAlign) || workspace_bytes < need))
        return ZIPLM_ERR_WORKSPACE;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    PhaseScope ps(PH_HESSIAN, static_cast<cudaStream_t>(cuda_stream));
    return run_hessian(H, X, x_dtype, false, L, d, n_tokens, ldx, alpha, beta, workspace,
                       workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

size_t ziplm_hessian_tokens_workspace_bytes(int L, int d, long long n_tokens, ziplm_dtype a_dtype) {
    if (L < 1 || d < 1 || n_tokens < 0) return 0;
    return hessian_workspace_bytes(L, d, n_tokens, a_dtype, true);
}

ziplm_status ziplm_hessian_accumulate_tokens(float* H, const void* A, ziplm_dtype a_dtype, int L,
                                             int d, long long n_tokens, long long lda, float alpha,
                                             float beta, void* workspace, size_t workspace_bytes,
                                             void* cuda_stream) {
    if (L < 1 || d < 1 || n_tokens < 0 || lda < d || !H) return ZIPLM_ERR_INVALID_ARG;
    if (a_dtype != ZIPLM_F32 && a_dtype != ZIPLM_BF16 && a_dtype != ZIPLM_F16) return ZIPLM_ERR_INVALID_ARG;
    if (!(beta == 0.f || beta == 1.f) || !isfinite(alpha)) return ZIPLM_ERR_INVALID_ARG;
    const size_t esz = (a_dtype == ZIPLM_F32) ? 4 : 2;
    if (n_tokens > 0 && (!A || !aligned(A, esz))) return ZIPLM_ERR_INVALID_ARG;
    const size_t need = hessian_workspace_bytes(L, d, n_tokens, a_dtype, true);
    if (need > 0 && (!workspace || !aligned(workspace, kAlign) || workspace_bytes < need))
        return ZIPLM_ERR_WORKSPACE;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    PhaseScope ps(PH_HESSIAN, static_cast<cudaStream_t>(cuda_stream));
    return run_hessian(H, A, a_dtype, true, L, d, n_tokens, lda, alpha, beta, workspace,
                       workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

size_t ziplm_inverse_workspace_bytes(int L, int d) {
    if (L < 1 || d < 1) return 0;
    return inverse_workspace_bytes(L, d);
}

ziplm_status ziplm_damped_inverse(const float* H, int L, int d, float damp_frac, double* Hinv,
                                  int* layer_status, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream) {
    if (L < 1 || d < 1 || !H || !Hinv || !layer_status) return ZIPLM_ERR_INVALID_ARG;
    if (!(damp_frac >= 0.f) || !isfinite(damp_frac)) return ZIPLM_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, kAlign) || workspace_bytes < inverse_workspace_bytes(L, d))
        return ZIPLM_ERR_WORKSPACE;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ZIPLM_CHECK_CUDA(cudaMemsetAsync(layer_status, 0, sizeof(int) * L, st));
    PhaseScope ps(PH_INVERSE, st);
    return run_damped_inverse(H, L, d, damp_frac, Hinv, nullptr, 0, nullptr, nullptr, layer_status,
                              workspace, workspace_bytes, st);
}

size_t ziplm_prune_workspace_bytes(int L, int d_row, int d_col, int group_size, int n_levels) {
    if (L < 1 || d_row < 1 || d_col < 1 || group_size < 1 || n_levels < 0) return 0;
    if (d_col % group_size != 0 || group_size > 128) return 0;
    if (group_size == 1 && !force_block_path())
        return neuron_workspace_bytes(L, d_row, d_col, n_levels);
    return block_workspace_bytes(L, d_row, d_col, group_size, n_levels);
}

ziplm_status ziplm_prune_layers(const float* W, const float* H, int L, int d_row, int d_col,
                                int group_size, float damp_frac, const int* levels, int n_levels,
                                float* W_snap, float* loss, float* base_loss, int* order,
                                float* saliency, int* layer_status, void* workspace,
                                size_t workspace_bytes, void* cuda_stream) {
    if (L < 1 || d_row < 1 || d_col < 1 || group_size < 1 || n_levels < 0) return ZIPLM_ERR_INVALID_ARG;
    if (d_col % group_size != 0) return ZIPLM_ERR_INVALID_ARG;
    if (!W || !H || !order || !layer_status) return ZIPLM_ERR_INVALID_ARG;
    if (!aligned(H, 16)) return ZIPLM_ERR_INVALID_ARG;      // H is read with 128-bit loads
    if (n_levels > 0 && (!levels || !W_snap || !loss)) return ZIPLM_ERR_INVALID_ARG;
    if (!(damp_frac >= 0.f) || !isfinite(damp_frac)) return ZIPLM_ERR_INVALID_ARG;
    const int G = d_col / group_size;
    for (int i = 0; i < n_levels; ++i) {
        if (levels[i] < 0 || levels[i] > G) return ZIPLM_ERR_INVALID_ARG;
        if (i > 0 && levels[i] >= levels[i - 1]) return ZIPLM_ERR_INVALID_ARG;
    }
    if (group_size > 128) return ZIPLM_ERR_UNSUPPORTED;
    const size_t need = ziplm_prune_workspace_bytes(L, d_row, d_col, group_size, n_levels);
    if (!workspace || !aligned(workspace, kAlign) || workspace_bytes < need) return ZIPLM_ERR_WORKSPACE;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ZIPLM_CHECK_CUDA(cudaMemsetAsync(layer_status, 0, sizeof(int) * L, st));
    if (group_size == 1 && !force_block_path())
        return run_prune_neurons(W, H, L, d_row, d_col, damp_frac, levels, n_levels, W_snap, loss,
                                 base_loss, order, saliency, layer_status, workspace,
                                 workspace_bytes, st);
    return run_prune_blocks(W, H, L, d_row, d_col, group_size, damp_frac, levels, n_levels, W_snap,
                            loss, base_loss, order, saliency, layer_status, workspace,
                            workspace_bytes, st);
}

ziplm_status ziplm_kept_structures(const int* order, int L, int G, int level, int* kept,
                                   int* layer_status, void* cuda_stream) {
    if (L < 1 || G < 1 || level < 0 || level > G || !order || !layer_status) return ZIPLM_ERR_INVALID_ARG;
    if (level > 0 && !kept) return ZIPLM_ERR_INVALID_ARG;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    return run_kept_structures(order, L, G, level, kept, layer_status, static_cast<cudaStream_t>(cuda_stream));
}

ziplm_status ziplm_gather_columns(const float* M, long long ld, long long layer_stride, const int* kept,
                                  int L, int rows, int G, int group_size, int level, float* out,
                                  void* cuda_stream) {
    if (L < 1 || rows < 0 || G < 1 || group_size < 1 || level < 0 || level > G) return ZIPLM_ERR_INVALID_ARG;
    if (ld < (long long)G * group_size || layer_stride < 0) return ZIPLM_ERR_INVALID_ARG;
    if (level > 0 && rows > 0 && (!M || !kept || !out)) return ZIPLM_ERR_INVALID_ARG;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    return run_gather_columns(M, ld, layer_stride, kept, L, rows, G, group_size, level, out,
                              static_cast<cudaStream_t>(cuda_stream));
}

ziplm_status ziplm_gather_rows(const float* M, long long ld, long long layer_stride, const int* kept,
                               int L, int cols, int G, int group_size, int level, float* out,
                               void* cuda_stream) {
    if (L < 1 || cols < 0 || G < 1 || group_size < 1 || level < 0 || level > G) return ZIPLM_ERR_INVALID_ARG;
    if (ld < cols || layer_stride < 0) return ZIPLM_ERR_INVALID_ARG;
    if (level > 0 && cols > 0 && (!M || !kept || !out)) return ZIPLM_ERR_INVALID_ARG;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    return run_gather_rows(M, ld, layer_stride, kept, L, cols, G, group_size, level, out,
                           static_cast<cudaStream_t>(cuda_stream));
}

size_t ziplm_select_workspace_bytes(int n_candidates, int n_modules, int n_buckets) {
    if (n_candidates < 1 || n_modules < 1 || n_buckets < 1) return 0;
    return select_workspace_bytes(n_candidates, n_modules, n_buckets);
}

ziplm_status ziplm_select_levels(const float* loss, const float* base_loss, const float* time,
                                 const int* n_options, int n_modules, int max_options,
                                 const float* coef, int n_candidates, double budget, int n_buckets,
                                 int* selected, double* cost, double* time_sum, int* candidate_status,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (n_modules < 1 || max_options < 1 || n_candidates < 1 || n_buckets < 1) return ZIPLM_ERR_INVALID_ARG;
    if (!(budget > 0.0) || !isfinite(budget)) return ZIPLM_ERR_INVALID_ARG;
    if (!loss || !base_loss || !time || !n_options || !coef || !selected || !cost || !time_sum ||
        !candidate_status)
        return ZIPLM_ERR_INVALID_ARG;
    if (max_options > 255 || n_buckets > 12000) return ZIPLM_ERR_UNSUPPORTED;
    const size_t need = select_workspace_bytes(n_candidates, n_modules, n_buckets);
    if (!workspace || !aligned(workspace, kAlign) || workspace_bytes < need) return ZIPLM_ERR_WORKSPACE;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    return run_select_levels(loss, base_loss, time, n_options, n_modules, max_options, coef, n_candidates,
                             budget, n_buckets, selected, cost, time_sum, candidate_status, workspace,
                             workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

size_t ziplm_search_workspace_bytes(int n_searches, int n_modules, int n_buckets) {
    if (n_searches < 1 || n_modules < 1 || n_buckets < 1) return 0;
    return search_workspace_bytes(n_searches, n_modules, n_buckets);
}

ziplm_status ziplm_search_levels(const float* loss, const float* base_loss, const float* time,
                                 const int* n_options, int n_modules, int max_options,
                                 const float* objective, const float* coef0, const double* budgets,
                                 int n_searches, int n_buckets, const unsigned char* mask,
                                 const float* values, int n_steps, int* best_selected, float* best_coef,
                                 double* best_objective, int* n_accepted, int* search_status,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (n_modules < 1 || max_options < 1 || n_searches < 1 || n_buckets < 1 || n_steps < 0)
        return ZIPLM_ERR_INVALID_ARG;
    if (!loss || !base_loss || !time || !n_options || !objective || !coef0 || !budgets || !best_selected ||
        !best_coef || !best_objective || !n_accepted || !search_status)
        return ZIPLM_ERR_INVALID_ARG;
    if (n_steps > 0 && (!mask || !values)) return ZIPLM_ERR_INVALID_ARG;
    if (max_options > 255 || n_buckets > 12000 || n_modules > 512) return ZIPLM_ERR_UNSUPPORTED;
    const size_t need = search_workspace_bytes(n_searches, n_modules, n_buckets);
    if (!workspace || !aligned(workspace, kAlign) || workspace_bytes < need) return ZIPLM_ERR_WORKSPACE;
    if (!have_device()) return ZIPLM_ERR_CUDA;
    return run_search_levels(loss, base_loss, time, n_options, n_modules, max_options, objective, coef0,
                             budgets, n_searches, n_buckets, mask, values, n_steps, best_selected, best_coef,
                             best_objective, n_accepted, search_status, workspace, workspace_bytes,
                             static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"
