// Shared host/device helpers for the ZipLM structured-OBS kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <atomic>
#include <stdint.h>

#include "ziplm.h"

namespace ziplm {

constexpr int kTile = 64;          // tile edge of the float64 factorisation kernels
constexpr size_t kAlign = 256;     // alignment of every carve-out of a workspace

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }
inline int round_up_int(int x, int a) { return (x + a - 1) / a * a; }

// Bump allocator over a caller-provided workspace; with base == nullptr it only measures.
struct Carver {
    char* base;
    size_t off;
    explicit Carver(void* b) : base(static_cast<char*>(b)), off(0) {}
    template <typename T>
    T* take(size_t count) {
        size_t start = off;
        off = align_up(off + count * sizeof(T));
        return base ? reinterpret_cast<T*>(base + start) : nullptr;
    }
};

// Number of kernels launched by this library since it was loaded (diagnostics).
extern std::atomic<long long> g_launches;

// Current value of a diagnostic option (ziplm_set_option); 0 is every option's default.
int option_value(int option);

// Phases reported by the optional event timing (ziplm_profile_begin / ziplm_profile_end).
enum Phase { PH_HESSIAN = 0, PH_INVERSE, PH_INIT, PH_PREP, PH_UPDATE, PH_SNAPSHOT, PH_BLOCK_SCORE,
             PH_BLOCK_UPDATE, PH_LAZY_STEPS, PH_LAZY_UPDATE_AQ, PH_LAZY_UPDATE_W, PH_INV_PRODUCTS,
             PH_INV_LEAVES, PH_INV_LAUUM, PH_LAZY_REFRESH, PH_COUNT };

// Brackets the launches issued during its lifetime with a pair of events when timing is on.
struct PhaseScope {
    PhaseScope(int phase, cudaStream_t st);
    ~PhaseScope();
    cudaStream_t st_;
    int idx_;
};

// Placed after every kernel launch: counts it and returns ZIPLM_ERR_CUDA from the caller if the
// launch failed.
#define ZIPLM_CHECK_LAUNCH()                                   \
    do {                                                       \
        ++::ziplm::g_launches;                                 \
        cudaError_t e__ = cudaGetLastError();                  \
        if (e__ != cudaSuccess) return ZIPLM_ERR_CUDA;         \
    } while (0)

#define ZIPLM_CHECK_CUDA(expr)                                 \
    do {                                                       \
        cudaError_t e__ = (expr);                              \
        if (e__ != cudaSuccess) return ZIPLM_ERR_CUDA;         \
    } while (0)

// A layer's status only ever moves from OK to the first error seen.
__device__ inline void set_layer_status(int* layer_status, int l, int code) {
    atomicCAS(layer_status + l, (int)ZIPLM_OK, code);
}

// ---- stages implemented in the other translation units (host-side planners) -----------------

// Workspace of the float64 damped inverse for L layers of width d.
size_t inverse_workspace_bytes(int L, int d);

// (H + lambda I)^-1 in float64.  out64 (may be null) receives the full symmetric [L, d, d]
// matrix; tri32/diag64 (may be null) receive the strictly lower triangle in fp32 with row pitch
// `pitch32` and the diagonal in float64; lam_out (may be null) receives lambda per layer.
ziplm_status run_damped_inverse(const float* H, int L, int d, float damp_frac, double* out64,
                                float* tri32, int pitch32, double* diag64, double* lam_out,
                                int* layer_status, void* ws, size_t ws_bytes, cudaStream_t st);

size_t neuron_workspace_bytes(int L, int r, int d, int n_levels);
ziplm_status run_prune_neurons(const float* W, const float* H, int L, int r, int d,
                               float damp_frac, const int* levels, int n_levels, float* W_snap,
                               float* loss, float* base_loss, int* order, float* saliency,
                               int* layer_status, void* ws, size_t ws_bytes, cudaStream_t st);

// Neuron path with delayed rank-B updates (prune_lazy.cu); chosen by run_prune_neurons.
bool lazy_path_supported(int d);
size_t lazy_workspace_bytes(int L, int r, int d, int n_levels);
ziplm_status run_prune_lazy(const float* W, const float* H, int L, int r, int d, float damp_frac,
                            const int* levels, int n_levels, float* W_snap, float* loss,
                            float* base_loss, int* order, float* saliency, int* layer_status,
                            void* ws, size_t ws_bytes, cudaStream_t st);

size_t block_workspace_bytes(int L, int r, int d, int g, int n_levels);
ziplm_status run_prune_blocks(const float* W, const float* H, int L, int r, int d, int g,
                              float damp_frac, const int* levels, int n_levels, float* W_snap,
                              float* loss, float* base_loss, int* order, float* saliency,
                              int* layer_status, void* ws, size_t ws_bytes, cudaStream_t st);

// base_loss[l] = 1/2 tr(W[l] H[l] W[l]^T) = ||W X||_F^2; acc64 is an [L] float64 scratch.
ziplm_status run_base_loss(const float* W, const float* H, int L, int r, int d, double* acc64,
                           float* base_loss, cudaStream_t st);

// Tensor-core route of the Hessian (hessian_tc.cu) and the route choice (hessian.cu).
// token_major = false: X is [L, d, ldx], token index contiguous; true: X is [L, N, ldx], one
// token per row, feature index contiguous.
size_t hessian_tc_workspace_bytes(int L, int d, long long n_tokens, ziplm_dtype dt, bool token_major);
ziplm_status run_hessian_tc(float* H, const void* X, ziplm_dtype dt, bool token_major, int L, int d,
                            long long N, long long ldx, float alpha, float beta, void* ws,
                            size_t ws_bytes, cudaStream_t st);
size_t hessian_workspace_bytes(int L, int d, long long n_tokens, ziplm_dtype dt, bool token_major);
ziplm_status run_hessian(float* H, const void* X, ziplm_dtype dt, bool token_major, int L, int d,
                         long long N, long long ldx, float alpha, float beta, void* ws,
                         size_t ws_bytes, cudaStream_t st);

// Model reshaping (reshape.cu): survivors of a level, and column / row gathers by that list.
ziplm_status run_kept_structures(const int* order, int L, int G, int level, int* kept, int* bad,
                                 cudaStream_t st);
ziplm_status run_gather_columns(const float* M, long long ld, long long layer_stride, const int* kept,
                                int L, int rows, int G, int g, int level, float* out, cudaStream_t st);
ziplm_status run_gather_rows(const float* M, long long ld, long long layer_stride, const int* kept,
                             int L, int cols, int G, int g, int level, float* out, cudaStream_t st);

// Budgeted level selection (select.cu): one level per module under a run-time budget, K
// coefficient vectors per launch.
size_t select_workspace_bytes(int K, int n_mod, int n_buckets);
ziplm_status run_select_levels(const float* loss, const float* base_loss, const float* time,
                               const int* n_opt, int n_mod, int max_opt, const float* coef, int K,
                               double budget, int n_buckets, int* selected, double* cost, double* time_sum,
                               int* status, void* ws, size_t ws_bytes, cudaStream_t st);

size_t search_workspace_bytes(int S, int n_mod, int n_buckets);
ziplm_status run_search_levels(const float* loss, const float* base_loss, const float* time,
                               const int* n_opt, int n_mod, int max_opt, const float* objective,
                               const float* coef0, const double* budgets, int S, int n_buckets,
                               const unsigned char* mask, const float* values, int n_steps, int* best_sel,
                               float* best_coef, double* best_obj, int* n_accepted, int* status, void* ws,
                               size_t ws_bytes, cudaStream_t st);

}  // namespace ziplm
