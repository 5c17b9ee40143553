/*
 * ziplm.h -- C ABI of the layer-wise structured Optimal-Brain-Surgeon solver of ZipLM
 * (arXiv 2302.04089, Sec. 3.1, Algorithm 1) for NVIDIA B200 (sm_100a).
 *
 * Conventions shared by every entry point
 *   - "dev" pointers are CUDA device pointers of the current device, "host" pointers are
 *     ordinary host memory.  All matrices are dense row-major.
 *   - The caller owns every buffer.  The library allocates no device memory and keeps no state
 *     between calls, apart from the diagnostics at the end of this file, the stream pool of
 *     ziplm_prune_layers described next and the built-in scratch of
 *     ziplm_damped_inverse_noalloc.  Calls may be made from several host threads.
 *   - All work is ordered on `cuda_stream` (a cudaStream_t passed as void*, NULL = the default
 *     stream) and the call returns without synchronising: it starts after everything already
 *     enqueued there and the stream continues only when it is complete.  Buffers must stay alive
 *     until the stream has drained.  ziplm_prune_layers may run groups of layers concurrently on
 *     up to eight internal non-blocking streams (created once per device, on first use), forked
 *     from and joined back to `cuda_stream` with events.  Calls on different streams with
 *     disjoint output and workspace buffers are independent and may overlap on the device
 *     (inputs may be shared): enqueueing the next batch of layers on a second stream lets its
 *     tensor-core and float64 phases run under the greedy loop of the first; with several
 *     batches in flight keep groups x batches at eight or fewer (ZIPLM_OPT_LAYER_GROUPS).
 *   - The return value reports what the host can see when the work is enqueued (bad arguments,
 *     workspace too small, a failed launch).  Failures that depend on the data (a Hessian that
 *     is not positive definite, non-finite values) are written to `layer_status[l]` on the
 *     device; the outputs of such a layer are unspecified but in bounds and the other layers
 *     are unaffected.
 *   - There is no CPU fallback: without a CUDA device the compute entry points return
 *     ZIPLM_ERR_CUDA.
 *
 * Notation (the paper's): W is d_row x d_col, X is d_col x n_tokens (one calibration token per
 * column), H = 2 X X^T, a structure is `group_size` consecutive columns of W (1 = FFN neuron,
 * 64 = attention head), G = d_col / group_size structures per layer, L same-shape layers are
 * processed together because the method treats every layer independently (Sec. 3.2).
 */
#ifndef ZIPLM_H_
#define ZIPLM_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ZIPLM_OK = 0,
    ZIPLM_ERR_INVALID_ARG = 1, /* shape, pointer or level list rejected on the host            */
    ZIPLM_ERR_WORKSPACE = 2,   /* workspace pointer NULL / misaligned / smaller than required  */
    ZIPLM_ERR_NOT_PD = 3,      /* damped Hessian not positive definite (per layer)             */
    ZIPLM_ERR_NONFINITE = 4,   /* NaN or Inf met in H, W or a saliency (per layer)             */
    ZIPLM_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out                           */
    ZIPLM_ERR_CUDA = 6,        /* a CUDA runtime call or kernel launch failed                  */
    ZIPLM_ERR_UNSUPPORTED = 7  /* valid request outside what this build implements            */
} ziplm_status;

typedef enum { ZIPLM_F32 = 0, ZIPLM_BF16 = 1, ZIPLM_F16 = 2 } ziplm_dtype;

/* Human-readable name of a status code (static storage, never NULL). */
const char* ziplm_status_string(ziplm_status s);

/* ---------------------------------------------------------------------------------------------
 * Calibration Hessian (caption of Algorithm 1: H = 2 X X^T; "Saliency scores and weight update").
 *
 *   H[l] = beta * H[l] + alpha * X[l] X[l]^T        for l = 0 .. L-1
 *
 * alpha = 2 gives the paper's Hessian; beta = 1 adds one more batch of tokens to a running sum,
 * beta = 0 overwrites.  Products are accumulated in fp32; fp32 inputs keep fp32 accuracy (on the
 * tensor-core route every feature row is scaled by a power of two and split into two fp16 parts,
 * three exact partial products per product, about 21 significant bits), bf16 and fp16 inputs are multiplied exactly
 * (an fp16 or bf16 product has at most 22 significant bits).
 *
 *   H          dev, [L, d, d] fp32, in/out; full symmetric matrix on return
 *   X          dev, [L, d, ldx] of x_dtype, token index contiguous; only the first n_tokens
 *              entries of each row are read; not modified.  The base address must be 16-byte
 *              aligned and ldx * sizeof(element) a multiple of 16.
 *   ldx        row pitch of X in elements, >= n_tokens
 *   workspace  dev scratch of at least ziplm_hessian_workspace_bytes(...) bytes, 256-byte
 *              aligned; may be NULL when that size is 0
 *
 * Errors: ZIPLM_ERR_INVALID_ARG for L, d < 1, n_tokens < 0, ldx < n_tokens, a NULL pointer,
 * misaligned X or beta outside {0, 1}; ZIPLM_ERR_WORKSPACE; ZIPLM_ERR_CUDA.
 * n_tokens = 0 scales H by beta and returns.
 * Every wait inside the tensor-core kernel is bounded.  Should one run out (it cannot on a healthy
 * device), the call has no status output of its own: H[l][0][0] of every layer is NaN on return,
 * so that ziplm_damped_inverse or ziplm_prune_layers on that H reports ZIPLM_ERR_NONFINITE for
 * every layer.  The same holds for ziplm_hessian_accumulate_tokens.
 */
size_t ziplm_hessian_workspace_bytes(int L, int d, long long n_tokens, ziplm_dtype x_dtype);

ziplm_status ziplm_hessian_accumulate(float* H, const void* X, ziplm_dtype x_dtype, int L, int d,
                                      long long n_tokens, long long ldx, float alpha, float beta,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Calibration Hessian from token-major activations, batch by batch (caption of Algorithm 1:
 * H = 2 X X^T; Sec. 3.1: X are the layer inputs collected on calibration data, which a forward
 * pass emits one token per row).
 *
 *   H[l] = beta * H[l] + alpha * A[l]^T A[l]        for l = 0 .. L-1
 *
 * A[l] is the n_tokens x d matrix whose rows are the layer's input vectors, i.e. A[l] = X[l]^T in
 * the paper's notation, so the result is the same matrix ziplm_hessian_accumulate computes from
 * X[l].  Calling it once per calibration batch with beta = 1 (beta = 0 on the first batch, or on a
 * zeroed H) builds the Hessian of the whole calibration set without ever holding all activations.
 * Arithmetic and accuracy are those of ziplm_hessian_accumulate: a pre-pass brings the batch into
 * the token-contiguous layout (for fp32 together with the fp16 split) and the same tensor-core
 * product kernel runs on it.
 *
 *   H          dev, [L, d, d] fp32, in/out; full symmetric matrix on return
 *   A          dev, [L, n_tokens, lda] of a_dtype, feature index contiguous; only the first d
 *              entries of each row are read; not modified.  Aligned to its element size.
 *   lda        row pitch of A in elements, >= d
 *   workspace  dev scratch of at least ziplm_hessian_tokens_workspace_bytes(...) bytes, 256-byte
 *              aligned; may be NULL when that size is 0
 *
 * Errors: ZIPLM_ERR_INVALID_ARG for L, d < 1, n_tokens < 0, lda < d, a NULL or misaligned
 * pointer or beta outside {0, 1}; ZIPLM_ERR_WORKSPACE; ZIPLM_ERR_CUDA.
 * n_tokens = 0 scales H by beta and returns.
 */
size_t ziplm_hessian_tokens_workspace_bytes(int L, int d, long long n_tokens, ziplm_dtype a_dtype);

ziplm_status ziplm_hessian_accumulate_tokens(float* H, const void* A, ziplm_dtype a_dtype, int L,
                                             int d, long long n_tokens, long long lda, float alpha,
                                             float beta, void* workspace, size_t workspace_bytes,
                                             void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Damped inverse (caption of Algorithm 1: H^-1 = (2 X X^T + lambda I)^-1).
 *
 *   lambda[l] = damp_frac * mean(diag H[l]);   Hinv[l] = (H[l] + lambda[l] I)^-1
 *
 * computed in float64 through a blocked Cholesky factorisation H + lambda I = C C^T, the inverse
 * of the triangular factor and the product C^-T C^-1.  This is the first stage of
 * ziplm_prune_layers, exported so that it can be used and checked on its own.
 *
 *   H             dev, [L, d, d] fp32, symmetric (only the lower triangle is read); not modified
 *   Hinv          dev, [L, d, d] fp64, full symmetric matrix on return
 *   layer_status  dev, [L] int: ZIPLM_OK, ZIPLM_ERR_NOT_PD (a pivot <= 0 or mean(diag) <= 0
 *                 with damp_frac > 0) or ZIPLM_ERR_NONFINITE
 *   workspace     dev scratch >= ziplm_inverse_workspace_bytes(L, d), 256-byte aligned
 */
size_t ziplm_inverse_workspace_bytes(int L, int d);

ziplm_status ziplm_damped_inverse(const float* H, int L, int d, float damp_frac, double* Hinv,
                                  int* layer_status, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Damped inverse without a workspace argument (the paper has no counterpart; this is a
 * convenience of the library).
 *
 * Some callers cannot obtain device memory at the point where they need the inverse: code that
 * runs inside a framework hook or a plugin callback where the allocator must not be entered, a
 * process whose whole device budget was handed to another allocator up front, or a real-time
 * loop where a cudaMalloc (which may synchronise the device) is not acceptable.  For them this
 * entry point computes exactly what ziplm_damped_inverse computes, with the same kernels, but
 * takes its scratch from a 12 MiB array that is compiled into the library.  It calls neither
 * cudaMalloc nor cudaFree nor any routine that allocates.
 *
 *   H, Hinv, layer_status, damp_frac, cuda_stream   as for ziplm_damped_inverse; the caller still
 *                 provides the input and both outputs.
 *
 * Limit: the request must satisfy ziplm_inverse_workspace_bytes(L, d) <= 12 MiB (12582912), e.g.
 * one layer up to d = 704, four layers of d = 320, sixteen layers of d = 128; anything larger
 * returns ZIPLM_ERR_UNSUPPORTED and does nothing.
 * Cost: every GPU that loads the library holds the 12 MiB until the process exits.
 * First call on a device: it looks up the device address of the built-in array (with that
 * device current) and remembers it; make this first call outside any stream capture.
 * Sharing: all calls on a device use the same array, and it keeps whatever the last call left
 * there.  No call relies on those leftovers (every region is rewritten before it is read), but
 * two calls whose kernels overlap on the GPU -- different streams, or different host threads
 * without ordering -- race on it and give wrong results: order such calls on one stream or with
 * events.
 * Errors: ZIPLM_ERR_INVALID_ARG as for ziplm_damped_inverse; ZIPLM_ERR_UNSUPPORTED beyond the
 * limit; ZIPLM_ERR_CUDA if the address lookup or a launch fails.
 */
ziplm_status ziplm_damped_inverse_noalloc(const float* H, int L, int d, float damp_frac,
                                          double* Hinv, int* layer_status, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Greedy structured pruning of L same-shape layers (Algorithm 1; Eq. 2, Eq. 3, Eq. 4) with a
 * snapshot at every requested level (the per-layer database of Sec. 3.2).
 *
 * For every layer: dampen and invert H as above; then, until min(levels) structures remain,
 * score every remaining structure S with
 *     rho_S = sum_i W[i,S] ((H^-1)[S,S])^-1 W[i,S]^T                           (Eq. 2)
 * remove the structure with the smallest rho (ties: lowest structure index), apply
 *     W <- W - W[:,S] ((H^-1)[S,S])^-1 (H^-1)[S,:]                             (Eq. 3)
 *     H^-1 <- H^-1 - (H^-1)[:,S] ((H^-1)[S,S])^-1 (H^-1)[S,:]                  (Eq. 4)
 * and, whenever the number of remaining structures equals an entry of `levels`, store the
 * weights with the removed columns set to exactly zero (last line of Algorithm 1) together with
 * the reconstruction loss of Eq. 1.
 *
 *   W            dev, [L, d_row, d_col] fp32; not modified
 *   H            dev, [L, d_col, d_col] fp32, the UNDAMPED 2 X X^T, symmetric; not modified;
 *                16-byte aligned (ZIPLM_ERR_INVALID_ARG otherwise)
 *   group_size   columns per structure; d_col % group_size == 0; 1 <= group_size <= 128
 *   damp_frac    lambda = damp_frac * mean(diag H[l]); >= 0
 *   levels       HOST, [n_levels] numbers of REMAINING structures, strictly decreasing, each in
 *                [0, G]; level 0 removes the whole module, level G is the unpruned layer
 *   W_snap       dev, [L, n_levels, d_row, d_col] fp32
 *   loss         dev, [L, n_levels] fp32:  ||(W - W_snap) X||_F^2  (no damping term)
 *   base_loss    dev, [L] fp32:  ||W X||_F^2 ; may be NULL
 *   order        dev, [L, G] int: structure removed at step t, -1 for steps that did not run
 *   saliency     dev, [L, G] fp32: rho of the structure removed at step t (0 past the end);
 *                may be NULL
 *   layer_status dev, [L] int, per-layer ziplm_status
 *   workspace    dev scratch >= ziplm_prune_workspace_bytes(...), 256-byte aligned
 *
 * The loss is evaluated through the identity  loss + lambda/2 ||W - W_snap||_F^2 = 1/2 * (sum of
 * the rho of the structures removed so far), which holds because every rho is twice the increase
 * of the damped least-squares objective; it needs no extra pass over H.
 *
 * Errors: ZIPLM_ERR_INVALID_ARG (shapes, NULL pointers, levels not strictly decreasing or out
 * of range, damp_frac < 0 or not finite), ZIPLM_ERR_UNSUPPORTED (group_size > 128),
 * ZIPLM_ERR_WORKSPACE, ZIPLM_ERR_CUDA.
 */
size_t ziplm_prune_workspace_bytes(int L, int d_row, int d_col, int group_size, int n_levels);

ziplm_status ziplm_prune_layers(const float* W, const float* H, int L, int d_row, int d_col,
                                int group_size, float damp_frac, const int* levels, int n_levels,
                                float* W_snap, float* loss, float* base_loss, int* order,
                                float* saliency, int* layer_status, void* workspace,
                                size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Model reshaping (Sec. 3.1, "Pruned structures": once the columns of the removed structures are
 * zero, the matching rows of the previous layer can be removed without any output change).
 *
 * A snapshot of ziplm_prune_layers keeps the original shape with zero columns.  These three calls
 * turn a level of the database into the smaller dense matrices a runtime executes:
 *
 *   ziplm_kept_structures   kept[l] = the `level` structures of layer l that order[l][0 .. G-level)
 *                           does not list, ascending
 *   ziplm_gather_columns    out[l][i][k*g + c] = M[l][i][kept[l][k]*g + c]     (this layer: FC2,
 *                           attention out-projection)
 *   ziplm_gather_rows       out[l][k*g + c][j] = M[l][kept[l][k]*g + c][j]     (previous layer: FC1
 *                           weight and, as a one-column matrix, its bias; the Q, K, V rows of a head)
 *
 * All three only move data; the outputs are bit-exact copies.
 *
 *   order         dev, [L, G] int, as written by ziplm_prune_layers; only the first G - level
 *                 entries of a row are read
 *   kept          dev, [L, level] int
 *   layer_status  dev, [L] int: ZIPLM_OK, or ZIPLM_ERR_INVALID_ARG when those entries are not
 *                 distinct indices in [0, G) (kept[l] is then unspecified)
 *   M             dev, fp32; layer l starts at M + l * layer_stride (elements), row pitch ld
 *                 (elements).  To read level slot s of W_snap [L, n_levels, d_row, d_col] pass
 *                 W_snap + s * d_row * d_col, ld = d_col, layer_stride = n_levels * d_row * d_col.
 *   rows / cols   number of rows of M (columns gather) / of columns of M that are copied (rows
 *                 gather)
 *   out           dev, dense [L, rows, level * g] (columns) or [L, level * g, cols] (rows)
 *
 * An entry of `kept` outside [0, G) produces zeros in the gathers.  level = 0 writes nothing.
 * Errors: ZIPLM_ERR_INVALID_ARG (sizes, NULL pointers, ld smaller than the matrix width),
 * ZIPLM_ERR_UNSUPPORTED (G beyond 1.6 million structures, rows beyond 1048560), ZIPLM_ERR_CUDA.
 */
ziplm_status ziplm_kept_structures(const int* order, int L, int G, int level, int* kept,
                                   int* layer_status, void* cuda_stream);

ziplm_status ziplm_gather_columns(const float* M, long long ld, long long layer_stride,
                                  const int* kept, int L, int rows, int G, int group_size, int level,
                                  float* out, void* cuda_stream);

ziplm_status ziplm_gather_rows(const float* M, long long ld, long long layer_stride, const int* kept,
                               int L, int cols, int G, int group_size, int level, float* out,
                               void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Budgeted choice of one database level per module (Sec. 3.2, "Runtime awareness", "Finding the
 * optimal sparsity configuration", "Structured SPDY search").
 *
 * For module m (an attention block or a fully-connected block) the database holds n_options[m]
 * levels; level s costs time[m][s] in the latency table and has the prior
 *     p[m][s] = loss[m][s] / base_loss[m]          (relative layer-wise squared error; 1 for a
 *                                                   dropped module, 0 for the unpruned one)
 * taken directly from the outputs of ziplm_prune_layers.  For each of n_candidates sensitivity
 * vectors c[k] the call finds the levels that minimise  sum_m c[k][m] * p[m][s_m]  subject to
 * sum_m time[m][s_m] <= budget.  The search of the paper solves this once per mutated coefficient
 * vector (1000 steps), which is why candidates are batched.
 *
 * Time is discretised into n_buckets units of budget / n_buckets and every option is rounded UP
 * (units = ceil(time * n_buckets / budget) in float64), so the selection never exceeds the budget
 * in real time; it is optimal for the discretised problem.  Costs are float64 sums formed in
 * module order; ties go to the lowest option index.
 *
 *   loss, time        dev, [n_modules, max_options] fp32; entries s >= n_options[m] are ignored
 *   base_loss         dev, [n_modules] fp32, > 0
 *   n_options         dev, [n_modules] int, each in [1, max_options]
 *   coef              dev, [n_candidates, n_modules] fp32
 *   budget            total run time allowed, same unit as `time`, > 0
 *   selected          dev, [n_candidates, n_modules] int: chosen option per module (-1 on failure)
 *   cost              dev, [n_candidates] fp64: the minimum
 *   time_sum          dev, [n_candidates] fp64: sum of the chosen options' times
 *   candidate_status  dev, [n_candidates] int: ZIPLM_OK; ZIPLM_ERR_INVALID_ARG when even the
 *                     fastest options exceed the budget; ZIPLM_ERR_NONFINITE for NaN inputs
 *   workspace         dev scratch >= ziplm_select_workspace_bytes(...), 256-byte aligned
 *
 * Errors: ZIPLM_ERR_INVALID_ARG; ZIPLM_ERR_UNSUPPORTED (max_options > 255 or n_buckets > 12000);
 * ZIPLM_ERR_WORKSPACE; ZIPLM_ERR_CUDA.
 */
size_t ziplm_select_workspace_bytes(int n_candidates, int n_modules, int n_buckets);

ziplm_status ziplm_select_levels(const float* loss, const float* base_loss, const float* time,
                                 const int* n_options, int n_modules, int max_options,
                                 const float* coef, int n_candidates, double budget, int n_buckets,
                                 int* selected, double* cost, double* time_sum, int* candidate_status,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Mutation search over the sensitivity coefficients (Sec. 3.2, "Structured SPDY search": a fixed
 * number of steps -- 1000 in the paper -- each mutating in expectation 10 % of the coefficients).
 *
 * For each of n_searches run-time budgets (speedup targets), starting from coef0[k]: step t
 * replaces the coefficients m with mask[k][t][m] != 0 by values[k][t][m], solves the selection
 * problem of ziplm_select_levels for the mutated vector, scores the selection, and keeps the
 * mutated vector when its score is strictly lower than the best so far (the unmutated coef0 is
 * scored first).  The random draws are the caller's: marks drawn with probability 0.1 per
 * coefficient give the paper's mutation rate.
 *
 * Score: the paper scores a candidate by the calibration loss of the stitched model, which only
 * the caller's model can give.  Here the score of a selection is sum_m objective[m][s_m], a
 * separable stand-in (for instance priors measured against a held-out calibration set); a caller
 * with a model uses ziplm_select_levels on a batch of mutated vectors and scores them itself.
 * Every selection the search evaluates meets its budget, as in the paper.
 *
 *   loss, base_loss, time, n_options, n_modules, max_options, n_buckets
 *                    as for ziplm_select_levels
 *   objective        dev, [n_modules, max_options] fp32
 *   coef0            dev, [n_searches, n_modules] fp32
 *   budgets          dev, [n_searches] fp64, each > 0
 *   mask             dev, [n_searches, n_steps, n_modules] bytes
 *   values           dev, [n_searches, n_steps, n_modules] fp32
 *   best_selected    dev, [n_searches, n_modules] int (-1 if no evaluated selection met the budget)
 *   best_coef        dev, [n_searches, n_modules] fp32: the coefficients that produced it
 *   best_objective   dev, [n_searches] fp64 (float64 sum in module order; inf if none)
 *   n_accepted       dev, [n_searches] int: mutations that were kept
 *   search_status    dev, [n_searches] int: ZIPLM_OK, ZIPLM_ERR_INVALID_ARG (budget below the
 *                    fastest configuration), ZIPLM_ERR_NONFINITE
 *   workspace        dev scratch >= ziplm_search_workspace_bytes(...), 256-byte aligned
 *
 * One thread block runs one whole search, so the call is efficient when many targets are searched
 * together.  Errors: as ziplm_select_levels; ZIPLM_ERR_UNSUPPORTED also for n_modules > 512.
 */
size_t ziplm_search_workspace_bytes(int n_searches, int n_modules, int n_buckets);

ziplm_status ziplm_search_levels(const float* loss, const float* base_loss, const float* time,
                                 const int* n_options, int n_modules, int max_options,
                                 const float* objective, const float* coef0, const double* budgets,
                                 int n_searches, int n_buckets, const unsigned char* mask,
                                 const float* values, int n_steps, int* best_selected, float* best_coef,
                                 double* best_objective, int* n_accepted, int* search_status,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Diagnostics (no counterpart in the paper): options, a launch counter and optional per-phase
 * timing.  This is the only process-wide state the library keeps besides an internal pool of
 * streams (see ziplm_prune_layers); no environment variable is read.
 *
 * ziplm_set_option         sets a process-wide option that later calls read when they start; every
 *                          option defaults to 0.  ZIPLM_ERR_INVALID_ARG for an unknown option or a
 *                          value outside its range.  Results never depend on an option beyond
 *                          rounding (every variant passes the same parity tests).
 *     ZIPLM_OPT_NEURON_PATH       0: delayed rank-32 updates where the shape allows them
 *                                 (d_col % 4 == 0, d_col <= 6144); 1: per-step streaming update.
 *     ZIPLM_OPT_LAYER_GROUPS      0: default (6); 1..8: number of layer groups that
 *                                 ziplm_prune_layers runs on internal streams (1 = none).
 *     ZIPLM_OPT_FORCE_BLOCK_PATH  1: group_size 1 takes the general block path (float64 state).
 *                                 The only option ziplm_prune_workspace_bytes depends on: set it
 *                                 before the query and leave it until the call.
 *     ZIPLM_OPT_HESSIAN_ROUTE     0: tensor cores from 32 tokens on; 1: CUDA-core kernel always.
 *     ZIPLM_OPT_SPIN_LIMIT        0: default; n > 0: poll limit of the Hessian kernel's wait for a
 *                                 free pipeline stage (tests make a bounded wait run out with it;
 *                                 see ziplm_hessian_accumulate for how that is reported).
 *     ZIPLM_OPT_COMPACT_EVERY_BLOCK  0: the delayed-update neuron path leaves removed positions in
 *                                 place for a few blocks (dense tensor-core update of H^-1 and Q)
 *                                 and squeezes them out when 128 of them, or a sixteenth of all
 *                                 positions, have gathered; 1: squeezes them out after every
 *                                 block (gathering CUDA-core update only).
 * ziplm_get_option         current value of an option.
 * ziplm_launch_count       kernels launched by this library since it was loaded.
 * ziplm_profile_begin      from now on every phase of every call is bracketed by a pair of CUDA
 *                          events on the caller's stream (process-wide switch, not re-entrant;
 *                          costs a few microseconds per phase, so timed runs leave it off).
 * ziplm_profile_end        switches timing off, waits for the recorded events and returns, per
 *                          phase, the summed milliseconds (host [n_phases] double, may be NULL)
 *                          and the number of bracketed spans (host [n_phases], may be NULL).
 * ziplm_profile_phase_count / ziplm_profile_phase_name   enumerate the phases ("hessian",
 *                          "inverse", "init", "prep", "update", "snapshot", "lazy_steps", ...).
 */
typedef enum {
    ZIPLM_OPT_NEURON_PATH = 0,
    ZIPLM_OPT_LAYER_GROUPS = 1,
    ZIPLM_OPT_FORCE_BLOCK_PATH = 2,
    ZIPLM_OPT_HESSIAN_ROUTE = 3,
    ZIPLM_OPT_SPIN_LIMIT = 4,
    ZIPLM_OPT_COMPACT_EVERY_BLOCK = 5,
    ZIPLM_OPT_COUNT = 6
} ziplm_option;
ziplm_status ziplm_set_option(ziplm_option option, int value);
int ziplm_get_option(ziplm_option option);
long long ziplm_launch_count(void);
ziplm_status ziplm_profile_begin(void);
ziplm_status ziplm_profile_end(double* phase_ms, long long* phase_spans, int n_phases);
int ziplm_profile_phase_count(void);
const char* ziplm_profile_phase_name(int phase);

#ifdef __cplusplus
}
#endif
#endif /* ZIPLM_H_ */
