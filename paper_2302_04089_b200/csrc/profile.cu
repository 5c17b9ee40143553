// Diagnostics: launch counter and optional per-phase CUDA-event timing.  Off by default; when
// switched on, every phase of the following calls is bracketed by a pair of events on the
// caller's stream, which costs a little time between kernels but no device memory.
#include <atomic>
#include <mutex>
#include <vector>

#include "common.cuh"

namespace ziplm {

std::atomic<long long> g_launches{0};

static std::atomic<int> g_options[ZIPLM_OPT_COUNT];

int option_value(int option) {
    return (option >= 0 && option < ZIPLM_OPT_COUNT) ? g_options[option].load(std::memory_order_relaxed) : 0;
}

namespace {
struct Span { int phase; cudaEvent_t a, b; };
std::mutex g_mu;
bool g_on = false;
std::vector<Span> g_spans;
const char* kPhaseNames[PH_COUNT] = {"hessian", "inverse", "init", "prep", "update", "snapshot",
                                     "block_score", "block_update", "lazy_steps", "lazy_update_aq",
                                     "lazy_update_w", "inverse_products", "inverse_leaves",
                                     "inverse_lauum", "lazy_refresh"};
}  // namespace

PhaseScope::PhaseScope(int phase, cudaStream_t st) : st_(st), idx_(-1) {
    if (!g_on) return;
    std::lock_guard<std::mutex> lk(g_mu);
    Span s;
    s.phase = phase;
    if (cudaEventCreate(&s.a) != cudaSuccess) return;
    if (cudaEventCreate(&s.b) != cudaSuccess) { cudaEventDestroy(s.a); return; }
    cudaEventRecord(s.a, st);
    g_spans.push_back(s);
    idx_ = (int)g_spans.size() - 1;
}

PhaseScope::~PhaseScope() {
    if (idx_ < 0) return;
    std::lock_guard<std::mutex> lk(g_mu);
    cudaEventRecord(g_spans[idx_].b, st_);
}

}  // namespace ziplm

using namespace ziplm;

extern "C" {

long long ziplm_launch_count(void) { return g_launches.load(); }

ziplm_status ziplm_set_option(ziplm_option option, int value) {
    if (option < 0 || option >= ZIPLM_OPT_COUNT || value < 0) return ZIPLM_ERR_INVALID_ARG;
    if ((option == ZIPLM_OPT_NEURON_PATH || option == ZIPLM_OPT_FORCE_BLOCK_PATH ||
         option == ZIPLM_OPT_HESSIAN_ROUTE || option == ZIPLM_OPT_COMPACT_EVERY_BLOCK) && value > 1)
        return ZIPLM_ERR_INVALID_ARG;
    if (option == ZIPLM_OPT_LAYER_GROUPS && value > 8) return ZIPLM_ERR_INVALID_ARG;
    ziplm::g_options[option].store(value, std::memory_order_relaxed);
    return ZIPLM_OK;
}

int ziplm_get_option(ziplm_option option) { return ziplm::option_value((int)option); }

int ziplm_profile_phase_count(void) { return PH_COUNT; }

const char* ziplm_profile_phase_name(int phase) {
    return (phase >= 0 && phase < PH_COUNT) ? kPhaseNames[phase] : "?";
}

ziplm_status ziplm_profile_begin(void) {
    std::lock_guard<std::mutex> lk(g_mu);
    for (auto& s : g_spans) { cudaEventDestroy(s.a); cudaEventDestroy(s.b); }
    g_spans.clear();
    g_on = true;
    return ZIPLM_OK;
}

ziplm_status ziplm_profile_end(double* phase_ms, long long* phase_spans, int n_phases) {
    std::lock_guard<std::mutex> lk(g_mu);
    g_on = false;
    for (int i = 0; i < n_phases; ++i) {
        if (phase_ms) phase_ms[i] = 0.0;
        if (phase_spans) phase_spans[i] = 0;
    }
    ziplm_status rc = ZIPLM_OK;
    for (auto& s : g_spans) {
        float ms = 0.f;
        if (cudaEventSynchronize(s.b) != cudaSuccess ||
            cudaEventElapsedTime(&ms, s.a, s.b) != cudaSuccess) {
            rc = ZIPLM_ERR_CUDA;
        } else if (s.phase < n_phases) {
            if (phase_ms) phase_ms[s.phase] += (double)ms;
            if (phase_spans) phase_spans[s.phase] += 1;
        }
        cudaEventDestroy(s.a);
        cudaEventDestroy(s.b);
    }
    g_spans.clear();
    return rc;
}

}  // extern "C"
