// Host-only entry points: version, status names, workspace sizes.
#include "common.cuh"

namespace tppo {
size_t egae_workspace_bytes(int64_t N);
size_t select_workspace_bytes(int64_t N);
size_t policy_workspace_bytes(int64_t R, int64_t n_max);
size_t value_workspace_bytes();
size_t lmhead_workspace_bytes(int64_t M, int32_t K, int32_t V);
}  // namespace tppo

// Test hooks (see tppo_test_hooks in the header): read by the launchers of the two look-back kernels.
namespace tppo {
static int32_t g_test_polls = -1;
static int32_t g_test_no_publish = 0;
uint32_t test_spin_limit(uint32_t normal) {
    const int32_t p = __atomic_load_n(&g_test_polls, __ATOMIC_RELAXED);
    return p < 0 ? normal : uint32_t(p);
}
int32_t test_no_publish() { return __atomic_load_n(&g_test_no_publish, __ATOMIC_RELAXED); }
}  // namespace tppo

TPPO_API void tppo_test_hooks(int32_t lookback_polls, int32_t no_publish) {
    __atomic_store_n(&tppo::g_test_polls, lookback_polls, __ATOMIC_RELAXED);
    __atomic_store_n(&tppo::g_test_no_publish, no_publish ? 1 : 0, __ATOMIC_RELAXED);
}

TPPO_API int tppo_version(void) { return 200; }

TPPO_API const char* tppo_status_string(int status) {
    switch (status) {
        case TPPO_OK: return "ok";
        case TPPO_ERR_INVALID_ARG: return "invalid argument";
        case TPPO_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case TPPO_ERR_UNSUPPORTED: return "unsupported";
        case TPPO_ERR_CUDA: return "CUDA runtime error";
        case TPPO_ERR_TOO_LARGE: return "problem larger than the built-in capacity of this entry point";
        default: return "unknown status";
    }
}

// N doubles as the number of logits rows R for TPPO_OP_POLICY_LOSS and as M for TPPO_OP_LMHEAD
// (B then carries K).
TPPO_API size_t tppo_workspace_bytes(int op, int64_t N, int32_t B, int64_t n_max, int32_t V) {
    if (N < 0 || n_max < 0) return 0;
    switch (op) {
        case TPPO_OP_EGAE: return tppo::egae_workspace_bytes(N);
        case TPPO_OP_SELECT_TOKENS: return tppo::select_workspace_bytes(N);
        case TPPO_OP_POLICY_LOSS: return tppo::policy_workspace_bytes(N, n_max);
        case TPPO_OP_VALUE_LOSS: return tppo::value_workspace_bytes();
        case TPPO_OP_LMHEAD: return tppo::lmhead_workspace_bytes(N, B, V);
        default: return 0;
    }
}
