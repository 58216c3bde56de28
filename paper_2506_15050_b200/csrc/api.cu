// Host-only entry points: version, status names, workspace sizes.
#include "common.cuh"

namespace tppo {
size_t egae_workspace_bytes(int64_t N);
size_t select_workspace_bytes(int64_t N);
size_t policy_workspace_bytes(int64_t R, int64_t n_max);
size_t value_workspace_bytes();
size_t lmhead_workspace_bytes(int64_t M, int32_t K, int32_t V);
}  // namespace tppo

TPPO_API int tppo_version(void) { return 100; }

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
