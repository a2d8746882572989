// Host-only entry points: workspace sizing, status names, version.
#include "mrl_common.cuh"

size_t mrl_policy_loss_workspace_bytes(long long N, int S);
size_t mrl_fused_lmhead_workspace_bytes(long long N, int V, int H, int S);

extern "C" size_t mrl_workspace_bytes(int32_t which, int64_t N, int32_t V, int32_t H, int32_t dtype, int32_t S) {
  (void)dtype;
  if (N < 0 || S < 0) return 0;
  switch (which) {
    case MRL_WS_TOKEN_LOGPROBS:
      return 0;
    case MRL_WS_POLICY_LOSS:
      return mrl_policy_loss_workspace_bytes(N, S);
    case MRL_WS_FUSED_LMHEAD:
      return mrl_fused_lmhead_workspace_bytes(N, V, H, S);
    default:
      return 0;
  }
}

extern "C" const char* mrl_status_string(int code) {
  switch (code) {
    case MRL_OK: return "MRL_OK";
    case MRL_ERR_INVALID_ARG: return "MRL_ERR_INVALID_ARG";
    case MRL_ERR_BAD_TOKEN_ID: return "MRL_ERR_BAD_TOKEN_ID";
    case MRL_ERR_UNSUPPORTED_DTYPE: return "MRL_ERR_UNSUPPORTED_DTYPE";
    case MRL_ERR_WORKSPACE_TOO_SMALL: return "MRL_ERR_WORKSPACE_TOO_SMALL";
    case MRL_ERR_CUDA: return "MRL_ERR_CUDA";
    case MRL_ERR_TIMEOUT: return "MRL_ERR_TIMEOUT";
    case MRL_ERR_UNSUPPORTED_SHAPE: return "MRL_ERR_UNSUPPORTED_SHAPE";
    default: return "MRL_ERR_UNKNOWN";
  }
}

extern "C" int mrl_version(void) { return MRL_VERSION; }
