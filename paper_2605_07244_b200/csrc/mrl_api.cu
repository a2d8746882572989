// Host-only entry points: workspace sizing, status names, version.
#include "mrl_common.cuh"

size_t mrl_policy_loss_workspace_bytes(long long N, int S);
size_t mrl_fused_lmhead_workspace_bytes(long long N, int V, int H, int S);
size_t mrl_thl_workspace_bytes(long long total_words);

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
    case MRL_WS_THL_WORD_ALIGN:
      return mrl_thl_workspace_bytes(N);
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
    case MRL_ERR_STATIC_SCRATCH_TOO_SMALL: return "MRL_ERR_STATIC_SCRATCH_TOO_SMALL";
    default: return "MRL_ERR_UNKNOWN";
  }
}

extern "C" int mrl_version(void) { return MRL_VERSION; }

namespace {
void** g_prof_start = nullptr;
void** g_prof_stop = nullptr;
int g_prof_n = 0;
long long g_prof_i = 0;
const char* g_prof_last = "";
}  // namespace

extern "C" const char* mrl_profile_last_kernel(void) { return g_prof_last; }

extern "C" int mrl_profile_dominant_kernel(void** start_events, void** stop_events, int32_t n) {
  if (n < 0) return MRL_ERR_INVALID_ARG;
  if (n == 0 || start_events == nullptr || stop_events == nullptr) {
    g_prof_start = g_prof_stop = nullptr;
    g_prof_n = 0;
  } else {
    g_prof_start = start_events;
    g_prof_stop = stop_events;
    g_prof_n = n;
  }
  g_prof_i = 0;
  return MRL_OK;
}

void mrl_profile_before(cudaStream_t st, const char* kernel_name) {
  if (g_prof_n > 0) g_prof_last = kernel_name;
  if (g_prof_n > 0) cudaEventRecord(static_cast<cudaEvent_t>(g_prof_start[g_prof_i % g_prof_n]), st);
}

void mrl_profile_after(cudaStream_t st) {
  if (g_prof_n > 0) {
    cudaEventRecord(static_cast<cudaEvent_t>(g_prof_stop[g_prof_i % g_prof_n]), st);
    ++g_prof_i;
  }
}
