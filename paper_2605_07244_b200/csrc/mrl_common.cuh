// Shared device/host helpers of libmrl (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "mrl.h"

#define MRL_LOG2E 1.4426950408889634f
// The base-2 domain of the running sums is x = z * MRL_LOG2E with the FLOAT constant above, so the way back to nats
// divides by that float: 1 / float(log2 e) = MRL_NAT_HI + MRL_NAT_LO (to 2e-16).  Multiplying by ln 2 instead is 1.06e-8
// off, a bias of 1e-7 in every log-sum-exp, which a response-level ratio adds up over the tokens of a response.
#define MRL_NAT_HI 0.6931471824645996f
#define MRL_NAT_LO 7.348693209507928e-09f
#define MRL_NAT_F64 0.6931471898132927

#define MRL_CUDA_OK(expr)                       \
  do {                                          \
    cudaError_t e__ = (expr);                   \
    if (e__ != cudaSuccess) return MRL_ERR_CUDA; \
  } while (0)

static inline size_t mrl_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Runs `set` (the cudaFuncSetAttribute calls of one kernel) once per device instead of on every launch: `done` holds
// one bit per device ordinal.  Two threads that race here both set the same attributes, which is harmless.
template <typename F>
static inline int mrl_once_per_device(std::atomic<uint64_t>& done, F set) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MRL_ERR_CUDA;
  const uint64_t bit = 1ull << (dev & 63);
  if (done.load(std::memory_order_acquire) & bit) return MRL_OK;
  if (set() != cudaSuccess) return MRL_ERR_CUDA;
  done.fetch_or(bit, std::memory_order_release);
  return MRL_OK;
}

// Carves sub-buffers out of the caller's workspace; every piece is 256-byte aligned.
struct MrlCarver {
  char* base;
  size_t off;
  explicit MrlCarver(void* p) : base(static_cast<char*>(p)), off(0) {}
  template <typename T>
  T* take(size_t n) {
    T* p = reinterpret_cast<T*>(base + off);
    off += mrl_align_up(n * sizeof(T), 256);
    return p;
  }
};

// Per-row scratch of the loss passes (carved from the caller's workspace) and the host steps around the row kernels.
struct MrlLossWs {
  float *rowA, *rowcu, *rowcn;        // A_t, c_t u_t, cn_t
  float* rowck;                       // beta c_t of the KL term (0 when the term is off)
  float* cscale;                      // [1] factor still to be applied to rowcu and rowck (1, or the token-mean 1 / D)
  float *row_m2, *row_s, *row_zt;     // base-2 running max, sum of 2^(x - max), target logit
  double *pg_term, *nll_term, *kl_term;  // per-row terms (response-level ratio only)
  double* partials;                      // [ceil(N / 256)][6] block sums of the terms and the row statistics
  uint8_t* rowstat;                   // MRL_ROW_* bits
  int32_t* seq_cnt;
  unsigned long long* totals;         // [0] valid tokens, [1] bad ids, [2] / [3] tickets of the last-block sums
  size_t bytes;
};
#define MRL_ROW_VALID 1
#define MRL_ROW_CLIPPED 2
#define MRL_ROW_READ 4
size_t mrl_policy_loss_workspace_bytes(long long N, int S);
int mrl_rows_prepare(void* workspace, long long N, int V, int S, const int32_t* ids, const uint8_t* mask,
                     const int32_t* cu_seqlens, const float* adv_seq, const float* tok_weight,
                     const float* nll_weight, const mrl_loss_params* lp, int32_t* status, cudaStream_t st,
                     MrlLossWs* out);
int mrl_rows_finish(const MrlLossWs& w, long long N, const float* logp_old, const mrl_loss_params* lp, float* logp,
                    float* loss, int64_t* stats, cudaStream_t st);

int mrl_rows_finish_sequence(const MrlLossWs& w, long long N, int S, const int32_t* cu_seqlens, const float* adv_seq,
                             const float* logp_old, const float* nll_weight, const mrl_loss_params* lp, float* logp,
                             float* loss, int64_t* stats, float* g_out, float* lse2_out, cudaStream_t st);

// The KL term's arguments are consistent (Eq. (1), beta R(theta)).
static inline bool mrl_kl_args_ok(const mrl_loss_params* lp) {
  if (lp->logp_ref == nullptr) return true;
  if (lp->kl_loss == nullptr) return false;
  return lp->kl_estimator == MRL_KL_K1 || lp->kl_estimator == MRL_KL_K2 || lp->kl_estimator == MRL_KL_K3;
}

// Benchmark instrumentation (mrl_profile_dominant_kernel): event pairs recorded around dominant kernels.
void mrl_profile_before(cudaStream_t st, const char* kernel_name);  // a static string naming the launch
void mrl_profile_after(cudaStream_t st);

namespace mrl {

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// base-2 log-sum-exp (in units of MRL_LOG2E) -> nats
__device__ __forceinline__ float lse2_to_nats(float lse2) { return fmaf(lse2, MRL_NAT_HI, lse2 * MRL_NAT_LO); }

__device__ __forceinline__ float bf16lo_to_f32(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t packed) { return __uint_as_float(packed & 0xffff0000u); }

// round-to-nearest-even pack of two floats: low half = a, high half = b
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
  return r;
}

// Running log-sum-exp state in the base-2 domain: sum_i 2^(x_i - m), x = z * log2(e).
struct Lse2 {
  float m;  // running maximum of the scaled values (-inf when empty)
  float s;  // sum of 2^(x - m)
};

__device__ __forceinline__ Lse2 lse2_empty() { return Lse2{-INFINITY, 0.f}; }

__device__ __forceinline__ Lse2 lse2_merge(Lse2 a, Lse2 b) {
  float m = fmaxf(a.m, b.m);
  if (m == -INFINITY) return Lse2{m, 0.f};
  return Lse2{m, a.s * ex2_approx(a.m - m) + b.s * ex2_approx(b.m - m)};
}

__device__ __forceinline__ Lse2 lse2_warp_reduce(Lse2 v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Lse2 w;
    w.m = __shfl_xor_sync(0xffffffffu, v.m, o);
    w.s = __shfl_xor_sync(0xffffffffu, v.s, o);
    v = lse2_merge(v, w);
  }
  return v;
}

// Block-wide merge in a fixed order; every thread gets the result.  `scratch` holds 2*32 floats.
template <int kThreads>
__device__ __forceinline__ Lse2 lse2_block_reduce(Lse2 v, float* scratch) {
  constexpr int kWarps = kThreads / 32;
  v = lse2_warp_reduce(v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) {
    scratch[warp] = v.m;
    scratch[32 + warp] = v.s;
  }
  __syncthreads();
  Lse2 r = lse2_empty();
  if (lane < kWarps) r = Lse2{scratch[lane], scratch[32 + lane]};
  r = lse2_warp_reduce(r);
  __syncthreads();
  return r;
}

// Per-row scalar inputs of the loss and what the row contributes.
struct RowIn {
  float A;         // advantage of the row's sequence
  float cu;        // c_t * u_t
  float cn;        // NLL coefficient
  float logp_old;  // behaviour trace (ignored when has_old is false)
  bool has_old;
  float ck;        // beta c_t of the KL term; 0: term off
  float logp_ref;  // reference trace (read only when ck != 0)
  int kl_est;      // MRL_KL_*
};

// k'(d) of the sampled-token KL estimators, d = logp - logp_ref
__device__ __forceinline__ float kl_slope(float d, int est) {
  return est == MRL_KL_K1 ? 1.0f : (est == MRL_KL_K2 ? d : -expm1f(-d));
}
__device__ __forceinline__ double kl_value(double d, int est) {
  return est == MRL_KL_K1 ? d : (est == MRL_KL_K2 ? 0.5 * d * d : expm1(-d) + d);
}

struct RowOut {
  float logp;
  float pg_term;   // -cu * min(rho A, clip(rho) A)
  float nll_term;  // -cn * logp
  float g;         // dlogits = g * (p - onehot)
  bool clipped;
};

// Ratio, clipped surrogate, KL slope and gradient multiplier of one valid row (Eq. (1), Eq. (2)).
__device__ __forceinline__ RowOut mrl_row_loss(float logp, const RowIn& in, float eps_lo, float eps_hi) {
  RowOut o;
  o.logp = logp;
  const float rho = in.has_old ? expf(logp - in.logp_old) : 1.0f;
  const float lo = 1.0f - eps_lo, hi = 1.0f + eps_hi;
  const bool live = (in.cu != 0.f) && (in.A != 0.f);
  o.clipped = (in.A > 0.f && rho > hi) || (in.A < 0.f && rho < lo);
  const float s = fminf(rho * in.A, fminf(fmaxf(rho, lo), hi) * in.A);
  o.pg_term = live ? -in.cu * s : 0.f;
  o.nll_term = (in.cn != 0.f) ? -in.cn * logp : 0.f;
  o.g = ((live && !o.clipped) ? in.cu * in.A * rho : 0.f) + in.cn;
  if (in.ck != 0.f) o.g -= in.ck * kl_slope(logp - in.logp_ref, in.kl_est);  // dL_KL/dlogp = beta c k'(d)
  return o;
}

}  // namespace mrl
