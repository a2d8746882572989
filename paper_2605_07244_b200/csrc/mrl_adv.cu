// mrl_group_advantages: group-relative advantages (Sec. 3), pooled baseline (Sec. 5.1, App. H),
// batch whitening (App. A) and the SGT rescue gate with selection of y* (Sec. 5.3, App. B).
// Latency-bound: a few thousand floats.  One warp per prompt, fixed reduction order.
#include "mrl_common.cuh"

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ unsigned long long warp_min_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
    v = w < v ? w : v;
  }
  return v;
}

// SplitMix64 output function (Steele, Lea, Flood 2014).
__device__ __forceinline__ unsigned long long splitmix64(unsigned long long x) {
  x += 0x9E3779B97F4A7C15ull;
  unsigned long long z = x;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// mean and sum of squared deviations of x[0..n) (strided by lane), two passes
__device__ __forceinline__ void warp_mean_ss(const float* x, int n, int lane, float& mean, float& ss) {
  float s = 0.f;
  for (int i = lane; i < n; i += 32) s += x[i];
  mean = warp_sum(s) / (float)n;
  float q = 0.f;
  for (int i = lane; i < n; i += 32) {
    float d = x[i] - mean;
    q += d * d;
  }
  ss = warp_sum(q);
}

__global__ void __launch_bounds__(32) adv_prompt_kernel(
    const float* __restrict__ rewards, const int32_t* __restrict__ seq_len, int M, int G, int learner,
    mrl_adv_params ap, float* __restrict__ adv_own, float* __restrict__ adv_pool,
    uint8_t* __restrict__ rescue, int32_t* __restrict__ pick, float* __restrict__ nll_w,
    int32_t* __restrict__ n_gated) {
  const int p = blockIdx.x, lane = threadIdx.x;
  const int MG = M * G;
  const float* r = rewards + (size_t)p * MG;
  const bool znorm = ap.mode == MRL_ADV_GROUP_ZNORM;

  if (adv_pool != nullptr) {
    float mean, ss;
    warp_mean_ss(r, MG, lane, mean, ss);
    const int den = max(MG - ap.ddof, 1);
    const float inv = znorm ? 1.0f / (sqrtf(ss / (float)den) + ap.eps) : 1.0f;
    for (int i = lane; i < MG; i += 32) adv_pool[(size_t)p * MG + i] = (r[i] - mean) * inv;
  }
  if (adv_own != nullptr) {
    for (int m = 0; m < M; ++m) {
      float mean, ss;
      warp_mean_ss(r + m * G, G, lane, mean, ss);
      const int den = max(G - ap.ddof, 1);
      const float inv = znorm ? 1.0f / (sqrtf(ss / (float)den) + ap.eps) : 1.0f;
      for (int g = lane; g < G; g += 32) adv_own[(size_t)p * MG + m * G + g] = (r[m * G + g] - mean) * inv;
    }
  }

  // ---- SGT gate for `learner` (strict configuration: every own rollout is a negative)
  if (rescue == nullptr && pick == nullptr && nll_w == nullptr && n_gated == nullptr) return;
  bool own_neg = true;
  for (int g = lane; g < G; g += 32) own_neg = own_neg && (r[learner * G + g] < ap.sgt_negative_thr);
  own_neg = __all_sync(0xffffffffu, own_neg);
  // key of the best peer success under the pick rule; ~0 = none
  unsigned long long best = ~0ull;
  int n_succ = 0;
  for (int i = lane; i < MG; i += 32) {
    const bool is_succ = (i / G != learner) && (r[i] > ap.sgt_success_thr);
    if (is_succ) {
      ++n_succ;
      unsigned long long len = (ap.sgt_pick == MRL_PICK_SHORTEST) ? (unsigned long long)(uint32_t)seq_len[(size_t)p * MG + i] : 0ull;
      unsigned long long key = (len << 32) | (unsigned long long)i;
      best = key < best ? key : best;
    }
  }
  best = warp_min_u64(best);
  n_succ = (int)warp_sum((float)n_succ);  // <= 1024: exact in float
  const bool fire = own_neg && n_succ > 0;
  int chosen = -1;
  if (fire && ap.sgt_pick != MRL_PICK_NONE) {
    chosen = (int)(best & 0xffffffffull);
    if (ap.sgt_pick == MRL_PICK_SEEDED) {
      const unsigned long long h = splitmix64(((ap.seed & 0xffffffffull) << 32) | (unsigned long long)(uint32_t)p);
      int k = (int)(h % (unsigned long long)n_succ);
      chosen = -1;
      for (int i = 0; i < MG; ++i) {  // every lane walks the same short list
        if ((i / G != learner) && (r[i] > ap.sgt_success_thr)) {
          if (k == 0) {
            chosen = i;
            break;
          }
          --k;
        }
      }
    }
  }
  if (nll_w != nullptr) {
    for (int i = lane; i < MG; i += 32) {
      float w = 0.f;
      if (fire) {
        if (ap.sgt_pick == MRL_PICK_ALL)
          w = ((i / G != learner) && (r[i] > ap.sgt_success_thr)) ? 1.f : 0.f;
        else
          w = (i == chosen) ? 1.f : 0.f;
      }
      nll_w[(size_t)p * MG + i] = w;
    }
  }
  if (lane == 0) {
    if (rescue != nullptr) rescue[p] = fire ? 1 : 0;
    if (pick != nullptr) pick[p] = chosen;
    if (n_gated != nullptr && chosen >= 0) atomicAdd(n_gated, ap.sgt_pick == MRL_PICK_ALL ? n_succ : 1);
  }
}

// App. A: divide the group-centred values by the batch standard deviation.  One block, fixed order.
// x is [P, M, G]; `per_policy` = 1: one std per policy over its P*G values; 0: one std over everything.
__global__ void __launch_bounds__(1024) adv_batch_whiten_kernel(float* __restrict__ x, int P, int M, int G,
                                                                int per_policy, int ddof, float eps) {
  __shared__ double red[32];
  __shared__ float inv_sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int groups = per_policy ? M : 1;
  const long long per = per_policy ? (long long)P * G : (long long)P * M * G;
  for (int m = 0; m < groups; ++m) {
    double mean = 0.0, ss = 0.0;
    for (int pass = 0; pass < 2; ++pass) {
      double acc = 0.0;
      for (long long i = tid; i < per; i += blockDim.x) {
        long long idx = per_policy ? ((i / G) * M + m) * (long long)G + (i % G) : i;
        double v = (double)x[idx];
        acc += pass == 0 ? v : (v - mean) * (v - mean);
      }
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (lane == 0) red[warp] = acc;
      __syncthreads();
      if (warp == 0) {
        double t = lane < (int)(blockDim.x >> 5) ? red[lane] : 0.0;
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0) red[0] = t;
      }
      __syncthreads();
      if (pass == 0) mean = red[0] / (double)per; else ss = red[0];
      __syncthreads();
    }
    if (tid == 0) {
      long long den = per - ddof > 1 ? per - ddof : 1;
      inv_sh = (float)(1.0 / (sqrt(ss / (double)den) + (double)eps));
    }
    __syncthreads();
    const float inv = inv_sh;
    for (long long i = tid; i < per; i += blockDim.x) {
      long long idx = per_policy ? ((i / G) * M + m) * (long long)G + (i % G) : i;
      x[idx] *= inv;
    }
    __syncthreads();
  }
}

}  // namespace

extern "C" int mrl_group_advantages(const float* rewards, const int32_t* seq_len, int32_t P, int32_t M, int32_t G,
                                    int32_t learner, const mrl_adv_params* ap, float* adv_own, float* adv_pool,
                                    uint8_t* rescue, int32_t* pick, float* nll_seq_weight, int32_t* n_gated,
                                    void* stream) {
  if (ap == nullptr || P < 0 || M < 1 || G < 1 || (long long)M * G > 1024) return MRL_ERR_INVALID_ARG;
  if (learner < 0 || learner >= M) return MRL_ERR_INVALID_ARG;
  if (ap->mode < MRL_ADV_MEAN_ONLY || ap->mode > MRL_ADV_BATCH_ZNORM) return MRL_ERR_INVALID_ARG;
  if (ap->sgt_pick < MRL_PICK_NONE || ap->sgt_pick > MRL_PICK_SEEDED) return MRL_ERR_INVALID_ARG;
  if (ap->ddof != 0 && ap->ddof != 1) return MRL_ERR_INVALID_ARG;
  const bool wants_gate = rescue || pick || nll_seq_weight || n_gated;
  if (wants_gate && ap->sgt_pick == MRL_PICK_SHORTEST && seq_len == nullptr) return MRL_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n_gated != nullptr) MRL_CUDA_OK(cudaMemsetAsync(n_gated, 0, sizeof(int32_t), st));
  if (P == 0) return MRL_OK;
  if (rewards == nullptr) return MRL_ERR_INVALID_ARG;
  adv_prompt_kernel<<<P, 32, 0, st>>>(rewards, seq_len, M, G, learner, *ap, adv_own, adv_pool, rescue, pick,
                                      nll_seq_weight, n_gated);
  MRL_CUDA_OK(cudaGetLastError());
  if (ap->mode == MRL_ADV_BATCH_ZNORM) {
    if (adv_own != nullptr) {
      adv_batch_whiten_kernel<<<1, 1024, 0, st>>>(adv_own, P, M, G, 1, ap->ddof, ap->eps);
      MRL_CUDA_OK(cudaGetLastError());
    }
    if (adv_pool != nullptr) {
      adv_batch_whiten_kernel<<<1, 1024, 0, st>>>(adv_pool, P, M, G, 0, ap->ddof, ap->eps);
      MRL_CUDA_OK(cudaGetLastError());
    }
  }
  return MRL_OK;
}
