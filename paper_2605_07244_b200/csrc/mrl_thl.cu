// THL word-level trace alignment (mrl_thl_word_align_logprobs): the source policy's per-token log-probs are summed
// per whitespace-delimited word and the word total is spread evenly over the learner's tokens of that word.
//
// One CTA per sequence.  Token-to-word maps come from a span-by-span tokenisation, so equal word ids are
// contiguous; a word's source sum and target count are therefore taken by the thread that sits on the first
// token of the run, walking the run in token order: no floating-point atomics, bitwise reproducible.  A word id
// that shows up in two separate runs, or lies outside the sequence's word range, raises MRL_DEV_BAD_WORD_MAP and
// is treated as "no word".
#include "mrl_common.cuh"

namespace {

constexpr int kAlignThreads = 256;

__device__ __forceinline__ float block_sum(float v, float* scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float r = lane < kAlignThreads / 32 ? scratch[lane] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
  return r;
}

__global__ void __launch_bounds__(kAlignThreads) thl_word_align_kernel(
    const float* __restrict__ src_logp, const int32_t* __restrict__ src_word, const int32_t* __restrict__ src_cu,
    const int32_t* __restrict__ tgt_word, const int32_t* __restrict__ tgt_cu, const int32_t* __restrict__ word_cu,
    float ignore_value, float* __restrict__ out, float* __restrict__ src_total, float* __restrict__ tgt_total,
    float* __restrict__ word_sum, int32_t* __restrict__ word_cnt, long long n_src, long long n_tgt,
    long long total_words, int32_t* status) {
  __shared__ float scratch[kAlignThreads / 32];
  __shared__ int any_source, bad;
  const int i = blockIdx.x, tid = threadIdx.x;
  // Offsets come from device memory the host cannot check: every range is cut to its array, so a corrupt offset
  // array raises MRL_DEV_BAD_WORD_MAP instead of reaching outside the buffers.
  const long long s_lo = src_cu[i], s_hi = src_cu[i + 1], t_lo = tgt_cu[i], t_hi = tgt_cu[i + 1];
  const long long w_lo = word_cu[i], w_hi = word_cu[i + 1];
  const bool bad_offsets = s_lo < 0 || s_hi < s_lo || s_hi > n_src || t_lo < 0 || t_hi < t_lo || t_hi > n_tgt ||
                           w_lo < 0 || w_hi < w_lo || w_hi > total_words;
  const int s0 = (int)min(max(s_lo, 0ll), n_src), ns = (int)(min(max(s_hi, (long long)s0), n_src) - s0);
  const int t0 = (int)min(max(t_lo, 0ll), n_tgt), nt = (int)(min(max(t_hi, (long long)t0), n_tgt) - t0);
  const int w0 = (int)min(max(w_lo, 0ll), total_words), nw = (int)(min(max(w_hi, (long long)w0), total_words) - w0);
  float* zsum = word_sum + w0;   // Z_w
  int32_t* cnt = word_cnt + w0;  // C_w; -1 while the word has not been seen on the source side either
  const int32_t* sw = src_word + s0;
  const int32_t* tw = tgt_word + t0;

  if (tid == 0) {
    any_source = 0;
    bad = bad_offsets ? 1 : 0;
  }
  for (int w = tid; w < nw; w += kAlignThreads) {
    zsum[w] = 0.f;
    cnt[w] = 0;
  }
  __syncthreads();

  // ---- pass 1: Z_w from the first token of every source run; every response token counts in the sequence total
  float total = 0.f;
  for (int p = tid; p < ns; p += kAlignThreads) {
    const int wid = sw[p];
    total += src_logp[s0 + p];
    if (wid < 0) continue;
    if (wid >= nw) { bad = 1; continue; }
    any_source = 1;
    if (p > 0 && sw[p - 1] == wid) continue;  // not the first token of its run
    float z = 0.f;
    int q = p;
    while (q < ns && sw[q] == wid) z += src_logp[s0 + q++];
    if (atomicAdd(&cnt[wid], 1) != 0) bad = 1;  // a second run of the same word: cnt is used as a "seen" mark here
    zsum[wid] = z;
  }
  total = block_sum(total, scratch);  // (contains the barriers that end pass 1)
  if (tid == 0 && src_total != nullptr) src_total[i] = total;
  for (int w = tid; w < nw; w += kAlignThreads) cnt[w] = 0;  // back to a count
  __syncthreads();

  // ---- pass 2: C_w from the first token of every target run
  for (int p = tid; p < nt; p += kAlignThreads) {
    const int wid = tw[p];
    if (wid < 0) continue;
    if (wid >= nw) { bad = 1; continue; }
    if (p > 0 && tw[p - 1] == wid) continue;
    int q = p;
    while (q < nt && tw[q] == wid) ++q;
    if (atomicAdd(&cnt[wid], q - p) != 0) bad = 1;
  }
  __syncthreads();

  // ---- pass 3: Z_w / C_w on every target token with a word; ignore_value elsewhere and in skipped sequences
  const bool skip = any_source == 0;
  float tsum = 0.f;
  for (int p = tid; p < nt; p += kAlignThreads) {
    const int wid = tw[p];
    float v = ignore_value;
    if (!skip && wid >= 0 && wid < nw) {
      v = zsum[wid] / (float)cnt[wid];  // cnt >= 1: this token was counted
      tsum += v;
    }
    out[t0 + p] = v;
  }
  tsum = block_sum(tsum, scratch);
  if (tid == 0) {
    if (tgt_total != nullptr) tgt_total[i] = tsum;
    if (bad && status != nullptr) atomicOr(status, MRL_DEV_BAD_WORD_MAP);
  }
}

}  // namespace

size_t mrl_thl_workspace_bytes(long long total_words) {
  if (total_words <= 0) return 0;
  return 2 * mrl_align_up((size_t)total_words * 4, 256);
}

extern "C" int mrl_thl_word_align_logprobs(const float* src_logp, const int32_t* src_word, const int32_t* src_cu,
                                           const int32_t* tgt_word, const int32_t* tgt_cu, const int32_t* word_cu,
                                           int32_t B, int64_t N_src, int64_t N_tgt, int64_t total_words,
                                           float ignore_value, float* out,
                                           float* src_total, float* tgt_total, int32_t* status, void* workspace,
                                           size_t workspace_bytes, void* stream) {
  if (B < 0 || total_words < 0 || N_src < 0 || N_tgt < 0 || N_src > 0x7fffffffll || N_tgt > 0x7fffffffll ||
      total_words > 0x7fffffffll)
    return MRL_ERR_INVALID_ARG;
  if (B == 0) return MRL_OK;
  if (src_word == nullptr || src_cu == nullptr || tgt_word == nullptr || tgt_cu == nullptr || word_cu == nullptr ||
      src_logp == nullptr || out == nullptr)
    return MRL_ERR_INVALID_ARG;
  const size_t need = mrl_thl_workspace_bytes(total_words);
  if (need > 0 && (workspace == nullptr || workspace_bytes < need)) return MRL_ERR_WORKSPACE_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MRL_ERR_INVALID_ARG;
  float* word_sum = static_cast<float*>(workspace);
  int32_t* word_cnt = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + need / 2);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  mrl_profile_before(st, "thl_word_align_kernel");
  thl_word_align_kernel<<<(unsigned)B, kAlignThreads, 0, st>>>(src_logp, src_word, src_cu, tgt_word, tgt_cu, word_cu,
                                                               ignore_value, out, src_total, tgt_total, word_sum,
                                                               word_cnt, N_src, N_tgt, total_words, status);
  mrl_profile_after(st);
  return cudaGetLastError() == cudaSuccess ? MRL_OK : MRL_ERR_CUDA;
}
