// mrl_policy_loss_fwd_bwd_host: the logits-in pass for a batch that lives in host memory.
//
// The batch is cut into micro-batches of whole sequences (App. A: log-prob micro-batches, the loss accumulated
// across them) and the three legs of a micro-batch -- host-to-device copy of its logits, the loss kernels in
// place on the staging buffer, device-to-host copy of its gradient -- run on three streams over three staging
// buffers, so that the bus carries data in both directions while the kernels work.  Everything the pass computes
// is computed by mrl_policy_loss_fwd_bwd; this file only plans the slabs and orders the copies.
#include <mutex>
#include <vector>

#include "mrl_common.cuh"

size_t mrl_policy_loss_workspace_bytes(long long N, int S);

namespace {

constexpr int kBufs = 3;
constexpr int kMaxDevices = 64;

// Copy streams and events of one device, created on first use and kept for the life of the process.
struct HostPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, small_in = nullptr;
  cudaEvent_t in_done[kBufs] = {}, comp_done[kBufs] = {}, out_done[kBufs] = {};
};
HostPipe g_pipe[kMaxDevices];
std::mutex g_pipe_mutex;  // guards the one-time creation (calls on one device must still not overlap: they share the pipe)

int pipe_for_current_device(HostPipe** out) {
  int dev = -1;
  MRL_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return MRL_ERR_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe& p = g_pipe[dev];
  if (!p.ready) {
    MRL_CUDA_OK(cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking));
    MRL_CUDA_OK(cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking));
    MRL_CUDA_OK(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
    MRL_CUDA_OK(cudaEventCreateWithFlags(&p.small_in, cudaEventDisableTiming));
    for (int b = 0; b < kBufs; ++b) {
      MRL_CUDA_OK(cudaEventCreateWithFlags(&p.in_done[b], cudaEventDisableTiming));
      MRL_CUDA_OK(cudaEventCreateWithFlags(&p.comp_done[b], cudaEventDisableTiming));
      MRL_CUDA_OK(cudaEventCreateWithFlags(&p.out_done[b], cudaEventDisableTiming));
    }
    p.ready = true;
  }
  *out = &p;
  return MRL_OK;
}

struct HostWs {
  int32_t *ids, *cu, *cu_local, *status;
  uint8_t* mask;
  float *logp_old, *tok_weight, *nll_weight, *logp_ref, *adv, *logp, *entropy, *loss, *kl;
  long long* stats;
  char* buf[kBufs];
  void* loss_ws;
  size_t loss_ws_bytes;
  size_t bytes;
};

HostWs carve_host_ws(void* ws, long long N, long long ld, int elem, int S, long long slab_rows) {
  MrlCarver c(ws);
  HostWs w;
  w.ids = c.take<int32_t>((size_t)N);
  w.mask = c.take<uint8_t>((size_t)N);
  w.logp_old = c.take<float>((size_t)N);
  w.tok_weight = c.take<float>((size_t)N);
  w.nll_weight = c.take<float>((size_t)N);
  w.logp_ref = c.take<float>((size_t)N);
  w.logp = c.take<float>((size_t)N);
  w.entropy = c.take<float>((size_t)N);
  w.cu = c.take<int32_t>((size_t)S + 1);
  w.cu_local = c.take<int32_t>((size_t)S + 1);
  w.adv = c.take<float>((size_t)S + 1);
  w.loss = c.take<float>(2);
  w.kl = c.take<float>(1);
  w.stats = c.take<long long>(4);
  w.status = c.take<int32_t>(1);
  for (int b = 0; b < kBufs; ++b) w.buf[b] = c.take<char>((size_t)slab_rows * (size_t)ld * (size_t)elem);
  w.loss_ws_bytes = mrl_policy_loss_workspace_bytes(slab_rows, S);
  w.loss_ws = c.take<char>(w.loss_ws_bytes);
  w.bytes = c.off;
  return w;
}

// cu_local[j] = cu[s0 + j] - cu[s0], j = 0 .. n
__global__ void __launch_bounds__(256) rebase_cu_kernel(const int32_t* __restrict__ cu, int s0, int n,
                                                         int32_t* __restrict__ cu_local) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j <= n) cu_local[j] = cu[s0 + j] - cu[s0];
}

int elem_size(int dtype) { return dtype == MRL_BF16 ? 2 : 4; }

}  // namespace

extern "C" size_t mrl_host_pipeline_workspace_bytes(int64_t N, int64_t ld, int32_t dtype, int32_t S,
                                                    int64_t slab_rows) {
  if (N < 0 || S < 0 || ld < 1 || slab_rows < 1 || (dtype != MRL_BF16 && dtype != MRL_F32)) return 0;
  return carve_host_ws(nullptr, N, ld, elem_size(dtype), S, slab_rows).bytes;
}

extern "C" int mrl_policy_loss_fwd_bwd_host(const void* h_logits, int32_t dtype, int64_t N, int32_t V, int64_t ld,
                                            const int32_t* h_ids, const uint8_t* h_mask,
                                            const int32_t* h_cu_seqlens, int32_t S, const float* h_adv_seq,
                                            const float* h_logp_old, const float* h_tok_weight,
                                            const float* h_nll_weight, const mrl_loss_params* lp, void* h_dlogits,
                                            int64_t ld_out, float* h_logp, float* h_loss, int64_t* h_stats,
                                            int32_t* h_status, int64_t slab_rows, void* workspace,
                                            size_t workspace_bytes, void* stream) {
  if (dtype != MRL_BF16 && dtype != MRL_F32) return MRL_ERR_UNSUPPORTED_DTYPE;
  if (lp == nullptr || h_loss == nullptr || N < 0 || S < 0 || V < 1 || ld < V || slab_rows < 1) return MRL_ERR_INVALID_ARG;
  if (h_dlogits != nullptr && ld_out < V) return MRL_ERR_INVALID_ARG;
  if (lp->flags & MRL_FLAG_ACCUMULATE_LOSS) return MRL_ERR_INVALID_ARG;  // the call always returns the whole step
  if (!mrl_kl_args_ok(lp)) return MRL_ERR_INVALID_ARG;
  if (N > 0 && S == 0) return MRL_ERR_INVALID_ARG;  // rows without a sequence
  if (N > 0 && (h_logits == nullptr || h_ids == nullptr || h_cu_seqlens == nullptr || h_adv_seq == nullptr))
    return MRL_ERR_INVALID_ARG;
  const int elem = elem_size(dtype);
  if (((size_t)ld * elem) % 32 != 0) return MRL_ERR_UNSUPPORTED_SHAPE;  // keeps every slab as aligned as the buffer
  const size_t need = carve_host_ws(nullptr, N, ld, elem, S, slab_rows).bytes;
  if (workspace == nullptr || workspace_bytes < need) return MRL_ERR_WORKSPACE_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MRL_ERR_INVALID_ARG;

  // ---- plan on the host: slabs of whole sequences, the step's denominators
  std::vector<int> slab_first;  // first sequence of every slab, then S
  if (S > 0) {
    if (h_cu_seqlens[0] != 0 || h_cu_seqlens[S] != N) return MRL_ERR_INVALID_ARG;
    int s0 = 0;
    while (s0 < S) {
      slab_first.push_back(s0);
      int s1 = s0;
      while (s1 < S && (long long)h_cu_seqlens[s1 + 1] - h_cu_seqlens[s0] <= slab_rows) {
        if (h_cu_seqlens[s1 + 1] < h_cu_seqlens[s1]) return MRL_ERR_INVALID_ARG;
        ++s1;
      }
      if (s1 == s0) return MRL_ERR_UNSUPPORTED_SHAPE;  // one sequence is longer than a staging buffer
      s0 = s1;
    }
  }
  slab_first.push_back(S);
  const int n_slabs = (int)slab_first.size() - 1;
  mrl_loss_params slp = *lp;
  slp.flags |= MRL_FLAG_ACCUMULATE_LOSS;
  if (slp.agg_mode == MRL_AGG_TOKEN_MEAN && !(slp.pg_denominator > 0)) {
    long long valid = 0;
    for (long long t = 0; t < N; ++t)
      valid += ((h_mask == nullptr || h_mask[t] != 0) && h_ids[t] >= 0 && h_ids[t] < V) ? 1 : 0;
    slp.pg_denominator = (double)valid;
    if (valid == 0) slp.pg_denominator = 1.0;  // nothing is valid: every coefficient is zero anyway
  }
  if (!(slp.seq_denominator > 0)) slp.seq_denominator = (double)(S > 0 ? S : 1);

  HostPipe* pp = nullptr;
  int rc = pipe_for_current_device(&pp);
  if (rc != MRL_OK) return rc;
  HostPipe& P = *pp;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const HostWs w = carve_host_ws(workspace, N, ld, elem, S, slab_rows);

  // ---- the small arrays go first, on the inbound stream, after whatever the caller's stream has queued
  MRL_CUDA_OK(cudaEventRecord(P.start, st));
  MRL_CUDA_OK(cudaStreamWaitEvent(P.in, P.start, 0));
  MRL_CUDA_OK(cudaStreamWaitEvent(P.out, P.start, 0));
  const size_t n4 = (size_t)N * 4;
  if (N > 0) {
    MRL_CUDA_OK(cudaMemcpyAsync(w.ids, h_ids, n4, cudaMemcpyHostToDevice, P.in));
    if (h_mask) MRL_CUDA_OK(cudaMemcpyAsync(w.mask, h_mask, (size_t)N, cudaMemcpyHostToDevice, P.in));
    if (h_logp_old) MRL_CUDA_OK(cudaMemcpyAsync(w.logp_old, h_logp_old, n4, cudaMemcpyHostToDevice, P.in));
    if (h_tok_weight) MRL_CUDA_OK(cudaMemcpyAsync(w.tok_weight, h_tok_weight, n4, cudaMemcpyHostToDevice, P.in));
    if (h_nll_weight) MRL_CUDA_OK(cudaMemcpyAsync(w.nll_weight, h_nll_weight, n4, cudaMemcpyHostToDevice, P.in));
    if (lp->logp_ref) MRL_CUDA_OK(cudaMemcpyAsync(w.logp_ref, lp->logp_ref, n4, cudaMemcpyHostToDevice, P.in));
    MRL_CUDA_OK(cudaMemcpyAsync(w.cu, h_cu_seqlens, ((size_t)S + 1) * 4, cudaMemcpyHostToDevice, P.in));
    MRL_CUDA_OK(cudaMemcpyAsync(w.adv, h_adv_seq, (size_t)S * 4, cudaMemcpyHostToDevice, P.in));
  }
  MRL_CUDA_OK(cudaEventRecord(P.small_in, P.in));
  MRL_CUDA_OK(cudaMemsetAsync(w.loss, 0, 2 * sizeof(float), st));
  MRL_CUDA_OK(cudaMemsetAsync(w.kl, 0, sizeof(float), st));
  MRL_CUDA_OK(cudaMemsetAsync(w.stats, 0, 4 * sizeof(long long), st));
  MRL_CUDA_OK(cudaMemsetAsync(w.status, 0, sizeof(int32_t), st));
  MRL_CUDA_OK(cudaStreamWaitEvent(st, P.small_in, 0));

  // ---- the slabs: copy in | kernels in place | copy out, three buffers in rotation
  const size_t row_bytes = (size_t)ld * elem;
  // If queueing fails half-way, what is already queued on the two copy streams is ordered before the end of the
  // caller's stream, so that a caller who synchronises its stream after the error return has nothing left in flight.
  auto give_up = [&](int code) {
    if (cudaEventRecord(P.small_in, P.in) == cudaSuccess) (void)cudaStreamWaitEvent(st, P.small_in, 0);
    if (cudaEventRecord(P.start, P.out) == cudaSuccess) (void)cudaStreamWaitEvent(st, P.start, 0);
    return code;
  };
  auto queue_slab = [&](int k) -> int {
    const int b = k % kBufs, s0 = slab_first[k], s1 = slab_first[k + 1];
    const long long a = h_cu_seqlens[s0], n = (long long)h_cu_seqlens[s1] - a;
    if (k >= kBufs) MRL_CUDA_OK(cudaStreamWaitEvent(P.in, P.out_done[b], 0));  // the buffer's last gradient has left
    if (n > 0)
      MRL_CUDA_OK(cudaMemcpyAsync(w.buf[b], static_cast<const char*>(h_logits) + (size_t)a * row_bytes,
                                  (size_t)n * row_bytes, cudaMemcpyHostToDevice, P.in));
    MRL_CUDA_OK(cudaEventRecord(P.in_done[b], P.in));

    MRL_CUDA_OK(cudaStreamWaitEvent(st, P.in_done[b], 0));
    rebase_cu_kernel<<<(s1 - s0 + 256) / 256, 256, 0, st>>>(w.cu, s0, s1 - s0, w.cu_local);
    MRL_CUDA_OK(cudaGetLastError());
    slp.entropy = lp->entropy ? w.entropy + a : nullptr;
    slp.logp_ref = lp->logp_ref ? w.logp_ref + a : nullptr;
    slp.kl_loss = lp->logp_ref ? w.kl : nullptr;
    rc = mrl_policy_loss_fwd_bwd(w.buf[b], dtype, n, V, ld, w.ids + a, h_mask ? w.mask + a : nullptr, w.cu_local,
                                 s1 - s0, w.adv + s0, h_logp_old ? w.logp_old + a : nullptr,
                                 h_tok_weight ? w.tok_weight + a : nullptr, h_nll_weight ? w.nll_weight + a : nullptr,
                                 &slp, h_dlogits ? w.buf[b] : nullptr, ld, w.logp + a, w.loss,
                                 reinterpret_cast<int64_t*>(w.stats), w.status, w.loss_ws, w.loss_ws_bytes, st);
    if (rc != MRL_OK) return rc;
    MRL_CUDA_OK(cudaEventRecord(P.comp_done[b], st));

    MRL_CUDA_OK(cudaStreamWaitEvent(P.out, P.comp_done[b], 0));
    if (h_dlogits != nullptr && n > 0)
      MRL_CUDA_OK(cudaMemcpy2DAsync(static_cast<char*>(h_dlogits) + (size_t)a * (size_t)ld_out * elem,
                                    (size_t)ld_out * elem, w.buf[b], row_bytes, (size_t)V * elem, (size_t)n,
                                    cudaMemcpyDeviceToHost, P.out));
    MRL_CUDA_OK(cudaEventRecord(P.out_done[b], P.out));
    return MRL_OK;
  };
  for (int k = 0; k < n_slabs; ++k) {
    rc = queue_slab(k);
    if (rc != MRL_OK) return give_up(rc);
  }
  // ---- the caller's stream ends after the last gradients have left, then the small results follow on it
  for (int k = n_slabs > kBufs ? n_slabs - kBufs : 0; k < n_slabs; ++k)
    MRL_CUDA_OK(cudaStreamWaitEvent(st, P.out_done[k % kBufs], 0));
  if (h_logp != nullptr && N > 0) MRL_CUDA_OK(cudaMemcpyAsync(h_logp, w.logp, n4, cudaMemcpyDeviceToHost, st));
  if (lp->entropy != nullptr && N > 0) MRL_CUDA_OK(cudaMemcpyAsync(lp->entropy, w.entropy, n4, cudaMemcpyDeviceToHost, st));
  MRL_CUDA_OK(cudaMemcpyAsync(h_loss, w.loss, 2 * sizeof(float), cudaMemcpyDeviceToHost, st));
  if (lp->logp_ref != nullptr) MRL_CUDA_OK(cudaMemcpyAsync(lp->kl_loss, w.kl, sizeof(float), cudaMemcpyDeviceToHost, st));
  if (h_stats != nullptr) MRL_CUDA_OK(cudaMemcpyAsync(h_stats, w.stats, 4 * sizeof(long long), cudaMemcpyDeviceToHost, st));
  if (h_status != nullptr) MRL_CUDA_OK(cudaMemcpyAsync(h_status, w.status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  return MRL_OK;
}
