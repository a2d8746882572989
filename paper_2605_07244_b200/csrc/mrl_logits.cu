// Logits-in path: mrl_token_logprobs and mrl_policy_loss_fwd_bwd.
//
// Fast kernel (bf16, 16-byte aligned rows): one thread-block cluster per logits row.  Each CTA of
// the cluster pulls its slice of the row into shared memory with bulk asynchronous copies (four
// chunks, one mbarrier each), reduces max / sum-of-exponentials as the chunks land while caching the
// exponentials in place, exchanges one (max, sum, target-logit) triple per CTA through distributed
// shared memory, evaluates the ratio / clip / loss scalars, and writes g * (softmax - onehot) from
// the cached slice.  The row is read from HBM exactly once and written exactly once; nothing is
// shared between clusters.
// General kernel (any dtype, any V, any alignment): one CTA per row, three passes over global
// memory; used for small or unaligned problems.
#include "mrl_common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kChunks = 4;            // bulk copies (and mbarriers) per CTA slice
constexpr int kUnroll = 4;            // 16-byte vectors in flight per thread
constexpr int kMaxCluster = 8;        // portable cluster size limit
constexpr int kMaxPartBytes = 76000;  // slice size that still lets three CTAs share an SM
constexpr uint32_t kSpinLimit = 1u << 20;

// rowstat bits
constexpr uint8_t kStatValid = MRL_ROW_VALID, kStatClipped = MRL_ROW_CLIPPED, kStatRead = MRL_ROW_READ;

struct RowParams {
  const void* logits;
  void* dlogits;
  long long ld, ld_out;
  long long N;
  int V;
  const int32_t* ids;
  const uint8_t* mask;
  const float* rowA;
  const float* rowcu;
  const float* rowcn;
  const float* logp_old;
  float eps_lo, eps_hi;
  uint32_t flags;
  int loss_mode;  // 0: log-probs only, 1: loss (+ gradient when dlogits != null)
  float* logp;
  float* lse;
  float* row_m2;  // loss mode: per-row (max, sum, target) of the base-2 log-sum-exp, finished in float64 later
  float* row_s;
  float* row_zt;
  uint8_t* rowstat;
  int32_t* status;
  int part_elems;  // elements per CTA slice (multiple of 8)
  int cluster;     // CTAs per row
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the copy did not land within the spin limit.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__device__ __forceinline__ void st_global_v4(void* p, uint4 v) {
  asm volatile("st.global.cs.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Everything the loss needs from one row besides the logits.
struct RowCtx {
  int id;
  bool valid;  // mask on and id in range
  bool dead;   // nothing to read: invalid, or skipped by MRL_FLAG_SKIP_ZERO_ROWS
  mrl::RowIn in;
};

__device__ __forceinline__ RowCtx load_row_ctx(const RowParams& p, long long row) {
  RowCtx c;
  c.id = p.ids[row];
  const bool m = p.mask == nullptr || p.mask[row] != 0;
  c.valid = m && c.id >= 0 && c.id < p.V;
  c.in.A = 0.f;
  c.in.cu = 0.f;
  c.in.cn = 0.f;
  c.in.logp_old = 0.f;
  c.in.has_old = false;
  if (p.loss_mode) {
    c.in.A = p.rowA[row];
    c.in.cu = p.rowcu[row];
    c.in.cn = p.rowcn[row];
    c.in.has_old = p.logp_old != nullptr;
    if (c.in.has_old) c.in.logp_old = p.logp_old[row];
  }
  c.dead = !c.valid;
  if (p.loss_mode && (p.flags & MRL_FLAG_SKIP_ZERO_ROWS) && (c.in.cu == 0.f || c.in.A == 0.f) && c.in.cn == 0.f)
    c.dead = true;
  return c;
}

// Log-probs mode: the float32 results.  Loss mode: the raw reduction triple and the row's status bits; the
// ratio, surrogate terms and the reported log-prob are finished in float64 by row_terms_kernel.
__device__ __forceinline__ void write_row_scalars(const RowParams& p, long long row, const RowCtx& c, float logp,
                                                  float lse, mrl::Lse2 tot, float zt, bool clipped, bool read) {
  if (p.loss_mode) {
    p.row_m2[row] = tot.m;
    p.row_s[row] = tot.s;
    p.row_zt[row] = zt;
    uint8_t st = 0;
    if (c.valid) st |= kStatValid;
    if (clipped && c.in.A != 0.f) st |= kStatClipped;
    if (read) st |= kStatRead;
    p.rowstat[row] = st;
  } else {
    p.logp[row] = logp;
    if (p.lse != nullptr) p.lse[row] = lse;
  }
}

// ------------------------------------------------------------------------------------------------
// Fast kernel: bf16, one thread-block cluster per row, each CTA's slice of the row resident in shared memory.
//
// A CTA pulls its slice in with four bulk asynchronous copies (an mbarrier each) and works on it as the copies
// land.  Pass 1, in steps of 1,024 vectors: each thread takes the maximum of its own 32 logits of the step as
// reference, turns them into 2^(x - ref), sums them in float32 and writes them back over the logits as bf16, so
// that pass 2 needs no exponential; the references stay in registers.  The CTA's (max, sum, target logit) is
// pushed to every other CTA of the cluster through distributed shared memory (a remote store and a remote
// mbarrier arrive per peer); warp 0 alone waits for the peers, forms the row's scalars and hands them to the
// block.  Pass 2: every cached value times g 2^(ref - lse) as two packed bf16 FMAs (scale = hi + lo, one
// rounding of the result), streamed out with 128-bit stores.  Full steps run without per-vector bounds checks;
// only the last step of a slice can be ragged.  Slices are at most 76,000 bytes, so three CTAs of different rows
// share an SM and one CTA's copy latency, exchange and stores overlap the others' arithmetic.
// A row is read from HBM once and written once; nothing is shared between clusters.
// Dynamic shared memory: [slice | 4 copy barriers, 1 exchange barrier | exchange | per-warp scratch | row scalars]
// ------------------------------------------------------------------------------------------------
constexpr int kStepVecs = kThreads * kUnroll;                                // vectors per step of a CTA
constexpr int kMaxSteps = (kMaxPartBytes / 16 + kStepVecs - 1) / kStepVecs;  // 5
constexpr int kWarps = kThreads / 32;
constexpr size_t kTailBytes = 64 + kMaxCluster * 16 + 2 * kWarps * 4 + 32;

__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// packed arithmetic on two bf16
__device__ __forceinline__ uint32_t hmax2_u32(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t hfma2_u32(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}

__global__ void __launch_bounds__(kThreads, 3) row_cluster_kernel(const RowParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int C = p.cluster;
  const long long row = blockIdx.x / C;
  const int rank = blockIdx.x % C;  // equals the rank in the cluster for a 1-D cluster
  const int part_off = rank * p.part_elems;
  const int part_len = max(0, min(p.V - part_off, p.part_elems));  // multiple of 8
  const int nvec = part_len >> 3;
  const size_t slice_bytes = (size_t)p.part_elems * 2;

  uint4* slice = reinterpret_cast<uint4*>(smem);
  unsigned char* tail = smem + slice_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tail);                    // [kChunks] copies, then the exchange
  float4* xchg = reinterpret_cast<float4*>(tail + 64);                   // [kMaxCluster]
  float* red = reinterpret_cast<float*>(tail + 64 + kMaxCluster * 16);   // [2][kWarps]
  float* fin = red + 2 * kWarps;                                         // lse2, g, target-column value, ok
  float* tgt = fin + 4;                                                  // target logit, has-target

  const bool want_grad = p.dlogits != nullptr;
  const __nv_bfloat16* grow = static_cast<const __nv_bfloat16*>(p.logits) + row * p.ld + part_off;
  __nv_bfloat16* orow = want_grad ? static_cast<__nv_bfloat16*>(p.dlogits) + row * p.ld_out + part_off : nullptr;

  // Rows that may be dead are decided before anything is fetched; otherwise fetch first.
  const bool may_be_dead = p.mask != nullptr || (p.flags & MRL_FLAG_SKIP_ZERO_ROWS);
  RowCtx ctx;
  if (may_be_dead) {
    ctx = load_row_ctx(p, row);
    if (ctx.dead) {
      if (orow != nullptr)
        for (int i = tid; i < nvec; i += kThreads) st_global_v4(orow + (size_t)i * 8, make_uint4(0, 0, 0, 0));
      if (rank == 0 && tid == 0) write_row_scalars(p, row, ctx, 0.f, 0.f, mrl::lse2_empty(), 0.f, false, false);
      return;  // the whole cluster takes this branch: no cluster barrier is left waiting
    }
  }

  const int vpc = (nvec + kChunks - 1) / kChunks;  // vectors per copy
  if (tid == 0) {
#pragma unroll
    for (int k = 0; k < kChunks; ++k) mbar_init(&bars[k], 1);
    mbar_init(&bars[kChunks], C > 1 ? C - 1 : 1);
    tgt[0] = 0.f;
    tgt[1] = 0.f;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
#pragma unroll
    for (int k = 0; k < kChunks; ++k) {
      const int lo = k * vpc, hi = min(nvec, lo + vpc);
      if (hi > lo) {
        const uint32_t bytes = (uint32_t)(hi - lo) * 16u;
        mbar_expect_tx(&bars[k], bytes);
        bulk_g2s(slice + lo, grow + (size_t)lo * 8, bytes, &bars[k]);
      }
    }
  }
  if (C > 1) cluster_arrive();  // "my exchange barrier exists": waited for just before the first remote access
  __syncthreads();
  if (!may_be_dead) ctx = load_row_ctx(p, row);

  // where the target logit lives in this CTA's slice: the step whose vectors hold it, for the thread that holds it
  const int rel = ctx.id - part_off;
  int owner_step = -1;
  if (ctx.valid && rel >= 0 && rel < part_len && ((rel >> 3) % kThreads) == tid) owner_step = (rel >> 3) / kStepVecs;
  const __nv_bfloat16* slice_elems = reinterpret_cast<const __nv_bfloat16*>(slice);

  // ---- pass 1
  bool timed_out = false;
  int waited = 0;  // copies known to have landed
  float ref[kMaxSteps], sums[kMaxSteps];
  float zt = 0.f;
  uint4* const mine = slice + tid;  // this thread's vectors: mine[step * kStepVecs + u * kThreads]
#pragma unroll
  for (int it = 0; it < kMaxSteps; ++it) {
    ref[it] = -INFINITY;
    sums[it] = 0.f;
    const int base = it * kStepVecs;
    if (base < nvec) {
      const int last = min(nvec - 1, base + (kUnroll - 1) * kThreads + tid);
      const int need = last / vpc + 1;
      while (waited < need) {
        if (!mbar_wait_bounded(&bars[waited], 0)) timed_out = true;
        ++waited;
      }
      if (owner_step == it) zt = __bfloat162float(slice_elems[rel]);  // before this thread overwrites it below
      const bool full = base + kStepVecs <= nvec;  // uniform: only the last step of a slice is ragged
      uint4 v[kUnroll];
      if (full) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = mine[base + u * kThreads];
      } else {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          v[u] = (base + u * kThreads + tid < nvec) ? mine[base + u * kThreads]
                                                    : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
      }
      uint32_t mx = hmax2_u32(hmax2_u32(v[0].x, v[0].y), hmax2_u32(v[0].z, v[0].w));
#pragma unroll
      for (int u = 1; u < kUnroll; ++u)
        mx = hmax2_u32(mx, hmax2_u32(hmax2_u32(v[u].x, v[u].y), hmax2_u32(v[u].z, v[u].w)));
      const float vmax = fmaxf(mrl::bf16lo_to_f32(mx), mrl::bf16hi_to_f32(mx));
      // a thread whose 32 logits are all -inf takes reference 0: every term is 2^-inf = 0
      const float r = vmax != -INFINITY ? vmax * MRL_LOG2E : 0.f, neg_r = -r;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
        uint32_t e[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float a = mrl::ex2_approx(fmaf(mrl::bf16lo_to_f32(w[j]), MRL_LOG2E, neg_r));
          const float b = mrl::ex2_approx(fmaf(mrl::bf16hi_to_f32(w[j]), MRL_LOG2E, neg_r));
          s0 += a;
          s1 += b;
          e[j] = mrl::pack_bf16x2(a, b);
        }
        v[u] = make_uint4(e[0], e[1], e[2], e[3]);
      }
      if (want_grad) {
        if (full) {
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) mine[base + u * kThreads] = v[u];
        } else {
#pragma unroll
          for (int u = 0; u < kUnroll; ++u)
            if (base + u * kThreads + tid < nvec) mine[base + u * kThreads] = v[u];
        }
      }
      ref[it] = vmax != -INFINITY ? r : -INFINITY;
      sums[it] = s0 + s1;
    }
  }
  while (waited < kChunks) {  // copies this thread had no vector in
    const int lo = waited * vpc;
    if (lo < nvec && !mbar_wait_bounded(&bars[waited], 0)) timed_out = true;
    ++waited;
  }

  // ---- (max, sum) of the warp: the maximum first, one rescale per step, then a plain sum
  if (owner_step >= 0) {  // at most one thread of the whole cluster
    tgt[0] = zt;
    tgt[1] = 1.f;
  }
  float m = -INFINITY;
#pragma unroll
  for (int it = 0; it < kMaxSteps; ++it) m = fmaxf(m, ref[it]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float sum = 0.f;
  if (m != -INFINITY) {
#pragma unroll
    for (int it = 0; it < kMaxSteps; ++it) sum = fmaf(sums[it], mrl::ex2_approx(ref[it] - m), sum);  // 2^-inf = 0
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) {
    red[warp] = m;
    red[kWarps + warp] = sum;
  }
  const bool any_timeout = __syncthreads_or(timed_out ? 1 : 0) != 0;

  // ---- warp 0: the CTA's triple to every peer, the peers' triples, the row's scalars
  if (warp == 0) {
    float wm = lane < kWarps ? red[lane] : -INFINITY;
    float ws = lane < kWarps ? red[kWarps + lane] : 0.f;
    float cm = wm;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
    float cs = (wm != -INFINITY) ? ws * mrl::ex2_approx(wm - cm) : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cs += __shfl_xor_sync(0xffffffffu, cs, o);
    bool wok = !any_timeout;
    if (C > 1) {
      cluster_wait();  // every CTA of the cluster has initialised its exchange barrier
      if (lane == 0) {
        const float zpart = tgt[0], opart = tgt[1];
        xchg[rank] = make_float4(cm, cs, zpart, opart);
        for (int r = 0; r < C; ++r) {
          if (r == rank) continue;
          const uint32_t dst = mapa_u32(smem_u32(&xchg[rank]), (uint32_t)r);
          asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(cm), "f"(cs), "f"(zpart),
                       "f"(opart)
                       : "memory");
          const uint32_t rbar = mapa_u32(smem_u32(&bars[kChunks]), (uint32_t)r);
          asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(rbar) : "memory");
        }
      }
      __syncwarp();
      bool got = false;
      for (uint32_t i = 0; i < (kSpinLimit << 2) && !got; ++i) got = mbar_try_wait_cluster(&bars[kChunks], 0);
      wok = wok && got;
    } else if (lane == 0) {
      xchg[0] = make_float4(cm, cs, tgt[0], tgt[1]);
    }
    __syncwarp();
    float4 o = make_float4(-INFINITY, 0.f, 0.f, 0.f);
    if (lane < C && wok) o = xchg[lane];
    float tm = o.x;
#pragma unroll
    for (int q = 16; q > 0; q >>= 1) tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, q));
    float ts = (o.x != -INFINITY) ? o.y * mrl::ex2_approx(o.x - tm) : 0.f;
    float ztot = o.w != 0.f ? o.z : 0.f;
#pragma unroll
    for (int q = 16; q > 0; q >>= 1) {
      ts += __shfl_xor_sync(0xffffffffu, ts, q);      // xor tree over the ranks: the same order in every CTA
      ztot += __shfl_xor_sync(0xffffffffu, ztot, q);  // one owner: exact
    }
    const float lse2 = tm + log2f(ts);
    const float lse = lse2 * MRL_LN2;
    float logp = 0.f, g = 0.f;
    bool clipped = false;
    if (ctx.valid && wok) {
      logp = ztot - lse;
      if (p.loss_mode) {
        const mrl::RowOut ro = mrl::mrl_row_loss(logp, ctx.in, p.eps_lo, p.eps_hi);
        g = ro.g;
        clipped = ro.clipped;
      }
    }
    if (lane == 0) {
      if (rank == 0 && wok)
        write_row_scalars(p, row, ctx, logp, ctx.valid ? lse : 0.f, mrl::Lse2{tm, ts}, ztot, clipped, true);
      if (!wok && p.status != nullptr) atomicOr(p.status, MRL_DEV_TIMEOUT);
      fin[0] = lse2;
      fin[1] = g;
      fin[2] = g * (mrl::ex2_approx(fmaf(ztot, MRL_LOG2E, -lse2)) - 1.0f);  // the target column
      fin[3] = wok ? 1.f : 0.f;
    }
  } else if (C > 1) {
    cluster_wait();  // pairs with the arrive above (every thread of the cluster takes part)
  }
  __syncthreads();
  const float lse2 = fin[0], g = fin[1], tfix = fin[2];
  const bool ok = fin[3] != 0.f;

  // ---- pass 2: dlogits slice = g * softmax - g * onehot, from the cached exponentials
  if (want_grad && ok) {
    uint4* const out = reinterpret_cast<uint4*>(orow) + tid;  // this thread's output vectors, indexed like `mine`
#pragma unroll
    for (int it = 0; it < kMaxSteps; ++it) {
      const int base = it * kStepVecs;
      if (base < nvec) {
        const bool full = base + kStepVecs <= nvec;
        uint4 o[kUnroll];
        if (g == 0.f) {  // uniform over the row
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) o[u] = make_uint4(0, 0, 0, 0);
        } else {
          // cached value times scale, as two packed bf16 FMAs: scale = hi + lo, one rounding of the result
          const float scale = ref[it] != -INFINITY ? g * mrl::ex2_approx(ref[it] - lse2) : 0.f;
          const float s_hi = __bfloat162float(__float2bfloat16_rn(scale));
          const uint32_t hi2 = mrl::pack_bf16x2(s_hi, s_hi), lo2 = mrl::pack_bf16x2(scale - s_hi, scale - s_hi);
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const uint4 e = (full || base + u * kThreads + tid < nvec) ? mine[base + u * kThreads] : make_uint4(0, 0, 0, 0);
            o[u].x = hfma2_u32(e.x, hi2, hfma2_u32(e.x, lo2, 0u));
            o[u].y = hfma2_u32(e.y, hi2, hfma2_u32(e.y, lo2, 0u));
            o[u].z = hfma2_u32(e.z, hi2, hfma2_u32(e.z, lo2, 0u));
            o[u].w = hfma2_u32(e.w, hi2, hfma2_u32(e.w, lo2, 0u));
          }
        }
        if (full) {
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) st_global_v4(out + base + u * kThreads, o[u]);
        } else {
#pragma unroll
          for (int u = 0; u < kUnroll; ++u)
            if (base + u * kThreads + tid < nvec) st_global_v4(out + base + u * kThreads, o[u]);
        }
        // the target column gets g (p - 1): a scalar store by the thread whose vector store just covered it, so
        // the two stores to that address are ordered by program order
        if (owner_step == it && g != 0.f) orow[rel] = __float2bfloat16_rn(tfix);
      }
    }
  }
  // Every peer's remote store and arrive has landed before warp 0 got past its wait, and this CTA's own remote
  // accesses were issued before it: nobody touches a CTA's shared memory after that CTA can have left.
}

// ------------------------------------------------------------------------------------------------
// General kernel: one CTA per row, any dtype / V / alignment.
// ------------------------------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ float ld_as_f32(const T* p);
template <>
__device__ __forceinline__ float ld_as_f32<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float ld_as_f32<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T>
__device__ __forceinline__ void st_from_f32(T* p, float v);
template <>
__device__ __forceinline__ void st_from_f32<float>(float* p, float v) { *p = v; }
template <>
__device__ __forceinline__ void st_from_f32<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(kThreads) row_general_kernel(const RowParams p) {
  __shared__ float scratch[64];
  const int tid = threadIdx.x;
  const long long row = blockIdx.x;
  const T* z = static_cast<const T*>(p.logits) + row * p.ld;
  T* dz = p.dlogits ? static_cast<T*>(p.dlogits) + row * p.ld_out : nullptr;
  const RowCtx ctx = load_row_ctx(p, row);
  if (ctx.dead) {
    if (dz != nullptr)
      for (int v = tid; v < p.V; v += kThreads) st_from_f32<T>(dz + v, 0.f);
    if (tid == 0) write_row_scalars(p, row, ctx, 0.f, 0.f, mrl::lse2_empty(), 0.f, false, false);
    return;
  }
  const float zt = ld_as_f32<T>(z + ctx.id);  // before any in-place write
  float mx = -INFINITY;
  for (int v = tid; v < p.V; v += kThreads) mx = fmaxf(mx, ld_as_f32<T>(z + v));
  mrl::Lse2 acc{mx * MRL_LOG2E, 0.f};
  if (mx != -INFINITY) {
    const float neg_m = -acc.m;
    float s = 0.f;
    for (int v = tid; v < p.V; v += kThreads) s += mrl::ex2_approx(fmaf(ld_as_f32<T>(z + v), MRL_LOG2E, neg_m));
    acc.s = s;
  }
  const mrl::Lse2 tot = mrl::lse2_block_reduce<kThreads>(acc, scratch);
  const float lse2 = tot.m + log2f(tot.s);
  const float lse = lse2 * MRL_LN2;
  const float logp = zt - lse;
  float g = 0.f;
  bool clipped = false;
  if (p.loss_mode) {
    const mrl::RowOut ro = mrl::mrl_row_loss(logp, ctx.in, p.eps_lo, p.eps_hi);
    g = ro.g;
    clipped = ro.clipped;
  }
  if (tid == 0) write_row_scalars(p, row, ctx, logp, lse, tot, zt, clipped, true);
  if (dz == nullptr) return;
  if (g == 0.f) {
    for (int v = tid; v < p.V; v += kThreads) st_from_f32<T>(dz + v, 0.f);
    return;
  }
  const float neg_k = -(lse2 - log2f(fabsf(g)));
  const float sgn = g < 0.f ? -1.f : 1.f;
  for (int v = tid; v < p.V; v += kThreads)
    st_from_f32<T>(dz + v, sgn * mrl::ex2_approx(fmaf(ld_as_f32<T>(z + v), MRL_LOG2E, neg_k)));
  __syncthreads();
  if (tid == 0) st_from_f32<T>(dz + ctx.id, g * (expf(zt - lse) - 1.0f));
}

// ------------------------------------------------------------------------------------------------
// Per-sequence bookkeeping around the row kernel.
// ------------------------------------------------------------------------------------------------
// valid-token count of each sequence, the total, and bad-id detection
__global__ void __launch_bounds__(128) seq_count_kernel(const int32_t* __restrict__ cu, int S, long long N, int V,
                                                         const int32_t* __restrict__ ids,
                                                         const uint8_t* __restrict__ mask, int32_t* seq_cnt,
                                                         unsigned long long* totals, int32_t* status) {
  __shared__ int red[2][4];
  const int s = blockIdx.x;
  const long long a = max(0ll, min((long long)cu[s], N)), b = max(a, min((long long)cu[s + 1], N));
  int cnt = 0, bad = 0;
  for (long long t = a + threadIdx.x; t < b; t += blockDim.x) {
    const bool m = mask == nullptr || mask[t] != 0;
    const int id = ids[t];
    const bool in_range = id >= 0 && id < V;
    cnt += (m && in_range) ? 1 : 0;
    bad += (m && !in_range) ? 1 : 0;
  }
  for (int o = 16; o > 0; o >>= 1) {
    cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    bad += __shfl_xor_sync(0xffffffffu, bad, o);
  }
  if ((threadIdx.x & 31) == 0) {
    red[0][threadIdx.x >> 5] = cnt;
    red[1][threadIdx.x >> 5] = bad;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    cnt = red[0][0] + red[0][1] + red[0][2] + red[0][3];
    bad = red[1][0] + red[1][1] + red[1][2] + red[1][3];
    seq_cnt[s] = cnt;
    atomicAdd(&totals[0], (unsigned long long)cnt);  // integer sums: order does not matter
    if (bad) {
      atomicAdd(&totals[1], (unsigned long long)bad);
      if (status != nullptr) atomicOr(status, MRL_DEV_BAD_TOKEN_ID);
    }
  }
}

// A_t, c_t u_t and cn_t of every row (Eq. (1) aggregation, Eq. (2) per-token average)
__global__ void __launch_bounds__(128) row_coef_kernel(const int32_t* __restrict__ cu, int S, long long N, int V,
                                                        const int32_t* __restrict__ ids,
                                                        const uint8_t* __restrict__ mask,
                                                        const float* __restrict__ adv_seq,
                                                        const float* __restrict__ tok_weight,
                                                        const float* __restrict__ nll_weight,
                                                        const int32_t* __restrict__ seq_cnt,
                                                        const unsigned long long* __restrict__ totals,
                                                        mrl_loss_params lp, float* rowA, float* rowcu, float* rowcn) {
  const int s = blockIdx.x;
  const long long a = max(0ll, min((long long)cu[s], N)), b = max(a, min((long long)cu[s + 1], N));
  const double len = (double)seq_cnt[s];
  const double D = lp.pg_denominator > 0 ? lp.pg_denominator : (double)totals[0];
  const double Sd = lp.seq_denominator > 0 ? lp.seq_denominator : (double)S;
  float c = 0.f, cn_base = 0.f;
  if (len > 0) {
    if (lp.agg_mode == MRL_AGG_TOKEN_MEAN)
      c = D > 0 ? (float)(1.0 / D) : 0.f;
    else
      c = (float)(1.0 / (Sd * len));
    cn_base = (float)((double)lp.nll_coeff / len);
  }
  const float A = adv_seq[s];
  for (long long t = a + threadIdx.x; t < b; t += blockDim.x) {
    const bool m = mask == nullptr || mask[t] != 0;
    const int id = ids[t];
    const bool valid = m && id >= 0 && id < V;
    rowA[t] = A;
    rowcu[t] = valid ? c * (tok_weight ? tok_weight[t] : 1.f) : 0.f;
    rowcn[t] = (valid && nll_weight) ? cn_base * nll_weight[t] : 0.f;
  }
}

// Ratio, clipped surrogate and NLL term of every row in float64, from the row kernel's reduction triple:
// lse = (m2 + log2 s) ln 2, logp = z_target - lse, rho = exp(logp - logp_old)  (Sec. 3; Eq. (1); Eq. (2)).
// The surrogate is continuous across the clip bound, so the float32 decision the gradient used and the
// float64 one here cannot disagree by more than rounding.
__global__ void __launch_bounds__(256) row_terms_kernel(long long N, const float* __restrict__ row_m2,
                                                         const float* __restrict__ row_s,
                                                         const float* __restrict__ row_zt,
                                                         const uint8_t* __restrict__ rowstat,
                                                         const float* __restrict__ rowA,
                                                         const float* __restrict__ rowcu,
                                                         const float* __restrict__ rowcn,
                                                         const float* __restrict__ logp_old, float eps_lo,
                                                         float eps_hi, double* __restrict__ pg_term,
                                                         double* __restrict__ nll_term, float* __restrict__ logp) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= N) return;
  const uint8_t st = rowstat[t];
  double pg = 0.0, nl = 0.0, lp = 0.0;
  if ((st & kStatValid) && (st & kStatRead)) {
    const double lse = ((double)row_m2[t] + log2((double)row_s[t])) * 0.693147180559945309417232121458;
    lp = (double)row_zt[t] - lse;
    const double A = rowA[t], cu = rowcu[t], cn = rowcn[t];
    if (cu != 0.0 && A != 0.0) {
      const double rho = logp_old ? exp(lp - (double)logp_old[t]) : 1.0;
      const double lo = 1.0 - (double)eps_lo, hi = 1.0 + (double)eps_hi;
      pg = -cu * fmin(rho * A, fmin(fmax(rho, lo), hi) * A);
    }
    if (cn != 0.0) nl = -cn * lp;
  }
  pg_term[t] = pg;
  nll_term[t] = nl;
  if (logp != nullptr) logp[t] = (float)lp;
}

// fixed-order float64 sums of the per-row terms and the row statistics
__global__ void __launch_bounds__(1024) finalize_kernel(const double* __restrict__ pg_term,
                                                         const double* __restrict__ nll_term,
                                                         const uint8_t* __restrict__ rowstat, long long N,
                                                         const unsigned long long* __restrict__ totals,
                                                         uint32_t flags, float* loss, long long* stats) {
  __shared__ double red[6][32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  double v[6] = {0, 0, 0, 0, 0, 0};
  for (long long t = tid; t < N; t += 1024) {
    v[0] += pg_term[t];
    v[1] += nll_term[t];
    const uint8_t st = rowstat[t];
    v[2] += (st & kStatValid) ? 1.0 : 0.0;
    v[3] += (st & kStatClipped) ? 1.0 : 0.0;
    v[4] += (st & kStatRead) ? 1.0 : 0.0;
  }
#pragma unroll
  for (int k = 0; k < 5; ++k) {
    for (int o = 16; o > 0; o >>= 1) v[k] += __shfl_xor_sync(0xffffffffu, v[k], o);
    if (lane == 0) red[k][warp] = v[k];
  }
  __syncthreads();
  if (warp == 0) {
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      double t = red[k][lane];
      for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
      v[k] = t;
    }
    if (lane == 0) {
      const bool accum = flags & MRL_FLAG_ACCUMULATE_LOSS;
      loss[0] = (accum ? loss[0] : 0.f) + (float)v[0];
      loss[1] = (accum ? loss[1] : 0.f) + (float)v[1];
      if (stats != nullptr) {
        stats[0] = (accum ? stats[0] : 0) + (long long)v[2];
        stats[1] = (accum ? stats[1] : 0) + (long long)v[3];
        stats[2] = (accum ? stats[2] : 0) + (long long)v[4];
        stats[3] = (accum ? stats[3] : 0) + (long long)totals[1];
      }
    }
  }
}

MrlLossWs carve_loss_ws(void* ws, long long N, int S) {
  MrlCarver c(ws);
  MrlLossWs w;
  w.totals = c.take<unsigned long long>(4);
  w.rowA = c.take<float>((size_t)N);
  w.rowcu = c.take<float>((size_t)N);
  w.rowcn = c.take<float>((size_t)N);
  w.row_m2 = c.take<float>((size_t)N);
  w.row_s = c.take<float>((size_t)N);
  w.row_zt = c.take<float>((size_t)N);
  w.pg_term = c.take<double>((size_t)N);
  w.nll_term = c.take<double>((size_t)N);
  w.rowstat = c.take<uint8_t>((size_t)N);
  w.seq_cnt = c.take<int32_t>((size_t)S + 1);
  w.bytes = c.off;
  return w;
}

// Picks the fast path when its alignment rules hold; returns the cluster size (0 = general kernel).
int pick_cluster(const RowParams& p, int dtype) {
  if (dtype != MRL_BF16) return 0;
  if (p.V % 8 != 0 || p.ld % 8 != 0) return 0;
  if ((reinterpret_cast<uintptr_t>(p.logits) & 15) != 0) return 0;
  if (p.dlogits != nullptr && (p.ld_out % 8 != 0 || (reinterpret_cast<uintptr_t>(p.dlogits) & 15) != 0)) return 0;
  if (p.V < 4096) return 0;  // short rows: the general kernel's three passes stay in cache
  int C = 1;
  while ((long long)p.V * 2 > (long long)C * kMaxPartBytes) C *= 2;
  return C <= kMaxCluster ? C : 0;
}

int launch_rows(RowParams p, int dtype, cudaStream_t st) {
  if (p.N == 0) return MRL_OK;
  if (p.N > 0x7fffffffll / kMaxCluster) return MRL_ERR_UNSUPPORTED_SHAPE;
  const int C = pick_cluster(p, dtype);
  if (C == 0) {
    mrl_profile_before(st);
    if (dtype == MRL_BF16)
      row_general_kernel<__nv_bfloat16><<<(unsigned)p.N, kThreads, 0, st>>>(p);
    else
      row_general_kernel<float><<<(unsigned)p.N, kThreads, 0, st>>>(p);
    mrl_profile_after(st);
    return cudaGetLastError() == cudaSuccess ? MRL_OK : MRL_ERR_CUDA;
  }
  const int vecs = (p.V / 8 + C - 1) / C;
  p.part_elems = vecs * 8;
  p.cluster = C;
  const size_t smem = (size_t)p.part_elems * 2 + kTailBytes;
  // per device and idempotent; set on every call so that a change of the current device is harmless
  MRL_CUDA_OK(cudaFuncSetAttribute(row_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(p.N * C));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  mrl_profile_before(st);
  MRL_CUDA_OK(cudaLaunchKernelEx(&cfg, row_cluster_kernel, p));
  mrl_profile_after(st);
  return MRL_OK;
}

bool dtype_ok(int dtype) { return dtype == MRL_BF16 || dtype == MRL_F32; }

}  // namespace

size_t mrl_policy_loss_workspace_bytes(long long N, int S) { return carve_loss_ws(nullptr, N, S).bytes; }

// Per-sequence bookkeeping shared by the logits-in and the hidden-in pass: carves the per-row scratch, counts the
// valid tokens of every sequence and fills A_t, c_t u_t and cn_t of every row.
int mrl_rows_prepare(void* workspace, long long N, int V, int S, const int32_t* ids, const uint8_t* mask,
                     const int32_t* cu_seqlens, const float* adv_seq, const float* tok_weight,
                     const float* nll_weight, const mrl_loss_params* lp, int32_t* status, cudaStream_t st,
                     MrlLossWs* out) {
  MrlLossWs w = carve_loss_ws(workspace, N, S);
  // rows no sequence covers must contribute nothing: clear the coefficient arrays and the totals
  MRL_CUDA_OK(cudaMemsetAsync(w.totals, 0, (size_t)((char*)w.row_m2 - (char*)w.totals), st));
  seq_count_kernel<<<S, 128, 0, st>>>(cu_seqlens, S, N, V, ids, mask, w.seq_cnt, w.totals, status);
  MRL_CUDA_OK(cudaGetLastError());
  row_coef_kernel<<<S, 128, 0, st>>>(cu_seqlens, S, N, V, ids, mask, adv_seq, tok_weight, nll_weight, w.seq_cnt,
                                     w.totals, *lp, w.rowA, w.rowcu, w.rowcn);
  MRL_CUDA_OK(cudaGetLastError());
  *out = w;
  return MRL_OK;
}

// Float64 loss terms from the per-row reduction triples, then the fixed-order sums into loss / stats.
int mrl_rows_finish(const MrlLossWs& w, long long N, const float* logp_old, const mrl_loss_params* lp, float* logp,
                    float* loss, int64_t* stats, cudaStream_t st) {
  row_terms_kernel<<<(unsigned)((N + 255) / 256), 256, 0, st>>>(N, w.row_m2, w.row_s, w.row_zt, w.rowstat, w.rowA,
                                                                w.rowcu, w.rowcn, logp_old, lp->eps_lo, lp->eps_hi,
                                                                w.pg_term, w.nll_term, logp);
  MRL_CUDA_OK(cudaGetLastError());
  finalize_kernel<<<1, 1024, 0, st>>>(w.pg_term, w.nll_term, w.rowstat, N, w.totals, lp->flags, loss,
                                      reinterpret_cast<long long*>(stats));
  MRL_CUDA_OK(cudaGetLastError());
  return MRL_OK;
}

extern "C" int mrl_token_logprobs(const void* logits, int32_t dtype, int64_t N, int32_t V, int64_t ld,
                                  const int32_t* ids, const uint8_t* mask, float* logp, float* lse, int32_t* status,
                                  void* workspace, size_t workspace_bytes, void* stream) {
  (void)workspace;
  (void)workspace_bytes;
  if (!dtype_ok(dtype)) return MRL_ERR_UNSUPPORTED_DTYPE;
  if (N < 0 || V < 1 || ld < V) return MRL_ERR_INVALID_ARG;
  if (N == 0) return MRL_OK;
  if (logits == nullptr || ids == nullptr || logp == nullptr) return MRL_ERR_INVALID_ARG;
  RowParams p = {};
  p.logits = logits;
  p.ld = ld;
  p.ld_out = ld;
  p.N = N;
  p.V = V;
  p.ids = ids;
  p.mask = mask;
  p.logp = logp;
  p.lse = lse;
  p.status = status;
  p.loss_mode = 0;
  return launch_rows(p, dtype, static_cast<cudaStream_t>(stream));
}

extern "C" int mrl_policy_loss_fwd_bwd(const void* logits, int32_t dtype, int64_t N, int32_t V, int64_t ld,
                                       const int32_t* ids, const uint8_t* mask, const int32_t* cu_seqlens, int32_t S,
                                       const float* adv_seq, const float* logp_old, const float* tok_weight,
                                       const float* nll_weight, const mrl_loss_params* lp, void* dlogits,
                                       int64_t ld_out, float* logp, float* loss, int64_t* stats, int32_t* status,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  if (!dtype_ok(dtype)) return MRL_ERR_UNSUPPORTED_DTYPE;
  if (lp == nullptr || loss == nullptr || N < 0 || S < 0 || V < 1 || ld < V) return MRL_ERR_INVALID_ARG;
  if (dlogits != nullptr && ld_out < V) return MRL_ERR_INVALID_ARG;
  if (lp->agg_mode != MRL_AGG_TOKEN_MEAN && lp->agg_mode != MRL_AGG_SEQ_MEAN_TOKEN_MEAN) return MRL_ERR_INVALID_ARG;
  if (!(lp->eps_lo >= 0.f) || !(lp->eps_hi >= 0.f)) return MRL_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool accum = lp->flags & MRL_FLAG_ACCUMULATE_LOSS;
  if (N == 0 || S == 0) {
    if (N != 0) return MRL_ERR_INVALID_ARG;  // rows without a sequence
    if (!accum) {
      MRL_CUDA_OK(cudaMemsetAsync(loss, 0, 2 * sizeof(float), st));
      if (stats != nullptr) MRL_CUDA_OK(cudaMemsetAsync(stats, 0, 4 * sizeof(int64_t), st));
    }
    return MRL_OK;
  }
  if (logits == nullptr || ids == nullptr || cu_seqlens == nullptr || adv_seq == nullptr) return MRL_ERR_INVALID_ARG;
  const size_t need = mrl_policy_loss_workspace_bytes(N, S);
  if (workspace == nullptr || workspace_bytes < need) return MRL_ERR_WORKSPACE_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MRL_ERR_INVALID_ARG;
  MrlLossWs w;
  int rc = mrl_rows_prepare(workspace, N, V, S, ids, mask, cu_seqlens, adv_seq, tok_weight, nll_weight, lp, status, st,
                            &w);
  if (rc != MRL_OK) return rc;

  RowParams p = {};
  p.logits = logits;
  p.dlogits = dlogits;
  p.ld = ld;
  p.ld_out = dlogits ? ld_out : ld;
  p.N = N;
  p.V = V;
  p.ids = ids;
  p.mask = mask;
  p.rowA = w.rowA;
  p.rowcu = w.rowcu;
  p.rowcn = w.rowcn;
  p.logp_old = logp_old;
  p.eps_lo = lp->eps_lo;
  p.eps_hi = lp->eps_hi;
  p.flags = lp->flags;
  p.loss_mode = 1;
  p.row_m2 = w.row_m2;
  p.row_s = w.row_s;
  p.row_zt = w.row_zt;
  p.rowstat = w.rowstat;
  p.status = status;
  rc = launch_rows(p, dtype, st);
  if (rc != MRL_OK) return rc;
  return mrl_rows_finish(w, N, logp_old, lp, logp, loss, stats, st);
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of mrl_policy_loss_fwd_bwd: the scratch lives in the library image.
// ------------------------------------------------------------------------------------------------
namespace {

// Per-row and per-sequence scratch of the loss pass for the largest problem the static entry point takes.
// Every device that loads the library keeps one copy of this array until the process exits.
constexpr size_t kStaticWsBytes = MRL_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_loss_ws[kStaticWsBytes];

constexpr int kMaxDevices = 64;
void* g_static_ws_ptr[kMaxDevices] = {};  // device address of the array, per device ordinal (0 = not looked up yet)

// In host code `g_static_loss_ws` is only a handle; the device address has to be asked for, with the
// device it is wanted on current.  Looked up once per device and cached.
int static_ws_address(void** out) {
  int dev = -1;
  MRL_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return MRL_ERR_UNSUPPORTED_SHAPE;
  if (g_static_ws_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    MRL_CUDA_OK(cudaGetSymbolAddress(&ptr, g_static_loss_ws));
    if (ptr == nullptr) return MRL_ERR_CUDA;
    g_static_ws_ptr[dev] = ptr;
  }
  *out = g_static_ws_ptr[dev];
  return MRL_OK;
}

}  // namespace

extern "C" int mrl_policy_loss_fwd_bwd_static(const void* logits, int32_t dtype, int64_t N, int32_t V, int64_t ld,
                                              const int32_t* ids, const uint8_t* mask, const int32_t* cu_seqlens,
                                              int32_t S, const float* adv_seq, const float* logp_old,
                                              const float* tok_weight, const float* nll_weight,
                                              const mrl_loss_params* lp, void* dlogits, int64_t ld_out, float* logp,
                                              float* loss, int64_t* stats, int32_t* status, void* stream) {
  if (N < 0 || S < 0) return MRL_ERR_INVALID_ARG;
  if (N > MRL_STATIC_MAX_ROWS || S > MRL_STATIC_MAX_SEQS) return MRL_ERR_STATIC_SCRATCH_TOO_SMALL;
  if (mrl_policy_loss_workspace_bytes(N, S) > kStaticWsBytes) return MRL_ERR_STATIC_SCRATCH_TOO_SMALL;
  void* ws = nullptr;
  if (N > 0 && S > 0) {  // the empty call needs no scratch and touches no symbol
    const int rc = static_ws_address(&ws);
    if (rc != MRL_OK) return rc;
  }
  // The callee clears the part of the scratch that has to start at zero on every call (the coefficient
  // arrays and the counters); everything else is overwritten before it is read.
  return mrl_policy_loss_fwd_bwd(logits, dtype, N, V, ld, ids, mask, cu_seqlens, S, adv_seq, logp_old, tok_weight,
                                 nll_weight, lp, dlogits, ld_out, logp, loss, stats, status, ws, kStaticWsBytes, stream);
}
