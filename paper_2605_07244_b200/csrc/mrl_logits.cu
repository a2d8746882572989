// Logits-in path: mrl_token_logprobs and mrl_policy_loss_fwd_bwd.
//
// Streaming kernel (bf16 or float32, 16- or 32-byte aligned rows of at least 4,096 columns): one CTA per logits
// row, two CTAs per SM.  Pass 1 streams the row from HBM with wide loads while keeping a running (max, sum of
// exponentials) per thread; after the block reduction and the ratio / clip / loss scalars, pass 2 takes the row
// again -- from registers, shared memory and L2 -- and writes g * (softmax - onehot) with streaming stores.  The row
// crosses the HBM interface once in each direction (plus what L2 has dropped); nothing is shared between CTAs.
// General kernel (any dtype, any V, any alignment): one CTA per row, three passes over global
// memory; used for short or unaligned rows.
#include <mutex>
#include <type_traits>

#include "mrl_common.cuh"

namespace {

constexpr int kThreads = 256;        // general kernel
constexpr int kStreamThreads = 512;  // streaming kernel: two CTAs per SM
constexpr long long kSplitRowBytes = 512 * 1024;  // rows at least this long are split over a cluster of two CTAs
// Shared memory per CTA that holds the oldest vectors of its row between the passes.  More is not better: the
// carve-out comes out of L1, and L1 is what keeps this kernel's loads in flight (measured on B200, ms per step on
// 34 k rows of 304 KB, half / all of them with a gradient: 0 KB 3.40 / 3.88, 32 KB 3.35 / 3.82, 48 KB 3.35 / 3.79,
// 64 KB 3.37 / 3.81, 80 KB 3.38 / 3.79, 96 KB 4.09 / 4.37).
constexpr int kParkBytes = 48 * 1024;

// internal bit of RowParams.flags (not part of the ABI): rows outside every sequence are not read and report an empty
// reduction triple, so the response-level pass, whose per-response kernel writes covered rows only, leaves them at g = 0
constexpr uint32_t kFlagSkipUncovered = 1u << 31;

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
  const float* rowck;     // KL term: beta c_t; read only when logp_ref is given
  const float* cscale;    // [1] common factor of rowcu and rowck (the token-mean 1 / D when it was not known up front, else 1)
  const float* logp_ref;  // nullable
  int kl_est;
  const float* logp_old;
  float eps_lo, eps_hi;
  uint32_t flags;
  int loss_mode;  // 0: log-probs only, 1: loss (+ gradient when dlogits != null)
  float* logp;
  float* lse;
  float* entropy;  // nullable: per-row entropy of softmax(z_t) (diagnostic)
  float* row_m2;  // loss mode: per-row (max, sum, target) of the base-2 log-sum-exp, finished in float64 later
  float* row_s;
  float* row_zt;
  uint8_t* rowstat;
  int32_t* status;
  int keep_q;  // streaming kernel: how many groups of blockDim vectors, the first ones pass 1 reads, are parked
};

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
  c.in.ck = 0.f;
  c.in.logp_ref = 0.f;
  c.in.kl_est = p.kl_est;
  if (p.loss_mode) {
    const float cs = p.cscale[0];
    c.in.A = p.rowA[row];
    c.in.cu = p.rowcu[row] * cs;
    c.in.cn = p.rowcn[row];
    c.in.has_old = p.logp_old != nullptr;
    if (c.in.has_old) c.in.logp_old = p.logp_old[row];
    if (p.logp_ref != nullptr) {
      c.in.ck = p.rowck[row] * cs;
      c.in.logp_ref = p.logp_ref[row];
    }
  }
  c.dead = !c.valid;
  if (p.loss_mode && (p.flags & MRL_FLAG_SKIP_ZERO_ROWS) && (c.in.cu == 0.f || c.in.A == 0.f) && c.in.cn == 0.f &&
      c.in.ck == 0.f)
    c.dead = true;
  // a row that no sequence covers has all its coefficients at zero (they were cleared before the sequences wrote theirs)
  if (p.loss_mode && (p.flags & kFlagSkipUncovered) && c.in.cu == 0.f && c.in.cn == 0.f && c.in.ck == 0.f) c.dead = true;
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

// scalar element access in either logits type
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

// packed maximum of two bf16 pairs
__device__ __forceinline__ uint32_t hmax2_u32(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// ------------------------------------------------------------------------------------------------
// Streaming kernel: one CTA per row; shared memory holds only the few vectors parked between the passes.
// Pass 1 streams the row from HBM with 128- or 256-bit loads (running maximum and rescaled sum per thread);
// pass 2 needs the same vectors again: the last group read is still in registers, the first 48 KB read were
// parked in shared memory, the rest comes from L2 -- the rows in flight (two per SM) are a fraction of its
// capacity, and the first read asks L2 to keep the lines -- and g * (softmax - onehot) leaves with streaming
// stores.  HBM sees one read and one write of the row (plus the second reads L2 misses).  Many small CTAs with
// deep unrolling keep far more bytes in flight per SM than a slice fetched into shared memory does, which is what
// this memory-bound pass needs.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
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
constexpr uint32_t kExchangeSpinLimit = 1u << 22;  // polls of the peer's triple before giving up (~a second)

template <int kWords>
struct StreamVec {
  uint32_t w[kWords];
};
enum { kHintKeep = 0, kHintLast = 1 };

template <int kWords, int kHint>
__device__ __forceinline__ StreamVec<kWords> stream_ld(const void* p) {
  StreamVec<kWords> v;
  if constexpr (kWords == 8) {
    if constexpr (kHint == kHintKeep)
      asm volatile("ld.global.L1::no_allocate.L2::evict_last.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]),
                     "=r"(v.w[7])
                   : "l"(p));
    else
      asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]),
                     "=r"(v.w[7])
                   : "l"(p));
  } else {
    asm volatile("ld.global.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "l"(p));
  }
  return v;
}
// Output lines are never read again: they are marked evict-first in L2 so that they do not push out the rows that
// wait for their second read (the `.cs` qualifier alone does not do that).
template <int kWords>
__device__ __forceinline__ void stream_st(void* p, const StreamVec<kWords>& v) {
  if constexpr (kWords == 8) {
    asm volatile("st.global.L2::evict_first.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v.w[0]),
                 "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7])
                 : "memory");
  } else {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]),
                 "r"(v.w[2]), "r"(v.w[3]), "l"(pol)
                 : "memory");
  }
}
// A thread's own vectors parked in shared memory between the passes (only the thread that wrote one reads it back,
// so no barrier is needed).  256-bit vectors are kept as two planes of 16-byte halves: every 16-byte access of a
// warp is then contiguous.
template <int kWords>
__device__ __forceinline__ void park_st(uint32_t base, uint32_t plane_bytes, uint32_t slot, const StreamVec<kWords>& v) {
  const uint32_t a = base + slot * 16u;
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3])
               : "memory");
  if constexpr (kWords == 8)
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a + plane_bytes), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]),
                 "r"(v.w[7])
                 : "memory");
}
template <int kWords>
__device__ __forceinline__ StreamVec<kWords> park_ld(uint32_t base, uint32_t plane_bytes, uint32_t slot) {
  StreamVec<kWords> v;
  const uint32_t a = base + slot * 16u;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "r"(a));
  if constexpr (kWords == 8)
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7])
                 : "r"(a + plane_bytes));
  return v;
}

template <int kWords>
__device__ __forceinline__ StreamVec<kWords> stream_fill(uint32_t x) {
  StreamVec<kWords> v;
#pragma unroll
  for (int j = 0; j < kWords; ++j) v.w[j] = x;
  return v;
}

// kC = 1: the CTA takes the whole row.  kC = 2: a cluster of two CTAs takes the row, half each, and the halves'
// (max, sum, target logit) cross through distributed shared memory: a remote store plus a remote mbarrier arrive.
// kF32: float32 logits (one element per 32-bit word) instead of bf16 (two).
template <int kT, int kU, int kWords, int kC, bool kEnt, bool kF32>
__global__ void __launch_bounds__(kT, 1024 / kT) row_stream_kernel(const RowParams p) {
  constexpr int kWarpsT = kT / 32;
  constexpr int kVecBytes = kWords * 4, kVecElems = kF32 ? kWords : kWords * 2;
  constexpr uint32_t kNegInf = kF32 ? 0xff800000u : 0xff80ff80u;  // -inf, or a pair of them
  using Elem = typename std::conditional<kF32, float, __nv_bfloat16>::type;
  using Vec = StreamVec<kWords>;
  __shared__ float red[3 * 32];
  __shared__ float fin[4];
  __shared__ __align__(16) float4 xchg[2];
  __shared__ __align__(8) uint64_t xbar;
  extern __shared__ __align__(16) unsigned char parked[];  // keep_q * kT vectors
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int keep_q = p.keep_q;
  const uint32_t park_base = smem_u32(parked), park_plane = (uint32_t)keep_q * kT * 16u;
  const long long row = blockIdx.x / kC;
  const int rank = blockIdx.x % kC;  // rank in the 1-D cluster
  const int row_nvec = p.V / kVecElems;
  const int part_nvec = (row_nvec + kC - 1) / kC;
  const int part_off = rank * part_nvec * kVecElems;               // first element of this CTA's part
  const int nvec = max(0, min(row_nvec - rank * part_nvec, part_nvec));
  const bool want_grad = p.dlogits != nullptr;
  const Elem* grow = static_cast<const Elem*>(p.logits) + row * p.ld + part_off;
  Elem* orow = want_grad ? static_cast<Elem*>(p.dlogits) + row * p.ld_out + part_off : nullptr;
  const char* in = reinterpret_cast<const char*>(grow) + (size_t)tid * kVecBytes;
  char* out = reinterpret_cast<char*>(orow) + (size_t)tid * kVecBytes;

  const RowCtx ctx = load_row_ctx(p, row);
  if (ctx.dead) {
    if (orow != nullptr)
      for (int i = tid; i < nvec; i += kT) stream_st<kWords>(out + (size_t)(i - tid) * kVecBytes, stream_fill<kWords>(0u));
    if (rank == 0 && tid == 0) {
      write_row_scalars(p, row, ctx, 0.f, 0.f, mrl::lse2_empty(), 0.f, false, false);
      if (kEnt) p.entropy[row] = 0.f;
    }
    return;  // both CTAs of a cluster take this branch: no cluster barrier is left waiting
  }
  if (kC > 1) {
    if (tid == 0) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&xbar)), "r"(kC - 1) : "memory");
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // "my exchange barrier exists": the peer waits for this just before its remote store
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  }
  const int rel = ctx.id - part_off;                               // target column relative to this part
  const bool owner = ctx.valid && rel >= 0 && rel < nvec * kVecElems;
  float zt = 0.f;
  if (tid == 0 && owner) zt = ld_as_f32<Elem>(grow + rel);         // before anything is written in place

  // ---- pass 1: running (max, sum) in the base-2 domain
  // The row is walked from its last group of kT * kU vectors (the ragged one) down to its first, so that the group
  // read last is a full one: its vectors stay in registers over the reduction and pass 2 starts from them.
  float m_run = -INFINITY, s_run = 0.f, u_run = 0.f;  // u: sum of 2^(x - m) z, for the entropy (kEnt only)
  const int last_base = ((nvec - 1) / (kT * kU)) * (kT * kU);
  Vec v[kU];
  for (int base = last_base; base >= 0; base -= kT * kU) {
    if (base + kT * kU <= nvec) {
#pragma unroll
      for (int u = 0; u < kU; ++u) v[u] = stream_ld<kWords, kHintKeep>(in + (size_t)(base + u * kT) * kVecBytes);
    } else {
#pragma unroll
      for (int u = 0; u < kU; ++u)
        v[u] = (base + u * kT + tid < nvec) ? stream_ld<kWords, kHintKeep>(in + (size_t)(base + u * kT) * kVecBytes)
                                            : stream_fill<kWords>(kNegInf);
    }
    // the first vectors read are the ones L2 is likeliest to have dropped by pass 2: park them
    const int q0 = ((last_base - base) / (kT * kU)) * kU;
    if (q0 < keep_q) {
#pragma unroll
      for (int u = 0; u < kU; ++u)
        if (q0 + u < keep_q && base + u * kT + tid < nvec)
          park_st<kWords>(park_base, park_plane, (uint32_t)((q0 + u) * kT + tid), v[u]);
    }
    float vmax;
    if constexpr (kF32) {
      vmax = -INFINITY;
#pragma unroll
      for (int u = 0; u < kU; ++u) {
#pragma unroll
        for (int j = 0; j < kWords; ++j) vmax = fmaxf(vmax, __uint_as_float(v[u].w[j]));
      }
    } else {
      uint32_t mx = kNegInf;
#pragma unroll
      for (int u = 0; u < kU; ++u) {
#pragma unroll
        for (int j = 0; j < kWords; ++j) mx = hmax2_u32(mx, v[u].w[j]);
      }
      vmax = fmaxf(mrl::bf16lo_to_f32(mx), mrl::bf16hi_to_f32(mx));
    }
    const float m_new = fmaxf(m_run, vmax * MRL_LOG2E);
    if (m_new > m_run) {  // also the first group (m_run = -inf, s_run = 0)
      const float f = mrl::ex2_approx(m_run - m_new);
      s_run *= f;
      if (kEnt) u_run *= f;
      m_run = m_new;
    }
    if (m_run != -INFINITY) {
      const float neg_m = -m_run;
      float s0 = 0.f, s1 = 0.f, u0 = 0.f, u1 = 0.f;
#pragma unroll
      for (int u = 0; u < kU; ++u) {
#pragma unroll
        for (int j = 0; j < kWords; ++j) {
          if constexpr (kF32) {
            const float z = __uint_as_float(v[u].w[j]);
            const float a = mrl::ex2_approx(fmaf(z, MRL_LOG2E, neg_m));
            if (j & 1) s1 += a; else s0 += a;
            if (kEnt) {  // a = 0 exactly where z = -inf: keep 0 * inf out of the sum
              if (j & 1) u1 = a != 0.f ? fmaf(a, z, u1) : u1; else u0 = a != 0.f ? fmaf(a, z, u0) : u0;
            }
          } else {
            const float zlo = mrl::bf16lo_to_f32(v[u].w[j]), zhi = mrl::bf16hi_to_f32(v[u].w[j]);
            const float a = mrl::ex2_approx(fmaf(zlo, MRL_LOG2E, neg_m)), b = mrl::ex2_approx(fmaf(zhi, MRL_LOG2E, neg_m));
            s0 += a;
            s1 += b;
            if (kEnt) {
              u0 = a != 0.f ? fmaf(a, zlo, u0) : u0;
              u1 = b != 0.f ? fmaf(b, zhi, u1) : u1;
            }
          }
        }
      }
      s_run += s0 + s1;
      if (kEnt) u_run += u0 + u1;
    }
  }
  // ---- block totals: maximum first, one rescale, then a plain sum (fixed order: reproducible)
  float m = m_run;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  const float rescale = m_run != -INFINITY ? mrl::ex2_approx(m_run - m) : 0.f;
  float sum = s_run * rescale, usum = kEnt ? u_run * rescale : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (kEnt) usum += __shfl_xor_sync(0xffffffffu, usum, o);
  }
  if (lane == 0) {
    red[warp] = m;
    red[32 + warp] = sum;
    if (kEnt) red[64 + warp] = usum;
  }
  __syncthreads();
  if (warp == 0) {
    const float wm = lane < kWarpsT ? red[lane] : -INFINITY, ws = lane < kWarpsT ? red[32 + lane] : 0.f;
    float tm = wm;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, o));
    const float wscale = wm != -INFINITY ? mrl::ex2_approx(wm - tm) : 0.f;
    float ts = ws * wscale, tu = (kEnt && lane < kWarpsT) ? red[64 + lane] * wscale : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ts += __shfl_xor_sync(0xffffffffu, ts, o);
      if (kEnt) tu += __shfl_xor_sync(0xffffffffu, tu, o);
    }
    bool ok = true;
    if (kC > 1) {
      asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // the peer's barrier is initialised
      if (lane == 0) {
        xchg[rank] = make_float4(tm, ts, zt, owner ? 1.f : 0.f);
        const uint32_t peer = (uint32_t)(rank ^ 1);
        const uint32_t dst = mapa_u32(smem_u32(&xchg[rank]), peer);
        asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(tm), "f"(ts), "f"(zt),
                     "f"(owner ? 1.f : 0.f)
                     : "memory");
        asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(mapa_u32(smem_u32(&xbar), peer))
                     : "memory");
        bool got = false;
        for (uint32_t i = 0; i < kExchangeSpinLimit && !got; ++i) got = mbar_try_wait_cluster(&xbar, 0);
        ok = got;
        if (got) {  // rank order, so both CTAs form the same sums
          const float4 a = xchg[0], b = xchg[1];
          tm = fmaxf(a.x, b.x);
          ts = (a.x != -INFINITY ? a.y * mrl::ex2_approx(a.x - tm) : 0.f) +
               (b.x != -INFINITY ? b.y * mrl::ex2_approx(b.x - tm) : 0.f);
          zt = a.w != 0.f ? a.z : (b.w != 0.f ? b.z : 0.f);
        } else if (p.status != nullptr) {
          atomicOr(p.status, MRL_DEV_TIMEOUT);
        }
      }
    }
    if (lane == 0) {
      const float lse2 = tm + log2f(ts);
      const float lse = mrl::lse2_to_nats(lse2);
      float logp = 0.f, g = 0.f;
      bool clipped = false;
      if (ctx.valid && ok) {
        logp = zt - lse;
        if (p.loss_mode) {
          const mrl::RowOut ro = mrl::mrl_row_loss(logp, ctx.in, p.eps_lo, p.eps_hi);
          g = ro.g;
          clipped = ro.clipped;
        }
      }
      if (rank == 0 && ok) write_row_scalars(p, row, ctx, logp, ctx.valid ? lse : 0.f, mrl::Lse2{tm, ts}, zt, clipped, true);
      if (kEnt) p.entropy[row] = ctx.valid ? lse - tu / ts : 0.f;  // H = lse - sum_v p_v z_v
      fin[0] = lse2;
      fin[1] = g;
      fin[2] = g * (mrl::ex2_approx(fmaf(zt, MRL_LOG2E, -lse2)) - 1.0f);
      fin[3] = ok ? 1.f : 0.f;
    }
  } else if (kC > 1) {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // pairs with the arrive above
  }
  __syncthreads();
  // Neither CTA of a pair may leave while its peer can still write into its shared memory (the exchange's remote
  // store and remote arrive).  Each CTA signals here, after its own remote accesses were issued, and waits for the
  // peer's signal just before it exits -- also when its bounded wait for the triple ran out.
  if (kC > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  auto leave = [] {
    if (kC > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  };
  if (!want_grad || fin[3] == 0.f) {
    leave();
    return;
  }
  const float lse2 = fin[0], g = fin[1], tfix = fin[2];

  // ---- pass 2: the same vectors again (L2), dlogits = g 2^(z log2e - lse2), the target column patched after
  if (g == 0.f) {
    for (int i = tid; i < nvec; i += kT) stream_st<kWords>(out + (size_t)(i - tid) * kVecBytes, stream_fill<kWords>(0u));
    leave();
    return;
  }
  const float neg_k = -(lse2 - log2f(fabsf(g)));  // 2^(z log2e - k) = |g| softmax(z)
  const uint32_t sign = g < 0.f ? (kF32 ? 0x80000000u : 0x80008000u) : 0u;
  // (the first group is still in registers; the others in the order pass 1 read them last-to-first, so the most
  // recently loaded lines, the likeliest to be still in L2, come first; the oldest come back from shared memory)
  for (int base = 0; base <= last_base; base += kT * kU) {
    const bool full = base + kT * kU <= nvec;
    if (base != 0) {
      const int q0 = ((last_base - base) / (kT * kU)) * kU;
#pragma unroll
      for (int u = 0; u < kU; ++u)
        v[u] = !(full || base + u * kT + tid < nvec) ? stream_fill<kWords>(0u)
               : (q0 + u < keep_q)                   ? park_ld<kWords>(park_base, park_plane, (uint32_t)((q0 + u) * kT + tid))
                                                     : stream_ld<kWords, kHintLast>(in + (size_t)(base + u * kT) * kVecBytes);
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      Vec r;
#pragma unroll
      for (int j = 0; j < kWords; ++j) {
        if constexpr (kF32) {
          r.w[j] = __float_as_uint(mrl::ex2_approx(fmaf(__uint_as_float(v[u].w[j]), MRL_LOG2E, neg_k))) ^ sign;
        } else {
          const float a = mrl::ex2_approx(fmaf(mrl::bf16lo_to_f32(v[u].w[j]), MRL_LOG2E, neg_k));
          const float b = mrl::ex2_approx(fmaf(mrl::bf16hi_to_f32(v[u].w[j]), MRL_LOG2E, neg_k));
          r.w[j] = mrl::pack_bf16x2(a, b) ^ sign;
        }
      }
      if (full || base + u * kT + tid < nvec) stream_st<kWords>(out + (size_t)(base + u * kT) * kVecBytes, r);
    }
  }
  // the thread whose vector store covered the target column patches it (program order on one address)
  if (owner && tid == (rel / kVecElems) % kT) st_from_f32<Elem>(orow + rel, tfix);
  leave();
}

// ------------------------------------------------------------------------------------------------
// General kernel: one CTA per row, any dtype / V / alignment.
// ------------------------------------------------------------------------------------------------

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
    if (tid == 0) {
      write_row_scalars(p, row, ctx, 0.f, 0.f, mrl::lse2_empty(), 0.f, false, false);
      if (p.entropy != nullptr) p.entropy[row] = 0.f;
    }
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
  const float lse = mrl::lse2_to_nats(lse2);
  const float logp = zt - lse;
  float g = 0.f;
  bool clipped = false;
  if (p.loss_mode) {
    const mrl::RowOut ro = mrl::mrl_row_loss(logp, ctx.in, p.eps_lo, p.eps_hi);
    g = ro.g;
    clipped = ro.clipped;
  }
  if (tid == 0) write_row_scalars(p, row, ctx, logp, lse, tot, zt, clipped, true);
  if (p.entropy != nullptr) {  // H = lse - sum_v p_v z_v, p_v = 2^(z_v log2e - lse2)
    float u = 0.f;
    for (int v = tid; v < p.V; v += kThreads) {
      const float zv = ld_as_f32<T>(z + v);
      const float pv = mrl::ex2_approx(fmaf(zv, MRL_LOG2E, -lse2));
      u = pv != 0.f ? fmaf(pv, zv, u) : u;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) u += __shfl_xor_sync(0xffffffffu, u, o);
    __syncthreads();
    if ((tid & 31) == 0) scratch[tid >> 5] = u;
    __syncthreads();
    if (tid == 0) {
      float t = 0.f;
      for (int k = 0; k < kThreads / 32; ++k) t += scratch[k];
      p.entropy[row] = lse - t;
    }
    __syncthreads();
  }
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
// Backward-only row kernels (response-level ratio): g_t is known only once the whole response has been scored, so
// the gradient is a launch of its own that reads the row again.
// ------------------------------------------------------------------------------------------------
template <int kT, int kU, int kWords, bool kF32>
__global__ void __launch_bounds__(kT, 1024 / kT) row_backward_stream_kernel(const RowParams p, const float* __restrict__ row_g,
                                                                            const float* __restrict__ row_lse2,
                                                                            const float* __restrict__ row_zt) {
  constexpr int kVecBytes = kWords * 4, kVecElems = kF32 ? kWords : kWords * 2;
  using Elem = typename std::conditional<kF32, float, __nv_bfloat16>::type;
  using Vec = StreamVec<kWords>;
  const int tid = threadIdx.x;
  const long long row = blockIdx.x;
  const int nvec = p.V / kVecElems;
  const char* in = reinterpret_cast<const char*>(static_cast<const Elem*>(p.logits) + row * p.ld) +
                   (size_t)tid * kVecBytes;
  Elem* orow = static_cast<Elem*>(p.dlogits) + row * p.ld_out;
  char* out = reinterpret_cast<char*>(orow) + (size_t)tid * kVecBytes;
  const float g = row_g[row];
  if (g == 0.f) {
    for (int i = tid; i < nvec; i += kT) stream_st<kWords>(out + (size_t)(i - tid) * kVecBytes, stream_fill<kWords>(0u));
    return;
  }
  const float lse2 = row_lse2[row];
  const float neg_k = -(lse2 - log2f(fabsf(g)));  // 2^(z log2e - k) = |g| softmax(z)
  const uint32_t sign = g < 0.f ? (kF32 ? 0x80000000u : 0x80008000u) : 0u;
  for (int base = 0; base < nvec; base += kT * kU) {
    const bool full = base + kT * kU <= nvec;
    Vec v[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u)
      v[u] = (full || base + u * kT + tid < nvec) ? stream_ld<kWords, kHintLast>(in + (size_t)(base + u * kT) * kVecBytes)
                                                  : stream_fill<kWords>(0u);
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      Vec r;
#pragma unroll
      for (int j = 0; j < kWords; ++j) {
        if constexpr (kF32) {
          r.w[j] = __float_as_uint(mrl::ex2_approx(fmaf(__uint_as_float(v[u].w[j]), MRL_LOG2E, neg_k))) ^ sign;
        } else {
          const float a = mrl::ex2_approx(fmaf(mrl::bf16lo_to_f32(v[u].w[j]), MRL_LOG2E, neg_k));
          const float b = mrl::ex2_approx(fmaf(mrl::bf16hi_to_f32(v[u].w[j]), MRL_LOG2E, neg_k));
          r.w[j] = mrl::pack_bf16x2(a, b) ^ sign;
        }
      }
      if (full || base + u * kT + tid < nvec) stream_st<kWords>(out + (size_t)(base + u * kT) * kVecBytes, r);
    }
  }
  const int id = p.ids[row];  // g != 0 only on valid rows: the id is in range
  if (tid == (id / kVecElems) % kT)
    st_from_f32<Elem>(orow + id, g * (mrl::ex2_approx(fmaf(row_zt[row], MRL_LOG2E, -lse2)) - 1.0f));
}

template <typename T>
__global__ void __launch_bounds__(kThreads) row_backward_general_kernel(const RowParams p, const float* __restrict__ row_g,
                                                                        const float* __restrict__ row_lse2,
                                                                        const float* __restrict__ row_zt) {
  const int tid = threadIdx.x;
  const long long row = blockIdx.x;
  const T* z = static_cast<const T*>(p.logits) + row * p.ld;
  T* dz = static_cast<T*>(p.dlogits) + row * p.ld_out;
  const float g = row_g[row];
  if (g == 0.f) {
    for (int v = tid; v < p.V; v += kThreads) st_from_f32<T>(dz + v, 0.f);
    return;
  }
  const float lse2 = row_lse2[row];
  const float neg_k = -(lse2 - log2f(fabsf(g)));
  const float sgn = g < 0.f ? -1.f : 1.f;
  for (int v = tid; v < p.V; v += kThreads)
    st_from_f32<T>(dz + v, sgn * mrl::ex2_approx(fmaf(ld_as_f32<T>(z + v), MRL_LOG2E, neg_k)));
  __syncthreads();
  if (tid == 0) st_from_f32<T>(dz + p.ids[row], g * (mrl::ex2_approx(fmaf(row_zt[row], MRL_LOG2E, -lse2)) - 1.0f));
}

// Response-level ratio (App. H, data-level coupling): one block per response.  L_theta - L_behavior over the valid
// tokens in float64 (fixed order), w = exp of it, the clip decision, the response's loss term (kept on its first
// row), and for every row the gradient multiplier g_t = A w / S_d [unclipped] + cn_t and the base-2 log-sum-exp the
// backward launch needs.  g_out / lse2_out may alias row_s / row_m2 (each thread reads its row before writing it).
__global__ void __launch_bounds__(256) seq_ratio_kernel(const int32_t* __restrict__ cu, int S, long long N,
                                                         const float* row_m2, const float* row_s,
                                                         const float* __restrict__ row_zt, uint8_t* __restrict__ rowstat,
                                                         const int32_t* __restrict__ seq_cnt,
                                                         const float* __restrict__ adv_seq,
                                                         const float* __restrict__ logp_old,
                                                         const float* __restrict__ nll_weight,
                                                         const float* __restrict__ rowck,
                                                         const float* __restrict__ cscale, mrl_loss_params lp,
                                                         double* __restrict__ pg_term, double* __restrict__ nll_term,
                                                         double* __restrict__ kl_term, float* __restrict__ logp,
                                                         float* g_out, float* lse2_out) {
  __shared__ double red[8];
  __shared__ double diff_sh;
  const int s = blockIdx.x, tid = threadIdx.x;
  const long long a = max(0ll, min((long long)cu[s], N)), b = max(a, min((long long)cu[s + 1], N));
  const double kNat = MRL_NAT_F64;  // nats per unit of the base-2 sums (1 / the float log2 e they were scaled with)
  double d = 0.0;
  for (long long t = a + tid; t < b; t += 256) {
    const uint8_t st = rowstat[t];
    if ((st & kStatValid) && (st & kStatRead)) {
      const double lpv = (double)row_zt[t] - ((double)row_m2[t] + log2((double)row_s[t])) * kNat;
      d += lpv - (logp_old ? (double)logp_old[t] : lpv);
    }
  }
  for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
  if ((tid & 31) == 0) red[tid >> 5] = d;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int k = 0; k < 8; ++k) t += red[k];
    diff_sh = t;
  }
  __syncthreads();
  const double len = (double)seq_cnt[s];
  const double Sd = lp.seq_denominator > 0 ? lp.seq_denominator : (double)S;
  const double A = adv_seq[s];
  const double w = exp(diff_sh);
  const double lo = 1.0 - (double)lp.eps_lo, hi = 1.0 + (double)lp.eps_hi;
  const bool live = len > 0 && A != 0.0;
  const bool clipped = live && ((A > 0 && w > hi) || (A < 0 && w < lo));
  const double term = live ? -fmin(w * A, fmin(fmax(w, lo), hi) * A) / Sd : 0.0;
  const float g_pg = (live && !clipped) ? (float)(A * w / Sd) : 0.f;
  const double cn_base = len > 0 ? (double)lp.nll_coeff / len : 0.0;
  for (long long t = a + tid; t < b; t += 256) {
    const uint8_t st = rowstat[t];
    const bool valid = (st & kStatValid) && (st & kStatRead);
    double lpv = 0.0;
    float l2 = 0.f, g = 0.f;
    double nl = 0.0, kl = 0.0;
    if (valid) {
      l2 = row_m2[t] + log2f(row_s[t]);
      lpv = (double)row_zt[t] - ((double)row_m2[t] + log2((double)row_s[t])) * kNat;
      const float cn = nll_weight ? (float)cn_base * nll_weight[t] : 0.f;
      g = g_pg + cn;
      if (cn != 0.f) nl = -(double)cn * lpv;
      const float ck = lp.logp_ref != nullptr ? rowck[t] * cscale[0] : 0.f;
      if (ck != 0.f) {  // the KL term stays per token (App. A)
        const double d = lpv - (double)lp.logp_ref[t];
        kl = (double)ck * mrl::kl_value(d, lp.kl_estimator);
        g -= ck * mrl::kl_slope((float)d, lp.kl_estimator);
      }
      if (clipped) rowstat[t] = st | kStatClipped;
    }
    pg_term[t] = t == a ? term : 0.0;
    nll_term[t] = nl;
    kl_term[t] = kl;
    if (logp != nullptr) logp[t] = (float)lpv;
    lse2_out[t] = l2;
    g_out[t] = g;
  }
}

// ------------------------------------------------------------------------------------------------
// Per-sequence bookkeeping around the row kernel.
// ------------------------------------------------------------------------------------------------
// One block per sequence: its valid-token count (and bad-id detection), then A_t, c_t u_t, cn_t and beta c_t of its
// rows (Eq. (1) aggregation and regulariser, Eq. (2) per-token average).  When the token-mean denominator is the valid
// tokens of this very call, it is only known once every block has counted: the rows then get u_t and beta, and the
// common factor 1 / D is published in cscale[0] by the block that finishes last; consumers multiply by cscale[0],
// which is exactly 1 in every other case (the products are the same floats either way).  Rows that no sequence
// covers (before cu[0], after cu[S]) get zero coefficients from the first and the last block.
__global__ void __launch_bounds__(128) seq_prepare_kernel(const int32_t* __restrict__ cu, int S, long long N, int V,
                                                           const int32_t* __restrict__ ids,
                                                           const uint8_t* __restrict__ mask,
                                                           const float* __restrict__ adv_seq,
                                                           const float* __restrict__ tok_weight,
                                                           const float* __restrict__ nll_weight, mrl_loss_params lp,
                                                           int32_t* seq_cnt, unsigned long long* totals, float* cscale,
                                                           float* rowA, float* rowcu, float* rowcn, float* rowck,
                                                           int32_t* status) {
  __shared__ int red[2][4];
  __shared__ int len_sh;
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
  const bool defer = lp.agg_mode == MRL_AGG_TOKEN_MEAN && !(lp.pg_denominator > 0);
  if (threadIdx.x == 0) {
    cnt = red[0][0] + red[0][1] + red[0][2] + red[0][3];
    bad = red[1][0] + red[1][1] + red[1][2] + red[1][3];
    seq_cnt[s] = cnt;
    len_sh = cnt;
    atomicAdd(&totals[0], (unsigned long long)cnt);  // integer sums: order does not matter
    if (bad) {
      atomicAdd(&totals[1], (unsigned long long)bad);
      if (status != nullptr) atomicOr(status, MRL_DEV_BAD_TOKEN_ID);
    }
    __threadfence();
    if (atomicAdd(&totals[3], 1ull) == (unsigned long long)S - 1) {  // every block has added its count
      __threadfence();
      const double D = (double)atomicAdd(&totals[0], 0ull);
      cscale[0] = defer ? (D > 0 ? (float)(1.0 / D) : 0.f) : 1.0f;
    }
  }
  __syncthreads();
  const double len = (double)len_sh;
  const double Sd = lp.seq_denominator > 0 ? lp.seq_denominator : (double)S;
  float c = 0.f, cn_base = 0.f;
  if (len > 0) {
    if (lp.agg_mode == MRL_AGG_TOKEN_MEAN)
      c = defer ? 1.0f : (float)(1.0 / lp.pg_denominator);
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
    rowck[t] = (valid && lp.logp_ref != nullptr) ? lp.kl_coeff * c : 0.f;
  }
  // rows outside every sequence must contribute nothing
  const long long z0 = s == 0 ? 0 : N, z1 = s == 0 ? a : N;
  for (long long t = z0 + threadIdx.x; t < z1; t += blockDim.x) rowA[t] = rowcu[t] = rowcn[t] = rowck[t] = 0.f;
  if (s == S - 1)
    for (long long t = b + threadIdx.x; t < N; t += blockDim.x) rowA[t] = rowcu[t] = rowcn[t] = rowck[t] = 0.f;
}

// Sum of six per-thread float64 values over a block of 256 threads in a fixed order (shuffle tree inside a warp, then
// the warps in turn); the result is in thread 0.
__device__ __forceinline__ void block_sum6(double (&v)[6], double (*red)[8]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < 6; ++k) {
    for (int o = 16; o > 0; o >>= 1) v[k] += __shfl_xor_sync(0xffffffffu, v[k], o);
    if (lane == 0) red[k][warp] = v[k];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int k = 0; k < 6; ++k) {
      double t = 0.0;
      for (int w = 0; w < 8; ++w) t += red[k][w];
      v[k] = t;
    }
  }
}

// Fixed-order float64 sums of the blocks' partial sums (terms and row statistics) into loss / stats, by the block that
// finishes last: every block publishes its six partial sums, then takes a ticket; the one that draws the last ticket
// sees all of them and adds them up in block order, so the result does not depend on which block that was.
struct FinalizeArgs {
  double* partials;            // [gridDim.x][6]
  unsigned long long* totals;  // [1]: rows with a bad id; [2]: the ticket counter (zero before the launch, zero after)
  uint32_t flags;
  float* loss;
  float* kl_loss;              // nullable
  long long* stats;            // nullable
};
__device__ __forceinline__ void publish_and_finalize(double (&v)[6], double (*red)[8], const FinalizeArgs& f) {
  __shared__ bool is_last;
  if (threadIdx.x == 0) {
    for (int k = 0; k < 6; ++k) f.partials[(long long)blockIdx.x * 6 + k] = v[k];
    __threadfence();
    is_last = atomicAdd(&f.totals[2], 1ull) == (unsigned long long)gridDim.x - 1;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  double t[6] = {0, 0, 0, 0, 0, 0};
  for (long long b = threadIdx.x; b < (long long)gridDim.x; b += 256) {
#pragma unroll
    for (int k = 0; k < 6; ++k) t[k] += __ldcg(&f.partials[b * 6 + k]);
  }
  block_sum6(t, red);
  if (threadIdx.x == 0) {
    const bool accum = f.flags & MRL_FLAG_ACCUMULATE_LOSS;
    f.loss[0] = (accum ? f.loss[0] : 0.f) + (float)t[0];
    f.loss[1] = (accum ? f.loss[1] : 0.f) + (float)t[1];
    if (f.kl_loss != nullptr) f.kl_loss[0] = (accum ? f.kl_loss[0] : 0.f) + (float)t[5];
    if (f.stats != nullptr) {
      f.stats[0] = (accum ? f.stats[0] : 0) + (long long)t[2];
      f.stats[1] = (accum ? f.stats[1] : 0) + (long long)t[3];
      f.stats[2] = (accum ? f.stats[2] : 0) + (long long)t[4];
      f.stats[3] = (accum ? f.stats[3] : 0) + (long long)__ldcg(&f.totals[1]);
    }
    f.totals[2] = 0;
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
                                                         const float* __restrict__ rowck,
                                                         const float* __restrict__ cscale,
                                                         const float* __restrict__ logp_ref, int kl_est,
                                                         const float* __restrict__ logp_old, float eps_lo,
                                                         float eps_hi, const FinalizeArgs fa,
                                                         float* __restrict__ logp) {
  __shared__ double red[6][8];
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const uint8_t st = t < N ? rowstat[t] : 0;
  double pg = 0.0, nl = 0.0, kl = 0.0, lp = 0.0;
  if ((st & kStatValid) && (st & kStatRead)) {
    const double lse = ((double)row_m2[t] + log2((double)row_s[t])) * 0.693147180559945309417232121458;
    lp = (double)row_zt[t] - lse;
    const float cs = cscale[0];
    const double A = rowA[t], cu = rowcu[t] * cs, cn = rowcn[t];  // (the float products the row kernel formed)
    const float ck = logp_ref != nullptr ? rowck[t] * cs : 0.f;
    if (cu != 0.0 && A != 0.0) {
      const double rho = logp_old ? exp(lp - (double)logp_old[t]) : 1.0;
      const double lo = 1.0 - (double)eps_lo, hi = 1.0 + (double)eps_hi;
      pg = -cu * fmin(rho * A, fmin(fmax(rho, lo), hi) * A);
    }
    if (cn != 0.0) nl = -cn * lp;
    if (ck != 0.f) kl = (double)ck * mrl::kl_value(lp - (double)logp_ref[t], kl_est);
  }
  if (t < N && logp != nullptr) logp[t] = (float)lp;
  double v[6] = {pg, nl, (st & kStatValid) ? 1.0 : 0.0, (st & kStatClipped) ? 1.0 : 0.0, (st & kStatRead) ? 1.0 : 0.0, kl};
  block_sum6(v, red);
  publish_and_finalize(v, red, fa);
}

// The same block partials from per-row term arrays (the response-level ratio writes those).
__global__ void __launch_bounds__(256) rows_partial_kernel(long long N, const double* __restrict__ pg_term,
                                                            const double* __restrict__ nll_term,
                                                            const double* __restrict__ kl_term,
                                                            const uint8_t* __restrict__ rowstat,
                                                            const FinalizeArgs fa) {
  __shared__ double red[6][8];
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const uint8_t st = t < N ? rowstat[t] : 0;
  double v[6] = {t < N ? pg_term[t] : 0.0, t < N ? nll_term[t] : 0.0, (st & kStatValid) ? 1.0 : 0.0,
                 (st & kStatClipped) ? 1.0 : 0.0, (st & kStatRead) ? 1.0 : 0.0, t < N ? kl_term[t] : 0.0};
  block_sum6(v, red);
  publish_and_finalize(v, red, fa);
}

MrlLossWs carve_loss_ws(void* ws, long long N, int S) {
  MrlCarver c(ws);
  MrlLossWs w;
  w.totals = c.take<unsigned long long>(4);  // (one 256-byte piece: cleared by a single small memset per call)
  w.cscale = reinterpret_cast<float*>(w.totals + 4);
  w.rowA = c.take<float>((size_t)N);
  w.rowcu = c.take<float>((size_t)N);
  w.rowcn = c.take<float>((size_t)N);
  w.rowck = c.take<float>((size_t)N);
  w.row_m2 = c.take<float>((size_t)N);
  w.row_s = c.take<float>((size_t)N);
  w.row_zt = c.take<float>((size_t)N);
  w.pg_term = c.take<double>((size_t)N);
  w.nll_term = c.take<double>((size_t)N);
  w.kl_term = c.take<double>((size_t)N);
  w.partials = c.take<double>((size_t)((N + 255) / 256) * 6);
  w.rowstat = c.take<uint8_t>((size_t)N);
  w.seq_cnt = c.take<int32_t>((size_t)S + 1);
  w.bytes = c.off;
  return w;
}

// Which kernel takes the rows: 0 = general, 4 = streaming with 128-bit accesses, 8 = with 256-bit accesses.
int pick_stream_words(const RowParams& p, int dtype) {
  if (p.V < 4096) return 0;  // short rows: the general kernel's three passes stay in cache
  const uintptr_t in = reinterpret_cast<uintptr_t>(p.logits), out = reinterpret_cast<uintptr_t>(p.dlogits);
  const bool grad = p.dlogits != nullptr;
  const int e32 = dtype == MRL_BF16 ? 16 : 8, e16 = e32 / 2;  // elements per 32- and 16-byte vector
  if (p.V % e32 == 0 && p.ld % e32 == 0 && (in & 31) == 0 && (!grad || (p.ld_out % e32 == 0 && (out & 31) == 0))) return 8;
  if (p.V % e16 == 0 && p.ld % e16 == 0 && (in & 15) == 0 && (!grad || (p.ld_out % e16 == 0 && (out & 15) == 0))) return 4;
  return 0;
}

int launch_rows(RowParams p, int dtype, cudaStream_t st) {
  if (p.N == 0) return MRL_OK;
  if (p.N > 0x7fffffffll) return MRL_ERR_UNSUPPORTED_SHAPE;
  const int words = pick_stream_words(p, dtype);
  const unsigned n = (unsigned)p.N;
  if (words == 0) {
    mrl_profile_before(st, "row_general_kernel");
    if (dtype == MRL_BF16)
      row_general_kernel<__nv_bfloat16><<<n, kThreads, 0, st>>>(p);
    else
      row_general_kernel<float><<<n, kThreads, 0, st>>>(p);
    mrl_profile_after(st);
    return cudaGetLastError() == cudaSuccess ? MRL_OK : MRL_ERR_CUDA;
  }
  // Two CTAs per SM stream one row each, or -- for rows so long that two rows per SM would be evicted from L2
  // before the second pass reads them back -- the two halves of one row as a cluster of two.  (At 300 KB rows the
  // split reads HBM 1.01x instead of 1.34x but is 4 % slower: its per-CTA fixed work is spread over half the bytes.)
  // (the entropy diagnostic is carried by the whole-row variant only)
  const bool f32 = dtype == MRL_F32;
  const bool split = (long long)p.V * (f32 ? 4 : 2) >= kSplitRowBytes && p.N <= 0x3fffffffll && p.entropy == nullptr;
  const bool ent = p.entropy != nullptr;
  const int C = split ? 2 : 1;
  // gradient launches park the vectors each CTA reads first (whole groups of blockDim vectors)
  p.keep_q = p.dlogits != nullptr ? kParkBytes / (kStreamThreads * words * 4) : 0;
  const size_t park_bytes = (size_t)p.keep_q * kStreamThreads * words * 4;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n * (unsigned)C);
  cfg.blockDim = dim3(kStreamThreads);
  cfg.dynamicSmemBytes = park_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  using Kernel = void (*)(const RowParams);
  const Kernel k = f32 ? (words == 8 ? (split ? row_stream_kernel<kStreamThreads, 4, 8, 2, false, true>
                                        : ent ? row_stream_kernel<kStreamThreads, 4, 8, 1, true, true>
                                              : row_stream_kernel<kStreamThreads, 4, 8, 1, false, true>)
                                     : (split ? row_stream_kernel<kStreamThreads, 8, 4, 2, false, true>
                                        : ent ? row_stream_kernel<kStreamThreads, 8, 4, 1, true, true>
                                              : row_stream_kernel<kStreamThreads, 8, 4, 1, false, true>))
                       : (words == 8 ? (split ? row_stream_kernel<kStreamThreads, 4, 8, 2, false, false>
                                        : ent ? row_stream_kernel<kStreamThreads, 4, 8, 1, true, false>
                                              : row_stream_kernel<kStreamThreads, 4, 8, 1, false, false>)
                                     : (split ? row_stream_kernel<kStreamThreads, 8, 4, 2, false, false>
                                        : ent ? row_stream_kernel<kStreamThreads, 8, 4, 1, true, false>
                                              : row_stream_kernel<kStreamThreads, 8, 4, 1, false, false>));
  if (park_bytes > 0) {
    // exactly the carve-out two CTAs per SM need, as a percentage of the 228 KB an SM can give: the rest stays L1.
    // (park_bytes is the same for every gradient launch of one kernel: kParkBytes rounded to whole groups.)
    static std::atomic<uint64_t> attr_done[12];
    const int slot = (f32 ? 6 : 0) + (words == 8 ? 0 : 3) + (split ? 0 : ent ? 1 : 2);
    const int rc = mrl_once_per_device(attr_done[slot], [&] {
      const int carve = (int)((2 * (park_bytes + 2048) * 100 + 228 * 1024 - 1) / (228 * 1024));
      const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)park_bytes);
      return e != cudaSuccess ? e : cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, carve < 100 ? carve : 100);
    });
    if (rc != MRL_OK) return rc;
  }
  mrl_profile_before(st, split ? "row_stream_kernel (row split over a CTA pair)" : "row_stream_kernel");
  const cudaError_t e = cudaLaunchKernelEx(&cfg, k, p);
  mrl_profile_after(st);
  return e == cudaSuccess ? MRL_OK : MRL_ERR_CUDA;
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
  MRL_CUDA_OK(cudaMemsetAsync(w.totals, 0, 64, st));  // the counters, the tickets, cscale
  seq_prepare_kernel<<<S, 128, 0, st>>>(cu_seqlens, S, N, V, ids, mask, adv_seq, tok_weight, nll_weight, *lp, w.seq_cnt,
                                        w.totals, w.cscale, w.rowA, w.rowcu, w.rowcn, w.rowck, status);
  MRL_CUDA_OK(cudaGetLastError());
  *out = w;
  return MRL_OK;
}

// Float64 loss terms from the per-row reduction triples, then the fixed-order sums into loss / stats.
int mrl_rows_finish(const MrlLossWs& w, long long N, const float* logp_old, const mrl_loss_params* lp, float* logp,
                    float* loss, int64_t* stats, cudaStream_t st) {
  const FinalizeArgs fa = {w.partials, w.totals, lp->flags, loss, lp->logp_ref != nullptr ? lp->kl_loss : nullptr,
                           reinterpret_cast<long long*>(stats)};
  row_terms_kernel<<<(unsigned)((N + 255) / 256), 256, 0, st>>>(N, w.row_m2, w.row_s, w.row_zt, w.rowstat, w.rowA,
                                                                w.rowcu, w.rowcn, w.rowck, w.cscale, lp->logp_ref,
                                                                lp->kl_estimator, logp_old, lp->eps_lo, lp->eps_hi, fa,
                                                                logp);
  MRL_CUDA_OK(cudaGetLastError());
  return MRL_OK;
}

// Response-level ratio: loss terms, per-row gradient multipliers and log-sum-exps from the forward pass's per-row
// triples, then the fixed-order sums.  Rows that no sequence covers keep g = 0 (the arrays are cleared first).
int mrl_rows_finish_sequence(const MrlLossWs& w, long long N, int S, const int32_t* cu_seqlens, const float* adv_seq,
                             const float* logp_old, const float* nll_weight, const mrl_loss_params* lp, float* logp,
                             float* loss, int64_t* stats, float* g_out, float* lse2_out, cudaStream_t st) {
  MRL_CUDA_OK(cudaMemsetAsync(w.pg_term, 0, (size_t)N * sizeof(double), st));
  MRL_CUDA_OK(cudaMemsetAsync(w.nll_term, 0, (size_t)N * sizeof(double), st));
  MRL_CUDA_OK(cudaMemsetAsync(w.kl_term, 0, (size_t)N * sizeof(double), st));
  if (logp != nullptr) MRL_CUDA_OK(cudaMemsetAsync(logp, 0, (size_t)N * sizeof(float), st));
  seq_ratio_kernel<<<S, 256, 0, st>>>(cu_seqlens, S, N, w.row_m2, w.row_s, w.row_zt, w.rowstat, w.seq_cnt, adv_seq,
                                      logp_old, nll_weight, w.rowck, w.cscale, *lp, w.pg_term, w.nll_term, w.kl_term, logp, g_out,
                                      lse2_out);
  MRL_CUDA_OK(cudaGetLastError());
  const FinalizeArgs fa = {w.partials, w.totals, lp->flags, loss, lp->logp_ref != nullptr ? lp->kl_loss : nullptr,
                           reinterpret_cast<long long*>(stats)};
  rows_partial_kernel<<<(unsigned)((N + 255) / 256), 256, 0, st>>>(N, w.pg_term, w.nll_term, w.kl_term, w.rowstat, fa);
  MRL_CUDA_OK(cudaGetLastError());
  return MRL_OK;
}

namespace {
int launch_rows_backward(const RowParams& p, int dtype, const float* g, const float* lse2, const float* zt,
                         cudaStream_t st) {
  if (p.N == 0) return MRL_OK;
  const int words = pick_stream_words(p, dtype);
  const unsigned n = (unsigned)p.N;
  mrl_profile_before(st, words != 0 ? "row_backward_stream_kernel" : "row_backward_general_kernel");
  if (words == 8 && dtype == MRL_BF16)
    row_backward_stream_kernel<kStreamThreads, 4, 8, false><<<n, kStreamThreads, 0, st>>>(p, g, lse2, zt);
  else if (words == 4 && dtype == MRL_BF16)
    row_backward_stream_kernel<kStreamThreads, 8, 4, false><<<n, kStreamThreads, 0, st>>>(p, g, lse2, zt);
  else if (words == 8)
    row_backward_stream_kernel<kStreamThreads, 4, 8, true><<<n, kStreamThreads, 0, st>>>(p, g, lse2, zt);
  else if (words == 4)
    row_backward_stream_kernel<kStreamThreads, 8, 4, true><<<n, kStreamThreads, 0, st>>>(p, g, lse2, zt);
  else if (dtype == MRL_BF16)
    row_backward_general_kernel<__nv_bfloat16><<<n, kThreads, 0, st>>>(p, g, lse2, zt);
  else
    row_backward_general_kernel<float><<<n, kThreads, 0, st>>>(p, g, lse2, zt);
  mrl_profile_after(st);
  return cudaGetLastError() == cudaSuccess ? MRL_OK : MRL_ERR_CUDA;
}
}  // namespace

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
  if (lp->ratio_level != MRL_RATIO_TOKEN && lp->ratio_level != MRL_RATIO_SEQUENCE) return MRL_ERR_INVALID_ARG;
  if (lp->ratio_level == MRL_RATIO_SEQUENCE && tok_weight != nullptr) return MRL_ERR_INVALID_ARG;
  if (!mrl_kl_args_ok(lp)) return MRL_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool accum = lp->flags & MRL_FLAG_ACCUMULATE_LOSS;
  if (N == 0 || S == 0) {
    if (N != 0) return MRL_ERR_INVALID_ARG;  // rows without a sequence
    if (!accum) {
      MRL_CUDA_OK(cudaMemsetAsync(loss, 0, 2 * sizeof(float), st));
      if (lp->logp_ref != nullptr) MRL_CUDA_OK(cudaMemsetAsync(lp->kl_loss, 0, sizeof(float), st));
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
  p.rowck = w.rowck;
  p.cscale = w.cscale;
  p.logp_ref = lp->logp_ref;
  p.kl_est = lp->kl_estimator;
  p.logp_old = logp_old;
  p.eps_lo = lp->eps_lo;
  p.eps_hi = lp->eps_hi;
  p.flags = lp->flags;
  p.loss_mode = 1;
  p.entropy = lp->entropy;
  p.row_m2 = w.row_m2;
  p.row_s = w.row_s;
  p.row_zt = w.row_zt;
  p.rowstat = w.rowstat;
  p.status = status;
  if (lp->ratio_level == MRL_RATIO_SEQUENCE) {
    // forward only (ratio one: no token-level clipping), then the responses' ratios, then the gradient launch
    p.dlogits = nullptr;
    p.logp_old = nullptr;
    p.flags &= ~MRL_FLAG_SKIP_ZERO_ROWS;  // every valid row is needed for its response's sum
    p.flags |= kFlagSkipUncovered;        // rows outside every sequence: empty triple, hence g = 0 below
    rc = launch_rows(p, dtype, st);
    if (rc != MRL_OK) return rc;
    // (g and the base-2 log-sum-exp overwrite the forward pass's sum and maximum row by row; the per-response
    // kernel writes covered rows only, and uncovered rows hold the empty triple's zero sum)
    rc = mrl_rows_finish_sequence(w, N, S, cu_seqlens, adv_seq, logp_old, nll_weight, lp, logp, loss, stats, w.row_s,
                                  w.row_m2, st);
    if (rc != MRL_OK || dlogits == nullptr) return rc;
    p.dlogits = dlogits;
    return launch_rows_backward(p, dtype, w.row_s, w.row_m2, w.row_zt, st);
  }
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
  static std::mutex lookup_mutex;  // the one-time look-up may be raced by threads; the array itself is still shared
  std::lock_guard<std::mutex> lock(lookup_mutex);
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
