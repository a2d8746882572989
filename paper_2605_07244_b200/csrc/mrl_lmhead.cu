// Hidden-in path (fused LM head): mrl_fused_lmhead_loss_fwd_bwd.
//
// Every product of the pass is  C[M, N] = A B^T  (bf16 operands, fp32 accumulation) on one persistent tcgen05
// kernel, specialised by its epilogue and by how each operand lies in memory (K-major, or MN-major = given as the
// [K, M] / [K, N] matrix, so that nothing ever has to be transposed in memory):
//   forward    z = hidden W^T, tile by tile; the epilogue folds each tile into per-row (max, sum 2^x) partials and
//              picks the target logit; the [N, V] logits are never stored
//   backward   per vocabulary chunk: recompute the z tile, write D = g (softmax - onehot) in bf16 as D[N, Vc];
//              dHidden (+)= D W_chunk  (W_chunk enters MN-major);  dW[chunk] = D^T hidden  (both enter MN-major)
// Kernel anatomy (one CTA per SM, 192 threads): warp 0 feeds a shared-memory ring with TMA tile loads
// (128-byte swizzle, no multicast), one thread of warp 1 issues tcgen05.mma into one of two TMEM accumulators,
// warps 2..5 drain the other accumulator with tcgen05.ld while the next tile's MMAs run.  Every mbarrier wait is
// bounded; when one runs out the CTA raises MRL_DEV_TIMEOUT in the status word, lets its copies land and frees
// its TMEM.
#include <cuda.h>

#include "mrl_common.cuh"

namespace {

constexpr int BM = 128, BN = 256, BK = 64;  // CTA tile; BK * 2 bytes = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int kAccStages = 2;
constexpr int kTmemCols = kAccStages * BN;  // 512: all of tensor memory
constexpr int kGemmThreads = 192;
constexpr uint32_t kABytes = BM * BK * 2;  // a CTA's A tile of one stage
// Epilogue staging: each of the four epilogue warps owns 32 rows of 128 bytes (+ 16 bytes of padding per row, which
// keeps both the row-wise writes and the line-wise reads free of bank conflicts).  A thread holds one row of the
// accumulator; written out directly, every warp store would touch 32 different lines with 16 bytes each, and those
// requests compete with the operand copies for the SM's path to L2 (the dZ product lost 8 % of its tensor time to
// them).  Staged through shared memory the same bytes leave as whole 128-byte lines.
constexpr uint32_t kEpiRowBytes = 144, kEpiWarpBytes = 32 * kEpiRowBytes, kEpiStageBytes = 4 * kEpiWarpBytes;
// kC CTAs share a tile of kC * 128 rows: each holds its own 128 rows of A and 256 / kC rows of B per stage.
// kR = 2 (single CTAs only): a CTA works on a tile of 256 rows as two 128-row halves that share the B tile -- two MMAs
// per K step, one into each half of tensor memory -- so a stage carries 64 KB for twice the flops (a third fewer
// operand bytes per flop from L2, like a pair, without the pair's traffic between shared memories); the accumulators
// are then not double-buffered, which suits products whose K is long against their epilogue.
template <int kC, int kR = 1>
struct GemmCfg {
  static_assert(kR == 1 || (kR == 2 && kC == 1), "tall tiles are a single-CTA shape");
  static constexpr int kBRows = BN / kC;
  static constexpr uint32_t kACtaBytes = kR * kABytes;
  static constexpr uint32_t kBBytes = kBRows * BK * 2, kStageBytes = kACtaBytes + kBBytes;
  static constexpr int kStages = (192 * 1024) / kStageBytes;  // 4 (128-row tiles), 6 (pairs), 3 (tall): 192 KB of stages
  static constexpr int kAccs = kAccStages / kR;               // accumulators a CTA cycles through
  static constexpr size_t kSmem = (size_t)kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ +
                                  kEpiStageBytes /*epilogue staging*/;
};
constexpr uint32_t kWaitLimit = 1u << 24;   // mbarrier polls before a wait gives up (of the order of a second)
constexpr int kVChunk = 16384;              // vocabulary columns per backward chunk (multiple of BN)

enum { EPI_LSE = 0, EPI_DZ = 1, EPI_STORE = 2, EPI_LSE_ENT = 3 };  // _ENT: also sum_v 2^(x_v - m) z_v, for the entropy
enum { C_BF16 = 0, C_F32 = 1, C_F32_ADD = 2, C_BF16_FROM_ACC = 3 };

struct GemmParams {
  int M, N, K;
  int m_tiles, n_tiles, k_blocks;
  int group_m;            // row-tiles per raster group
  int a_blocks, b_blocks; // MN-major operand with a three-dimensional map (make_tmap_mn_blocks): fetched by one copy
  // Optional compaction (device arrays; the counts are read by the kernel, so the host never waits for them):
  const int* m_list;      // ascending indices of the row-tiles (of BM * kC rows) to work on; null = all of them
  const int* m_count;     // [1] how many
  const int* k_list;      // ascending indices of the K-blocks (of BK) to sum over; null = all of them
  const int* k_count;     // [1]
  int32_t* status;
  // EPI_LSE
  float2* partial;        // [n_tiles][part_ld]: (running max, sum) of the tile's columns, base-2 domain
  float* partial_u;       // EPI_LSE_ENT: [n_tiles][part_ld] sum of 2^(x - max) z over the tile's columns
  long long part_ld;
  const int32_t* ids;     // [M]
  float* zt;              // [M] target logit
  int col0;               // vocabulary index of column 0 of this product
  // EPI_DZ
  const float* g;         // [M] gradient multiplier g_t
  const float* lse2;      // [M] log2 sum_v 2^(z log2 e)
  __nv_bfloat16* D;       // [M, ldD]
  long long ldD;
  // EPI_STORE
  void* C;                // bf16 or fp32 [M, ldc]
  float* Cacc;            // fp32 [M, ldacc] running sum (C_BF16_FROM_ACC reads it, C_F32 / C_F32_ADD write C)
  long long ldc, ldacc;
  int c_mode;
};

// ------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  False when the limit ran out here (the abort flag is raised) or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kWaitLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// the same for a three-dimensional box (an MN-major operand fetched as several 64-wide blocks by one instruction)
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// arrive on an mbarrier of another CTA of the cluster (address from mapa)
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load of a CTA pair: the bytes land in this CTA, the completion is counted on `bar`, which may live in
// the other CTA of the pair (a shared::cluster address)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
// commit of a CTA pair's MMAs: one arrival on the barrier at this offset in every CTA of `mask`
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T, one 256 x 256 x 16 step of a CTA pair (issued by the leader CTA)
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
      : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, one 128 x 256 x 16 step
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
      : "memory");
}
// 32 lanes x 32 consecutive fp32 columns of tensor memory: thread i gets lane (base + i), columns [col, col + 32)
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile stored as 128-byte rows with the 128-byte swizzle (what the
// TMA tile load writes): 8-row groups 1024 bytes apart, descriptor version 1 (sm_100), layout type SWIZZLE_128B.
__device__ __forceinline__ uint64_t smem_desc_k128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                    // leading byte offset (unused by swizzled K-major layouts)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                    // descriptor version
  d |= (uint64_t)2 << 61;                    // SWIZZLE_128B
  return d;
}
// The same for an MN-major tile: the operand is stored with its M (or N) index contiguous, and the TMA brings it in as
// boxes of 64 such elements (128 bytes) by BK rows of K.  Inside a box, 8 K-rows of 128 bytes form one swizzle atom
// (1024 bytes apart: the stride byte offset); boxes of consecutive groups of 64 follow each other BK * 128 bytes
// apart (the leading byte offset).  One MMA step of K = 16 is two atoms: + 2048 bytes in the start address.
__device__ __forceinline__ uint64_t smem_desc_mn128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);
  d |= (uint64_t)((BK * 128) >> 4) << 16;     // leading byte offset: next group of 64 along M / N
  d |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset: next group of 8 along K
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// kind::f16 instruction descriptor: fp32 accumulator, bf16 x bf16, N = 256, M = 128 per CTA
// (bits 15 / 16: A / B is MN-major)
template <int kC, bool kAMn, bool kBMn>
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kAMn ? 1u : 0u) << 15) | ((kBMn ? 1u : 0u) << 16) |
                            ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((BM * kC) >> 4) << 24);

// tile t -> (row-tile, column-tile): row-tiles run fastest inside a group of group_m, so that the CTAs of one wave
// share a handful of A and B tiles
__device__ __forceinline__ void tile_coords(int t, int m_tiles, int n_tiles, int group_m, int& m, int& n) {
  const int per_group = group_m * n_tiles;
  const int grp = t / per_group, r = t - grp * per_group;
  const int m0 = grp * group_m;
  const int gm = min(group_m, m_tiles - m0);
  n = r / gm;
  m = m0 + (r - n * gm);
}

// ------------------------------------------------------------------------------------------ epilogues
// one thread = one row of the tile; v[] = 32 consecutive accumulator columns starting at tile column c

struct LseRow {
  float m, s, zt;
  bool has;
  float u;  // sum of 2^(x - m) z (kEnt only)
};

template <bool kEnt>
__device__ __forceinline__ void epi_lse_batch(const float* v, int c, int ncols_valid, int rel_id, LseRow& st) {
  float bm = -INFINITY;
#pragma unroll
  for (int j = 0; j < 32; ++j)
    if (c + j < ncols_valid) bm = fmaxf(bm, v[j]);
  if (bm == -INFINITY) return;  // no valid column in this batch
  const float m_new = fmaxf(st.m, bm * MRL_LOG2E);
  const float f = mrl::ex2_approx(st.m - m_new);  // first batch: 0 * 2^-inf = 0
  st.s *= f;
  if (kEnt) st.u *= f;
  st.m = m_new;
  float s0 = 0.f, s1 = 0.f, u0 = 0.f, u1 = 0.f;
#pragma unroll
  for (int j = 0; j < 32; j += 2) {
    if (c + j < ncols_valid) {
      const float e = mrl::ex2_approx(fmaf(v[j], MRL_LOG2E, -m_new));
      s0 += e;
      if (kEnt) u0 = e != 0.f ? fmaf(e, v[j], u0) : u0;  // e = 0 exactly where z = -inf: keep 0 * inf out
    }
    if (c + j + 1 < ncols_valid) {
      const float e = mrl::ex2_approx(fmaf(v[j + 1], MRL_LOG2E, -m_new));
      s1 += e;
      if (kEnt) u1 = e != 0.f ? fmaf(e, v[j + 1], u1) : u1;
    }
  }
  st.s += s0 + s1;
  if (kEnt) st.u += u0 + u1;
  if (rel_id >= c && rel_id < c + 32) {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (rel_id == c + j) st.zt = v[j];
    st.has = true;
  }
}

__device__ __forceinline__ void store_bf16x32(__nv_bfloat16* dst, const float* d, int nvalid) {
  if (nvalid >= 32 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint4 u;
      u.x = mrl::pack_bf16x2(d[q * 8 + 0], d[q * 8 + 1]);
      u.y = mrl::pack_bf16x2(d[q * 8 + 2], d[q * 8 + 3]);
      u.z = mrl::pack_bf16x2(d[q * 8 + 4], d[q * 8 + 5]);
      u.w = mrl::pack_bf16x2(d[q * 8 + 6], d[q * 8 + 7]);
      reinterpret_cast<uint4*>(dst)[q] = u;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < nvalid) dst[j] = __float2bfloat16_rn(d[j]);
  }
}

__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 u;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "r"(addr));
  return u;
}

// ------------------------------------------------------------------------------------------ the GEMM kernel
// kAMn / kBMn: the operand is stored MN-major (its M / N index contiguous, K strided) instead of K-major.
template <int EPI, int kC, bool kAMn, bool kBMn, int kR = 1>
__global__ void __launch_bounds__(kGemmThreads, 1)
lmhead_gemm_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                   const GemmParams p) {
  using Cfg = GemmCfg<kC, kR>;
  constexpr int kAccs = Cfg::kAccs;
  constexpr int kStages = Cfg::kStages;
  constexpr uint32_t kStageBytes = Cfg::kStageBytes;
  constexpr bool kLse = EPI == EPI_LSE || EPI == EPI_LSE_ENT;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_addr(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
  unsigned char* tiles_ptr = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles_ptr + (size_t)kStages * kStageBytes);
  // bars[0..kStages): full, [kStages..2kStages): empty, then tmem_full[2], tmem_empty[2]
  const uint32_t bar0 = smem_addr(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + kAccStages + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 2 * kAccStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t epi_stage0 = bar0 + 256u;  // after the 256 bytes reserved for barriers and flags

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // a pair of CTAs (kC = 2) works on one tile of 256 rows: rank 0 leads (arms the barriers, issues the MMAs)
  const int rank = kC == 2 ? (int)(blockIdx.x & 1u) : 0;
  const int unit = (int)blockIdx.x / kC, n_units = (int)gridDim.x / kC;
  const int m_tiles = p.m_list != nullptr ? min(*p.m_count, p.m_tiles) : p.m_tiles;
  const int k_blocks = p.k_list != nullptr ? min(*p.k_count, p.k_blocks) : p.k_blocks;
  const int total_tiles = m_tiles * p.n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < kAccStages; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 4 * kC);  // one arrival per epilogue warp of every CTA of the pair
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {  // the same warp in both CTAs of a pair, the same shared-memory slot
    if (kC == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)),
                   "r"((uint32_t)kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)),
                   "r"((uint32_t)kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (kC == 2) cluster_sync_all();  // the peer's barriers exist before anything is signalled across the pair
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer: this CTA's 128 rows of A and its 256 / kC rows of B
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = unit; t < total_tiles && ok; t += n_units) {
        int m, n;
        tile_coords(t, m_tiles, p.n_tiles, p.group_m, m, n);
        if (p.m_list != nullptr) m = p.m_list[m];
        const int a_row = (m * kC + rank) * (BM * kR), b_row = n * BN + rank * Cfg::kBRows;
        // K-block indices come from the list (when there is one) eight at a time and one group ahead, so that their
        // loads never sit between two copies
        auto k_index = [&](int kb) { return (p.k_list != nullptr && kb < k_blocks) ? __ldg(p.k_list + kb) : kb; };
        int k_next[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) k_next[j] = k_index(j);
        for (int kb0 = 0; kb0 < k_blocks && ok; kb0 += 8) {
          int k_cur[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            k_cur[j] = k_next[j];
            k_next[j] = k_index(kb0 + 8 + j);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (kb0 + j >= k_blocks) break;
            const int kx = k_cur[j] * BK;
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = tiles + (uint32_t)stage * kStageBytes;
            // the leader's barrier counts the bytes of both CTAs of a pair; only the leader arms it
            const uint32_t bar = kC == 2 ? mapa_u32(full_bar(stage), 0u) : full_bar(stage);
            if (rank == 0) mbar_expect_tx(full_bar(stage), (uint32_t)kC * kStageBytes);
            auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y) {
              if (kC == 2) tma_load_2d_pair(dst, map, x, y, bar); else tma_load_2d(dst, map, x, y, bar);
            };
            auto load_blocks = [&](uint32_t dst, const CUtensorMap* map, int block0, int y) {
              if (kC == 2) tma_load_3d_pair(dst, map, 0, y, block0, bar); else tma_load_3d(dst, map, 0, y, block0, bar);
            };
            if (kAMn) {  // blocks of 64 rows-of-the-tile x BK: one copy, or one per block
              if (p.a_blocks) {
                load_blocks(a_dst, &tmapA, a_row / 64, kx);
              } else {
#pragma unroll
                for (int q = 0; q < kR * BM / 64; ++q) load(a_dst + (uint32_t)q * (BK * 128), &tmapA, a_row + 64 * q, kx);
              }
            } else {
              load(a_dst, &tmapA, kx, a_row);
            }
            if (kBMn) {
              if (p.b_blocks) {
                load_blocks(a_dst + Cfg::kACtaBytes, &tmapB, b_row / 64, kx);
              } else {
#pragma unroll
                for (int q = 0; q < Cfg::kBRows / 64; ++q)
                  load(a_dst + Cfg::kACtaBytes + (uint32_t)q * (BK * 128), &tmapB, b_row + 64 * q, kx);
              }
            } else {
              load(a_dst + Cfg::kACtaBytes, &tmapB, kx, b_row);
            }
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (the leader CTA of a pair)
    if (lane == 0 && rank == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int t = unit; t < total_tiles && ok; t += n_units) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kR) * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = tiles + (uint32_t)stage * kStageBytes;
          const uint64_t adesc = kAMn ? smem_desc_mn128(a_src) : smem_desc_k128(a_src);
          const uint64_t bdesc = kBMn ? smem_desc_mn128(a_src + Cfg::kACtaBytes) : smem_desc_k128(a_src + Cfg::kACtaBytes);
          // one step of K = 16: 32 bytes along a K-major swizzle row, two 1024-byte atoms of an MN-major tile
          constexpr uint64_t a_step = kAMn ? (2048 >> 4) : 2, b_step = kBMn ? (2048 >> 4) : 2;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            if (kC == 2)
              tc_mma_pair(d_tmem, adesc + a_step * k, bdesc + b_step * k, kIdesc<kC, kAMn, kBMn>, (kb | k) != 0);
            else
              for (int h = 0; h < kR; ++h)  // the 128-row halves of a tall tile: 16 KB further in A, BN columns further in D
                tc_mma(d_tmem + (uint32_t)h * BN, adesc + a_step * k + (uint64_t)h * (kABytes >> 4), bdesc + b_step * k,
                       kIdesc<kC, kAMn, kBMn>, (kb | k) != 0);
          }
          // the stage is free (in both CTAs) once these MMAs have read it
          if (kC == 2) tc_commit_pair(empty_bar(stage), 3); else tc_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (kC == 2) tc_commit_pair(tfull_bar(acc), 3); else tc_commit(tfull_bar(acc));
        if (++acc == kAccs) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue: warps 2..5 own TMEM lanes 32 * (warp % 4) .. + 31
    const int quad = warp & 3;
    const int row_in_tile = quad * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = unit; t < total_tiles && ok; t += n_units) {
      int m, n;
      tile_coords(t, m_tiles, p.n_tiles, p.group_m, m, n);
      if (p.m_list != nullptr) m = p.m_list[m];
      const int ncols_valid = min(BN, p.N - n * BN);
#pragma unroll 1
      for (int h = 0; h < kR; ++h) {  // the 128-row halves of a tall tile, one after the other
      const int half_row0 = ((m * kC + rank) * kR + h) * BM;
      const int row = half_row0 + row_in_tile;
      const bool row_ok = row < p.M;
      // per-row inputs before the accumulator is ready
      LseRow st = {-INFINITY, 0.f, 0.f, false, 0.f};
      int rel_id = -1;
      float g = 0.f, neg_k = 0.f, l2 = 0.f, sgn = 1.f;
      if (kLse) {
        if (row_ok) rel_id = p.ids[row] - (p.col0 + n * BN);
      } else if (EPI == EPI_DZ) {
        if (row_ok) {
          g = p.g[row];
          l2 = p.lse2[row];
          rel_id = p.ids[row] - (p.col0 + n * BN);
        }
        neg_k = -(l2 - log2f(fabsf(g)));  // 2^(z log2e - k) = |g| softmax(z); unused when g = 0
        sgn = g < 0.f ? -1.f : 1.f;
      }
      if (h == 0) {
        if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
      }
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kR + h) * BN;
      // staging area of this warp, and which of its 16-byte pieces this lane moves when a staged block is written out:
      // piece i of the lane is bytes [16 (lane % 8), + 16) of row lane / 8 + 4 i, so a warp instruction covers four
      // whole rows of 128 bytes
      const uint32_t stg = epi_stage0 + (uint32_t)quad * kEpiWarpBytes;
      const uint32_t stg_mine = stg + (uint32_t)lane * kEpiRowBytes;
      const int piece_row = lane >> 3, piece_col = lane & 7;
      const long long tile_row0 = (long long)half_row0 + quad * 32;
#pragma unroll 1
      for (int c = 0; c < BN; c += 32) {
        if (c >= ncols_valid) break;  // uniform across the CTA
        float v[32];
        tc_ld32(t_row + (uint32_t)c, v);
        if (kLse) {
          epi_lse_batch<EPI == EPI_LSE_ENT>(v, c, ncols_valid, rel_id, st);
        } else if (EPI == EPI_DZ) {
          float d[32];
          if (g == 0.f) {
#pragma unroll
            for (int j = 0; j < 32; ++j) d[j] = 0.f;
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) d[j] = sgn * mrl::ex2_approx(fmaf(v[j], MRL_LOG2E, neg_k));
            if (rel_id >= c && rel_id < c + 32) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (rel_id == c + j) d[j] = g * (mrl::ex2_approx(fmaf(v[j], MRL_LOG2E, -l2)) - 1.0f);
            }
          }
          // whole blocks of 64 columns with 128-byte aligned rows leave through the staging area as whole lines
          const bool lines = (ncols_valid & 63) == 0 && (p.ldD & 63) == 0 && (reinterpret_cast<uintptr_t>(p.D) & 127) == 0;
          if (lines) {
            const uint32_t dst = stg_mine + (uint32_t)(c & 32) * 2u;
#pragma unroll
            for (int q = 0; q < 4; ++q)
              sts_v4(dst + 16u * q, mrl::pack_bf16x2(d[q * 8 + 0], d[q * 8 + 1]), mrl::pack_bf16x2(d[q * 8 + 2], d[q * 8 + 3]),
                     mrl::pack_bf16x2(d[q * 8 + 4], d[q * 8 + 5]), mrl::pack_bf16x2(d[q * 8 + 6], d[q * 8 + 7]));
            if (c & 32) {  // 64 columns of 32 rows are staged: 4 KB, eight 16-byte pieces per lane
              __syncwarp();
              __nv_bfloat16* base = p.D + (long long)n * BN + (c - 32) + piece_col * 8;
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int r = piece_row + 4 * i;
                const uint4 u = lds_v4(stg + (uint32_t)r * kEpiRowBytes + (uint32_t)piece_col * 16u);
                if (tile_row0 + r < p.M) *reinterpret_cast<uint4*>(base + (tile_row0 + r) * p.ldD) = u;
              }
              __syncwarp();
            }
          } else if (row_ok) {
            const int nvalid = ncols_valid - c;
            store_bf16x32(p.D + (long long)row * p.ldD + (long long)n * BN + c, d, nvalid);
          }
        } else {
          const int nvalid = ncols_valid - c;
          const long long col = (long long)n * BN + c;
          const bool f32_out = p.c_mode == C_F32 || p.c_mode == C_F32_ADD;
          // float32 accumulator traffic (read-modify-write of C, or the read of the running sum): one staged block is
          // 32 rows x 32 floats = 32 whole lines
          const float* acc_in = p.c_mode == C_F32_ADD ? static_cast<const float*>(p.C) : p.Cacc;
          const long long ld_in = p.c_mode == C_F32_ADD ? p.ldc : p.ldacc;
          const bool lines = p.c_mode != C_BF16 && nvalid >= 32 && (ld_in & 3) == 0 &&
                             (reinterpret_cast<uintptr_t>(acc_in) & 15) == 0 &&
                             (f32_out ? ((p.ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(p.C) & 15) == 0)
                                      : ((p.ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(p.C) & 7) == 0));
          if (lines) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              sts_v4(stg_mine + 16u * q, __float_as_uint(v[4 * q + 0]), __float_as_uint(v[4 * q + 1]),
                     __float_as_uint(v[4 * q + 2]), __float_as_uint(v[4 * q + 3]));
            __syncwarp();
            // (all eight reads of the running sum are issued before the first of them is used: one round trip to
            // memory per block, not eight)
            const long long off = col + piece_col * 4;
            float4 o[8];
            if (p.c_mode != C_F32) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const long long rr = tile_row0 + piece_row + 4 * i;
                o[i] = rr < p.M ? *reinterpret_cast<const float4*>(acc_in + rr * ld_in + off) : make_float4(0.f, 0.f, 0.f, 0.f);
              }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r = piece_row + 4 * i;
              const uint4 u = lds_v4(stg + (uint32_t)r * kEpiRowBytes + (uint32_t)piece_col * 16u);
              if (tile_row0 + r < p.M) {
                float4 t = make_float4(__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w));
                if (p.c_mode != C_F32) {
                  t.x += o[i].x;
                  t.y += o[i].y;
                  t.z += o[i].z;
                  t.w += o[i].w;
                }
                if (f32_out) {
                  *reinterpret_cast<float4*>(static_cast<float*>(p.C) + (tile_row0 + r) * p.ldc + off) = t;
                } else {
                  uint2 w;
                  w.x = mrl::pack_bf16x2(t.x, t.y);
                  w.y = mrl::pack_bf16x2(t.z, t.w);
                  *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.C) + (tile_row0 + r) * p.ldc + off) = w;
                }
              }
            }
            __syncwarp();
          } else if (row_ok) {
            if (p.c_mode == C_BF16) {
              store_bf16x32(static_cast<__nv_bfloat16*>(p.C) + (long long)row * p.ldc + col, v, nvalid);
            } else if (p.c_mode == C_BF16_FROM_ACC) {
              const float* a = p.Cacc + (long long)row * p.ldacc + col;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j < nvalid) v[j] += a[j];
              store_bf16x32(static_cast<__nv_bfloat16*>(p.C) + (long long)row * p.ldc + col, v, nvalid);
            } else {
              float* o = static_cast<float*>(p.C) + (long long)row * p.ldc + col;
              const bool add = p.c_mode == C_F32_ADD;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j < nvalid) o[j] = add ? o[j] + v[j] : v[j];
            }
          }
        }
      }
      if (h == kR - 1) {  // the accumulator has been read: hand it back to the MMA warp
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {  // the leader's barrier collects the epilogue warps of both CTAs
          if (kC == 2 && rank != 0) mbar_arrive_remote(mapa_u32(tempty_bar(acc), 0u)); else mbar_arrive(tempty_bar(acc));
        }
      }
      if (kLse && row_ok) {
        p.partial[(long long)n * p.part_ld + row] = make_float2(st.m, st.s);
        if (EPI == EPI_LSE_ENT) p.partial_u[(long long)n * p.part_ld + row] = st.u;
        if (st.has) p.zt[row] = st.zt;
      }
      }  // halves
      if (++acc == kAccs) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ---------------- teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0 && p.status != nullptr) atomicOr(p.status, MRL_DEV_TIMEOUT);
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies and MMAs still in flight land before the CTA goes
    __syncthreads();
  }
  if (kC == 2) cluster_sync_all();  // no CTA leaves while its peer may still signal into its shared memory
  if (warp == 1) {
    tc_fence_after();
    if (kC == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                   : "memory");
  }
}

// ------------------------------------------------------------------------------------------ small kernels
// Does the forward product have to produce this (unmasked, in-range) row?
__device__ __forceinline__ bool row_needs_forward(long long t, const float* rowA, const float* rowcu, const float* rowcn,
                                                  const float* rowck, bool has_ref, uint32_t flags) {
  if (!(flags & MRL_FLAG_SKIP_ZERO_ROWS)) return true;
  const bool zero = (rowcu[t] == 0.f || rowA[t] == 0.f) && rowcn[t] == 0.f && (!has_ref || rowck[t] == 0.f);
  return !zero;
}

// Liveness of every block of 256 rows.  mode 0 (backward): some row has g != 0.  mode 1 (forward): some row is
// unmasked with an id in range and needs the forward product.  One warp per block of rows.
__global__ void __launch_bounds__(256) tile_live_kernel(long long N, int n256, int mode, const float* __restrict__ g,
                                                         const int32_t* __restrict__ ids,
                                                         const uint8_t* __restrict__ mask, int V,
                                                         const float* __restrict__ rowA,
                                                         const float* __restrict__ rowcu,
                                                         const float* __restrict__ rowcn,
                                                         const float* __restrict__ rowck, bool has_ref, uint32_t flags,
                                                         uint8_t* __restrict__ live) {
  const int tile = (int)((blockIdx.x * 256u + threadIdx.x) >> 5), lane = threadIdx.x & 31;
  if (tile >= n256) return;
  bool any = false;
  for (int r = lane; r < 256; r += 32) {
    const long long t = (long long)tile * 256 + r;
    if (t >= N) break;
    if (mode == 0) {
      any |= g[t] != 0.f;
    } else {
      const int id = ids[t];
      const bool in_batch = (mask == nullptr || mask[t] != 0) && id >= 0 && id < V;
      any |= in_batch && row_needs_forward(t, rowA, rowcu, rowcn, rowck, has_ref, flags);
    }
  }
  any = __any_sync(0xffffffffu, any);
  if (lane == 0) live[tile] = any ? 1 : 0;
}

// Ascending lists of the live blocks at the three granularities the products use: 256-row tiles (CTA pairs),
// 128-row tiles, 64-row K-blocks; counts[0..2] = their lengths.  A batch without any live block lists block 0, so
// that no product runs empty (its rows then contribute zeros).  One block; ordered, hence reproducible.
__global__ void __launch_bounds__(1024) tile_lists_kernel(int n256, int n128, int n64, const uint8_t* __restrict__ live,
                                                           int* __restrict__ m256, int* __restrict__ m128,
                                                           int* __restrict__ k64, int* __restrict__ counts) {
  __shared__ int warp_tot[32];
  __shared__ int base_sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) base_sh = 0;
  __syncthreads();
  for (int c0 = 0; c0 < n256; c0 += 1024) {
    const int t = c0 + tid;
    const bool f = t < n256 && live[t] != 0;
    const unsigned bal = __ballot_sync(0xffffffffu, f);
    if (lane == 0) warp_tot[warp] = __popc(bal);
    __syncthreads();
    int off = base_sh;
    for (int wi = 0; wi < warp; ++wi) off += warp_tot[wi];
    if (f) {
      const int pos = off + __popc(bal & ((1u << lane) - 1u));
      m256[pos] = t;
      for (int j = 0; j < 2; ++j) if (2 * t + j < n128) m128[2 * pos + j] = 2 * t + j;
      for (int j = 0; j < 4; ++j) if (4 * t + j < n64) k64[4 * pos + j] = 4 * t + j;
    }
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int wi = 0; wi < 32; ++wi) tot += warp_tot[wi];
      base_sh += tot;
    }
    __syncthreads();
  }
  if (tid == 0) {
    int cnt = base_sh;
    if (cnt == 0) {
      m256[0] = 0;
      for (int j = 0; j < 2 && j < n128; ++j) m128[j] = j;
      for (int j = 0; j < 4 && j < n64; ++j) k64[j] = j;
      cnt = 1;
    }
    // only the batch's last block of 256 rows can be short of 128- or 64-row blocks
    const bool has_last = m256[cnt - 1] == n256 - 1;
    counts[0] = cnt;
    counts[1] = 2 * cnt - (has_last ? 2 * n256 - n128 : 0);
    counts[2] = 4 * cnt - (has_last ? 4 * n256 - n64 : 0);
  }
}

// Merges the per-tile partials of every row in tile order, then the row's ratio / clip / gradient multiplier.
__global__ void __launch_bounds__(256) lmhead_rows_kernel(long long N, int V, int n_tiles, const float2* __restrict__ partial,
                                                           const float* __restrict__ partial_u, float* __restrict__ entropy,
                                                           long long part_ld, const float* __restrict__ zt,
                                                           const int32_t* __restrict__ ids,
                                                           const uint8_t* __restrict__ mask,
                                                           const float* __restrict__ rowA,
                                                           const float* __restrict__ rowcu,
                                                           const float* __restrict__ rowcn,
                                                           const float* __restrict__ rowck,
                                                           const float* __restrict__ cscale,
                                                           const float* __restrict__ logp_ref, int kl_est,
                                                           const float* __restrict__ logp_old, float eps_lo,
                                                           float eps_hi, float* __restrict__ row_m2,
                                                           float* __restrict__ row_s, float* __restrict__ row_zt,
                                                           uint8_t* __restrict__ rowstat, float* __restrict__ g_out,
                                                           float* __restrict__ lse2_out, uint32_t flags) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= N) return;
  const int id = ids[t];
  const bool in_batch = (mask == nullptr || mask[t] != 0) && id >= 0 && id < V;
  // under MRL_FLAG_SKIP_ZERO_ROWS a row whose multiplier is known to be zero is not read (its tile may not even
  // have been computed): it reports logp = 0 and still counts in the denominators
  const bool valid = in_batch && row_needs_forward(t, rowA, rowcu, rowcn, rowck, logp_ref != nullptr, flags);
  mrl::Lse2 acc = mrl::lse2_empty();
  float usum = 0.f;  // sum_v 2^(x_v - acc.m) z_v, carried along when the entropy is asked for
  if (valid)
    for (int n = 0; n < n_tiles; ++n) {
      const float2 q = partial[(long long)n * part_ld + t];
      if (entropy != nullptr) {
        const float m = fmaxf(acc.m, q.x);
        if (m != -INFINITY)
          usum = usum * mrl::ex2_approx(acc.m - m) + partial_u[(long long)n * part_ld + t] * mrl::ex2_approx(q.x - m);
      }
      acc = mrl::lse2_merge(acc, mrl::Lse2{q.x, q.y});
    }
  float g = 0.f, l2 = 0.f;
  uint8_t st = 0;
  if (valid) {
    l2 = acc.m + log2f(acc.s);
    const float logp = zt[t] - mrl::lse2_to_nats(l2);
    mrl::RowIn in;
    in.A = rowA[t];
    in.cu = rowcu[t] * cscale[0];
    in.cn = rowcn[t];
    in.has_old = logp_old != nullptr;
    in.logp_old = in.has_old ? logp_old[t] : 0.f;
    in.ck = logp_ref != nullptr ? rowck[t] * cscale[0] : 0.f;
    in.logp_ref = logp_ref != nullptr ? logp_ref[t] : 0.f;
    in.kl_est = kl_est;
    const mrl::RowOut ro = mrl::mrl_row_loss(logp, in, eps_lo, eps_hi);
    g = ro.g;
    st = MRL_ROW_VALID | MRL_ROW_READ;
    if (ro.clipped && in.A != 0.f) st |= MRL_ROW_CLIPPED;
  }
  if (entropy != nullptr) entropy[t] = valid ? mrl::lse2_to_nats(l2) - usum / acc.s : 0.f;  // H = lse - sum_v p_v z_v
  row_m2[t] = acc.m;
  row_s[t] = acc.s;
  row_zt[t] = valid ? zt[t] : 0.f;
  rowstat[t] = in_batch ? (st | MRL_ROW_VALID) : st;
  g_out[t] = g;
  lse2_out[t] = l2;
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Tensor map of a row-major bf16 matrix [rows, cols] (ld elements between rows) read in [box_rows x 64] tiles.
int make_tmap(CUtensorMap* map, const void* base, long long rows, long long cols, long long ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return MRL_ERR_CUDA;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MRL_OK : MRL_ERR_CUDA;
}

// Tensor map of an MN-major operand -- a row-major bf16 matrix [k_rows, mn] (ld elements between rows) whose mn is a
// multiple of 64 -- as a three-dimensional tensor {64 elements, k_rows, mn / 64 blocks}: one box of {64, 64, blocks}
// then lands in shared memory as `blocks` consecutive 8 KB atoms of 64 K-rows x 128 bytes, which is the layout the
// MMA reads an MN-major operand from, with a single copy instruction instead of one per block.
int make_tmap_mn_blocks(CUtensorMap* map, const void* base, long long k_rows, long long mn, long long ld, int blocks) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return MRL_ERR_CUDA;
  const cuuint64_t dims[3] = {64, (cuuint64_t)k_rows, (cuuint64_t)(mn / 64)};
  const cuuint64_t strides[2] = {(cuuint64_t)ld * 2, 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)BK, (cuuint32_t)blocks};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MRL_OK : MRL_ERR_CUDA;
}

int sm_count() {
  static int n[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (n[dev] == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    n[dev] = v;
  }
  return n[dev];
}

// CTA pairs of the two-CTA kernel that can be resident together on the current device (0: use single CTAs).
template <int EPI, bool kAMn, bool kBMn>
int resident_pairs(cudaLaunchConfig_t* cfg) {
  static int cache[64] = {};
  int dev = 0;
  const bool cacheable = cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64;
  if (cacheable && cache[dev] != 0) return cache[dev] > 0 ? cache[dev] : 0;
  cfg->gridDim = dim3((unsigned)(sm_count() / 2 * 2));
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, lmhead_gemm_kernel<EPI, 2, kAMn, kBMn>, cfg) != cudaSuccess || n < 1) {
    (void)cudaGetLastError();
    n = 0;
  }
  if (cacheable) cache[dev] = n > 0 ? n : -1;
  return n;
}

// C[M, N] = A B^T.  A K-major operand is a row-major [rows = M or N, K] matrix; an MN-major one is a row-major
// [K, rows] matrix (what the other one would be transposed), `ld` elements between its rows either way.
// Compact lists of the blocks of rows that carry work (device arrays, see tile_lists_kernel).
struct TileLists {
  int *m256, *m128, *k64, *counts;
};

// Whether a product with both operands MN-major (dW) takes tall tiles: its K must be long enough to pay for the
// epilogue, which a tall tile cannot overlap with the next tile's MMAs, and there must be a tall tile per SM.
// Measured on B200, one 16,384 x 4,096 product, tall against 128-row tiles (ms): bf16 store K = 2,048 0.199 / 0.199,
// 4,096 0.359 / 0.379, 8,192 0.689 / 0.768, 65,536 6.08 / 6.77; float32 accumulate (read-modify-write epilogue)
// 8,192 0.808 / 0.800, 16,384 1.483 / 1.536, 65,536 5.95 / 6.62 -- at a clock only 3 % lower inside the step, where
// pairs of CTAs gain the same activity and lose it to clock.  The dHidden product (K = 16,384, float32 read-modify-write
// of a tile as large as its mainloop is short) measured slower with tall tiles and keeps 128 rows.
bool tall_policy(const GemmParams& p) {
  const long long tall_tiles = (long long)((p.M + 2 * BM - 1) / (2 * BM)) * ((p.N + BN - 1) / BN);
  const int min_k = p.c_mode == C_BF16 ? 4096 : 16384;
  return p.K >= min_k && tall_tiles >= sm_count();
}

// `m_rows` / `k_rows`: the M (resp. K) dimension of the product is the batch's rows and only the listed blocks count.
template <int EPI, bool kAMn, bool kBMn>
int launch_gemm(const void* A, long long lda, const void* B, long long ldb, GemmParams p, bool pair_tiles,
                cudaStream_t st, const TileLists* m_rows = nullptr, const TileLists* k_rows = nullptr) {
  if (p.M <= 0 || p.N <= 0 || p.K <= 0) return MRL_OK;
  p.n_tiles = (p.N + BN - 1) / BN;
  p.k_blocks = (p.K + BK - 1) / BK;
  // two-CTA tiles (256 rows) when asked for and pairs can be scheduled, else one CTA per 128-row tile
  static std::atomic<uint64_t> attr_done;  // one per instantiation: both tile shapes' shared-memory limits, once per device
  const int arc = mrl_once_per_device(attr_done, [] {
    const cudaError_t e = cudaFuncSetAttribute(lmhead_gemm_kernel<EPI, 2, kAMn, kBMn>,
                                               cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GemmCfg<2>::kSmem);
    if (e != cudaSuccess) return e;
    if constexpr (EPI == EPI_STORE && kAMn && kBMn) {
      const cudaError_t e2 = cudaFuncSetAttribute(lmhead_gemm_kernel<EPI, 1, kAMn, kBMn, 2>,
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GemmCfg<1, 2>::kSmem);
      if (e2 != cudaSuccess) return e2;
    }
    return cudaFuncSetAttribute(lmhead_gemm_kernel<EPI, 1, kAMn, kBMn>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)GemmCfg<1>::kSmem);
  });
  if (arc != MRL_OK) return arc;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = GemmCfg<2>::kSmem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int pairs = pair_tiles ? resident_pairs<EPI, kAMn, kBMn>(&cfg) : 0;
  const int kC = pairs > 0 ? 2 : 1;
  // tall tiles (256 rows in one CTA, accumulators not double-buffered)
  constexpr bool kTallShape = EPI == EPI_STORE && kAMn && kBMn;
  const bool tall = kTallShape && kC == 1 && tall_policy(p);
  const int kR = tall ? 2 : 1;
  CUtensorMap ta, tb;
  // K-major: tiles of [box rows x 64 of K]; MN-major: boxes of [64 of K rows x 64 of M / N]
  // (an MN-major operand whose M / N extent is a multiple of 64 gets the three-dimensional map: one copy per stage)
  p.a_blocks = (kAMn && p.M % 64 == 0) ? kR * BM / 64 : 0;
  p.b_blocks = (kBMn && p.N % 64 == 0) ? BN / kC / 64 : 0;
  int rc = !kAMn        ? make_tmap(&ta, A, p.M, p.K, lda, kR * BM)
           : p.a_blocks ? make_tmap_mn_blocks(&ta, A, p.K, p.M, lda, p.a_blocks)
                        : make_tmap(&ta, A, p.K, p.M, lda, BK);
  if (rc != MRL_OK) return rc;
  rc = !kBMn        ? make_tmap(&tb, B, p.N, p.K, ldb, BN / kC)
       : p.b_blocks ? make_tmap_mn_blocks(&tb, B, p.K, p.N, ldb, p.b_blocks)
                    : make_tmap(&tb, B, p.K, p.N, ldb, BK);
  if (rc != MRL_OK) return rc;
  p.m_tiles = (p.M + BM * kC * kR - 1) / (BM * kC * kR);
  if (m_rows != nullptr) {
    p.m_list = kC * kR == 2 ? m_rows->m256 : m_rows->m128;
    p.m_count = m_rows->counts + (kC * kR == 2 ? 0 : 1);
  }
  if (k_rows != nullptr) {
    p.k_list = k_rows->k64;
    p.k_count = k_rows->counts + 2;
  }
  // rows of A per raster group: the group's rows of A stay in L2 while B streams past them, so B is fetched from
  // DRAM once per group -- the taller the group the better, as long as its A panel (rows x K) fits L2 beside the
  // stream (measured: 4,096 rows at K = 4,096, 2,048 rows at K >= 16,384; DRAM traffic costs clock under the power cap)
  p.group_m = (p.K <= 8192 ? 4096 : 2048) / (BM * kC * kR);
  const long long tiles = (long long)p.m_tiles * p.n_tiles;
  if (tiles > 0x7fffffffll) return MRL_ERR_UNSUPPORTED_SHAPE;
  if (kC == 2) {
    const long long units = tiles < pairs ? tiles : pairs;
    cfg.gridDim = dim3((unsigned)(2 * units));
    mrl_profile_before(st, "lmhead_gemm_kernel (pair tiles)");
    const cudaError_t e = cudaLaunchKernelEx(&cfg, lmhead_gemm_kernel<EPI, 2, kAMn, kBMn>, ta, tb, p);
    mrl_profile_after(st);
    return e == cudaSuccess ? MRL_OK : MRL_ERR_CUDA;
  }
  const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
  if constexpr (kTallShape) {
    if (tall) {
      mrl_profile_before(st, "lmhead_gemm_kernel (tall tiles)");
      lmhead_gemm_kernel<EPI, 1, kAMn, kBMn, 2><<<grid, kGemmThreads, GemmCfg<1, 2>::kSmem, st>>>(ta, tb, p);
      mrl_profile_after(st);
      MRL_CUDA_OK(cudaGetLastError());
      return MRL_OK;
    }
  }
  mrl_profile_before(st, "lmhead_gemm_kernel");
  lmhead_gemm_kernel<EPI, 1, kAMn, kBMn><<<grid, kGemmThreads, GemmCfg<1>::kSmem, st>>>(ta, tb, p);
  mrl_profile_after(st);
  MRL_CUDA_OK(cudaGetLastError());
  return MRL_OK;
}

long long pad_to(long long x, long long a) { return (x + a - 1) / a * a; }

struct LmheadWs {
  void* rows;            // per-row scratch of the loss (MrlLossWs)
  float *g, *lse2, *zt;
  float2* partial;
  float* partial_u;      // the entropy's third partial
  __nv_bfloat16* D;      // one vocabulary chunk of dZ, [N, ldD]
  float* dH_acc;
  uint8_t* live;         // per block of 256 rows
  TileLists fwd, bwd;    // rows the forward product has to produce / rows with a gradient
  int n256, n128, n64;
  long long part_ld, ldD;
  int n_tiles_fwd, vchunk, n_chunks;
  size_t bytes;
};

LmheadWs carve_lmhead_ws(void* ws, long long N, int V, int H, int S) {
  LmheadWs w;
  MrlCarver c(ws);
  w.rows = c.take<unsigned char>(mrl_policy_loss_workspace_bytes(N, S));
  w.g = c.take<float>((size_t)N);
  w.lse2 = c.take<float>((size_t)N);
  w.zt = c.take<float>((size_t)N);
  w.n_tiles_fwd = (V + BN - 1) / BN;
  w.part_ld = pad_to(N, BM);
  w.partial = c.take<float2>((size_t)w.n_tiles_fwd * (size_t)w.part_ld);
  w.partial_u = c.take<float>((size_t)w.n_tiles_fwd * (size_t)w.part_ld);
  w.vchunk = V < kVChunk ? (int)pad_to(V, BN) : kVChunk;
  w.n_chunks = (V + w.vchunk - 1) / w.vchunk;
  w.ldD = w.vchunk;
  w.D = c.take<__nv_bfloat16>((size_t)N * (size_t)w.ldD);
  w.dH_acc = w.n_chunks > 1 ? c.take<float>((size_t)N * (size_t)H) : nullptr;
  w.n256 = (int)((N + 255) / 256);
  w.n128 = (int)((N + 127) / 128);
  w.n64 = (int)((N + 63) / 64);
  w.live = c.take<uint8_t>((size_t)w.n256);
  for (TileLists* l : {&w.fwd, &w.bwd}) {
    l->m256 = c.take<int>((size_t)w.n256);
    l->m128 = c.take<int>((size_t)2 * w.n256);
    l->k64 = c.take<int>((size_t)4 * w.n256);
    l->counts = c.take<int>(4);
  }
  w.bytes = c.off;
  return w;
}

}  // namespace

size_t mrl_fused_lmhead_workspace_bytes(long long N, int V, int H, int S) {
  if (N <= 0 || V <= 0 || H <= 0) return 0;
  return carve_lmhead_ws(nullptr, N, V, H, S).bytes;
}

// C[M, N] = A B^T with a plain store (bf16 or fp32, optionally added to): the building block of the two backward
// products, also reachable on its own for checks of the tensor-core mainloop.  a_mn / b_mn: the operand is given
// MN-major, i.e. as the row-major [K, M] (resp. [K, N]) matrix.
static int lmhead_gemm_rows(const void* A, long long lda, bool a_mn, const void* B, long long ldb, bool b_mn, int M,
                            int N, int K, void* C, long long ldc, int c_mode, float* Cacc, long long ldacc,
                            int32_t* status, bool pair_tiles, cudaStream_t st, const TileLists* m_rows,
                            const TileLists* k_rows) {
  GemmParams p = {};
  p.M = M;
  p.N = N;
  p.K = K;
  p.C = C;
  p.ldc = ldc;
  p.c_mode = c_mode;
  p.Cacc = Cacc;
  p.ldacc = ldacc;
  p.status = status;
  if (a_mn && b_mn) return launch_gemm<EPI_STORE, true, true>(A, lda, B, ldb, p, pair_tiles, st, m_rows, k_rows);
  if (b_mn) return launch_gemm<EPI_STORE, false, true>(A, lda, B, ldb, p, pair_tiles, st, m_rows, k_rows);
  if (a_mn) return MRL_ERR_INVALID_ARG;  // not needed by the pass: not instantiated
  return launch_gemm<EPI_STORE, false, false>(A, lda, B, ldb, p, pair_tiles, st, m_rows, k_rows);
}

int mrl_lmhead_gemm(const void* A, long long lda, bool a_mn, const void* B, long long ldb, bool b_mn, int M, int N, int K,
                    void* C, long long ldc, int c_mode, float* Cacc, long long ldacc, int32_t* status, bool pair_tiles,
                    cudaStream_t st) {
  return lmhead_gemm_rows(A, lda, a_mn, B, ldb, b_mn, M, N, K, C, ldc, c_mode, Cacc, ldacc, status, pair_tiles, st,
                          nullptr, nullptr);
}

extern "C" int mrl_fused_lmhead_loss_fwd_bwd(const void* hidden, const void* W, int64_t N, int32_t H, int32_t V,
                                             const int32_t* ids, const uint8_t* mask, const int32_t* cu_seqlens,
                                             int32_t S, const float* adv_seq, const float* logp_old,
                                             const float* tok_weight, const float* nll_weight,
                                             const mrl_loss_params* lp, void* dHidden, void* dW, float* logp,
                                             float* loss, int64_t* stats, int32_t* status, void* workspace,
                                             size_t workspace_bytes, void* stream) {
  if (lp == nullptr || loss == nullptr || N < 0 || S < 0 || V < 1 || H < 1) return MRL_ERR_INVALID_ARG;
  if (H % 64 != 0) return MRL_ERR_UNSUPPORTED_SHAPE;
  if (N > 0x7fffff00ll) return MRL_ERR_UNSUPPORTED_SHAPE;
  if (lp->agg_mode != MRL_AGG_TOKEN_MEAN && lp->agg_mode != MRL_AGG_SEQ_MEAN_TOKEN_MEAN) return MRL_ERR_INVALID_ARG;
  if (!(lp->eps_lo >= 0.f) || !(lp->eps_hi >= 0.f)) return MRL_ERR_INVALID_ARG;
  if (lp->ratio_level != MRL_RATIO_TOKEN && lp->ratio_level != MRL_RATIO_SEQUENCE) return MRL_ERR_INVALID_ARG;
  if (lp->ratio_level == MRL_RATIO_SEQUENCE && tok_weight != nullptr) return MRL_ERR_INVALID_ARG;
  if (!mrl_kl_args_ok(lp)) return MRL_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool accum_loss = lp->flags & MRL_FLAG_ACCUMULATE_LOSS;
  const bool accum_dw = lp->flags & MRL_FLAG_ACCUMULATE_DW;
  const bool pair = lp->flags & MRL_FLAG_PAIR_TILES;
  if (N == 0 || S == 0) {
    if (N != 0) return MRL_ERR_INVALID_ARG;
    if (!accum_loss) {
      MRL_CUDA_OK(cudaMemsetAsync(loss, 0, 2 * sizeof(float), st));
      if (lp->logp_ref != nullptr) MRL_CUDA_OK(cudaMemsetAsync(lp->kl_loss, 0, sizeof(float), st));
      if (stats != nullptr) MRL_CUDA_OK(cudaMemsetAsync(stats, 0, 4 * sizeof(int64_t), st));
    }
    if (dW != nullptr && !accum_dw) MRL_CUDA_OK(cudaMemsetAsync(dW, 0, (size_t)V * H * 2, st));
    return MRL_OK;
  }
  if (hidden == nullptr || W == nullptr || ids == nullptr || cu_seqlens == nullptr || adv_seq == nullptr)
    return MRL_ERR_INVALID_ARG;
  if ((dHidden == nullptr) != (dW == nullptr)) return MRL_ERR_INVALID_ARG;  // both gradients or forward only
  if ((reinterpret_cast<uintptr_t>(hidden) & 15) || (reinterpret_cast<uintptr_t>(W) & 15) ||
      (reinterpret_cast<uintptr_t>(dHidden) & 15) || (reinterpret_cast<uintptr_t>(dW) & 15))
    return MRL_ERR_INVALID_ARG;
  const size_t need = mrl_fused_lmhead_workspace_bytes(N, V, H, S);
  if (workspace == nullptr || workspace_bytes < need) return MRL_ERR_WORKSPACE_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MRL_ERR_INVALID_ARG;
  const LmheadWs w = carve_lmhead_ws(workspace, N, V, H, S);
  const __nv_bfloat16* hid = static_cast<const __nv_bfloat16*>(hidden);
  const __nv_bfloat16* Wm = static_cast<const __nv_bfloat16*>(W);

  MrlLossWs rw;
  int rc = mrl_rows_prepare(w.rows, N, V, S, ids, mask, cu_seqlens, adv_seq, tok_weight, nll_weight, lp, status, st,
                            &rw);
  if (rc != MRL_OK) return rc;
  MRL_CUDA_OK(cudaMemsetAsync(w.zt, 0, (size_t)N * sizeof(float), st));
  const bool seq_ratio = lp->ratio_level == MRL_RATIO_SEQUENCE;
  // a response-level ratio needs every valid row of a response for its sum: nothing is skipped on the way forward
  const uint32_t row_flags = seq_ratio ? (lp->flags & ~MRL_FLAG_SKIP_ZERO_ROWS) : lp->flags;
  const bool has_ref = !seq_ratio && lp->logp_ref != nullptr;
  const unsigned live_grid = (unsigned)((w.n256 + 7) / 8);

  // ---- which blocks of rows the forward product has to produce (all-masked blocks never; zero-multiplier blocks
  // not under MRL_FLAG_SKIP_ZERO_ROWS)
  tile_live_kernel<<<live_grid, 256, 0, st>>>(N, w.n256, 1, nullptr, ids, mask, V, rw.rowA, rw.rowcu, rw.rowcn, rw.rowck,
                                              has_ref, row_flags, w.live);
  MRL_CUDA_OK(cudaGetLastError());
  tile_lists_kernel<<<1, 1024, 0, st>>>(w.n256, w.n128, w.n64, w.live, w.fwd.m256, w.fwd.m128, w.fwd.k64, w.fwd.counts);
  MRL_CUDA_OK(cudaGetLastError());

  // ---- forward: per-tile log-sum-exp partials and the target logit, logits never stored
  {
    GemmParams p = {};
    p.M = (int)N;
    p.N = V;
    p.K = H;
    p.status = status;
    p.partial = w.partial;
    p.partial_u = w.partial_u;
    p.part_ld = w.part_ld;
    p.ids = ids;
    p.zt = w.zt;
    p.col0 = 0;
    rc = lp->entropy != nullptr ? launch_gemm<EPI_LSE_ENT, false, false>(hid, H, Wm, H, p, pair, st, &w.fwd)
                                : launch_gemm<EPI_LSE, false, false>(hid, H, Wm, H, p, pair, st, &w.fwd);
    if (rc != MRL_OK) return rc;
  }
  lmhead_rows_kernel<<<(unsigned)((N + 255) / 256), 256, 0, st>>>(N, V, w.n_tiles_fwd, w.partial, w.partial_u, lp->entropy,
                                                                  w.part_ld, w.zt, ids,
                                                                  mask, rw.rowA, rw.rowcu, rw.rowcn, rw.rowck, rw.cscale,
                                                                  seq_ratio ? nullptr : lp->logp_ref, lp->kl_estimator,
                                                                  seq_ratio ? nullptr : logp_old, lp->eps_lo,
                                                                  lp->eps_hi, rw.row_m2, rw.row_s, rw.row_zt,
                                                                  rw.rowstat, w.g, w.lse2, row_flags);
  MRL_CUDA_OK(cudaGetLastError());
  if (seq_ratio)  // response-level ratio: g_t comes from the whole response (App. H)
    rc = mrl_rows_finish_sequence(rw, N, S, cu_seqlens, adv_seq, logp_old, nll_weight, lp, logp, loss, stats, w.g,
                                  w.lse2, st);
  else
    rc = mrl_rows_finish(rw, N, logp_old, lp, logp, loss, stats, st);
  if (rc != MRL_OK) return rc;
  if (dHidden == nullptr) return MRL_OK;

  // ---- blocks of rows with a gradient: the rest (zero advantage, clipped, masked) is left out of all three backward
  // products -- their dHidden rows are zero, and they add nothing to dW
  tile_live_kernel<<<live_grid, 256, 0, st>>>(N, w.n256, 0, w.g, nullptr, nullptr, V, nullptr, nullptr, nullptr, nullptr,
                                              false, 0u, w.live);
  MRL_CUDA_OK(cudaGetLastError());
  tile_lists_kernel<<<1, 1024, 0, st>>>(w.n256, w.n128, w.n64, w.live, w.bwd.m256, w.bwd.m128, w.bwd.k64, w.bwd.counts);
  MRL_CUDA_OK(cudaGetLastError());
  MRL_CUDA_OK(cudaMemsetAsync(dHidden, 0, (size_t)N * H * 2, st));

  // ---- backward, per vocabulary chunk.  No operand is transposed in memory: W and hidden enter the two products
  // MN-major, D enters dHidden's K-major and dW's MN-major.
  for (int ch = 0; ch < w.n_chunks; ++ch) {
    const int v0 = ch * w.vchunk;
    const int vc = V - v0 < w.vchunk ? V - v0 : w.vchunk;
    {  // D = g (softmax - onehot) of the chunk's columns
      GemmParams p = {};
      p.M = (int)N;
      p.N = vc;
      p.K = H;
      p.status = status;
      p.ids = ids;
      p.col0 = v0;
      p.g = w.g;
      p.lse2 = w.lse2;
      p.D = w.D;
      p.ldD = w.ldD;
      rc = launch_gemm<EPI_DZ, false, false>(hid, H, Wm + (size_t)v0 * H, H, p, pair, st, &w.bwd);
      if (rc != MRL_OK) return rc;
    }
    {  // dHidden[N, H] (+)= D[N, vc] * W[v0 : v0 + vc, :]   (A = D K-major; B = the chunk of W, [K = vc, N = H])
      int mode = C_BF16;
      if (w.n_chunks > 1) mode = ch == 0 ? C_F32 : (ch == w.n_chunks - 1 ? C_BF16_FROM_ACC : C_F32_ADD);
      void* C = (mode == C_BF16 || mode == C_BF16_FROM_ACC) ? dHidden : static_cast<void*>(w.dH_acc);
      rc = lmhead_gemm_rows(w.D, w.ldD, false, Wm + (size_t)v0 * H, H, true, (int)N, H, vc, C, H, mode, w.dH_acc, H,
                            status, pair, st, &w.bwd, nullptr);
      if (rc != MRL_OK) return rc;
    }
    {  // dW[v0 : v0 + vc, :] = D^T hidden   (A = D as [K = N, M = vc]; B = hidden as [K = N, N = H])
      void* C = accum_dw ? static_cast<void*>(static_cast<float*>(dW) + (size_t)v0 * H)
                         : static_cast<void*>(static_cast<__nv_bfloat16*>(dW) + (size_t)v0 * H);
      rc = lmhead_gemm_rows(w.D, w.ldD, true, hid, H, true, vc, H, (int)N, C, H, accum_dw ? C_F32_ADD : C_BF16, nullptr,
                            0, status, pair, st, nullptr, &w.bwd);
      if (rc != MRL_OK) return rc;
    }
  }
  return MRL_OK;
}
