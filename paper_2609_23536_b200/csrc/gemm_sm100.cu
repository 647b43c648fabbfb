// FP8 GEMM for sm_100a: D[M,N] = (A[M,Kc] . B[N,Kc]^T) * alpha, A and B bytes (E4M3 or E5M2, mixed freely), each
// stored contraction-major ([rows, Kc]) or, in the paired variant, MN-major ([Kc, rows]: the transposed view of a
// row-major tensor, read by the tensor cores directly), FP32 accumulation in tensor memory.
//
// Structure (one persistent CTA per SM, 320 threads):
//   warp 0      TMA producer: cp.async.bulk.tensor 2D tiles (128-byte swizzle) into a shared-memory ring (6 stages
//               of 32 KB in the paired variant, 4 of 48 KB in the single-CTA one)
//   warp 1      allocates tensor memory, then one lane issues tcgen05.mma (128 x 256 x 32 per instruction) and
//               tcgen05.commit to release ring stages / publish a finished accumulator
//   warps 2-9   epilogue: tcgen05.ld the 128 x 256 FP32 accumulator (two warps per 32-lane quadrant, 128 columns
//               each) in 32 x 32 blocks, scale, write each block into a swizzled per-warp shared-memory tile and
//               hand it to the bulk-store unit: a bulk tensor store for bf16 (+ max|D| reduced by warp shuffles,
//               one atomicMax per warp and tile) and for FP32 overwrite; a bulk tensor reduction (.add) for FP32
//               accumulation straight into the destination (direct gradient placement): the addition is done in
//               L2, one per element and launch, and the destination tile is prefetched into L2 while the tile's
//               main loop runs.  The reduction is a plain round-to-nearest FP32 addition (subnormal values kept).
//   The launch may also carry up to eight independent problems (grouped launch): tiles are numbered problem after
//   problem and each role looks its tile's problem up, so that one set of persistent CTAs packs them all.
// When asked to, the last CTA to finish folds the pending amax values into their histories and updates the scales
// (the commit that ends F and dI), so that no extra launch is needed for it.
// Two accumulators (2 x 256 tensor-memory columns) let the epilogue of tile i overlap the main loop of tile i+1.
//
// Two variants share the code below.  The single-CTA one computes 128 x 256 tiles.  The paired one (used whenever M
// is a multiple of 256) runs as clusters of two CTAs on neighbouring SMs that compute one 256 x 256 tile together
// with tcgen05.mma.cta_group::2: each CTA loads its own 128 rows of A and its own 128 rows of B (32 KB per stage
// instead of 48 KB), the even CTA issues the MMAs for the pair, tcgen05.commit multicasts stage-free and
// accumulator-ready arrivals to both CTAs, and each CTA drains its own 128 accumulator rows.  That halves the
// B-operand shared-memory traffic per SM, which is what bounds the single-CTA variant.  No TMA multicast is used.
// Each output element is produced by exactly one thread with a fixed contraction order and reaches its destination
// by exactly one store or one addition per launch, so results do not depend on the grid size or on how tiles are
// scheduled (no split-K; launches that add to the same destination are ordered by their stream).
//
// Every wait on an mbarrier is bounded by a clock budget; on expiry the thread ORs an error bit into the status
// word, raises a CTA-wide abort flag that all other waits observe, and the CTA falls through to its common exit
// where tensor memory is released.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "commit.cuh"
#include "kernels.h"

namespace qe {
namespace {

constexpr int BM = 128, BN = 256, BK = 128;  // per-CTA rows, tile columns, bytes (= FP8 elements) per stage along K
constexpr int UMMA_K = 32;
constexpr uint32_t A_BYTES = BM * BK;
constexpr uint32_t TMEM_COLS = 512;
constexpr int MAX_STAGES = 6;
constexpr uint32_t EPI_BUF_BYTES = 4096;                     // per epilogue warp: one FP32 or two bf16 32 x 32 output tiles
                                                             // (1 KB-aligned, swizzled) that the bulk-store unit reads
template <bool TWO>
struct Cfg {
  static constexpr int STAGES = TWO ? 6 : 4;
  static constexpr uint32_t B_ROWS = TWO ? 128 : 256;  // rows of B this CTA loads per stage
  static constexpr uint32_t B_BYTES = B_ROWS * BK;
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr uint32_t TILE_M = TWO ? 256 : 128;  // rows of D per tile (per cluster)
  static constexpr uint32_t CTAS = TWO ? 2 : 1;
};
constexpr int THREADS = 320;
constexpr int EPI_WARPS = 8, EPI_THREADS = EPI_WARPS * 32;
static_assert(EPI_WARPS == 8, "shared-memory budget below assumes 8 epilogue warps");
constexpr uint32_t SMEM_BYTES = 6 * (A_BYTES + 128 * BK) + 1024 /*alignment slack*/ + 256 /*barriers, flags*/ +
                                8 * EPI_BUF_BYTES;  // 192 KB of stages in either variant
constexpr long long WAIT_BUDGET_CYCLES = 4000000000ll;  // ~2 s at the maximum SM clock

constexpr uint32_t ERR_PRODUCER = 1u, ERR_MMA = 2u, ERR_EPILOGUE = 4u;

// ------------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

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
// Bounded wait.  Returns false if the budget ran out or another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t err_bit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > WAIT_BUDGET_CYCLES) {
      *abort_flag = 1u;
      atomicOr(status, err_bit);
      return false;
    }
  }
}

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {  // barrier may live in the peer CTA
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster (shared::cluster window).
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load whose completion is credited to a barrier that may live in the peer CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {  // arrives on `bar` in both CTAs of the pair
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3)
               : "memory");
}
__device__ __forceinline__ void tc_mma_f8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int c0, int c1) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(c0), "r"(c1) : "memory");
}

// Bulk tensor store of a shared-memory tile (issued by one lane), with group tracking.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Bulk tensor reduction: global tile += shared-memory tile, added element by element where the data lives (L2).
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void tma_store_wait_read() {  // at most N groups may still be reading shared memory
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Shared-memory matrix descriptor for a contraction-major tile whose rows are 128 bytes, 128-byte swizzle:
// start address (>>4) in bits 0-13; leading byte offset (unused for this layout) 1 in bits 16-29; stride byte
// offset = 1024 (eight 128-byte rows) >>4 in bits 32-45; descriptor version 1 in bits 46-47; swizzle mode 2
// (128 B) in bits 61-63.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);  // .x = a in the low half
  return *reinterpret_cast<uint32_t*>(&v);
}

// Tile order.  The CTAs running at the same time take consecutive tiles.  Walking the dimension of the SMALLER
// operand fastest means that operand is swept again and again (from L2, where it fits) while the larger one is
// streamed from HBM once.
__device__ __forceinline__ void tile_coords(uint32_t tile, uint32_t tiles_m, uint32_t tiles_n, bool m_fastest,
                                            uint32_t tile_m, uint32_t& m0, uint32_t& n0) {
  if (m_fastest) {
    m0 = (tile % tiles_m) * tile_m;
    n0 = (tile / tiles_m) * BN;
  } else {
    n0 = (tile % tiles_n) * BN;
    m0 = (tile / tiles_n) * tile_m;
  }
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory"); }

// Which tile cluster `first` of `step` clusters takes in wave w: the clusters walk the tile list back and forth, so
// that with tiles sorted by decreasing duration the cluster that got the longest tile of one wave gets the shortest
// of the next (a static approximation of longest-processing-time-first).
__device__ __forceinline__ uint32_t snake_tile(uint32_t w, uint32_t first, uint32_t step) {
  return w * step + ((w & 1u) ? step - 1u - first : first);
}

// ------------------------------------------------------------------------------------------------ problem lookup
// A launch computes one GEMM, or (grouped launch) up to four independent ones whose tiles are numbered one after the
// other, so that one set of persistent CTAs packs them into common waves and the launch overhead is paid once.
struct OneProblem {
  const GemmParams& p;
  __device__ __forceinline__ uint32_t total_tiles(uint32_t tile_m) const { return (p.M / tile_m) * ((p.N + BN - 1) / BN); }
  __device__ __forceinline__ const GemmParams& at(uint32_t tile, uint32_t& local) const {
    local = tile;
    return p;
  }
  __device__ __forceinline__ const GemmParams& first() const { return p; }
  __device__ __forceinline__ uint32_t count() const { return 1; }
  __device__ __forceinline__ const CommitParams& commit(uint32_t) const { return p.commit; }
  __device__ __forceinline__ uint32_t* status_of(uint32_t) const { return p.status; }
};
struct ProblemGroup {
  const GemmGroupParams& g;
  __device__ __forceinline__ uint32_t total_tiles(uint32_t) const { return g.tile_end[g.n - 1]; }
  __device__ __forceinline__ const GemmParams& at(uint32_t tile, uint32_t& local) const {
    uint32_t i = 0, base = 0;
    while (i + 1 < g.n && tile >= g.tile_end[i]) base = g.tile_end[i++];
    local = tile - base;
    return g.prob[i];
  }
  __device__ __forceinline__ const GemmParams& first() const { return g.prob[0]; }
  __device__ __forceinline__ uint32_t count() const { return g.n; }
  __device__ __forceinline__ const CommitParams& commit(uint32_t i) const { return g.prob[i].commit; }
  __device__ __forceinline__ uint32_t* status_of(uint32_t i) const { return g.prob[i].status; }
};

// ------------------------------------------------------------------------------------------------ kernel
template <bool TWO, class PS>
__device__ __forceinline__ void gemm_body(const PS& ps) {
  using C = Cfg<TWO>;
  constexpr int STAGES = C::STAGES;
  constexpr uint32_t STAGE_BYTES = C::STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t epi_base = smem_base + STAGES * STAGE_BYTES;  // 1 KB-aligned
  const uint32_t bar_base = epi_base + 8 * EPI_BUF_BYTES;
  // barrier block: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], then tmem address + abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + 2 + a); };
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + STAGES * STAGE_BYTES + 8 * EPI_BUF_BYTES + 8 * (2 * MAX_STAGES + 4));
  volatile uint32_t* abort_flag = tmem_slot + 1;
  uint32_t* last_flag = tmem_slot + 2;
  uint32_t* red = tmem_slot + 4;  // 8 words for the commit's reduction

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = TWO ? cluster_ctarank() : 0u;  // position in the CTA pair; rank 0 issues the MMAs
  const uint32_t num_tiles = ps.total_tiles(C::TILE_M);
  const uint32_t first_tile = blockIdx.x / C::CTAS, tile_step = gridDim.x / C::CTAS;
  uint32_t* const status = ps.first().status;
// per tile: which problem it belongs to (`p`), its index inside that problem and the problem's tiling
#define QE_TILE_PROBLEM()                                                                      \
  uint32_t local_tile;                                                                         \
  const GemmParams& p = ps.at(tile, local_tile);                                               \
  const uint32_t tiles_m = p.M / C::TILE_M, tiles_n = (p.N + BN - 1) / BN, num_kb = p.Kc / BK; \
  const bool m_fastest = p.M <= p.N

  if (threadIdx.x == 32) {  // descriptor fetch overlaps the rest of the prologue (and the predecessor's tail)
    const GemmParams& q = ps.first();  // (a group's other descriptors are fetched on first use)
    asm volatile("prefetch.tensormap [%0];" ::"l"(&q.tmA) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&q.tmB) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&q.tmD) : "memory");
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), EPI_WARPS * C::CTAS);  // the epilogue warps of every CTA of the pair
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (TWO) {  // same warp in both CTAs of the pair
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (TWO) cluster_sync_all();  // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (warp == 0 && lane == 0 && first_tile < num_tiles) {
    // While the predecessor drains: pull the first ring-full of B tiles of this CTA's first tile towards L2.  A
    // prefetch moves no data into the SM, so it is harmless even if the predecessor is still writing that operand.
    const uint32_t tile = first_tile;
    QE_TILE_PROBLEM();
    uint32_t m0, n0;
    tile_coords(local_tile, tiles_m, tiles_n, m_fastest, C::TILE_M, m0, n0);
    const int rb = (int)(n0 + (TWO ? rank * C::B_ROWS : 0u));
    for (uint32_t kb = 0; kb < num_kb && kb < (uint32_t)STAGES; ++kb) {
      const int ka = (int)(kb * BK);
      if (p.b_mn) tma_prefetch_2d(&p.tmB, rb, ka);
      else tma_prefetch_2d(&p.tmB, ka, rb);
    }
  }
  // Everything above (barriers, tensor memory) touched no data a predecessor produces and may overlap the previous
  // kernel's tail; operands, scales and the destination may come from it, so wait for it here.
  grid_dep_wait();
  grid_dep_launch();
  if (blockIdx.x == 0 && threadIdx.x == 64) {  // FP8 hand-off: the consumer's tape snapshot of its inverse scale
    const GemmParams& q = ps.first();
    if (q.epi == 3 && q.sinv_dst) *q.sinv_dst = *q.sinv_src;
  }

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (uint32_t wave = 0, tile = first_tile; ok && tile < num_tiles; ++wave, tile = snake_tile(wave, first_tile, tile_step)) {
        QE_TILE_PROBLEM();
        uint32_t m0, n0;
        tile_coords(local_tile, tiles_m, tiles_n, m_fastest, C::TILE_M, m0, n0);
        for (uint32_t kb = 0; kb < num_kb; ++kb) {
          if (!(ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, status, ERR_PRODUCER))) break;
          const uint32_t a_dst = smem_base + s * STAGE_BYTES, b_dst = a_dst + A_BYTES;
          if (TWO) {
            // both CTAs credit the even CTA's barrier, which expects the bytes of the whole pair
            if (rank == 0) mbar_expect_tx(full_bar(s), 2 * STAGE_BYTES);
            const uint32_t bar = map_to_cta(full_bar(s), 0);
            // contraction-major operand: box = 128 K-bytes x 128 rows at (k, row); MN-major operand (stored as
            // [Kc, rows]): box = 128 row-bytes x 128 K-rows at (row, k).  Either way 16 KB land in shared memory.
            const int ka = (int)(kb * BK), ra = (int)(m0 + rank * BM), rb = (int)(n0 + rank * C::B_ROWS);
            if (p.a_mn) tma_load_2d_pair(a_dst, &p.tmA, bar, ra, ka);
            else tma_load_2d_pair(a_dst, &p.tmA, bar, ka, ra);
            if (p.b_mn) tma_load_2d_pair(b_dst, &p.tmB, bar, rb, ka);
            else tma_load_2d_pair(b_dst, &p.tmB, bar, ka, rb);
          } else {
            mbar_expect_tx(full_bar(s), STAGE_BYTES);
            tma_load_2d(a_dst, &p.tmA, full_bar(s), (int)(kb * BK), (int)m0);
            tma_load_2d(b_dst, &p.tmB, full_bar(s), (int)(kb * BK), (int)n0);
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        // give copies already in flight a bounded chance to land before the CTA's shared memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0 && rank == 0) {
      int s = 0;
      uint32_t ph = 0, acc = 0, acc_ph = 0;
      bool ok = true;
      for (uint32_t wave = 0, tile = first_tile; ok && tile < num_tiles; ++wave, tile = snake_tile(wave, first_tile, tile_step)) {
        QE_TILE_PROBLEM();
        (void)tiles_m; (void)tiles_n; (void)m_fastest;
        if (!(ok = mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, status, ERR_MMA))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * (uint32_t)BN;
        for (uint32_t kb = 0; kb < num_kb; ++kb) {
          if (!(ok = mbar_wait(full_bar(s), ph, abort_flag, status, ERR_MMA))) break;
          tc_fence_after();
          const uint32_t a_src = smem_base + s * STAGE_BYTES, b_src = a_src + A_BYTES;
          const uint64_t adesc = make_desc(a_src), bdesc = make_desc(b_src);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 32 along the contraction: 32 bytes inside the 128-byte swizzle row for a contraction-major
            // tile (+2 in the address field), 32 rows of 128 bytes for an MN-major one (+256)
            if (TWO) tc_mma_f8_pair(d_tmem, adesc + (p.a_mn ? 256u : 2u) * k, bdesc + (p.b_mn ? 256u : 2u) * k, p.idesc, (kb | (uint32_t)k) != 0u);
            else tc_mma_f8(d_tmem, adesc + 2u * k, bdesc + 2u * k, p.idesc, (kb | (uint32_t)k) != 0u);
          }
          if (TWO) tc_commit_pair(empty_bar(s));  // stage reusable (in both CTAs) once these MMAs have read it
          else tc_commit(empty_bar(s));
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        if (TWO) tc_commit_pair(tfull_bar(acc));  // accumulator complete (each CTA holds its 128 rows)
        else tc_commit(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue (warps 2..9)
    const uint32_t quad = (uint32_t)warp & 3u;          // tensor-memory lane quadrant this warp may read
    const uint32_t half = ((uint32_t)warp - 2u) >> 2;   // which 128 of the tile's 256 columns
    const int etid = (int)threadIdx.x - 64;
    const uint32_t epi_smem = epi_base + (uint32_t)(warp - 2) * EPI_BUF_BYTES;  // this warp's two output tiles
    uint32_t n_groups = 0;  // bulk-store groups this warp has committed (buffer parity)
    uint32_t acc = 0, acc_ph = 0;
    bool ok = true;
    const uint32_t tempty_leader0 = TWO ? map_to_cta(tempty_bar(0), 0) : tempty_bar(0);
    const uint32_t tempty_leader1 = TWO ? map_to_cta(tempty_bar(1), 0) : tempty_bar(1);
    for (uint32_t wave = 0, tile = first_tile; ok && tile < num_tiles; ++wave, tile = snake_tile(wave, first_tile, tile_step)) {
      QE_TILE_PROBLEM();
      (void)num_kb;
      const float alpha = __fmul_rn(*p.alpha_a, *p.alpha_b);
      uint32_t m0, n0;
      tile_coords(local_tile, tiles_m, tiles_n, m_fastest, C::TILE_M, m0, n0);
      const uint32_t row = m0 + rank * BM + quad * 32u + (uint32_t)lane;
      const uint32_t col0 = n0 + half * 128u;
      if (p.epi == 2 && col0 < p.N) {
        // accumulate: pull this thread's 512 destination bytes into L2, where the reduction will add to them, while
        // the MMAs of the tile run
        const char* d = reinterpret_cast<const char*>(reinterpret_cast<const float*>(p.out) + (size_t)row * p.ldo + col0);
#pragma unroll
        for (int j = 0; j < 4; ++j) asm volatile("prefetch.global.L2 [%0];" ::"l"(d + 128 * j));
      }
      const uint32_t blk_row0 = m0 + rank * BM + quad * 32u;
      const uint32_t nch = col0 >= p.N ? 0u : min(4u, (p.N - col0) / 32u);  // ragged last column tile; warp-uniform
      uint32_t r[2][32];
      if (!(ok = mbar_wait(tfull_bar(acc), acc_ph, abort_flag, status, ERR_EPILOGUE))) break;
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((quad * 32u) << 16) + acc * (uint32_t)BN + half * 128u;
      uint32_t amax_bits = 0;
      // Software pipeline over the warp's four 32 x 32 blocks: the tensor-memory load of block ch+1 is in flight
      // while block ch is scaled, written to shared memory and handed to the bulk-store unit.
      if (nch) tmem_ld32(t_row, r[0]);
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        if ((uint32_t)ch >= nch) break;
        const uint32_t col = col0 + ch * 32u;
        tmem_ld_wait();
        if ((uint32_t)ch + 1 < nch) tmem_ld32(t_row + (ch + 1) * 32u, r[(ch + 1) & 1]);
        const uint32_t(&rc)[32] = r[ch & 1];
        // Each lane (= row) writes its 32 columns into a swizzled shared-memory tile (conflict-free); one lane hands
        // the 32 x 32 tile to the bulk-store unit, which writes full rows to global memory (bf16, FP32 overwrite) or
        // adds them to the destination where it lives, in L2 (FP32 accumulate: one addition per element and launch).
        if (p.epi == 0) {
          const uint32_t buf = epi_smem + (n_groups & 1u) * 2048u;  // two tiles: the previous store may still read
          if (lane == 0) tma_store_wait_read<1>();
          __syncwarp();
          uint32_t o[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            o[j] = pack_bf16(__fmul_rn(__uint_as_float(rc[2 * j]), alpha), __fmul_rn(__uint_as_float(rc[2 * j + 1]), alpha));
            amax_bits = __vmaxu2(amax_bits, o[j] & 0x7fff7fffu);  // packed magnitudes of the rounded values stored
          }
#pragma unroll
          for (int c = 0; c < 4; ++c) {  // 64-byte rows, 64-byte swizzle: 16-byte chunk c of row r sits at c ^ ((r >> 1) & 3)
            const uint32_t dst = buf + (uint32_t)lane * 64u + (((uint32_t)c ^ (((uint32_t)lane >> 1) & 3u)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(o[4 * c]), "r"(o[4 * c + 1]),
                         "r"(o[4 * c + 2]), "r"(o[4 * c + 3])
                         : "memory");
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) tma_store_2d(&p.tmD, buf, (int)col, (int)blk_row0);
        } else if (p.epi == 3) {
          // FP8 hand-off to the consuming linear: round to bf16 (the value that linear would have read), take its
          // magnitude for the amax, multiply by the consumer's scale in FP32 and convert -- the consumer's cast
          // kernel, applied to registers.  32 bytes per row; two 1 KB tiles per warp.
          const uint32_t buf = epi_smem + (n_groups & 1u) * 1024u;
          if (lane == 0) tma_store_wait_read<1>();
          __syncwarp();
          const float qs = *p.out_scale;
          uint32_t q[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint32_t w[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              w[h] = pack_bf16(__fmul_rn(__uint_as_float(rc[4 * j + 2 * h]), alpha), __fmul_rn(__uint_as_float(rc[4 * j + 2 * h + 1]), alpha));
              amax_bits = __vmaxu2(amax_bits, w[h] & 0x7fff7fffu);
            }
            const float2 f01 = make_float2(__fmul_rn(__uint_as_float(w[0] << 16), qs), __fmul_rn(__uint_as_float(w[0] & 0xffff0000u), qs));
            const float2 f23 = make_float2(__fmul_rn(__uint_as_float(w[1] << 16), qs), __fmul_rn(__uint_as_float(w[1] & 0xffff0000u), qs));
            const uint32_t lo = p.out_fmt == 0 ? __nv_cvt_float2_to_fp8x2(f01, __NV_SATFINITE, __NV_E4M3)
                                               : __nv_cvt_float2_to_fp8x2(f01, __NV_SATFINITE, __NV_E5M2);
            const uint32_t hi = p.out_fmt == 0 ? __nv_cvt_float2_to_fp8x2(f23, __NV_SATFINITE, __NV_E4M3)
                                               : __nv_cvt_float2_to_fp8x2(f23, __NV_SATFINITE, __NV_E5M2);
            q[j] = lo | (hi << 16);
          }
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const uint32_t dst = buf + (uint32_t)lane * 32u + ((uint32_t)c << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(q[4 * c]), "r"(q[4 * c + 1]),
                         "r"(q[4 * c + 2]), "r"(q[4 * c + 3])
                         : "memory");
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) tma_store_2d(&p.tmD, buf, (int)col, (int)blk_row0);
        } else {
          // one tile: waiting for the previous block's store to have read it paces the FP32 traffic, which measured
          // faster than two tiles in flight per warp
          const uint32_t buf = epi_smem;
          if (lane == 0) tma_store_wait_read<0>();
          __syncwarp();
#pragma unroll
          for (int c = 0; c < 8; ++c) {  // 128-byte rows, 128-byte swizzle: chunk c of row r sits at c ^ (r & 7)
            const uint32_t dst = buf + (uint32_t)lane * 128u + (((uint32_t)c ^ ((uint32_t)lane & 7u)) << 4);
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst),
                         "f"(__fmul_rn(__uint_as_float(rc[4 * c]), alpha)), "f"(__fmul_rn(__uint_as_float(rc[4 * c + 1]), alpha)),
                         "f"(__fmul_rn(__uint_as_float(rc[4 * c + 2]), alpha)), "f"(__fmul_rn(__uint_as_float(rc[4 * c + 3]), alpha))
                         : "memory");
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (p.epi == 2) tma_reduce_add_2d(&p.tmD, buf, (int)col, (int)blk_row0);
            else tma_store_2d(&p.tmD, buf, (int)col, (int)blk_row0);
          }
        }
        ++n_groups;
      }
      // accumulator drained: hand it back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (TWO) mbar_arrive_cluster(acc ? tempty_leader1 : tempty_leader0);  // the MMA issuer waits in the even CTA
        else mbar_arrive(tempty_bar(acc));
      }
      if ((p.epi == 0 || p.epi == 3) && (p.amax_bits || p.amax_bits2)) {
        // two packed bf16 magnitudes -> FP32 bit pattern of the larger
        const uint32_t w = __reduce_max_sync(0xffffffffu, max(amax_bits & 0xffffu, amax_bits >> 16) << 16);
        if (lane == 0 && w) {
          if (p.amax_bits) atomicMax(p.amax_bits, w);
          if (p.amax_bits2) atomicMax(p.amax_bits2, w);
        }
      }
      if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
    }
    // Every epilogue thread of every CTA gets here (also after a timeout); the last CTA commits the scale state of
    // every problem that asks for it.  The commit needs the amax atomics only, so it runs while this CTA's last
    // bulk stores are still draining.
    uint32_t* ticket = nullptr;
    for (uint32_t i = 0; i < ps.count(); ++i)
      if (!ticket && ps.commit(i).st) ticket = &ps.commit(i).st->ticket;
    if (ticket && last_block(ticket, gridDim.x, etid, last_flag, epi_bar_sync)) {
      if (ps.count() == 1) {
        if (ps.commit(0).st) commit_classes(ps.commit(0), etid, red, epi_bar_sync);
      } else {
        // one epilogue warp per problem, side by side
        for (uint32_t i = (uint32_t)warp - 2u; i < ps.count(); i += EPI_WARPS)
          if (ps.commit(i).st) commit_classes_warp(ps.commit(i), lane);
      }
    }
    if (lane == 0) tma_store_wait_all();  // this warp's bulk stores have reached global memory
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // a wait gave up in this CTA: the error bits went to the first problem's status word; every other problem of a
    // shared launch gets them too, since any of their tiles may be missing
    const uint32_t bits = atomicOr(status, 0u);
    for (uint32_t i = 1; i < ps.count(); ++i)
      if (ps.status_of(i) && ps.status_of(i) != status) atomicOr(ps.status_of(i), bits);
  }
  if (TWO) cluster_sync_all();  // no arrival may still be on its way to a CTA that has left
  if (warp == 1) {
    tc_fence_after();
    if (TWO)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

#undef QE_TILE_PROBLEM

__global__ void __launch_bounds__(THREADS, 1) gemm_fp8_kernel(const __grid_constant__ GemmParams p) {
  gemm_body<false>(OneProblem{p});
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
    gemm_fp8_pair_kernel(const __grid_constant__ GemmParams p) {
  gemm_body<true>(OneProblem{p});
}

// Up to eight independent GEMMs (each eligible for the paired variant) in one launch.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
    gemm_fp8_pair_group_kernel(const __grid_constant__ GemmGroupParams g) {
  gemm_body<true>(ProblemGroup{g});
}

}  // namespace

bool gemm_uses_pair(uint32_t M) { return M % 256 == 0; }

uint32_t gemm_b_box_rows(uint32_t M) { return gemm_uses_pair(M) ? 128u : 256u; }

uint32_t gemm_idesc(int a_fmt, int b_fmt, uint32_t M, bool a_mn, bool b_mn) {
  // bits 4-5: accumulator format (1 = FP32); 7-9 / 10-12: A / B format (0 = E4M3, 1 = E5M2); 15 / 16: A / B major
  // (0 = contraction-major); 17-22: N >> 3; 24-28: M >> 4 (128 per CTA, 256 for a CTA pair).
  const uint32_t mma_m = gemm_uses_pair(M) ? 256u : 128u;
  return (1u << 4) | ((uint32_t)a_fmt << 7) | ((uint32_t)b_fmt << 10) | ((a_mn ? 1u : 0u) << 15) |
         ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((mma_m >> 4) << 24);
}

cudaError_t gemm_prepare() {
  cudaError_t e = cudaFuncSetAttribute((const void*)gemm_fp8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)SMEM_BYTES);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute((const void*)gemm_fp8_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute((const void*)gemm_fp8_pair_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)SMEM_BYTES);
}

bool make_gemm_group(const GemmParams* probs, uint32_t n, int num_sms, Launch* out) {
  if (n < 2 || n > 8) return false;
  GemmGroupParams g{};
  uint32_t tiles = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (!gemm_uses_pair(probs[i].M)) return false;  // paired variant only
    tiles += (probs[i].M / 256u) * ((probs[i].N + BN - 1) / BN);
    g.tile_end[i] = tiles;
    g.prob[i] = probs[i];
  }
  g.n = n;
  Launch l;
  l.func = (const void*)gemm_fp8_pair_group_kernel;
  const uint32_t ctas = 2u * tiles, cap = (uint32_t)num_sms & ~1u;
  l.grid = dim3(ctas < cap ? ctas : cap, 1, 1);
  l.block = dim3(THREADS, 1, 1);
  l.smem = SMEM_BYTES;
  l.set(g);
  *out = l;
  return true;
}

Launch make_gemm(const GemmParams& p, int num_sms) {
  Launch l;
  if (gemm_uses_pair(p.M)) {
    l.func = (const void*)gemm_fp8_pair_kernel;
    const uint32_t ctas = 2u * (p.M / 256u) * ((p.N + BN - 1) / BN);
    const uint32_t cap = (uint32_t)num_sms & ~1u;
    l.grid = dim3(ctas < cap ? ctas : cap, 1, 1);
    l.block = dim3(THREADS, 1, 1);
    l.smem = SMEM_BYTES;
    l.set(p);
    return l;
  }
  l.func = (const void*)gemm_fp8_kernel;
  const uint32_t tiles = (p.M / BM) * ((p.N + BN - 1) / BN);
  l.grid = dim3(tiles < (uint32_t)num_sms ? tiles : (uint32_t)num_sms, 1, 1);
  l.block = dim3(THREADS, 1, 1);
  l.smem = SMEM_BYTES;
  l.set(p);
  return l;
}

}  // namespace qe
