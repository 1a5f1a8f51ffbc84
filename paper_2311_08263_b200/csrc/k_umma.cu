// Weight-streaming skinny GEMM for sm_100a:  y[R, N] (+)= pro(x)[R, K] . W[N, K]^T,  R = batch * c rows,
// for up to four projections of a decoder layer in one persistent launch.
//
// The contraction is computed "swapped": a 128-row tile of W is the M operand of tcgen05.mma, a block of
// BN rows is the N operand, and the fp32 accumulator lives in tensor memory.  W tiles (128 rows x 64 k, 16 KB)
// arrive by TMA into a 128B-swizzled shared-memory ring.  The activation operand is a bf16 pair high + low
// (low = bf16(x - high)) in the same swizzled K-major layout: up to 16 rows four staging warps read the fp32
// activations, apply the fused transform (RMSNorm gain, or SwiGLU of the gate/up accumulators) and store both
// tiles; with more rows all CTAs convert the activations once per projection into a panel in global memory and
// one thread streams panel tiles by TMA.  Work is claimed dynamically in chunks of a few k-blocks of one tile;
// every partial accumulator is added to y with fp32 reductions in L2, so no second pass is needed and HBM
// traffic is W exactly once.
//
// Warp roles (320 threads): 0 = chunk claims + TMA producer, 1 = MMA issuer + TMEM owner, 2-5 = activation
// staging, 6-9 = epilogue (TMEM -> registers -> global).  Two accumulators alternate so the epilogue of one
// segment overlaps the MMAs of the next.  Every wait is bounded; on expiry the CTA records an error word,
// drains its own copies and MMAs (bounded too), frees TMEM and returns.
#include <cuda.h>

#include <cstdio>
#include <cstring>

#include "fc_internal.h"

namespace fc {

constexpr int kTileM = 128;       // weight rows per tile
constexpr int kTileK = 64;        // k elements per stage (128 bytes of bf16 = one swizzle row)
constexpr int kWBytes = kTileM * kTileK * 2;
constexpr int kThreads = 320;
constexpr unsigned long long kSpinBudget = 400000000ull;    // clock64 ticks (~0.2 s)

// Activations are staged as a bf16 pair hi + lo (lo = bf16(x - hi)), which removes the bf16 rounding of the
// activations; the two tiles are multiplied by one MMA of twice the width.  More than 128 rows run as blocks of
// 128 on the same weight chunk, back to back.
__host__ __device__ constexpr int x_parts(int bn) { return 2; }

constexpr int kMaxPhases = kChainMax;   // projections chained in one launch (O -> gate/up halves -> down halves -> next QKV)

struct PhaseDesc {
  GemmArgs g;
  int pro;                        // ProOp applied while the activations are staged
  int n_tiles, nkb;               // weight tiles over all matrices; 64-wide k blocks
  int tile_rows;                  // weight rows per tile: 128, or 256 when a pair of CTAs shares a tile (each CTA 128 of them)
  int tiles_m[kMaxMats];
  int tx_bytes[kMaxMats];         // bytes one TMA box of matrix m delivers
  int chunk_kb, cpt, nrb, n_chunks;   // work is claimed in chunks of chunk_kb k-blocks of one tile for one block of rows:
                                      // chunks per tile, row blocks, total
  int k_major;                        // claim order: all tiles of one k range before the next k range
  // Synchronisation with the other phases of a chained launch.  Either a grid barrier (wait_bar: index of the
  // barrier this phase waits on before its first activation load; sig_bar: index of the one it arrives on; -1: none)
  // or, between tile-major phases and the k-major phase that consumes their sum, one completion counter per
  // 128-column output tile: the producers' epilogue warps count each finished chunk on tile_done[tile]; the consumer
  // stages k-block kb once dep_done[kb / 2] has reached dep_need.
  int wait_bar, sig_bar;
  int epi_bar;                        // grid barrier the epilogue warps pass before their first reduction (-1: none)
  unsigned int *tile_done;
  const unsigned int *dep_done;
  unsigned int dep_need;
  int dep_tiles;                      // number of counters behind dep_done
  int pre_panel;                      // panel mode: the panel was filled by the kernel before this launch
};

struct MapPack {
  CUtensorMap m[kMaxPhases * kMaxMats];   // weights
  CUtensorMap x[kMaxPhases];              // activation panels (rows beyond 16)
};

struct UmmaParams {
  PhaseDesc ph[kMaxPhases];
  int n_phases;
  int stages;
  int pdl;                        // launched as a programmatic dependent of the previous kernel
  unsigned int *err;              // device error word (0 = ok)
  unsigned int *bar;              // [n_phases - 1] grid-barrier counters, zero when the kernel starts
  unsigned int *claim;            // [n_phases] work-claim counters, zero when the kernel starts
  unsigned int *bar_b;            // [n_phases] panel-ready barriers (panel mode), zero when the kernel starts
  ZeroList z;                     // buffers the epilogue warps clear once the previous kernel is complete
};

struct UmmaPlan {
  PhaseDesc d;
  CUtensorMap maps[kMaxMats];
  CUtensorMap xmap[3];            // activation panel [2 * pan_rows, K], boxes of 64 k x 32 / 64 / 128 rows
  bool has_xmap;
  int epi, n_sms;
  unsigned int *err;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false if the budget ran out or another role raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = clock64();
  unsigned int spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 0xFFu) == 0u) {
      if (*abort_flag) return false;
      if ((unsigned long long)(clock64() - t0) > kSpinBudget) { *abort_flag = 1; return false; }
    }
  }
  return true;
}
// Same for a converged warp: every lane waits, and the verdict is made uniform so that the lanes of a
// warp can never part ways around a later warp-level synchronisation.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
  const bool ok = mbar_wait(bar, parity, abort_flag);
  return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// ---- CTA pairs (cta_group::2): a cluster of two CTAs multiplies one 256-row weight tile; each CTA stages its 128
// weight rows and its half of the activation operand, the leader (cluster rank 0) issues the MMAs for both, and the
// accumulator rows of a CTA's 128 weight rows land in that CTA's tensor memory.
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrival on a barrier of any CTA of the cluster (address from map_to_cta)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
// TMA load into this CTA's shared memory whose bytes are counted on a barrier of the pair's leader
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// completion of the pair's MMAs so far, signalled on the barrier at this offset in both CTAs
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 B apart, 8-row groups
// 1024 B apart (the tile base is 1024-byte aligned; k sub-blocks advance the start address by 32 B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);          // start address
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024u >> 4) << 32;                 // stride byte offset
  d |= (uint64_t)1 << 46;                            // descriptor version for sm_100
  d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = bn.
__host__ __device__ constexpr uint32_t make_idesc(int bn, int m = kTileM) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ unsigned int ordered_key_u(float v) {
  if (v != v) return 0u;
  unsigned int u = __float_as_uint(v);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int *p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Grid barrier between two phases of a chained launch.  Every CTA of the grid is resident (the grid is
// sized to the SM count times the CTAs that fit per SM), so the wait ends; it is bounded all the same.
// signal: each participating warp calls it once after its last global write of the phase.
// The kWarpsSignalling warps of a CTA count up in shared memory; the last one posts the CTA's single arrival.
constexpr unsigned int kWarpsSignalling = 8;    // 4 staging + 4 epilogue warps
// Release increments instead of full fences: the warp barrier orders the other lanes' writes before lane 0's
// release, the acquire-release count in shared memory chains the warps of the CTA, and the release on the global
// counter publishes all of it to whoever acquires that counter.
__device__ __forceinline__ void red_release_gpu(unsigned int *p, unsigned int v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void grid_bar_signal(unsigned int *ctr, unsigned int *cta_count, int lane) {
  __syncwarp();
  if (lane == 0) {
    unsigned int prev;
    asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;" : "=r"(prev) : "r"(smem_u32(cta_count)) : "memory");
    if (prev == kWarpsSignalling - 1u) red_release_gpu(ctr, 1u);
  }
}
__device__ __forceinline__ bool grid_bar_wait(const unsigned int *ctr, unsigned int target, int lane,
                                              volatile int *abort_flag) {
  int ok = 1;
  if (lane == 0) {
    const unsigned long long t0 = clock64();
    unsigned int spins = 0;
    while (ld_acquire_u32(ctr) < target) {
      if ((++spins & 0x3Fu) == 0u) {
        if (*abort_flag) { ok = 0; break; }
        if ((unsigned long long)(clock64() - t0) > kSpinBudget) { *abort_flag = 1; ok = 0; break; }
      }
    }
  }
  return __shfl_sync(0xffffffffu, ok, 0) != 0;     // also orders the other lanes after lane 0's acquire
}

struct Segment { int tile, kb0, kb1; };

// Work distribution.  SMs do not all see the same memory bandwidth, so equal static shares finish microseconds
// apart and every grid barrier waits for the slowest.  Instead the producer warp of each CTA claims chunks
// (chunk_kb consecutive k-blocks of one 128-row tile, for one block of rows) from a per-phase global counter
// and publishes them to the other warps of its CTA through a small shared-memory queue; fast CTAs simply
// claim more.  A queue entry with tile < 0 ends the phase.
constexpr int kSegQ = 8;           // queue slots (power of two)
__device__ __forceinline__ void chunk_decode(const PhaseDesc &d, unsigned int id, Segment &s, int &rb) {
  // row blocks vary fastest: the blocks of one weight chunk are claimed one after the other, so the chunk is
  // streamed from HBM once and found in L2 by the later blocks
  if (d.k_major) {
    // with many rows the partial sums of one chunk are a lot of reductions; CTAs that claim one after the other
    // then work on different tiles, so their reductions do not meet on the same addresses
    const int per_k = d.n_tiles * d.nrb;
    const int kc = (int)(id / (unsigned)per_k);
    const int rem = (int)(id - (unsigned)kc * (unsigned)per_k);
    s.tile = rem / d.nrb;
    rb = rem - s.tile * d.nrb;
    s.kb0 = kc * d.chunk_kb;
    s.kb1 = min(d.nkb, s.kb0 + d.chunk_kb);
    return;
  }
  const int per_tile = d.cpt * d.nrb;
  s.tile = (int)(id / (unsigned)per_tile);
  const int rem = (int)(id - (unsigned)s.tile * (unsigned)per_tile);
  const int kc = rem / d.nrb;
  rb = rem - kc * d.nrb;
  s.kb0 = kc * d.chunk_kb;
  s.kb1 = min(d.nkb, s.kb0 + d.chunk_kb);
}

__device__ __forceinline__ void tile_info(const PhaseDesc &d, int tile, int &m, int &row0, int &rows_valid, int &ycol0) {
  m = 0;
  int lt = tile;
  while (m + 1 < d.g.n_mats && lt >= d.tiles_m[m]) { lt -= d.tiles_m[m]; ++m; }
  row0 = lt * d.tile_rows;
  rows_valid = min(d.tile_rows, d.g.n_rows[m] - row0);
  ycol0 = d.g.y_off[m] + row0;
}

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Four fp32 reductions in one instruction (16-byte aligned address).
__device__ __forceinline__ void red_add_v4(float *p, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
// 4 x 4 transpose across the four lanes of a quad and four registers: afterwards lane i holds in register j what
// lane j held in register i.
__device__ __forceinline__ void quad_transpose(float &r0, float &r1, float &r2, float &r3, int lane) {
  const bool b0 = lane & 1, b1 = lane & 2;
  float t;
  t = b0 ? r0 : r1; t = __shfl_xor_sync(0xffffffffu, t, 1); if (b0) r0 = t; else r1 = t;
  t = b0 ? r2 : r3; t = __shfl_xor_sync(0xffffffffu, t, 1); if (b0) r2 = t; else r3 = t;
  t = b1 ? r0 : r2; t = __shfl_xor_sync(0xffffffffu, t, 2); if (b1) r0 = t; else r2 = t;
  t = b1 ? r1 : r3; t = __shfl_xor_sync(0xffffffffu, t, 2); if (b1) r1 = t; else r3 = t;
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o);
    v = t > v ? t : v;
  }
  return v;
}

// Widths up to 32 rows run two CTAs per SM (the grid barrier needs the whole grid resident).
// PANEL: the activations come from a bf16 hi/lo panel in global memory, converted once per projection by all
// CTAs together and streamed by TMA, instead of being converted by every CTA for every weight tile.
// PAIR: launched as clusters of two CTAs that share 256-row weight tiles (panel mode, 128-row blocks): per k-block each
// CTA stages 16 KB of weights and ONE of the two activation tiles (the leader the high one, its peer the low one)
// for 2 x 128 x 256 x 64 products - half of the shared-memory traffic per product of the single-CTA form.  Chunks are
// dealt statically (pair i takes chunks i, i + pairs, ...), so both CTAs of a pair walk the same list without talking.
template <int EPI, int BN, bool PANEL, bool PAIR = false>
__global__ void __launch_bounds__(kThreads, (BN <= 32 ? 2 : 1))
gemm_umma_kernel(const __grid_constant__ MapPack maps, const __grid_constant__ UmmaParams p) {
  static_assert(!PAIR || (PANEL && BN == 128 && EPI == EPI_ATOMIC_ADD), "CTA pairs: panel mode, 128-row blocks, reductions");
  constexpr int kXParts = x_parts(BN);
  constexpr int kXBytes = BN * 128;                 // one staged activation tile (bf16, 64 k)
  constexpr int kStageBytes = kWBytes + (PAIR ? 1 : kXParts) * kXBytes;
  // The high and the low activation tiles lie back to back in a stage, which is exactly a K-major tile of 2 * BN
  // rows: one MMA of N = 2 * BN multiplies both (columns 0..BN-1 of the accumulator take the high part's products,
  // BN..2BN-1 the low part's; the epilogue adds them).  The issuing thread is the kernel's critical path at small
  // N - an MMA costs it a fixed ~200 cycles whatever its width - so half as many instructions matter.
  constexpr int kAccCols = kXParts * BN;                        // TMEM columns of one accumulator
  constexpr uint32_t kCols = (uint32_t)(2 * kAccCols);          // two accumulators: 64 .. 512, a power of two
  constexpr uint32_t kIdesc = PAIR ? make_idesc(kAccCols, 2 * kTileM) : make_idesc(kAccCols);

  extern __shared__ unsigned char smem_dyn[];
  __shared__ __align__(8) unsigned long long full_w[8], full_x[8], empty_b[8], accum_full[2], tmem_empty[2], ss_ready[2], drain_bar, go_bar[kMaxPhases], seg_full[kSegQ], seg_empty[kSegQ];
  __shared__ int4 seg_q[kSegQ];          // (tile, kb0, kb1, row block)
  __shared__ unsigned int bar_cnt_s[kMaxPhases], bar_cnt_b[kMaxPhases];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  __shared__ float ss_part[2][4][BN];   // per accumulator, per staging warp: partial sums of squares

  const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = p.stages;
  volatile int *abort_flag = &abort_s;
  const uint32_t rank = PAIR ? cluster_rank() : 0u;          // 0: the pair's leader

  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int i = 0; i < 8; ++i) { mbar_init(smem_u32(&full_w[i]), 1); mbar_init(smem_u32(&full_x[i]), 1); mbar_init(smem_u32(&empty_b[i]), 1); }
    // an accumulator is free again once the epilogue warps of the CTA (of both CTAs of a pair) have read it
    for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&accum_full[i]), 1); mbar_init(smem_u32(&tmem_empty[i]), PAIR ? 8 : 4); mbar_init(smem_u32(&ss_ready[i]), 4); }
    mbar_init(smem_u32(&drain_bar), 1);
    for (int i = 0; i < kMaxPhases; ++i) { mbar_init(smem_u32(&go_bar[i]), 1); bar_cnt_s[i] = 0u; bar_cnt_b[i] = 0u; }
    // a queue slot is read by the MMA thread, four staging warps and four epilogue warps
    for (int i = 0; i < kSegQ; ++i) { mbar_init(smem_u32(&seg_full[i]), 1); mbar_init(smem_u32(&seg_empty[i]), 9); }
    fence_barrier_init();
  }
  if (warp == 1) {
    if constexpr (PAIR) tmem_alloc_pair(smem_u32(&tmem_base_s), kCols);
    else tmem_alloc(smem_u32(&tmem_base_s), kCols);
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();      // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  // Let the next kernel of the stream start its own set-up and weight prefetch as soon as every CTA of
  // this grid has got this far (it still waits for this grid to finish before it touches any activation).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  int issued = 0;   // producer: k-block loads issued (for the drain on abort)

  // Next queue entry for a whole warp (take_warp) or for a single thread (take_lane): 1 = a segment,
  // 0 = end of the phase, -1 = a bounded wait gave up.
  auto take_warp = [&](int &sq, Segment &s, int &rb) -> int {
    const int slot = sq & (kSegQ - 1);
    if (!mbar_wait_warp(smem_u32(&seg_full[slot]), (uint32_t)(sq / kSegQ) & 1u, abort_flag)) return -1;
    const int4 d = seg_q[slot];
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&seg_empty[slot]));
    ++sq;
    if (d.x < 0) return 0;
    s.tile = d.x; s.kb0 = d.y; s.kb1 = d.z; rb = d.w;
    return 1;
  };
  auto take_lane = [&](int &sq, Segment &s, int &rb) -> int {
    const int slot = sq & (kSegQ - 1);
    if (!mbar_wait(smem_u32(&seg_full[slot]), (uint32_t)(sq / kSegQ) & 1u, abort_flag)) return -1;
    const int4 d = seg_q[slot];
    mbar_arrive(smem_u32(&seg_empty[slot]));
    ++sq;
    if (d.x < 0) return 0;
    s.tile = d.x; s.kb0 = d.y; s.kb1 = d.z; rb = d.w;
    return 1;
  };

  // Panel mode, step 1 of a phase: all CTAs together convert pro(x) into the bf16 panel [high | low] once.  A warp
  // takes 32 consecutive (row, 8-wide chunk) units at a time, four such groups per pass so that the loads overlap; the
  // warp's arrival on the panel-ready barrier follows.  The four staging warps of every CTA convert; when that is more
  // than one pass for them, the four epilogue warps (which have nothing else to do between two phases) join in
  // (wslot 4..7) - with less work their extra arrivals only cost time.
  // Only with 128-row blocks: measured at 64 rows the step is slower with it (4.68 -> 4.85 ms), and with 32-row blocks
  // two CTAs share an SM and the kernel has no registers to spare for a second copy of the conversion.
  auto conv_warps = [&](const PhaseDesc &P) -> int {
    if constexpr (BN < 128) return 4;
    const int n_groups = (P.g.R * (P.g.K >> 3) + 31) >> 5;
    return n_groups > (int)gridDim.x * 16 ? 8 : 4;
  };
  auto convert_share = [&](const PhaseDesc &P, int pi, int wslot) {
    const GemmArgs &g = P.g;
    const int pro = P.pro;
    const int kConvWarps = conv_warps(P);
    {
      const int kc8 = g.K >> 3;
      const int units = g.R * kc8;                       // the host keeps R * K / 8 below 2^31
      const int n_groups = (units + 31) >> 5;
      const int warps_total = (int)gridDim.x * kConvWarps;
      __nv_bfloat16 *pan_hi = (__nv_bfloat16 *)g.pan;
      __nv_bfloat16 *pan_lo = pan_hi + (long long)g.pan_rows * g.K;
      const bool want_ss = pro == PRO_GAIN && g.ss_out != nullptr;
      for (int g0 = (int)blockIdx.x * kConvWarps + wslot; g0 < n_groups; g0 += 4 * warps_total) {
        float4 xa[4], xb[4], ua[4], ubv[4];
        float ssr[4];
        uint4 gq[4];
        int un[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          un[j] = g0 + j * warps_total < n_groups ? ((g0 + j * warps_total) << 5) + lane : units;
          xa[j] = xb[j] = ua[j] = ubv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          ssr[j] = 0.f; gq[j] = make_uint4(0, 0, 0, 0);
          if (un[j] < units) {
            const int r = un[j] / kc8, k = (un[j] - r * kc8) << 3;
            const float *px = g.x + (long long)r * g.ldx + k;
            xa[j] = __ldcg(reinterpret_cast<const float4 *>(px));
            xb[j] = __ldcg(reinterpret_cast<const float4 *>(px + 4));
            if (pro == PRO_GAIN) gq[j] = *reinterpret_cast<const uint4 *>((const __nv_bfloat16 *)g.gain + k);
            if (pro == PRO_SILU_MUL) {
              const float *pu = g.x2 + (long long)r * g.ldx + k;
              ua[j] = __ldcg(reinterpret_cast<const float4 *>(pu));
              ubv[j] = __ldcg(reinterpret_cast<const float4 *>(pu + 4));
              ssr[j] = __ldcg(g.ss_in + r);
            }
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const bool live = un[j] < units;
          const int r = live ? un[j] / kc8 : -1;
          float v[8] = {xa[j].x, xa[j].y, xa[j].z, xa[j].w, xb[j].x, xb[j].y, xb[j].z, xb[j].w};
          float sq = 0.f;
          if (pro == PRO_GAIN) {
            const __nv_bfloat162 *gp = reinterpret_cast<const __nv_bfloat162 *>(&gq[j]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 gf = __bfloat1622float2(gp[i]);
              sq = fmaf(v[2 * i], v[2 * i], sq); sq = fmaf(v[2 * i + 1], v[2 * i + 1], sq);
              v[2 * i] *= gf.x; v[2 * i + 1] *= gf.y;
            }
          } else if (pro == PRO_SILU_MUL) {
            const float sr = rsqrtf(ssr[j] / (float)g.dn + g.eps);
            const float uu[8] = {ua[j].x, ua[j].y, ua[j].z, ua[j].w, ubv[j].x, ubv[j].y, ubv[j].z, ubv[j].w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float gt = sr * v[i];
              v[i] = __fdividef(gt, 1.0f + __expf(-gt)) * (sr * uu[i]);
            }
          }
          if (want_ss) {
            // lanes of a group usually share the row: one reduction per group, else one per lane
            const int r0 = __shfl_sync(0xffffffffu, r, 0);
            if (__all_sync(0xffffffffu, r == r0)) {
              const float t = warp_sum_f(sq);
              if (lane == 0 && r0 >= 0) atomicAdd(&g.ss_out[r0], t);
            } else if (live) {
              atomicAdd(&g.ss_out[r], sq);
            }
          }
          if (live) {
            const int k = (un[j] - r * kc8) << 3;
            uint4 pk;
            __nv_bfloat162 b0 = __floats2bfloat162_rn(v[0], v[1]), b1 = __floats2bfloat162_rn(v[2], v[3]);
            __nv_bfloat162 b2 = __floats2bfloat162_rn(v[4], v[5]), b3 = __floats2bfloat162_rn(v[6], v[7]);
            pk.x = *reinterpret_cast<uint32_t *>(&b0); pk.y = *reinterpret_cast<uint32_t *>(&b1);
            pk.z = *reinterpret_cast<uint32_t *>(&b2); pk.w = *reinterpret_cast<uint32_t *>(&b3);
            *reinterpret_cast<uint4 *>(pan_hi + (long long)r * g.K + k) = pk;
            const float2 h0 = __bfloat1622float2(b0), h1 = __bfloat1622float2(b1);
            const float2 h2 = __bfloat1622float2(b2), h3 = __bfloat1622float2(b3);
            b0 = __floats2bfloat162_rn(v[0] - h0.x, v[1] - h0.y); b1 = __floats2bfloat162_rn(v[2] - h1.x, v[3] - h1.y);
            b2 = __floats2bfloat162_rn(v[4] - h2.x, v[5] - h2.y); b3 = __floats2bfloat162_rn(v[6] - h3.x, v[7] - h3.y);
            pk.x = *reinterpret_cast<uint32_t *>(&b0); pk.y = *reinterpret_cast<uint32_t *>(&b1);
            pk.z = *reinterpret_cast<uint32_t *>(&b2); pk.w = *reinterpret_cast<uint32_t *>(&b3);
            *reinterpret_cast<uint4 *>(pan_lo + (long long)r * g.K + k) = pk;
          }
        }
      }
    }
    asm volatile("fence.proxy.async;" ::: "memory");      // generic-proxy stores before the TMA reads that follow the barrier
    __threadfence();
    __syncwarp();
    if (lane == 0 && atomicAdd(&bar_cnt_b[pi], 1u) == (unsigned int)(kConvWarps - 1)) { __threadfence(); atomicAdd(p.bar_b + pi, 1u); }
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // Weights depend on nothing that runs on the device, so the producer never waits for a grid barrier
    // or for the previous kernel: it streams phase after phase, limited only by free ring slots.
    if (lane == 0) {
      int it = 0, sq = 0;
      int stage = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int pi = 0; pi < p.n_phases && ok; ++pi) {
        const PhaseDesc &P = p.ph[pi];
        int dealt = 0;
        (void)dealt;
        for (;;) {
          const int slot = sq & (kSegQ - 1);
          if (!mbar_wait(smem_u32(&seg_empty[slot]), ((uint32_t)(sq / kSegQ) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          unsigned int id;
          if constexpr (PAIR) { id = (blockIdx.x >> 1) + (unsigned int)dealt * (gridDim.x >> 1); ++dealt; }
          else id = atomicAdd(p.claim + pi, 1u);
          if (id >= (unsigned int)P.n_chunks) {                 // nothing left in this phase
            seg_q[slot] = make_int4(-1, 0, 0, 0);
            mbar_arrive(smem_u32(&seg_full[slot]));
            ++sq;
            break;
          }
          Segment s;
          int rb;
          chunk_decode(P, id, s, rb);
          seg_q[slot] = make_int4(s.tile, s.kb0, s.kb1, rb);
          mbar_arrive(smem_u32(&seg_full[slot]));
          ++sq;
          int m, row0, rows_valid, ycol0;
          tile_info(P, s.tile, m, row0, rows_valid, ycol0);
          const CUtensorMap *mp = &maps.m[pi * kMaxMats + m];
          for (int kb = s.kb0; kb < s.kb1; ++kb, ++it) {
            if (!mbar_wait(smem_u32(&empty_b[stage]), ph ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t bar = smem_u32(&full_w[stage]);
            if constexpr (PAIR) {
              // the leader's barrier counts both CTAs' 16 KB; the peer's copy may land before the leader has announced
              // it (the byte count of a phase may run negative for a while)
              if (rank == 0) mbar_expect_tx(bar, 2u * (uint32_t)kWBytes);
              tma_load_2d_pair(smem_base + stage * kStageBytes, mp, kb * kTileK, row0 + (int)rank * kTileM, map_to_cta(bar, 0));
            } else {
              mbar_expect_tx(bar, (uint32_t)P.tx_bytes[m]);
              tma_load_2d(smem_base + stage * kStageBytes, mp, kb * kTileK, row0, bar);
            }
            issued = it + 1;
            if (++stage == S) { stage = 0; ph ^= 1u; }
          }
          if (!ok) break;
        }
      }
      if constexpr (PAIR) {
        // the leader's MMA completions arrive on this CTA's ring barriers too: all of them have landed before it leaves
        for (int i = (it > S ? it - S : 0); i < it && ok; ++i)
          ok = mbar_wait(smem_u32(&empty_b[i % S]), (uint32_t)(i / S) & 1u, abort_flag);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // This thread is the kernel's critical path up to 16 rows (the weights are usually there before it asks):
    // the ring position is kept incrementally and the operand descriptors are advanced by plain additions.
    if (lane == 0) {
      int seg = 0, sq = 0;
      int stage = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int pi = 0; pi < p.n_phases && ok; ++pi) {
        {
          Segment s;
          int rb = 0;
          while (ok) {
            const int got = take_lane(sq, s, rb);
            if (got <= 0) { ok = got == 0; break; }
            if (PAIR && rank != 0) { ++seg; continue; }       // the leader issues for the pair
            const int acc = seg & 1;
            if (!mbar_wait(smem_u32(&tmem_empty[acc]), (((uint32_t)seg >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccCols);
            for (int kb = s.kb0; kb < s.kb1; ++kb) {
              if (!mbar_wait(smem_u32(&full_w[stage]), ph, abort_flag) ||
                  !mbar_wait(smem_u32(&full_x[stage]), ph, abort_flag)) { ok = false; break; }
              tc_fence_after();
              const uint32_t a_base = smem_base + stage * kStageBytes;
              const uint64_t a_desc = smem_desc_sw128(a_base), b_desc = smem_desc_sw128(a_base + kWBytes);
#pragma unroll
              for (int kk = 0; kk < kTileK / 16; ++kk) {    // 32 bytes along k: the start-address field counts 16-byte units
                if constexpr (PAIR) umma_bf16_pair(d_tmem, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), kIdesc, (kb > s.kb0 || kk > 0) ? 1u : 0u);
                else umma_bf16(d_tmem, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), kIdesc, (kb > s.kb0 || kk > 0) ? 1u : 0u);
              }
              if constexpr (PAIR) umma_commit_pair(smem_u32(&empty_b[stage]));
              else umma_commit(smem_u32(&empty_b[stage]));
              if (++stage == S) { stage = 0; ph ^= 1u; }
            }
            if (ok) {
              if constexpr (PAIR) umma_commit_pair(smem_u32(&accum_full[acc]));
              else umma_commit(smem_u32(&accum_full[acc]));
            }
            ++seg;
          }
        }
      }
      if constexpr (PAIR) {
        // the peer's epilogue warps arrive on this CTA's accumulator barriers: wait for the last two rounds
        if (rank == 0)
          for (int sg = (seg > 2 ? seg - 2 : 0); sg < seg && ok; ++sg)
            ok = mbar_wait(smem_u32(&tmem_empty[sg & 1]), ((uint32_t)sg >> 1) & 1u, abort_flag);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------ activation staging
    // Each of the four staging warps owns every fourth k-block, so four blocks are in flight at once and
    // the L2 latency of the activation loads is hidden.  A lane handles kUW (row, 16-byte chunk) units.
    // Weights never depend on the previous kernel, so the producer warp is already streaming them; the
    // activations do, so wait here for the previous grid to complete.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int sw = warp - 2;
    constexpr int kUW = BN / 4;
    const int chunk = lane & 7;
    int it = 0, seg = 0, sq = 0;
    bool ok = true;
    for (int pi = 0; pi < p.n_phases && ok; ++pi) {
      const PhaseDesc &P = p.ph[pi];
      const GemmArgs &g = P.g;
      const int pro = P.pro;
      // the activations of this phase are the previous phase's outputs, reduced by every CTA of the grid
      // (one staging warp polls the grid-wide counter and releases the other three through shared memory)
      if (P.wait_bar >= 0) {
        if (sw == 0) {
          ok = grid_bar_wait(p.bar + P.wait_bar, gridDim.x, lane, abort_flag);
          if (ok && lane == 0) mbar_arrive(smem_u32(&go_bar[pi]));
        } else {
          ok = mbar_wait_warp(smem_u32(&go_bar[pi]), 0u, abort_flag);
        }
        if (!ok) break;
      }
      if constexpr (PANEL) {
        if (!P.pre_panel) {
          // ---- (1) this warp's share of the panel conversion
          convert_share(P, pi, sw);
          // ---- (2) panel-ready barrier: the converting warps of every CTA have stored their share
          if (sw == 0) {
            ok = grid_bar_wait(p.bar_b + pi, gridDim.x, lane, abort_flag);
            asm volatile("fence.proxy.async;" ::: "memory");
          }
        } else if (sw == 0) {
          asm volatile("fence.proxy.async;" ::: "memory");    // the previous kernel's stores, complete since griddepcontrol.wait
        }
        // ---- (3) warp 0 streams the activation tiles of every claimed k-block into the ring; the other three
        // staging warps only follow the queue
        {
          Segment s;
          int rb = 0;
          while (ok) {
            const int got = take_warp(sq, s, rb);
            if (got <= 0) { ok = got == 0; break; }
            if (sw != 0) { it += s.kb1 - s.kb0; ++seg; continue; }
            for (int kb = s.kb0; kb < s.kb1; ++kb, ++it) {
              const int stage = it % S;
              const uint32_t ph = (uint32_t)(it / S) & 1u;
              if (!mbar_wait_warp(smem_u32(&empty_b[stage]), ph ^ 1u, abort_flag)) { ok = false; break; }
              if (lane == 0) {
                const uint32_t bar = smem_u32(&full_x[stage]);
                const uint32_t xs = smem_base + stage * kStageBytes + kWBytes;
                if constexpr (PAIR) {
                  // the leader stages the high tile, its peer the low one: the two halves of the N = 256 operand
                  if (rank == 0) mbar_expect_tx(bar, (uint32_t)(kXParts * kXBytes));
                  tma_load_2d_pair(xs, &maps.x[pi], kb * kTileK, (int)rank * g.pan_rows + rb * BN, map_to_cta(bar, 0));
                } else {
                  mbar_expect_tx(bar, (uint32_t)(kXParts * kXBytes));
#pragma unroll
                  for (int part = 0; part < kXParts; ++part)
                    tma_load_2d(xs + part * kXBytes, &maps.x[pi], kb * kTileK, part * g.pan_rows + rb * BN, bar);
                }
              }
            }
            ++seg;
          }
        }
        if (ok && P.sig_bar >= 0) grid_bar_signal(p.bar + P.sig_bar, &bar_cnt_s[P.sig_bar], lane);
        continue;
      }
      {
        Segment s;
        int rb = 0;
        while (ok) {
          const int got = take_warp(sq, s, rb);
          if (got <= 0) { ok = got == 0; break; }
          const int acc = seg & 1;
          const bool need_ss = pro == PRO_GAIN && (EPI == EPI_ARGMAX || (g.ss_out != nullptr && s.tile == 0));
          float *my_ss = &ss_part[acc][sw][0];
          if (need_ss) {
            if (EPI == EPI_ARGMAX) {   // the epilogue two segments back must have let go of this buffer
              if (!mbar_wait_warp(smem_u32(&tmem_empty[acc]), (((uint32_t)seg >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            }
            for (int row = lane; row < BN; row += 32) my_ss[row] = 0.f;
            __syncwarp();
          }
          for (int kb = s.kb0; kb < s.kb1; ++kb, ++it) {
            if ((it & 3) != sw) continue;
            const int stage = it % S;
            const uint32_t ph = (uint32_t)(it / S) & 1u;
            if (!mbar_wait_warp(smem_u32(&empty_b[stage]), ph ^ 1u, abort_flag)) { ok = false; break; }
            // dataflow transition: these 64 columns of the input are final once every chunk of the previous
            // phase's tile kb / 2 has been reduced into them
            if (P.dep_done && !grid_bar_wait(P.dep_done + (kb >> 1), P.dep_need, lane, abort_flag)) { ok = false; break; }
            unsigned char *xs = smem_dyn + (smem_base - smem_u32(smem_dyn)) + stage * kStageBytes + kWBytes;
            const int k = kb * kTileK + chunk * 8;
            // Loads first, arithmetic and shared-memory stores after: a store between two units would keep the
            // compiler from hoisting the next unit's loads, and every unit would pay its own L2 round trip.
            const bool k_in = k < g.K;
            uint4 gq = make_uint4(0, 0, 0, 0);
            if (pro == PRO_GAIN && k_in) gq = *reinterpret_cast<const uint4 *>((const __nv_bfloat16 *)g.gain + k);
            for (int ub = 0; ub < kUW; ub += 4) {
              float4 xa[4], xb[4], ua[4], ubv[4];
              float ssr[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int r = rb * BN + (ub + j) * 4 + (lane >> 3);
                xa[j] = xb[j] = ua[j] = ubv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                ssr[j] = 0.f;
                if (r < g.R && k_in) {
                  const float *px = g.x + (long long)r * g.ldx + k;
                  xa[j] = __ldcg(reinterpret_cast<const float4 *>(px));        // L2 only: other CTAs wrote these
                  xb[j] = __ldcg(reinterpret_cast<const float4 *>(px + 4));
                  if (pro == PRO_SILU_MUL) {
                    const float *pu = g.x2 + (long long)r * g.ldx + k;
                    ua[j] = __ldcg(reinterpret_cast<const float4 *>(pu));
                    ubv[j] = __ldcg(reinterpret_cast<const float4 *>(pu + 4));
                    ssr[j] = __ldcg(g.ss_in + r);
                  }
                }
              }
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int row = (ub + j) * 4 + (lane >> 3);
                float v[8] = {xa[j].x, xa[j].y, xa[j].z, xa[j].w, xb[j].x, xb[j].y, xb[j].z, xb[j].w};
                float sq = 0.f;
                if (pro == PRO_GAIN) {
                  const __nv_bfloat162 *gp = reinterpret_cast<const __nv_bfloat162 *>(&gq);
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    const float2 gf = __bfloat1622float2(gp[i]);
                    sq = fmaf(v[2 * i], v[2 * i], sq); sq = fmaf(v[2 * i + 1], v[2 * i + 1], sq);
                    v[2 * i] *= gf.x; v[2 * i + 1] *= gf.y;
                  }
                } else if (pro == PRO_SILU_MUL) {
                  const float sr = rsqrtf(ssr[j] / (float)g.dn + g.eps);
                  const float uu[8] = {ua[j].x, ua[j].y, ua[j].z, ua[j].w, ubv[j].x, ubv[j].y, ubv[j].z, ubv[j].w};
#pragma unroll
                  for (int i = 0; i < 8; ++i) {
                    const float gt = sr * v[i];
                    v[i] = __fdividef(gt, 1.0f + __expf(-gt)) * (sr * uu[i]);
                  }
                }
                if (need_ss) {      // uniform across the warp
                  sq += __shfl_xor_sync(0xffffffffu, sq, 1);
                  sq += __shfl_xor_sync(0xffffffffu, sq, 2);
                  sq += __shfl_xor_sync(0xffffffffu, sq, 4);
                  if (chunk == 0) my_ss[row] += sq;
                }
                const int soff = (row >> 3) * 1024 + (row & 7) * 128 + ((chunk ^ (row & 7)) << 4);
                uint4 pk;
                __nv_bfloat162 b0 = __floats2bfloat162_rn(v[0], v[1]), b1 = __floats2bfloat162_rn(v[2], v[3]);
                __nv_bfloat162 b2 = __floats2bfloat162_rn(v[4], v[5]), b3 = __floats2bfloat162_rn(v[6], v[7]);
                pk.x = *reinterpret_cast<uint32_t *>(&b0); pk.y = *reinterpret_cast<uint32_t *>(&b1);
                pk.z = *reinterpret_cast<uint32_t *>(&b2); pk.w = *reinterpret_cast<uint32_t *>(&b3);
                *reinterpret_cast<uint4 *>(xs + soff) = pk;
                if (kXParts == 2) {      // low part: what the first rounding lost
                  const float2 h0 = __bfloat1622float2(b0), h1 = __bfloat1622float2(b1);
                  const float2 h2 = __bfloat1622float2(b2), h3 = __bfloat1622float2(b3);
                  __nv_bfloat162 l0 = __floats2bfloat162_rn(v[0] - h0.x, v[1] - h0.y), l1 = __floats2bfloat162_rn(v[2] - h1.x, v[3] - h1.y);
                  __nv_bfloat162 l2 = __floats2bfloat162_rn(v[4] - h2.x, v[5] - h2.y), l3 = __floats2bfloat162_rn(v[6] - h3.x, v[7] - h3.y);
                  pk.x = *reinterpret_cast<uint32_t *>(&l0); pk.y = *reinterpret_cast<uint32_t *>(&l1);
                  pk.z = *reinterpret_cast<uint32_t *>(&l2); pk.w = *reinterpret_cast<uint32_t *>(&l3);
                  *reinterpret_cast<uint4 *>(xs + kXBytes + soff) = pk;
                }
              }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&full_x[stage]));
          }
          if (!ok) break;
          if (need_ss) {
            __syncwarp();
            if (EPI == EPI_ARGMAX) {
              if (lane == 0) mbar_arrive(smem_u32(&ss_ready[acc]));
            } else {
              for (int row = lane; row < BN; row += 32) {
                const int r = rb * BN + row;
                if (r < g.R) atomicAdd(&g.ss_out[r], my_ss[row]);
              }
            }
          }
          ++seg;
        }
      }
      // this warp has finished reading the phase's inputs and adding its sums of squares
      if (ok && P.sig_bar >= 0) grid_bar_signal(p.bar + P.sig_bar, &bar_cnt_s[P.sig_bar], lane);
    }
  } else {
    // ------------------------------------------------------------ epilogue
    asm volatile("griddepcontrol.wait;" ::: "memory");   // outputs may still be read by the previous grid
    const int q = warp & 3;
    const int n_local = q * 32 + lane;
    // Side clearing: buffers the previous kernel has finished reading and that a later phase of this launch (one
    // that lies behind a grid barrier these warps arrive on) accumulates into.
    {
      const unsigned long long gtid = ((unsigned long long)blockIdx.x * 4 + q) * 32 + lane;
      const unsigned long long nth = (unsigned long long)gridDim.x * 128;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (!p.z.p[i]) continue;
        const unsigned long long n4 = p.z.n[i] >> 2;
        float4 *p4 = reinterpret_cast<float4 *>(p.z.p[i]);
        for (unsigned long long e = gtid; e < n4; e += nth) p4[e] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (unsigned long long e = (n4 << 2) + gtid; e < p.z.n[i]; e += nth) p.z.p[i][e] = 0.f;
      }
    }
    int seg = 0, sq = 0;
    bool ok = true;
    for (int pi = 0; pi < p.n_phases && ok; ++pi) {
      const PhaseDesc &P = p.ph[pi];
      const GemmArgs &g = P.g;
      bool epi_bar_passed = P.epi_bar < 0;
      if constexpr (PANEL && BN == 128) {
        // the previous phase's sums are complete (a staging warp polls the grid barrier and opens go_bar): this warp's
        // share of the panel conversion
        if (!P.pre_panel && conv_warps(P) == 8) {
          if (P.wait_bar >= 0 && !mbar_wait_warp(smem_u32(&go_bar[pi]), 0u, abort_flag)) { ok = false; break; }
          convert_share(P, pi, 4 + q);
        }
      }
      {
        Segment s;
        int rb = 0;
        while (ok) {
          const int got = take_warp(sq, s, rb);
          if (got <= 0) { ok = got == 0; break; }
          // the output is also the input of a projection this phase does not wait for otherwise (the residual read
          // by the second gate/up half while the first down half is ready to add to it): its readers must be done
          if (!epi_bar_passed) {
            if (!grid_bar_wait(p.bar + P.epi_bar, gridDim.x, lane, abort_flag)) { ok = false; break; }
            epi_bar_passed = true;
          }
          int m, row0, rows_valid, ycol0;
          tile_info(P, s.tile, m, row0, rows_valid, ycol0);
          if constexpr (PAIR) { ycol0 += (int)rank * kTileM; rows_valid = kTileM; }     // this CTA's 128 weight rows of the pair's 256
          const int acc = seg & 1;
          const uint32_t ph = ((uint32_t)seg >> 1) & 1u;
          if (!mbar_wait_warp(smem_u32(&accum_full[acc]), ph, abort_flag)) { ok = false; break; }
          if (EPI == EPI_ARGMAX && !PANEL && !mbar_wait_warp(smem_u32(&ss_ready[acc]), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const bool valid = n_local < rows_valid;
          const int col = ycol0 + n_local;
          for (int c0 = 0; c0 < BN; c0 += 16) {
            if (rb * BN + c0 >= g.R) break;
            float v[16];
            float ssum[16];
            if (EPI == EPI_ARGMAX) {      // all sixteen loads before the first use
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const int r = rb * BN + c0 + j;
                ssum[j] = PANEL ? (r < g.R ? __ldcg(g.ss_out + r) : 0.f)
                                : ss_part[acc][0][c0 + j] + ss_part[acc][1][c0 + j] + ss_part[acc][2][c0 + j] + ss_part[acc][3][c0 + j];
              }
            }
            tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kAccCols + c0), v);
            {
              float vl[16];
              tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kAccCols + BN + c0), vl);
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] += vl[j];
            }
            if (EPI == EPI_ATOMIC_ADD) {
              // A lane holds one output column (weight row) for 16 rows.  A reduction instruction costs the warp
              // ~100 cycles here whatever its width, so the quads are transposed first: lane i of a quad then holds
              // rows i, i + 4, i + 8, i + 12 for the quad's four adjacent columns - four 16-byte reductions instead
              // of sixteen scalar ones.  (Columns come in multiples of 8, so a quad is valid or invalid as a whole.)
              float *ybase = g.y + (ycol0 + q * 32 + (lane & ~3));
              const bool quad_valid = (q * 32 + (lane & ~3)) < rows_valid;
#pragma unroll
              for (int k4 = 0; k4 < 4; ++k4) {
                quad_transpose(v[4 * k4], v[4 * k4 + 1], v[4 * k4 + 2], v[4 * k4 + 3], lane);
                const int r = rb * BN + c0 + 4 * k4 + (lane & 3);
                if (quad_valid && r < g.R) red_add_v4(ybase + (long long)r * g.ldy, v[4 * k4], v[4 * k4 + 1], v[4 * k4 + 2], v[4 * k4 + 3]);
              }
            } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int r = rb * BN + c0 + j;
              if (r >= g.R) break;
              {
                float logit = v[j] * rsqrtf(ssum[j] / (float)g.dn + g.eps);
                unsigned long long key = 0ull;
                if (valid) {
                  if (g.perm && g.perm[g.tokens[r]] == col) logit += g.beta;
                  if (g.logits) g.logits[(long long)r * g.vocab + col] = logit;
                  key = ((unsigned long long)ordered_key_u(logit) << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned int)col);
                }
                key = warp_max_u64(key);
                if (lane == 0) atomicMax(&g.amax[r], key);
              }
            }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tmem_empty[acc]), 0));
            else mbar_arrive(smem_u32(&tmem_empty[acc]));
          }
          if (EPI == EPI_ATOMIC_ADD && P.tile_done) {       // this warp's share of the chunk is reduced into the tile
            __syncwarp();
            if (lane == 0) red_release_gpu(P.tile_done + s.tile, 1u);
          }
          ++seg;
        }
      }
      // all partial sums of this phase that this warp owns are on their way to L2
      if (ok && P.sig_bar >= 0) grid_bar_signal(p.bar + P.sig_bar, &bar_cnt_s[P.sig_bar], lane);
    }
  }

  // ---------------------------------------------------------------- teardown
  __syncthreads();
  if (abort_s) {
    if (threadIdx.x == 0) {
      atomicExch(p.err, 1u);
      // wait (bounded) for this CTA's own TMA copies still in flight (a pair's copies are counted by its leader, and
      // the peer stays until the leader has passed the cluster barrier below)
      const unsigned long long t0 = clock64();
      for (int i = (issued > S ? issued - S : 0); i < issued && rank == 0; ++i) {
        const uint32_t bar = smem_u32(&full_w[i % S]);
        while (!mbar_try(bar, (uint32_t)(i / S) & 1u))
          if ((unsigned long long)(clock64() - t0) > kSpinBudget / 4) break;
      }
    }
    if (warp == 1 && lane == 0) {
      // and for MMAs already issued
      umma_commit(smem_u32(&drain_bar));
      const unsigned long long t0 = clock64();
      while (!mbar_try(smem_u32(&drain_bar), 0u))
        if ((unsigned long long)(clock64() - t0) > kSpinBudget / 4) break;
    }
    __syncthreads();
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();      // neither CTA leaves, or frees tensor memory, while its peer still works
  if (warp == 1) {
    tc_fence_after();
    if constexpr (PAIR) tmem_dealloc_pair(tmem_base, kCols);
    else tmem_dealloc(tmem_base, kCols);
  }
}

// ------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)sym;
  }
  return fn;
}

// accumulator width, ring depth and resident CTAs per SM for a row count
static void bn_config(int R, int &bn, int &stages, int &ctas_per_sm) {
  if (R <= 16) { bn = 16; stages = 5; ctas_per_sm = 2; }          // 5 x (16 + 2 x 2) KB
  else if (R <= 32) { bn = 32; stages = 4; ctas_per_sm = 2; }     // 4 x (16 + 2 x 4) KB
  else if (R <= 64) { bn = 64; stages = 6; ctas_per_sm = 1; }     // 6 x (16 + 2 x 8) KB
  else { bn = 128; stages = 4; ctas_per_sm = 1; }                 // 4 x (16 + 2 x 16) KB; more rows: blocks of 128
}

UmmaPlan *umma_plan_create(const GemmArgs &a, int pro, int epi, int n_sms, unsigned int *err_word,
                           char *err, int errlen) {
  auto fail = [&](const char *msg) -> UmmaPlan * { if (err) snprintf(err, errlen, "%s", msg); return nullptr; };
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return fail("cuTensorMapEncodeTiled entry point not available");
  if (a.K < kTileK || a.K % 8) return fail("tensor-core path needs K >= 64 and K % 8 == 0");
  if (a.n_mats < 1 || a.n_mats > kMaxMats) return fail("bad matrix count");
  UmmaPlan *pl = new UmmaPlan();
  memset(pl, 0, sizeof(*pl));
  pl->d.g = a;
  pl->d.pro = pro;
  pl->epi = epi; pl->n_sms = n_sms; pl->err = err_word;
  pl->d.nkb = (a.K + kTileK - 1) / kTileK;
  pl->d.tile_rows = kTileM;
  pl->d.n_tiles = 0;
  for (int m = 0; m < a.n_mats; ++m) {
    if (a.n_rows[m] < 1) { delete pl; return fail("empty weight matrix"); }
    pl->d.tiles_m[m] = (a.n_rows[m] + kTileM - 1) / kTileM;
    pl->d.n_tiles += pl->d.tiles_m[m];
    const cuuint32_t box_rows = (cuuint32_t)(a.n_rows[m] < kTileM ? a.n_rows[m] : kTileM);
    pl->d.tx_bytes[m] = (int)(box_rows * kTileK * 2);
    cuuint64_t gdim[2] = {(cuuint64_t)a.K, (cuuint64_t)a.n_rows[m]};
    cuuint64_t gstr[1] = {(cuuint64_t)(a.ldw ? a.ldw : a.K) * 2};
    cuuint32_t box[2] = {(cuuint32_t)kTileK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(&pl->maps[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(a.w[m]), gdim, gstr, box,
                     estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { delete pl; return fail("cuTensorMapEncodeTiled failed (weight pointer must be 16-byte aligned)"); }
  }
  for (int m = a.n_mats; m < kMaxMats; ++m) pl->maps[m] = pl->maps[0];
  if (a.pan) {
    // activation panel [high rows | low rows] x K, one map per accumulator width (the box is bn rows high)
    if (a.pan_rows < 1 || a.pan_rows % kTileM || (long long)a.pan_rows * (a.K / 8) > 0x7fffffffLL) { delete pl; return fail("bad activation panel"); }
    const int widths[3] = {32, 64, 128};
    for (int i = 0; i < 3; ++i) {
      cuuint64_t gdim[2] = {(cuuint64_t)a.K, (cuuint64_t)2 * a.pan_rows};
      cuuint64_t gstr[1] = {(cuuint64_t)a.K * 2};
      cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)widths[i]};
      cuuint32_t estr[2] = {1, 1};
      CUresult r = enc(&pl->xmap[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.pan, gdim, gstr, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) { delete pl; return fail("cuTensorMapEncodeTiled failed (activation panel)"); }
    }
    pl->has_xmap = true;
  }
  return pl;
}

void umma_plan_destroy(UmmaPlan *p) { delete p; }

template <int EPI, int BN, bool PANEL>
static cudaError_t launch_one(const MapPack &maps, const UmmaParams &p, int grid, cudaStream_t st) {
  const size_t smem = (size_t)p.stages * (kWBytes + x_parts(BN) * BN * 128) + 1024;
  static size_t attr_smem[kMaxDevices] = {0};
  const int dev = current_device_slot();
  if (smem > attr_smem[dev]) {
    cudaError_t e = cudaFuncSetAttribute(gemm_umma_kernel<EPI, BN, PANEL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_smem[dev] = smem;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = p.pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, gemm_umma_kernel<EPI, BN, PANEL>, maps, p);
}

// CTA pairs: clusters of two, one CTA per SM, six stages of 16 KB weights + 16 KB activations.
constexpr int kPairStages = 6;
static size_t pair_smem_bytes() { return (size_t)kPairStages * (kWBytes + 128 * 128) + 1024; }
static void pair_launch_config(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, int grid, int pdl, cudaStream_t st) {
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = pair_smem_bytes(); cfg.stream = st;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pdl ? 2 : 1;
}
// Number of CTAs (an even number) that are certainly resident together as pairs; 0 if pairs cannot be launched.
static int pair_grid(int n_sms) {
  static int cached[kMaxDevices] = {0};
  const int dev = current_device_slot();
  if (cached[dev] == 0) {
    auto kern = gemm_umma_kernel<EPI_ATOMIC_ADD, 128, true, true>;
    cached[dev] = -1;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pair_smem_bytes()) == cudaSuccess) {
      cudaLaunchConfig_t cfg;
      cudaLaunchAttribute attr[2];
      pair_launch_config(cfg, attr, (n_sms / 2) * 2, 0, nullptr);
      int clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg) == cudaSuccess && clusters > 0)
        cached[dev] = 2 * (clusters < n_sms / 2 ? clusters : n_sms / 2);
      else
        (void)cudaGetLastError();
    } else {
      (void)cudaGetLastError();
    }
  }
  return cached[dev] > 0 ? cached[dev] : 0;
}
static cudaError_t launch_pair(const MapPack &maps, const UmmaParams &p, int grid, cudaStream_t st) {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  pair_launch_config(cfg, attr, grid, p.pdl, st);
  return cudaLaunchKernelEx(&cfg, gemm_umma_kernel<EPI_ATOMIC_ADD, 128, true, true>, maps, p);
}

template <int EPI>
static cudaError_t launch_bn(const MapPack &maps, const UmmaParams &p, int bn, bool panel, int grid, cudaStream_t st) {
  if (panel) {
    switch (bn) {
      case 32: return launch_one<EPI, 32, true>(maps, p, grid, st);
      case 64: return launch_one<EPI, 64, true>(maps, p, grid, st);
      case 128: return launch_one<EPI, 128, true>(maps, p, grid, st);
      default: return cudaErrorInvalidValue;
    }
  }
  switch (bn) {
    case 16: return launch_one<EPI, 16, false>(maps, p, grid, st);
    case 32: return launch_one<EPI, 32, false>(maps, p, grid, st);
    case 64: return launch_one<EPI, 64, false>(maps, p, grid, st);
    default: return launch_one<EPI, 128, false>(maps, p, grid, st);
  }
}

// One launch that runs plans[0..n-1] back to back on the same rows; plan i+1 consumes what plan i reduced
// into its output, separated by a grid barrier on bar[i] (zero at launch).  args[i] carries the per-launch
// buffers and the row count; weights, K and the matrix split stay as planned.
// Beyond 16 rows, plans that own an activation panel run in panel mode: bar_b[i] (zero at launch) is the
// panel-ready barrier of phase i.  Without `sync` (and always in panel mode) every phase waits at a grid barrier
// for the one before it.
cudaError_t launch_gemm_chain(const UmmaPlan *const *plans, const GemmArgs *args, int n, unsigned int *bar,
                              unsigned int *claim, unsigned int *bar_b, const ChainSync *sync, unsigned int *tile_done,
                              int td_stride, const ZeroList *zero, int pdl, cudaStream_t st, int cta_pairs) {
  if (n < 1 || n > kMaxPhases || !claim) return cudaErrorInvalidValue;
  if (n > 1 && !bar) return cudaErrorInvalidValue;
  MapPack maps;
  UmmaParams p;
  memset(&p, 0, sizeof p);
  const int epi = plans[0]->epi;
  int bn, cps;
  bn_config(args[0].R, bn, p.stages, cps);
  const int nrb = (args[0].R + bn - 1) / bn;
  const int tile_mode = (epi == EPI_ARGMAX) ? 1 : 0;
  bool panel = bar_b != nullptr && args[0].R > 16;
  for (int i = 0; i < n; ++i) panel = panel && plans[i]->has_xmap && args[0].R <= plans[i]->d.g.pan_rows;
  if (panel && epi == EPI_ARGMAX && !args[0].ss_out) return cudaErrorInvalidValue;
  if (args[0].pan_ready && !panel) return cudaErrorInvalidValue;     // the caller wrote the panel instead of the fp32 input
  if (args[0].R > 16 && !panel && n > 1 && sync) return cudaErrorInvalidValue;   // the caller plans `sync` for <= 16 rows
  const bool explicit_sync = sync && tile_done && !panel && !tile_mode && args[0].R <= 16;
  // CTA pairs: 128-row blocks in panel mode, every matrix a whole number of 256-row tiles
  bool pair = cta_pairs && panel && bn == 128 && !tile_mode;
  for (int i = 0; i < n && pair; ++i)
    for (int m = 0; m < plans[i]->d.g.n_mats; ++m) pair = pair && plans[i]->d.g.n_rows[m] % (2 * kTileM) == 0;
  const int pgrid = pair ? pair_grid(plans[0]->n_sms) : 0;
  pair = pair && pgrid >= 2;
  if (pair) p.stages = kPairStages;
  long long max_chunks = 1;
  for (int i = 0; i < n; ++i) {
    const UmmaPlan *pl = plans[i];
    const GemmArgs &a = args[i];
    if (pl->epi != epi || (epi == EPI_ARGMAX && n != 1) || a.R != args[0].R) return cudaErrorInvalidValue;
    PhaseDesc &d = p.ph[i];
    d = pl->d;
    d.g.x = a.x; d.g.x2 = a.x2; d.g.ldx = a.ldx; d.g.ss_in = a.ss_in; d.g.ss_out = a.ss_out;
    d.g.y = a.y; d.g.ldy = a.ldy; d.g.R = a.R; d.g.tokens = a.tokens; d.g.amax = a.amax; d.g.logits = a.logits;
    for (int m = 0; m < kMaxMats; ++m) maps.m[i * kMaxMats + m] = pl->maps[m];
    maps.x[i] = pl->xmap[bn == 32 ? 0 : bn == 64 ? 1 : 2];
    // the argmax epilogue needs whole tiles; partial sums may be split along k: chunks of four k-blocks (one per
    // staging warp) up to 16 rows, where fine chunks balance the CTAs best; longer chunks for more rows, where every
    // chunk ends in 128 x rows reductions (measured on the 7B shape: 8 k-blocks best at 32 rows, 16 at 64 and 128)
    d.chunk_kb = tile_mode ? d.nkb : !panel ? 4 : bn == 32 ? 8 : 16;
    d.k_major = panel && !tile_mode;
    d.wait_bar = i > 0 ? i - 1 : -1;
    d.sig_bar = i + 1 < n ? i : -1;
    d.epi_bar = -1;
    d.tile_done = nullptr; d.dep_done = nullptr; d.dep_need = 0; d.dep_tiles = 0;
    d.pre_panel = panel && i == 0 && a.pan_ready;
    if (pair) {
      d.tile_rows = 2 * kTileM;
      d.n_tiles = 0;
      for (int m = 0; m < d.g.n_mats; ++m) { d.tiles_m[m] = d.g.n_rows[m] / (2 * kTileM); d.n_tiles += d.tiles_m[m]; }
    }
    d.cpt = (d.nkb + d.chunk_kb - 1) / d.chunk_kb;
    const long long chunks = (long long)nrb * d.n_tiles * d.cpt;
    if (chunks > 0x7fffffffLL) return cudaErrorInvalidValue;
    d.n_chunks = (int)chunks;
    d.nrb = nrb;
    if (chunks > max_chunks) max_chunks = chunks;
  }
  if (explicit_sync) {
    for (int i = 0; i < n; ++i) {
      PhaseDesc &d = p.ph[i];
      const ChainSync &c = sync[i];
      if (c.wait_bar >= n || c.sig_bar >= n || c.epi_bar >= n || c.td_prod > 1 || c.td_cons > 1) return cudaErrorInvalidValue;
      d.wait_bar = c.wait_bar; d.sig_bar = c.sig_bar; d.epi_bar = c.epi_bar;
      if (c.td_prod >= 0) {          // tile-major producer: its tiles complete one after the other
        if (d.g.n_mats != 1 || d.g.y_off[0] != 0 || d.n_tiles > td_stride) return cudaErrorInvalidValue;
        d.tile_done = tile_done + (size_t)c.td_prod * td_stride;
      }
      if (c.td_cons >= 0) {          // k-major consumer: its first chunks need only the first tiles
        unsigned int need = 0;
        int tiles = 0;
        for (int j = 0; j < i; ++j)
          if (sync[j].td_prod == c.td_cons) {
            if (p.ph[j].g.n_rows[0] != d.g.K || p.ph[j].g.y != d.g.x) return cudaErrorInvalidValue;
            need += (unsigned int)(p.ph[j].cpt * p.ph[j].nrb * 4);     // four epilogue warps count every chunk
            tiles = p.ph[j].n_tiles;
          }
        if (!need) return cudaErrorInvalidValue;
        d.k_major = 1;
        d.dep_done = tile_done + (size_t)c.td_cons * td_stride;
        d.dep_need = need;
        d.dep_tiles = tiles;
      }
    }
  }
  for (int i = n; i < kMaxPhases; ++i) {
    for (int m = 0; m < kMaxMats; ++m) maps.m[i * kMaxMats + m] = plans[0]->maps[0];
    maps.x[i] = plans[0]->xmap[0];
  }
  p.n_phases = n; p.pdl = pdl; p.err = plans[0]->err; p.bar = bar; p.claim = claim; p.bar_b = bar_b;
  if (zero) p.z = *zero;
  // Staging warps own every fourth k-block and run ahead of each other; the parity waits on the ring
  // are only unambiguous while the ring is at least as deep as the number of staging warps.
  if (p.stages < 4 || p.stages > 8) return cudaErrorInvalidValue;
  if (pair) {
    // one chunk per pair at least; the grid barriers need every pair resident
    const long long want = 2 * max_chunks;
    return launch_pair(maps, p, (int)(want < pgrid ? want : pgrid), st);
  }
  const long long resident = (long long)plans[0]->n_sms * cps;     // the grid barrier needs every CTA resident
  const int grid = (int)(resident < max_chunks ? resident : max_chunks);
  if (epi == EPI_ARGMAX) return launch_bn<EPI_ARGMAX>(maps, p, bn, panel, grid, st);
  return launch_bn<EPI_ATOMIC_ADD>(maps, p, bn, panel, grid, st);
}

cudaError_t launch_gemm_umma(const UmmaPlan *pl, const GemmArgs &a, unsigned int *claim, unsigned int *bar_b,
                             const ZeroList *zero, int pdl, cudaStream_t st, int cta_pairs) {
  return launch_gemm_chain(&pl, &a, 1, nullptr, claim, bar_b, nullptr, nullptr, 0, zero, pdl, st, cta_pairs);
}

}  // namespace fc
