// Fused rotary embedding + in-place K/V write + split-KV window attention for bf16 (head_dim 64/128).
//
// grid (splits, kv heads x query-tile groups, sequences); the splits of one (sequence, kv head, query-tile group)
// form one thread-block cluster (at most 8).  A CTA owns a run of consecutive 64-key tiles of the cached keys of its
// kv head and QT 16-row tiles of the queries that map to that kv head (group heads x c window rows).
//   - Cached K/V tiles arrive by TMA (one 3-d tensor map over the K/V slab, boxes of 64 keys x 64 elements, 128-byte
//     swizzle) into a ring of NS stages; the first NS tiles are requested before the kernel waits for the QKV
//     projection, because cached keys were written by earlier steps.  No stage has a consumer barrier: a stage is
//     free again when every warp has passed the next tile's first CTA barrier, and thread 0 refills it there.
//   - The last split also owns the window's own keys (slots kv_len .. kv_len+c-1): it takes them straight from the
//     fp32 QKV accumulators, applies the deferred 1/rms factor and the rotation, stores them as bf16 in shared
//     memory (same swizzled layout as a TMA tile) and in the cache.  Window tiles are causal.
//   - Per tile, warp w computes S = Q.K^T for keys 8w..8w+7 on mma.sync m16n8k16 (q as a bf16 pair high + low, fp32
//     accumulation), the row maxima are exchanged through shared memory (quad shuffles inside the warp first), the
//     probabilities go to shared memory as bf16 high + low, and warp w accumulates O[:, its HD/8 columns] += P.V over
//     all keys of the tile.  So a warp holds 8 * QT * HD/64 output registers instead of a whole 16 x HD tile, there
//     is no merge of warps, and the register count stays low enough for a CTA of the following projection kernel
//     to be resident beside this one (its weight ring fills while the attention runs).
//   - The splits are merged through distributed shared memory: every CTA leaves its un-normalised output and its
//     (max, sum) per row in its own shared memory, a cluster barrier, then each CTA combines a share of the rows'
//     columns from all splits and writes fp32 output rows.
// Row j of sequence b sees keys 0 .. kv_len[b] + j (cache + causal part of the window).
// Every wait is bounded: a tile that does not arrive within the budget raises the error word and the CTA skips its
// remaining tiles (all CTAs still meet at the cluster barriers).
#include <cuda.h>

#include <cstring>

#include "fc_internal.h"

namespace fc {

namespace {

constexpr int kTK = 64;          // keys per tile
constexpr int kAttnThreads = 256;
constexpr unsigned long long kAttnSpin = 400000000ull;   // clock64 ticks (~0.2 s)

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2_t(uint32_t addr, uint32_t &r0, uint32_t &r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ float bf16_round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
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
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = clock64();
  unsigned int spins = 0;
  while (!mbar_try(bar, parity))
    if ((++spins & 0xFFu) == 0u && (unsigned long long)(clock64() - t0) > kAttnSpin) return false;
  return true;
}
// One box of a 3-d tensor map (elements, keys, planes) into shared memory, completion counted on an mbarrier.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_dsmem_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 ld_dsmem_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}

// Byte offset of 16-byte piece `ch` of row `r` in a tile stored as sub-tiles of [rows][128 B] (64 bf16 per row and
// sub-tile, sub-tiles `sub_stride` bytes apart), pieces permuted inside each 8-row group as the 128-byte TMA swizzle
// does it: piece index ^= row & 7.  TMA tiles start on a 1024-byte boundary, so the formula matches the hardware's.
__device__ __forceinline__ uint32_t tile_off(int r, int ch, uint32_t sub_stride) {
  return (uint32_t)(ch >> 3) * sub_stride + (uint32_t)r * 128u + (uint32_t)(((ch & 7) ^ (r & 7)) << 4);
}

// Window tile geometry shared by host and device: rows per window tile and number of window tiles.
__host__ __device__ inline int win_rows(int c) { return c <= kTK ? (c + 15) / 16 * 16 : kTK; }
__host__ __device__ inline int win_tiles(int c) { return (c + kTK - 1) / kTK; }

template <int HD>
struct AttnCfg {
  static constexpr int SUB = HD / 64;                       // 128-byte sub-tiles per row
  static constexpr int NS = HD == 128 ? 3 : 4;              // ring stages when one CTA has an SM to itself
  static constexpr int NS_MAX = 4;
  static constexpr uint32_t kSubBytes = kTK * 128;          // one sub-tile of a TMA tile
  static constexpr uint32_t kKBytes = SUB * kSubBytes;      // K (or V) part of a stage
  static constexpr uint32_t kStage = 2 * kKBytes;
  static constexpr uint32_t kQTile = 2u * SUB * 2048u;      // 16 query rows: high sub-tiles, then low sub-tiles
};

template <int HD>
size_t attn_smem_bytes(int c, int qt, int stages) {
  using C = AttnCfg<HD>;
  const size_t wstage = 2ull * C::SUB * win_rows(c) * 128;
  const size_t rows = (size_t)qt * 16;
  return 1024 + (size_t)stages * C::kStage + (size_t)win_tiles(c) * wstage + (size_t)qt * C::kQTile + (size_t)qt * 4096 +
         8 * rows * 4 /* per-warp maxima / sums */ + rows * 8 /* (max, sum) */;
}

}  // namespace

template <int HD, int QT>
__global__ void __maxnreg__(128)
attn_tma_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, const FusedAttnArgs a) {
  using C = AttnCfg<HD>;
  constexpr int SUB = C::SUB, HALF = HD / 2;
  const int NS = a.stages;                   // ring stages (2 .. 4)
  constexpr int NDW = HD / 64;               // 8-wide output blocks per warp (8 warps x NDW x 8 columns = HD)
  constexpr int ROWS = QT * 16;
  constexpr uint32_t kSubBytes = C::kSubBytes, kKBytes = C::kKBytes, kStage = C::kStage;

  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long full_bar[C::NS_MAX];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g4 = lane >> 2, t4 = lane & 3;
  const int split = blockIdx.x, ns = gridDim.x;
  const int group = a.hq / a.hkv;
  const int nq = group * a.c;
  const int nqg = ((nq + 15) / 16 + QT - 1) / QT;
  const int kvh = blockIdx.y / nqg, qg = blockIdx.y - kvh * nqg;
  const int bl = blockIdx.z, b = a.seq_map ? a.seq_map[bl] : a.b0 + bl;
  const int c = a.c;
  const int qd = a.hq * HD, kvd = a.hkv * HD;
  const unsigned int c_magic = a.c_magic;
  auto div_c = [&](int q) -> int { return c == 1 ? q : (int)__umulhi((unsigned int)q, c_magic); };

  // ---- shared-memory layout (byte offsets from a 1024-byte boundary)
  const uint32_t base = (smem_addr(smem_raw) + 1023u) & ~1023u;
  unsigned char *gen = smem_raw + (base - smem_addr(smem_raw));
  const int wrows = win_rows(c), nwt = win_tiles(c);
  const uint32_t wsub = (uint32_t)wrows * 128u, wk = SUB * wsub, wstage = 2u * wk;
  const uint32_t off_win = (uint32_t)NS * kStage;
  const uint32_t off_q = off_win + (uint32_t)nwt * wstage;
  const uint32_t off_p = off_q + QT * C::kQTile;
  const uint32_t off_wmax = off_p + QT * 4096u;
  const uint32_t off_ml = off_wmax + 8u * ROWS * 4u;
  float *wmax = reinterpret_cast<float *>(gen + off_wmax);    // [ROWS][8 warps]
  float *ml = reinterpret_cast<float *>(gen + off_ml);        // [ROWS][2]
  float *obuf = reinterpret_cast<float *>(gen);               // [ROWS][HD], over ring stage 0 once the tiles are consumed

  const int L = a.kv_len[b];
  const int n_ct = (L + kTK - 1) / kTK;                       // tiles of cached keys
  // tiles per split: the last split also turns the accumulators into the window's keys and runs the window tile(s),
  // which costs it about two tiles' time, so the cached tiles are dealt as if there were two more of them
  const int tps = (n_ct + (ns > 1 ? 2 : 0) + ns - 1) / ns;
  const int t_begin = min(n_ct, split * tps);
  const int n_cached = min(n_ct, t_begin + tps) - t_begin;
  const int n_win = split == ns - 1 ? nwt : 0;
  const int plane_k = a.k_plane0 + b * a.hkv + kvh, plane_v = a.v_plane0 + b * a.hkv + kvh;

  auto issue_tile = [&](int it) {                              // thread 0 only
    const int stage = it % NS;
    const uint32_t bar = smem_addr(&full_bar[stage]);
    const uint32_t dst = base + stage * kStage;
    const int y = (t_begin + it) * kTK;
    mbar_expect_tx(bar, kStage);
#pragma unroll
    for (int s = 0; s < SUB; ++s) tma_load_3d(dst + s * kSubBytes, &kmap, s * 64, y, plane_k, bar);
#pragma unroll
    for (int s = 0; s < SUB; ++s) tma_load_3d(dst + kKBytes + s * kSubBytes, &vmap, s * 64, y, plane_v, bar);
  };

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) mbar_init(smem_addr(&full_bar[i]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // cached keys were written by earlier steps: request the first tiles before waiting for the QKV projection
    for (int it = 0; it < NS && it < n_cached; ++it) issue_tile(it);
  }
  __syncthreads();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- side clearing of buffers nobody reads during this kernel
  {
    const unsigned long long gtid =
        ((unsigned long long)(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * blockDim.x + tid;
    const unsigned long long nth = (unsigned long long)gridDim.x * gridDim.y * gridDim.z * blockDim.x;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (!a.z.p[i]) continue;
      const unsigned long long n4 = a.z.n[i] >> 2;
      float4 *p4 = reinterpret_cast<float4 *>(a.z.p[i]);
      for (unsigned long long e = gtid; e < n4; e += nth) p4[e] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (unsigned long long e = (n4 << 2) + gtid; e < a.z.n[i]; e += nth) a.z.p[i][e] = 0.f;
    }
  }

  // ---- queries (1/rms, rotation, bf16 high + low) and, in the last split, the window's own keys (rotated, stored to
  // shared memory and to the cache) come from the fp32 accumulators.  A thread keeps one pair index i and walks the rows
  // four at a time; the first batch of window-key loads is issued together with the first batch of query loads, so that
  // both share one trip to L2.
  constexpr int RPP = kAttnThreads / HALF;                    // rows per pass
  const int pi_ = tid % HALF, rsub = tid / HALF;
  __nv_bfloat16 *kbase = (__nv_bfloat16 *)a.kcache + (long long)b * a.stride_b + (long long)kvh * a.stride_h;
  __nv_bfloat16 *vbase = (__nv_bfloat16 *)a.vcache + (long long)b * a.stride_b + (long long)kvh * a.stride_h;
  struct QRegs { float x0[4], x1[4], ss[4]; float2 rot[4]; };
  struct WRegs { float k0[4], k1[4], v0[4], v1[4], ss[4]; float2 rot[4]; };
  auto q_load = [&](int r0, QRegs &q) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int rl = r0 + u * RPP + rsub;
      const int qrow = qg * ROWS + rl;
      q.x0[u] = q.x1[u] = q.ss[u] = 0.f; q.rot[u] = make_float2(1.f, 0.f);
      if (rl < ROWS && qrow < nq) {
        const int g = div_c(qrow), j = qrow - g * c;
        const int r = bl * c + j, h = kvh * group + g;
        const float *qacc = a.qkv + (long long)r * a.ldq + h * HD;
        q.ss[u] = __ldcg(a.ss + r);
        q.x0[u] = __ldcg(qacc + pi_); q.x1[u] = __ldcg(qacc + pi_ + HALF);
        q.rot[u] = __ldg(a.rope + (long long)(L + j) * HALF + pi_);
      }
    }
  };
  auto q_store = [&](int r0, const QRegs &q) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int rl = r0 + u * RPP + rsub;
      if (rl >= ROWS) continue;
      const float sc = rsqrtf(q.ss[u] / (float)a.dn + a.eps);
      const float a0 = q.x0[u] * sc, a1 = q.x1[u] * sc;
      const float q0 = a0 * q.rot[u].x - a1 * q.rot[u].y, q1 = a0 * q.rot[u].y + a1 * q.rot[u].x;
      const __nv_bfloat16 h0 = __float2bfloat16_rn(q0), h1 = __float2bfloat16_rn(q1);
      unsigned char *qt_base = gen + off_q + (uint32_t)(rl >> 4) * C::kQTile;
      const int row = rl & 15;
      const uint32_t o0 = tile_off(row, pi_ >> 3, 2048u) + (uint32_t)(pi_ & 7) * 2u;
      const uint32_t o1 = tile_off(row, (pi_ + HALF) >> 3, 2048u) + (uint32_t)(pi_ & 7) * 2u;
      *reinterpret_cast<__nv_bfloat16 *>(qt_base + o0) = h0;
      *reinterpret_cast<__nv_bfloat16 *>(qt_base + o1) = h1;
      *reinterpret_cast<__nv_bfloat16 *>(qt_base + SUB * 2048u + o0) = __float2bfloat16_rn(q0 - __bfloat162float(h0));
      *reinterpret_cast<__nv_bfloat16 *>(qt_base + SUB * 2048u + o1) = __float2bfloat16_rn(q1 - __bfloat162float(h1));
    }
  };
  auto w_load = [&](int j0, WRegs &w) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = j0 + u * RPP + rsub;
      w.k0[u] = w.k1[u] = w.v0[u] = w.v1[u] = w.ss[u] = 0.f; w.rot[u] = make_float2(1.f, 0.f);
      if (j < c) {
        const int r = bl * c + j;
        const float *kacc = a.qkv + (long long)r * a.ldq + qd + kvh * HD;
        w.ss[u] = __ldcg(a.ss + r);
        w.k0[u] = __ldcg(kacc + pi_); w.k1[u] = __ldcg(kacc + pi_ + HALF);
        w.v0[u] = __ldcg(kacc + kvd + pi_); w.v1[u] = __ldcg(kacc + kvd + pi_ + HALF);
        w.rot[u] = __ldg(a.rope + (long long)(L + j) * HALF + pi_);
      }
    }
  };
  auto w_store = [&](int j0, const WRegs &w) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = j0 + u * RPP + rsub;
      if (j >= c) continue;
      const int pos = L + j;
      const float sc = rsqrtf(w.ss[u] / (float)a.dn + a.eps);
      const float x0 = w.k0[u] * sc, x1 = w.k1[u] * sc;
      const __nv_bfloat16 o0 = __float2bfloat16_rn(x0 * w.rot[u].x - x1 * w.rot[u].y);
      const __nv_bfloat16 o1 = __float2bfloat16_rn(x0 * w.rot[u].y + x1 * w.rot[u].x);
      const __nv_bfloat16 w0 = __float2bfloat16_rn(w.v0[u] * sc), w1 = __float2bfloat16_rn(w.v1[u] * sc);
      unsigned char *wt_base = gen + off_win + (uint32_t)(j / kTK) * wstage;
      const int row = j % kTK;
      const uint32_t f0 = tile_off(row, pi_ >> 3, wsub) + (uint32_t)(pi_ & 7) * 2u;
      const uint32_t f1 = tile_off(row, (pi_ + HALF) >> 3, wsub) + (uint32_t)(pi_ & 7) * 2u;
      *reinterpret_cast<__nv_bfloat16 *>(wt_base + f0) = o0;
      *reinterpret_cast<__nv_bfloat16 *>(wt_base + f1) = o1;
      *reinterpret_cast<__nv_bfloat16 *>(wt_base + wk + f0) = w0;
      *reinterpret_cast<__nv_bfloat16 *>(wt_base + wk + f1) = w1;
      kbase[(long long)pos * HD + pi_] = o0; kbase[(long long)pos * HD + pi_ + HALF] = o1;
      vbase[(long long)pos * HD + pi_] = w0; vbase[(long long)pos * HD + pi_ + HALF] = w1;
    }
  };
  {
    QRegs q;
    WRegs w;
    q_load(0, q);
    if (n_win > 0) w_load(0, w);
    q_store(0, q);
    for (int r0 = RPP * 4; r0 < ROWS; r0 += RPP * 4) { q_load(r0, q); q_store(r0, q); }
    if (n_win > 0) {
      w_store(0, w);
      for (int j0 = RPP * 4; j0 < c; j0 += RPP * 4) { w_load(j0, w); w_store(j0, w); }
    }
  }
  if (n_win > 0) {
    // rows of the last window tile beyond the window: zero, so that a zero probability never meets a stale NaN pattern
    {
      const int wt = nwt - 1;
      const int nv = c - wt * kTK;
      unsigned char *wt_base = gen + off_win + (uint32_t)wt * wstage;
      for (int e = tid; e < (wrows - nv) * (HD / 8); e += kAttnThreads) {
        const int row = nv + e / (HD / 8), ch = e % (HD / 8);
        *reinterpret_cast<uint4 *>(wt_base + tile_off(row, ch, wsub)) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4 *>(wt_base + wk + tile_off(row, ch, wsub)) = make_uint4(0, 0, 0, 0);
      }
    }
  }

  // ---- per-lane row bookkeeping: window row of query rows g4 and g4 + 8 of each tile (-1: no such query)
  int jrow[QT][2];
#pragma unroll
  for (int qt = 0; qt < QT; ++qt)
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int qrow = qg * ROWS + qt * 16 + g4 + hh * 8;
      jrow[qt][hh] = qrow < nq ? qrow - div_c(qrow) * c : -1;
    }

  const float scale = rsqrtf((float)HD);
  float m_run[QT][2], l_run[QT][2], oacc[QT][NDW][4];
#pragma unroll
  for (int qt = 0; qt < QT; ++qt) {
    m_run[qt][0] = m_run[qt][1] = -INFINITY;
    l_run[qt][0] = l_run[qt][1] = 0.f;
#pragma unroll
    for (int nd = 0; nd < NDW; ++nd)
#pragma unroll
      for (int i = 0; i < 4; ++i) oacc[qt][nd][i] = 0.f;
  }

  __syncthreads();                                            // queries and window keys staged
  // With one query tile per CTA the high parts of the query fragments stay in registers for the whole run of tiles
  // (every warp multiplies the whole 16 x HD query tile by its 8 keys of every tile; re-reading it from shared memory
  // for every tile is half of this kernel's shared-memory traffic); the low parts are still read per tile.
  constexpr bool kQRegs = QT == 1;
  uint32_t qh[kQRegs ? HD / 16 : 1][4];
  if (kQRegs) {
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks)
      ldsm_x4(base + off_q + tile_off(lane & 15, ks * 2 + (lane >> 4), 2048u), qh[ks][0], qh[ks][1], qh[ks][2], qh[ks][3]);
  }
  bool all_ok = true;
  const int n_tiles = n_cached + n_win;
  for (int ti = 0; ti < n_tiles; ++ti) {
    uint32_t kb, vb, sstride;
    int koff, nvalid, rows_t;                                 // key offset relative to L for window tiles
    bool ok = true;
    const bool causal = ti >= n_cached;
    if (!causal) {
      const int stage = ti % NS;
      ok = mbar_wait_bounded(smem_addr(&full_bar[stage]), (uint32_t)(ti / NS) & 1u);
      kb = base + stage * kStage; vb = kb + kKBytes; sstride = kSubBytes;
      const int key0 = (t_begin + ti) * kTK;
      koff = 0; nvalid = min(kTK, L - key0); rows_t = kTK;
      if (nvalid < kTK) {
        // the tile's rows beyond the cached keys hold whatever the slab holds there: zero the V rows (the K rows are
        // masked by a select, a zero probability would still multiply a NaN pattern in V)
        unsigned char *vg = gen + (vb - base);
        for (int e = tid; e < (kTK - nvalid) * (HD / 8); e += kAttnThreads) {
          const int row = nvalid + e / (HD / 8), ch = e % (HD / 8);
          *reinterpret_cast<uint4 *>(vg + tile_off(row, ch, kSubBytes)) = make_uint4(0, 0, 0, 0);
        }
      }
    } else {
      const int wt = ti - n_cached;
      kb = base + off_win + (uint32_t)wt * wstage; vb = kb + wk; sstride = wsub;
      koff = wt * kTK; nvalid = min(kTK, c - koff); rows_t = wrows;
    }

    // ---- S = Q.K^T for this warp's 8 keys
    float s[QT][4];
#pragma unroll
    for (int qt = 0; qt < QT; ++qt)
#pragma unroll
      for (int i = 0; i < 4; ++i) s[qt][i] = 0.f;
    const bool my_keys = warp * 8 < rows_t;
    if (my_keys) {
#pragma unroll
      for (int ks2 = 0; ks2 < HD / 32; ++ks2) {
        uint32_t kf[4];
        ldsm_x4(kb + tile_off(warp * 8 + (lane & 7), ks2 * 4 + (lane >> 3), sstride), kf[0], kf[1], kf[2], kf[3]);
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
          const uint32_t qoff = tile_off(lane & 15, (ks2 * 2 + h2) * 2 + (lane >> 4), 2048u);
#pragma unroll
          for (int qt = 0; qt < QT; ++qt) {
            uint32_t al[4];
            const uint32_t qb = base + off_q + (uint32_t)qt * C::kQTile + qoff;
            ldsm_x4(qb + SUB * 2048u, al[0], al[1], al[2], al[3]);
            if (kQRegs) {
              mma_bf16(s[qt], qh[ks2 * 2 + h2], kf[h2 * 2], kf[h2 * 2 + 1]);
            } else {
              uint32_t ah[4];
              ldsm_x4(qb, ah[0], ah[1], ah[2], ah[3]);
              mma_bf16(s[qt], ah, kf[h2 * 2], kf[h2 * 2 + 1]);
            }
            mma_bf16(s[qt], al, kf[h2 * 2], kf[h2 * 2 + 1]);
          }
        }
      }
    }
    // ---- mask, scale, maxima over this warp's keys
#pragma unroll
    for (int qt = 0; qt < QT; ++qt) {
      float mx[2] = {-INFINITY, -INFINITY};
      if (!causal && nvalid == rows_t) {          // a full tile of cached keys: every key is visible to every query row
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int hh = i >> 1;
          const float v = (my_keys && jrow[qt][hh] >= 0) ? s[qt][i] * scale : -INFINITY;
          s[qt][i] = v;
          mx[hh] = fmaxf(mx[hh], v);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int hh = i >> 1;
          const int kl = warp * 8 + t4 * 2 + (i & 1);
          const bool vis = my_keys && jrow[qt][hh] >= 0 && kl < nvalid && (!causal || koff + kl <= jrow[qt][hh]);
          const float v = vis ? s[qt][i] * scale : -INFINITY;
          s[qt][i] = v;
          mx[hh] = fmaxf(mx[hh], v);
        }
      }
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
        if (t4 == 0) wmax[(qt * 16 + g4 + hh * 8) * 8 + warp] = mx[hh];      // [row][warp]: a row's eight values in 32 bytes
      }
    }
    all_ok = __syncthreads_and(ok ? 1 : 0) != 0;              // maxima published; every warp is past the previous tile
    if (!all_ok) break;
    // the stage of the previous cached tile is free: request the tile NS ahead of it
    if (tid == 0 && ti >= 1 && ti - 1 + NS < n_cached) issue_tile(ti - 1 + NS);

    // ---- probabilities (bf16 high + low) to shared memory; running maximum and this warp's share of the sum
#pragma unroll
    for (int qt = 0; qt < QT; ++qt) {
      float mnew[2], corr[2], lsum[2] = {0.f, 0.f};
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int row = qt * 16 + g4 + hh * 8;
        float mx = m_run[qt][hh];
        {
          const float4 w0 = *reinterpret_cast<const float4 *>(wmax + row * 8), w1 = *reinterpret_cast<const float4 *>(wmax + row * 8 + 4);
          mx = fmaxf(mx, fmaxf(fmaxf(fmaxf(w0.x, w0.y), fmaxf(w0.z, w0.w)), fmaxf(fmaxf(w1.x, w1.y), fmaxf(w1.z, w1.w))));
        }
        mnew[hh] = mx;
        corr[hh] = (m_run[qt][hh] == -INFINITY) ? 0.f : __expf(m_run[qt][hh] - mx);
        m_run[qt][hh] = mx;
      }
      float p[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int hh = i >> 1;
        p[i] = (s[qt][i] == -INFINITY) ? 0.f : __expf(s[qt][i] - mnew[hh]);
        lsum[hh] += p[i];
      }
      if (my_keys) {
        unsigned char *pb = gen + off_p + (uint32_t)qt * 4096u;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int row = g4 + hh * 8;
          const uint32_t o = tile_off(row, warp, 2048u) + (uint32_t)t4 * 4u;
          const float p0 = p[hh * 2], p1 = p[hh * 2 + 1];
          *reinterpret_cast<uint32_t *>(pb + o) = pack_bf16(p0, p1);
          *reinterpret_cast<uint32_t *>(pb + 2048u + o) = pack_bf16(p0 - bf16_round(p0), p1 - bf16_round(p1));
        }
      }
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        lsum[hh] += __shfl_xor_sync(0xffffffffu, lsum[hh], 1);
        lsum[hh] += __shfl_xor_sync(0xffffffffu, lsum[hh], 2);
        l_run[qt][hh] = l_run[qt][hh] * corr[hh] + lsum[hh];
      }
#pragma unroll
      for (int nd = 0; nd < NDW; ++nd) {
        oacc[qt][nd][0] *= corr[0]; oacc[qt][nd][1] *= corr[0];
        oacc[qt][nd][2] *= corr[1]; oacc[qt][nd][3] *= corr[1];
      }
    }
    __syncthreads();                                          // probabilities staged (and stale V rows zeroed)

    // ---- O[:, this warp's columns] += P.V over the tile's keys
    for (int kt = 0; kt < rows_t / 16; ++kt) {
      uint32_t vf[4];
      const int key = kt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
      if (NDW == 2) ldsm_x4_t(vb + tile_off(key, warp * 2 + (lane >> 4), sstride), vf[0], vf[1], vf[2], vf[3]);
      else { ldsm_x2_t(vb + tile_off(key, warp, sstride), vf[0], vf[1]); vf[2] = vf[3] = 0u; }
      const uint32_t poff = tile_off(lane & 15, kt * 2 + (lane >> 4), 2048u);
#pragma unroll
      for (int qt = 0; qt < QT; ++qt) {
        uint32_t ph[4], pl[4];
        const uint32_t pb = base + off_p + (uint32_t)qt * 4096u + poff;
        ldsm_x4(pb, ph[0], ph[1], ph[2], ph[3]);
        ldsm_x4(pb + 2048u, pl[0], pl[1], pl[2], pl[3]);
#pragma unroll
        for (int nd = 0; nd < NDW; ++nd) {
          mma_bf16(oacc[qt][nd], ph, vf[nd * 2], vf[nd * 2 + 1]);
          mma_bf16(oacc[qt][nd], pl, vf[nd * 2], vf[nd * 2 + 1]);
        }
      }
    }
  }
  if (!all_ok && tid == 0) atomicExch(a.err, 1u);

  // ---- this CTA's result: un-normalised output rows and (max, sum) per row, in its own shared memory
  __syncthreads();                                            // all warps are done with the tiles and with wmax
#pragma unroll
  for (int qt = 0; qt < QT; ++qt)
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
      if (t4 == 0) wmax[(qt * 16 + g4 + hh * 8) * 8 + warp] = l_run[qt][hh];
#pragma unroll
  for (int qt = 0; qt < QT; ++qt)
#pragma unroll
    for (int nd = 0; nd < NDW; ++nd) {
      const int col = warp * (8 * NDW) + nd * 8 + t4 * 2;
      *reinterpret_cast<float2 *>(obuf + (qt * 16 + g4) * HD + col) = make_float2(oacc[qt][nd][0], oacc[qt][nd][1]);
      *reinterpret_cast<float2 *>(obuf + (qt * 16 + g4 + 8) * HD + col) = make_float2(oacc[qt][nd][2], oacc[qt][nd][3]);
    }
  __syncthreads();
  if (tid < ROWS) {
    float lt = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) lt += wmax[tid * 8 + w];
    // every warp holds the same running maximum; take it from the lane that owns this row in warp tid / 32's layout
    ml[tid * 2 + 1] = lt;
  }
  if (warp == 0 && t4 == 0) {
#pragma unroll
    for (int qt = 0; qt < QT; ++qt) {
      ml[(qt * 16 + g4) * 2] = m_run[qt][0];
      ml[(qt * 16 + g4 + 8) * 2] = m_run[qt][1];
    }
  }
  if (ns > 1) cluster_sync_all(); else __syncthreads();

  // ---- merge of the splits: every CTA combines its share of the output.  A thread fetches the (max, sum) pairs and
  // the partial outputs of all splits in one go (independent loads, one trip through the cluster's shared memory)
  // and derives the split weights of its row itself.
  for (int u = split * kAttnThreads + tid; u < ROWS * (HD / 4); u += ns * kAttnThreads) {
    const int row = u / (HD / 4), c4 = u - row * (HD / 4);
    const int qrow = qg * ROWS + row;
    if (qrow >= nq) continue;
    float2 mlv[8];
    float4 ov[8];
#pragma unroll
    for (int sp = 0; sp < 8; ++sp) {
      mlv[sp] = make_float2(-INFINITY, 0.f);
      ov[sp] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (sp < ns) {
        if (ns > 1) {
          mlv[sp] = ld_dsmem_f2(map_to_rank(base + off_ml + (uint32_t)row * 8u, (uint32_t)sp));
          ov[sp] = ld_dsmem_f4(map_to_rank(base + (uint32_t)(row * HD + c4 * 4) * 4u, (uint32_t)sp));
        } else {
          mlv[sp] = make_float2(ml[row * 2], ml[row * 2 + 1]);
          ov[sp] = *reinterpret_cast<const float4 *>(obuf + row * HD + c4 * 4);
        }
      }
    }
    float M = -INFINITY;
#pragma unroll
    for (int sp = 0; sp < 8; ++sp)
      if (mlv[sp].y > 0.f) M = fmaxf(M, mlv[sp].x);
    float den = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int sp = 0; sp < 8; ++sp) {
      const float w = mlv[sp].y > 0.f ? __expf(mlv[sp].x - M) : 0.f;
      den = fmaf(mlv[sp].y, w, den);
      acc.x = fmaf(w, ov[sp].x, acc.x); acc.y = fmaf(w, ov[sp].y, acc.y);
      acc.z = fmaf(w, ov[sp].z, acc.z); acc.w = fmaf(w, ov[sp].w, acc.w);
    }
    const float inv = den > 0.f ? 1.0f / den : 0.f;
    const int g = div_c(qrow), j = qrow - g * c;
    const int r = bl * c + j, h = kvh * group + g;
    const float o0 = acc.x * inv, o1 = acc.y * inv, o2 = acc.z * inv, o3 = acc.w * inv;
    if (a.out_pan) {
      __nv_bfloat16 *ph = (__nv_bfloat16 *)a.out_pan + (long long)r * qd + h * HD + c4 * 4;
      *reinterpret_cast<uint2 *>(ph) = make_uint2(pack_bf16(o0, o1), pack_bf16(o2, o3));
      *reinterpret_cast<uint2 *>(ph + (long long)a.pan_rows * qd) =
          make_uint2(pack_bf16(o0 - bf16_round(o0), o1 - bf16_round(o1)), pack_bf16(o2 - bf16_round(o2), o3 - bf16_round(o3)));
    } else {
      *reinterpret_cast<float4 *>(a.out + (long long)r * qd + h * HD + c4 * 4) = make_float4(o0, o1, o2, o3);
    }
  }
  if (ns > 1) cluster_sync_all();                             // the other splits may still be reading this CTA's memory
}

// ------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t make_kv_tensor_map(KvTensorMap *out, const void *base, int hd, int max_seq, long long planes) {
  static_assert(sizeof(CUtensorMap) <= sizeof(KvTensorMap), "tensor map storage");
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
    enc = (EncodeTiledFn)sym;
  }
  if ((hd != 64 && hd != 128) || max_seq < 1 || planes < 1 || ((uintptr_t)base & 15)) return cudaErrorInvalidValue;
  cuuint64_t gdim[3] = {(cuuint64_t)hd, (cuuint64_t)max_seq, (cuuint64_t)planes};
  cuuint64_t gstr[2] = {(cuuint64_t)hd * 2, (cuuint64_t)max_seq * hd * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)kTK, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(reinterpret_cast<CUtensorMap *>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), gdim,
                   gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

void fused_attn_plan(int max_len, int c, int hq, int hkv, int nb, int hd, int n_sms, int &nsplit, int &qt) {
  const int nqt = ((hq / hkv) * c + 15) / 16;
  // Query tiles per CTA.  One is the rule: more CTAs, each small enough for two to share an SM, hide each other's
  // waits best (measured: 13B, batch 8, c = 32: 5.2 -> 4.8 ms of attention per step against two tiles per CTA).  Only
  // when that makes more than six waves of CTAs do several query tiles share a CTA (and with it every key tile and
  // its barriers) - as long as two such CTAs still fit on an SM, which is what decides there (7B, K/V 8192, batch 16:
  // c = 32, where they fit, 40.7 ms with two tiles per CTA against 43.1; c = 64, where they do not, 90.1 against 80.0).
  auto two_fit = [&](int q) {
    const size_t per_sm = 228 * 1024, reserve = 1024 + 256;
    const size_t need = hd == 128 ? attn_smem_bytes<128>(c, q, 2) : attn_smem_bytes<64>(c, q, 2);
    return 2 * (need + reserve) <= per_sm;
  };
  qt = 1;
  while (qt < 4 && qt < nqt && (long long)nb * hkv * ((nqt + qt - 1) / qt) > 6ll * n_sms && two_fit(qt * 2)) qt *= 2;
  const long long units = (long long)nb * hkv * ((nqt + qt - 1) / qt);
  const int n_ct = (max_len + kTK - 1) / kTK;
  // Short caches: one CTA per SM, so that the projection kernel's CTAs come in beside them while the attention runs.
  // Long caches (more than 8 tiles per CTA that way) are a streaming problem: two CTAs per SM hide each other's waits.
  long long s = n_sms / units;
  if (s < 1) s = 1;
  if (n_ct > 8 * s) s = 2ll * n_sms / units;
  if (s > 8) s = 8;
  if (s > n_ct) s = n_ct;
  if (s < 1) s = 1;
  nsplit = (int)s;
}

template <int HD, int QT>
static cudaError_t launch_fused_t(const KvTensorMap &kmap, const KvTensorMap &vmap, const FusedAttnArgs &a, cudaStream_t st) {
  // Ring depth: the deep ring when every CTA has an SM to itself (the following projection kernel's CTAs come in beside
  // it); with more CTAs than SMs two of them share an SM and hide each other's waits, so the ring is made as deep as
  // still lets two fit (at least two stages).
  const int nqt_ = ((a.hq / a.hkv) * a.c + 15) / 16;
  const long long ctas = (long long)a.nsplit * a.hkv * ((nqt_ + QT - 1) / QT) * a.nb;
  int dev_id = 0, n_sms = 0;
  if (cudaGetDevice(&dev_id) != cudaSuccess || cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev_id) != cudaSuccess)
    return cudaErrorInvalidValue;
  FusedAttnArgs args = a;
  args.stages = AttnCfg<HD>::NS;
  if (ctas > n_sms) {
    const size_t per_sm = 228 * 1024, reserve = 1024 + 256;    // per CTA: the system's kilobyte and the static part
    while (args.stages > 2 && 2 * (attn_smem_bytes<HD>(a.c, QT, args.stages) + reserve) > per_sm) --args.stages;
  }
  const size_t smem = attn_smem_bytes<HD>(a.c, QT, args.stages);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  static size_t attr_smem[kMaxDevices] = {0};
  const int dev = current_device_slot();
  if (smem > attr_smem[dev]) {
    cudaError_t e = cudaFuncSetAttribute(attn_tma_kernel<HD, QT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_smem[dev] = smem;
  }
  const int nqt = ((a.hq / a.hkv) * a.c + 15) / 16;
  const int nqg = (nqt + QT - 1) / QT;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(a.nsplit, a.hkv * nqg, a.nb); cfg.blockDim = dim3(kAttnThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (a.pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (a.nsplit > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = (unsigned)a.nsplit; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, attn_tma_kernel<HD, QT>, *reinterpret_cast<const CUtensorMap *>(&kmap),
                            *reinterpret_cast<const CUtensorMap *>(&vmap), args);
}

cudaError_t launch_attn_fused(const KvTensorMap &kmap, const KvTensorMap &vmap, const FusedAttnArgs &a, int hd, cudaStream_t st) {
  if (a.nsplit < 1 || a.nsplit > 8 || a.c < 1 || a.c > 2 * kTK || !a.err) return cudaErrorInvalidValue;
  if ((long long)a.hkv * (((a.hq / a.hkv) * a.c + 15) / 16) > 65535 || a.nb > 65535) return cudaErrorInvalidValue;
  if (hd == 128) {
    if (a.qt == 1) return launch_fused_t<128, 1>(kmap, vmap, a, st);
    if (a.qt == 2) return launch_fused_t<128, 2>(kmap, vmap, a, st);
    if (a.qt == 4) return launch_fused_t<128, 4>(kmap, vmap, a, st);
  } else if (hd == 64) {
    if (a.qt == 1) return launch_fused_t<64, 1>(kmap, vmap, a, st);
    if (a.qt == 2) return launch_fused_t<64, 2>(kmap, vmap, a, st);
    if (a.qt == 4) return launch_fused_t<64, 4>(kmap, vmap, a, st);
  }
  return cudaErrorInvalidValue;
}

int attn_fused_max_rows() { return 2 * kTK; }

}  // namespace fc
