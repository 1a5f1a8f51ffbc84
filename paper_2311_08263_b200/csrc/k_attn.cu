// Fused rotary embedding + in-place K/V write + split-KV window attention for bf16 (head_dim 64/128).
//
// grid (splits, kv heads, sequences); one CTA owns a run of consecutive 128-key chunks (one chunk when the problem is
// small, several - with running softmax statistics - when there are more chunks than the GPU
// holds CTAs) of one kv head of one sequence.
// It stages a chunk's K and V in shared memory - cached keys by 16-byte copies; the window's own keys
// (slots kv_len .. kv_len+c-1) straight from the fp32 QKV accumulators with the deferred 1/rms factor and
// the rotation applied, writing them to the cache on the way (each window key has exactly one owner CTA).
// Then, for every 16-row tile of the queries that map to this kv head (group heads x c window rows), the
// four warps each take 32 keys: S = Q.K^T and P.V run on mma.sync m16n8k16 (bf16 in, fp32 accumulate),
// softmax statistics by warp shuffles, the four warps are merged through shared memory and one partial
// (max, sum, out) per (row, head, split) goes to scratch.  The last CTA of a (sequence, kv head) merges the
// splits and clears the accumulators it owns; the last CTA of the grid clears the per-row sums of squares.
// Row j of sequence b sees keys 0 .. kv_len[b] + j (cache + causal part of the window).
#include <cstring>

#include "fc_internal.h"

namespace fc {

namespace {

constexpr int kChunk = 128;      // keys per CTA
constexpr int kAttnThreads = 128;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
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
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

}  // namespace

template <int HD>
__global__ void __launch_bounds__(kAttnThreads) attn_fused_kernel(FusedAttnArgs a) {
  constexpr int LD = HD + 8;                 // padded row (elements): ldmatrix rows land in distinct banks
  constexpr int HALF = HD / 2;
  constexpr int ND = HD / 8;                 // 8-wide output blocks
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // One K/V buffer even when the CTA walks over several chunks: two CTAs share an SM, and while one waits for its
  // next chunk the other computes (measured against two buffers and one CTA per SM: 3.5 vs 5.0 ms of attention at
  // batch 16, K/V 8192, 8 layers of the 7B shape).
  __nv_bfloat16 *Ks = reinterpret_cast<__nv_bfloat16 *>(smem_raw);       // [kChunk][LD]
  __nv_bfloat16 *Vs = Ks + kChunk * LD;                                  // [kChunk][LD]
  __nv_bfloat16 *Qs = Vs + kChunk * LD;                                  // [16][LD]  high part of q
  __nv_bfloat16 *Ql = Qs + 16 * LD;                                      // [16][LD]  low part: q - bf16(q)
  float *Om = reinterpret_cast<float *>(Ql + 16 * LD);                   // [4][16][HD]
  float *mls = Om + 4 * 16 * HD;                                         // [4][16][2]
  __shared__ unsigned int s_last, s_last_grid;

  // blockIdx.x = split * qsplit + query tile: with several chunks per CTA every 16-row query tile gets CTAs of its own
  // (they produce the same window keys and write the same values to the cache)
  const int split = blockIdx.x / a.qsplit, kvh = blockIdx.y, bl = blockIdx.z;
  const int b = a.b0 + bl;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int L = a.kv_len[b];
  const int ltot = L + a.c;
  // this CTA's chunks: ch_first .. ch_first + n_iter - 1 (one iteration with no keys for a surplus CTA)
  const int ch_first = split * a.cpc;
  const int n_live = min(a.cpc, (ltot - ch_first * kChunk + kChunk - 1) / kChunk);
  const int n_iter = max(1, n_live);
  const int group = a.hq / a.hkv;
  const int nq = group * a.c;
  const int qd = a.hq * HD, kvd = a.hkv * HD;
  const unsigned int c_magic = a.c_magic;
  auto div_c = [&](int q) -> int { return a.c == 1 ? q : (int)__umulhi((unsigned int)q, c_magic); };
  __nv_bfloat16 *kbase = (__nv_bfloat16 *)a.kcache + (long long)b * a.stride_b + (long long)kvh * a.stride_h;
  __nv_bfloat16 *vbase = (__nv_bfloat16 *)a.vcache + (long long)b * a.stride_b + (long long)kvh * a.stride_h;

  // ---- cached keys of a chunk: 16-byte asynchronous copies (one group per chunk); the first chunk's are issued
  // before anything else
  constexpr int CPR = HD / 8;                                // 16-byte pieces per row
  auto issue_chunk = [&](int ch) {
    const int k0c = ch * kChunk;
    const int nkc = min(kChunk, ltot - k0c);
    const int n_cached_c = nkc > 0 ? min(nkc, max(0, L - k0c)) : 0;
    for (int e = tid; e < n_cached_c * CPR; e += kAttnThreads) {
      const int t = e / CPR, p = e % CPR;
      cp_async16(smem_addr(Ks + t * LD + p * 8), kbase + (long long)(k0c + t) * HD + p * 8);
      cp_async16(smem_addr(Vs + t * LD + p * 8), vbase + (long long)(k0c + t) * HD + p * 8);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  issue_chunk(ch_first);
  // The cached keys above were written by earlier steps; everything below depends on the previous kernel
  // (the QKV projection), so let the next kernel start its prefetch and wait for the previous one here.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // Q tile registers: a thread keeps one pair index and walks the 16 rows of a tile; all loads of a tile are
  // issued together.  The first tile's loads are issued here so that their latency overlaps the prologue.
  constexpr int QRPI = kAttnThreads / HALF;                  // rows covered per pass
  constexpr int QNIT = 16 / QRPI;
  const int qi_pair = tid % HALF, q_rsub = tid / HALF;
  float qx0[QNIT], qx1[QNIT], qss[QNIT];
  float2 qrot[QNIT];
  auto q_load = [&](int qt) {
#pragma unroll
    for (int it = 0; it < QNIT; ++it) {
      const int qrow = qt * 16 + q_rsub + it * QRPI;
      qx0[it] = qx1[it] = 0.f; qss[it] = 0.f; qrot[it] = make_float2(1.f, 0.f);
      if (qrow < nq) {
        const int g = div_c(qrow), j = qrow - g * a.c;
        const int r = bl * a.c + j, h = kvh * group + g;
        const float *qacc = a.qkv + (long long)r * a.ldq + h * HD;
        qss[it] = __ldcg(a.ss + r);
        qx0[it] = __ldcg(qacc + qi_pair); qx1[it] = __ldcg(qacc + qi_pair + HALF);
        qrot[it] = __ldg(a.rope + (long long)(L + j) * HALF + qi_pair);
      }
    }
  };
  const int qt_first = a.qsplit > 1 ? (int)(blockIdx.x % a.qsplit) : 0;
  q_load(qt_first);

  // side clearing of buffers nobody reads during this kernel
  {
    const unsigned long long gtid =
        ((unsigned long long)(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * blockDim.x + tid;
    const unsigned long long nth = (unsigned long long)gridDim.x * gridDim.y * gridDim.z * blockDim.x;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (!a.z.p[i]) continue;
      // 16-byte stores over the aligned bulk, scalar stores for the tail (buffers are 256-byte aligned)
      const unsigned long long n4 = a.z.n[i] >> 2;
      float4 *p4 = reinterpret_cast<float4 *>(a.z.p[i]);
      for (unsigned long long e = gtid; e < n4; e += nth) p4[e] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (unsigned long long e = (n4 << 2) + gtid; e < a.z.n[i]; e += nth) a.z.p[i][e] = 0.f;
    }
  }

  const float scale = rsqrtf((float)HD);
  const int qt_end = a.qsplit > 1 ? qt_first + 1 : (nq + 15) / 16;   // all query tiles, or this CTA's own
  const int g4 = lane >> 2, t4 = lane & 3;
  // running softmax statistics and output of this warp's keys over the CTA's chunks (rows g4 and g4 + 8)
  float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f}, oacc[ND][4];
  for (int ci = 0; ci < n_iter; ++ci) {
  const int k0 = (ch_first + ci) * kChunk;
  const int nk = min(kChunk, ltot - k0);                     // <= 0 for a surplus CTA
  const int n_cached = nk > 0 ? min(nk, max(0, L - k0)) : 0;
  const bool has_next = ci + 1 < n_iter;
  if (nk > 0) {
    // ---- window keys owned by this chunk: from the accumulators, rotated, stored to smem and to the cache.
    // A thread keeps one pair index i and walks the window rows in passes; the loads of a pass are all issued
    // before the first use so that they share one trip to L2.
    {
      constexpr int RPI = kAttnThreads / HALF;               // rows covered per pass
      constexpr int NB = 16 / RPI;                           // passes batched together: 16 window rows per trip
      const int i = tid % HALF, rsub = tid / HALF;
      const int n_win = nk - n_cached;
      for (int t0 = 0; t0 < n_win; t0 += RPI * NB) {
        float k0v[NB], k1v[NB], v0v[NB], v1v[NB], ssv[NB];
        float2 rot[NB];
#pragma unroll
        for (int u = 0; u < NB; ++u) {
          const int tw = t0 + u * RPI + rsub;
          k0v[u] = k1v[u] = v0v[u] = v1v[u] = ssv[u] = 0.f; rot[u] = make_float2(1.f, 0.f);
          if (tw < n_win) {
            const int pos = k0 + n_cached + tw, j = pos - L;
            const int r = bl * a.c + j;
            const float *kacc = a.qkv + (long long)r * a.ldq + qd + kvh * HD;
            ssv[u] = __ldcg(a.ss + r);
            k0v[u] = __ldcg(kacc + i); k1v[u] = __ldcg(kacc + i + HALF);
            v0v[u] = __ldcg(kacc + kvd + i); v1v[u] = __ldcg(kacc + kvd + i + HALF);
            rot[u] = __ldg(a.rope + (long long)pos * HALF + i);
          }
        }
#pragma unroll
        for (int u = 0; u < NB; ++u) {
          const int tw = t0 + u * RPI + rsub;
          if (tw >= n_win) continue;
          const int t = n_cached + tw, pos = k0 + t;
          const float sc = rsqrtf(ssv[u] / (float)a.dn + a.eps);
          const float x0 = k0v[u] * sc, x1 = k1v[u] * sc;
          const __nv_bfloat16 o0 = __float2bfloat16_rn(x0 * rot[u].x - x1 * rot[u].y);
          const __nv_bfloat16 o1 = __float2bfloat16_rn(x0 * rot[u].y + x1 * rot[u].x);
          const __nv_bfloat16 w0 = __float2bfloat16_rn(v0v[u] * sc), w1 = __float2bfloat16_rn(v1v[u] * sc);
          Ks[t * LD + i] = o0; Ks[t * LD + i + HALF] = o1;
          Vs[t * LD + i] = w0; Vs[t * LD + i + HALF] = w1;
          kbase[(long long)pos * HD + i] = o0; kbase[(long long)pos * HD + i + HALF] = o1;
          vbase[(long long)pos * HD + i] = w0; vbase[(long long)pos * HD + i + HALF] = w1;
        }
      }
    }
    // rows beyond nk: zero so that stale shared memory (possibly NaN patterns) never meets a zero weight
    for (int e = tid; e < (kChunk - nk) * CPR; e += kAttnThreads) {
      const int t = nk + e / CPR, p = e % CPR;
      *reinterpret_cast<uint4 *>(Ks + t * LD + p * 8) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4 *>(Vs + t * LD + p * 8) = make_uint4(0, 0, 0, 0);
    }
  }

  asm volatile("cp.async.wait_group 0;" ::: "memory");
  for (int qt = qt_first; qt < qt_end; ++qt) {
    __syncthreads();                                          // K/V staged; previous tile's Qs/Om/mls free
    // ---- Q tile: 1/rms, rotation, bf16 (loads were issued earlier for the first tile); staged once per tile
    if (ci == 0) {
    if (qt > qt_first) q_load(qt);
#pragma unroll
    for (int it = 0; it < QNIT; ++it) {
      const int row = q_rsub + it * QRPI;
      const float sc = rsqrtf(qss[it] / (float)a.dn + a.eps);
      const float a0 = qx0[it] * sc, a1 = qx1[it] * sc;
      // q and the probabilities go through the tensor cores as a bf16 pair hi + lo, so that only the cached
      // K and V (stored in the model dtype) carry bf16 rounding
      const float r0 = a0 * qrot[it].x - a1 * qrot[it].y, r1 = a0 * qrot[it].y + a1 * qrot[it].x;
      const __nv_bfloat16 h0 = __float2bfloat16_rn(r0), h1 = __float2bfloat16_rn(r1);
      Qs[row * LD + qi_pair] = h0; Qs[row * LD + qi_pair + HALF] = h1;
      Ql[row * LD + qi_pair] = __float2bfloat16_rn(r0 - __bfloat162float(h0));
      Ql[row * LD + qi_pair + HALF] = __float2bfloat16_rn(r1 - __bfloat162float(h1));
    }
    __syncthreads();
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) { mrun[hh] = -INFINITY; lrun[hh] = 0.f; }
#pragma unroll
    for (int d = 0; d < ND; ++d)
#pragma unroll
      for (int i = 0; i < 4; ++i) oacc[d][i] = 0.f;
    }

    // ---- S = Q.K^T for this warp's 32 keys
    float sacc[4][4];
#pragma unroll
    for (int nb = 0; nb < 4; ++nb)
#pragma unroll
      for (int i = 0; i < 4; ++i) sacc[nb][i] = 0.f;
    if (nk > 0) {
#pragma unroll
      for (int ks = 0; ks < HD / 16; ++ks) {
        uint32_t af[4], al[4];
        ldsm_x4(smem_addr(Qs + (lane & 15) * LD + ks * 16 + (lane >> 4) * 8), af[0], af[1], af[2], af[3]);
        ldsm_x4(smem_addr(Ql + (lane & 15) * LD + ks * 16 + (lane >> 4) * 8), al[0], al[1], al[2], al[3]);
#pragma unroll
        for (int nb = 0; nb < 4; nb += 2) {
          // two key blocks (8 keys each) x one 16-wide k step
          uint32_t b0, b1, b2, b3;
          const int key = warp * 32 + nb * 8 + (lane & 7) + ((lane >> 4) & 1) * 8;
          ldsm_x4(smem_addr(Ks + key * LD + ks * 16 + ((lane >> 3) & 1) * 8), b0, b1, b2, b3);
          mma_bf16(sacc[nb], af, b0, b1);
          mma_bf16(sacc[nb + 1], af, b2, b3);
          mma_bf16(sacc[nb], al, b0, b1);
          mma_bf16(sacc[nb + 1], al, b2, b3);
        }
      }
    }
    // ---- mask, scale, softmax statistics over this warp's keys (rows g4 and g4 + 8)
    float mrow[2] = {-INFINITY, -INFINITY};
    int jrow[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int qrow = qt * 16 + g4 + hh * 8;
      jrow[hh] = (qrow < nq) ? (qrow - div_c(qrow) * a.c) : -1;
    }
#pragma unroll
    for (int nb = 0; nb < 4; ++nb)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int hh = i >> 1;
        const int key = k0 + warp * 32 + nb * 8 + t4 * 2 + (i & 1);
        const bool ok = jrow[hh] >= 0 && key < ltot && key <= L + jrow[hh];
        const float s = ok ? sacc[nb][i] * scale : -INFINITY;
        sacc[nb][i] = s;
        mrow[hh] = fmaxf(mrow[hh], s);
      }
    float lrow[2] = {0.f, 0.f};
    float corr[2];                                            // rescales what earlier chunks contributed
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      mrow[hh] = fmaxf(mrow[hh], __shfl_xor_sync(0xffffffffu, mrow[hh], 1));
      mrow[hh] = fmaxf(mrow[hh], __shfl_xor_sync(0xffffffffu, mrow[hh], 2));
      mrow[hh] = fmaxf(mrow[hh], mrun[hh]);                   // running maximum including this chunk
      corr[hh] = (mrun[hh] == -INFINITY) ? 0.f : __expf(mrun[hh] - mrow[hh]);
      mrun[hh] = mrow[hh];
    }
    uint32_t pf[2][4], pl[2][4];                              // P (high and low parts) as A fragments: two 16-key steps
#pragma unroll
    for (int nb = 0; nb < 4; ++nb) {
      float p[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int hh = i >> 1;
        p[i] = (sacc[nb][i] == -INFINITY) ? 0.f : __expf(sacc[nb][i] - mrow[hh]);
        lrow[hh] += p[i];
      }
      pf[nb >> 1][(nb & 1) * 2 + 0] = pack_bf16(p[0], p[1]);
      pf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(p[2], p[3]);
      float pr[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) pr[i] = p[i] - __bfloat162float(__float2bfloat16_rn(p[i]));
      pl[nb >> 1][(nb & 1) * 2 + 0] = pack_bf16(pr[0], pr[1]);
      pl[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(pr[2], pr[3]);
    }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      lrow[hh] += __shfl_xor_sync(0xffffffffu, lrow[hh], 1);
      lrow[hh] += __shfl_xor_sync(0xffffffffu, lrow[hh], 2);
      lrun[hh] = lrun[hh] * corr[hh] + lrow[hh];
    }
    // ---- O = O * corr + P.V
    if (ci > 0) {
#pragma unroll
      for (int d = 0; d < ND; ++d) {
        oacc[d][0] *= corr[0]; oacc[d][1] *= corr[0];
        oacc[d][2] *= corr[1]; oacc[d][3] *= corr[1];
      }
    }
    if (nk > 0) {
#pragma unroll
      for (int kt = 0; kt < 2; ++kt) {
#pragma unroll
        for (int d = 0; d < ND; d += 2) {
          uint32_t b0, b1, b2, b3;
          const int key = warp * 32 + kt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          ldsm_x4_t(smem_addr(Vs + key * LD + d * 8 + (lane >> 4) * 8), b0, b1, b2, b3);
          mma_bf16(oacc[d], pf[kt], b0, b1);
          mma_bf16(oacc[d + 1], pf[kt], b2, b3);
          mma_bf16(oacc[d], pl[kt], b0, b1);
          mma_bf16(oacc[d + 1], pl[kt], b2, b3);
        }
      }
    }
    if (ci < n_iter - 1) continue;                            // more chunks to come: keep accumulating
    // ---- merge the four warps (after the CTA's last chunk)
    if (t4 == 0) {
      mls[(warp * 16 + g4) * 2] = mrun[0]; mls[(warp * 16 + g4) * 2 + 1] = lrun[0];
      mls[(warp * 16 + g4 + 8) * 2] = mrun[1]; mls[(warp * 16 + g4 + 8) * 2 + 1] = lrun[1];
    }
    __syncthreads();
    float fac[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int row = g4 + hh * 8;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < 4; ++w) M = fmaxf(M, mls[(w * 16 + row) * 2]);
      fac[hh] = (mrun[hh] == -INFINITY) ? 0.f : __expf(mrun[hh] - M);
    }
#pragma unroll
    for (int d = 0; d < ND; ++d) {
      float *o0 = Om + (warp * 16 + g4) * HD + d * 8 + t4 * 2;
      float *o1 = Om + (warp * 16 + g4 + 8) * HD + d * 8 + t4 * 2;
      *reinterpret_cast<float2 *>(o0) = make_float2(oacc[d][0] * fac[0], oacc[d][1] * fac[0]);
      *reinterpret_cast<float2 *>(o1) = make_float2(oacc[d][2] * fac[1], oacc[d][3] * fac[1]);
    }
    __syncthreads();
    for (int e = tid; e < 16 * (HD / 4); e += kAttnThreads) {
      const int row = e / (HD / 4), d4 = e % (HD / 4);
      const int qrow = qt * 16 + row;
      if (qrow >= nq) continue;
      const int g = div_c(qrow), j = qrow - g * a.c;
      const int r = bl * a.c + j, h = kvh * group + g;
      const long long pidx = ((long long)r * a.hq + h) * a.nsplit + split;
      const float4 p0 = *reinterpret_cast<const float4 *>(Om + row * HD + d4 * 4);
      const float4 p1 = *reinterpret_cast<const float4 *>(Om + (16 + row) * HD + d4 * 4);
      const float4 p2 = *reinterpret_cast<const float4 *>(Om + (32 + row) * HD + d4 * 4);
      const float4 p3 = *reinterpret_cast<const float4 *>(Om + (48 + row) * HD + d4 * 4);
      *reinterpret_cast<float4 *>(a.part_o + pidx * HD + d4 * 4) =
          make_float4(p0.x + p1.x + p2.x + p3.x, p0.y + p1.y + p2.y + p3.y, p0.z + p1.z + p2.z + p3.z, p0.w + p1.w + p2.w + p3.w);
      if (d4 == 0) {
        float M = -INFINITY;
        for (int w = 0; w < 4; ++w) M = fmaxf(M, mls[(w * 16 + row) * 2]);
        float lsum = 0.f;
        for (int w = 0; w < 4; ++w) {
          const float mw = mls[(w * 16 + row) * 2];
          if (mw != -INFINITY) lsum += mls[(w * 16 + row) * 2 + 1] * __expf(mw - M);
        }
        *reinterpret_cast<float2 *>(a.part_ml + pidx * 2) = make_float2(M, lsum);
      }
    }
  }
  if (has_next) {
    __syncthreads();                                          // every warp is done with this chunk's buffer
    issue_chunk(ch_first + ci + 1);                           // the co-resident CTA computes meanwhile
  }
  }

  // ---- merge the splits of this (sequence, kv head) and clear the accumulators of its heads.
  // Cluster launch (the splits of one kv head form one thread-block cluster): a hardware cluster barrier, then
  // every CTA of the cluster merges its share of the queries.  Otherwise the last CTA to arrive merges them all.
  int q_first, q_step;
  unsigned int ctas_counted;
  if (a.cluster) {
    __threadfence();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    q_first = (int)blockIdx.x * 4 + warp; q_step = (int)gridDim.x * 4;
    ctas_counted = gridDim.x * gridDim.y * gridDim.z;
  } else {
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const unsigned int prev = atomicAdd(&a.counters[b * a.hkv + kvh], 1u);
      s_last = (prev == gridDim.x - 1u);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    q_first = warp; q_step = 4;
    ctas_counted = gridDim.y * gridDim.z;
  }
  for (int qi = q_first; qi < nq; qi += q_step) {
    const int g = div_c(qi), j = qi - g * a.c;
    const int r = bl * a.c + j, h = kvh * group + g;
    const long long base = ((long long)r * a.hq + h) * a.nsplit;
    // lanes take one split each for the (max, sum) pairs; the output loads below are independent
    const float2 *ml2 = reinterpret_cast<const float2 *>(a.part_ml) + base;
    float M = -INFINITY;
    for (int s0 = 0; s0 < a.nsplit; s0 += 32) {
      const int s = s0 + lane;
      if (s < a.nsplit) { const float2 ml = __ldcg(ml2 + s); if (ml.y > 0.f) M = fmaxf(M, ml.x); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float den = 0.f, o[HD / 32];
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) o[i] = 0.f;
    for (int s0 = 0; s0 < a.nsplit; s0 += 32) {
      const int s = s0 + lane;
      float wl = 0.f, wgt = 0.f;
      if (s < a.nsplit) {
        const float2 ml = __ldcg(ml2 + s);
        if (ml.y > 0.f) { wgt = __expf(ml.x - M); wl = ml.y * wgt; }
      }
#pragma unroll
      for (int sh = 16; sh > 0; sh >>= 1) wl += __shfl_xor_sync(0xffffffffu, wl, sh);
      den += wl;
      const int ns = min(32, a.nsplit - s0);
      const float *po = a.part_o + (base + s0) * HD + lane;
#pragma unroll 8
      for (int t = 0; t < ns; ++t) {
        const float w = __shfl_sync(0xffffffffu, wgt, t);
#pragma unroll
        for (int i = 0; i < HD / 32; ++i) o[i] = fmaf(w, __ldcg(po + (long long)t * HD + i * 32), o[i]);
      }
    }
    const float inv = 1.0f / den;
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) a.out[(long long)r * qd + h * HD + i * 32 + lane] = o[i] * inv;
    // this head's q accumulator (and, once per row, the kv head's k and v) are no longer needed
    float *qacc = a.qkv + (long long)r * a.ldq + h * HD;
    for (int i = lane; i < HD; i += 32) qacc[i] = 0.f;
    if (g == 0) {
      float *kacc = a.qkv + (long long)r * a.ldq + qd + kvh * HD;
      for (int i = lane; i < HD; i += 32) { kacc[i] = 0.f; kacc[kvd + i] = 0.f; }
    }
  }
  // the last CTA (of those counted) clears the per-row sums of squares: every reader is done by then
  __syncthreads();
  if (tid == 0) {
    if (!a.cluster) a.counters[b * a.hkv + kvh] = 0u;
    const unsigned int prev = atomicAdd(a.grid_counter, 1u);
    s_last_grid = (prev == ctas_counted - 1u);
  }
  __syncthreads();
  if (s_last_grid) {
    for (int i = tid; i < a.nb * a.c; i += kAttnThreads) a.ss[i] = 0.f;
    if (tid == 0) *a.grid_counter = 0u;
  }
}

template <int HD>
static cudaError_t launch_fused_t(const FusedAttnArgs &a, cudaStream_t st) {
  constexpr int LD = HD + 8;
  const int nqt = ((a.hq / a.hkv) * a.c + 15) / 16;
  if (a.cpc < 1 || (a.qsplit != 1 && a.qsplit != nqt) || (a.cpc > 1 && a.qsplit != nqt)) return cudaErrorInvalidValue;
  const size_t smem = sizeof(__nv_bfloat16) * (size_t)(2 * kChunk * LD + 2 * 16 * LD) +
                      sizeof(float) * (size_t)(4 * 16 * HD + 4 * 16 * 2);
  static size_t attr_smem[kMaxDevices] = {0};
  const int dev = current_device_slot();
  if (smem > attr_smem[dev]) {
    cudaError_t e = cudaFuncSetAttribute(attn_fused_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_smem[dev] = smem;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(a.nsplit * a.qsplit, a.hkv, a.nb); cfg.blockDim = dim3(kAttnThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (a.pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  // Largest cluster this kernel can be scheduled with: 16 (non-portable size) if the device takes it, else 8.
  static int max_cluster_dev[kMaxDevices] = {0};
  int &max_cluster = max_cluster_dev[dev];
  if (max_cluster == 0) {
    max_cluster = 8;
    if (cudaFuncSetAttribute(attn_fused_kernel<HD>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
      cudaLaunchConfig_t q;
      memset(&q, 0, sizeof q);
      q.gridDim = dim3(16, 1, 1); q.blockDim = dim3(kAttnThreads); q.dynamicSmemBytes = smem;
      cudaLaunchAttribute qa[1];
      qa[0].id = cudaLaunchAttributeClusterDimension;
      qa[0].val.clusterDim.x = 16; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
      q.attrs = qa; q.numAttrs = 1;
      int n_clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&n_clusters, attn_fused_kernel<HD>, &q) == cudaSuccess && n_clusters > 0)
        max_cluster = 16;
    }
    (void)cudaGetLastError();
  }
  FusedAttnArgs args = a;
  const int cta_x = a.nsplit * a.qsplit;
  args.cluster = (cta_x >= 2 && cta_x <= max_cluster) ? 1 : 0;
  if (args.cluster) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = (unsigned)cta_x; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, attn_fused_kernel<HD>, args);
}

cudaError_t launch_attn_fused(const FusedAttnArgs &a, int hd, cudaStream_t st) {
  if (hd == 64) return launch_fused_t<64>(a, st);
  if (hd == 128) return launch_fused_t<128>(a, st);
  return cudaErrorInvalidValue;
}

int attn_fused_chunk() { return kChunk; }

}  // namespace fc
