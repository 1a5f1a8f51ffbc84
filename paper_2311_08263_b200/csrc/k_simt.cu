// FMA (non-tensor-core) kernels of the Jacobi-window decode step: embedding gather, the plain
// projection kernel used by the fp32 configuration, rotary embedding + K/V write, split-KV window
// attention, and the accept / commit / shift / refill kernel.
#include "fc_internal.h"

namespace fc {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ void zero_side(const ZeroList &z) {
  const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  const unsigned long long nth = (unsigned long long)gridDim.x * blockDim.x;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (z.p[i])
      for (unsigned long long j = tid; j < z.n[i]; j += nth) z.p[i][j] = 0.f;
}

// Monotone map float -> uint32 (larger float -> larger key); NaN maps to 0 so it never wins.
__device__ __forceinline__ unsigned int ordered_key(float v) {
  if (v != v) return 0u;
  unsigned int u = __float_as_uint(v);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ unsigned long long pack_max(float v, int idx) {
  return ((unsigned long long)ordered_key(v) << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned int)idx);
}

// ------------------------------------------------------------------------------------ embed
template <typename T>
__global__ void embed_kernel(EmbedArgs a) {
  const T *emb = (const T *)a.emb;
  const long long total = (long long)a.R * a.d;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    int r = (int)(i / a.d), k = (int)(i % a.d);
    a.x[i] = to_f32(emb[(long long)a.tokens[r] * a.d + k]);
  }
  zero_side(a.z);
}

cudaError_t launch_embed(const EmbedArgs &a, int dtype, cudaStream_t st) {
  int blocks = 148 * 2;
  if (dtype == FC_F32) embed_kernel<float><<<blocks, 256, 0, st>>>(a);
  else embed_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(a);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ FMA projection
// One warp per output feature n; lanes stride over k; rows in chunks of RC.  No split-K, so every
// output receives exactly one addition and the result is deterministic.
template <typename T, int PRO>
__device__ __forceinline__ float pro_apply(const GemmArgs &a, int r, int k, float s_r) {
  float x = a.x[(long long)r * a.ldx + k];
  if (PRO == PRO_GAIN) return x * to_f32(((const T *)a.gain)[k]);
  if (PRO == PRO_SILU_MUL) {
    float g = s_r * x, u = s_r * a.x2[(long long)r * a.ldx + k];
    return (g / (1.0f + expf(-g))) * u;
  }
  return x;
}

template <typename T, int PRO, int EPI>
__global__ void gemm_simt_kernel(GemmArgs a) {
  constexpr int RC = 8;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_total = a.n_rows[0] + (a.n_mats > 1 ? a.n_rows[1] : 0) + (a.n_mats > 2 ? a.n_rows[2] : 0);
  const int n = blockIdx.x * (blockDim.x >> 5) + warp;
  if (n >= n_total) return;
  int m = 0, nl = n;
  while (m + 1 < a.n_mats && nl >= a.n_rows[m]) { nl -= a.n_rows[m]; ++m; }
  const T *wrow = (const T *)a.w[m] + (long long)nl * a.K;
  const int ycol = a.y_off[m] + nl;

  for (int r0 = 0; r0 < a.R; r0 += RC) {
    float acc[RC], ssq[RC], srow[RC];
#pragma unroll
    for (int i = 0; i < RC; ++i) {
      acc[i] = 0.f; ssq[i] = 0.f; srow[i] = 1.f;
      if (PRO == PRO_SILU_MUL && r0 + i < a.R) srow[i] = rsqrtf(a.ss_in[r0 + i] / (float)a.dn + a.eps);
    }
    for (int k = lane; k < a.K; k += 32) {
      const float wv = to_f32(wrow[k]);
#pragma unroll
      for (int i = 0; i < RC; ++i) {
        if (r0 + i < a.R) {
          acc[i] = fmaf(wv, pro_apply<T, PRO>(a, r0 + i, k, srow[i]), acc[i]);
          if (PRO == PRO_GAIN) { float x = a.x[(long long)(r0 + i) * a.ldx + k]; ssq[i] = fmaf(x, x, ssq[i]); }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < RC; ++i) {
      const int r = r0 + i;
      if (r >= a.R) break;
      float v = warp_sum(acc[i]);
      float ss = (PRO == PRO_GAIN) ? warp_sum(ssq[i]) : 0.f;
      if (lane == 0) {
        if (EPI == EPI_ATOMIC_ADD) {
          atomicAdd(&a.y[(long long)r * a.ldy + ycol], v);
          if (PRO == PRO_GAIN && a.ss_out && n == 0) atomicAdd(&a.ss_out[r], ss);
        } else {
          float logit = v * rsqrtf(ss / (float)a.dn + a.eps);
          if (a.perm && a.perm[a.tokens[r]] == ycol) logit += a.beta;
          if (a.logits) a.logits[(long long)r * a.vocab + ycol] = logit;
          atomicMax(&a.amax[r], pack_max(logit, ycol));
        }
      }
    }
  }
}

template <typename T>
static cudaError_t launch_gemm_simt_t(const GemmArgs &a, int pro, int epi, cudaStream_t st) {
  int n_total = 0;
  for (int m = 0; m < a.n_mats; ++m) n_total += a.n_rows[m];
  dim3 block(256), grid((n_total + 7) / 8);
  if (epi == EPI_ARGMAX) {
    if (pro != PRO_GAIN) return cudaErrorInvalidValue;
    gemm_simt_kernel<T, PRO_GAIN, EPI_ARGMAX><<<grid, block, 0, st>>>(a);
  } else if (pro == PRO_NONE) gemm_simt_kernel<T, PRO_NONE, EPI_ATOMIC_ADD><<<grid, block, 0, st>>>(a);
  else if (pro == PRO_GAIN) gemm_simt_kernel<T, PRO_GAIN, EPI_ATOMIC_ADD><<<grid, block, 0, st>>>(a);
  else gemm_simt_kernel<T, PRO_SILU_MUL, EPI_ATOMIC_ADD><<<grid, block, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gemm_simt(const GemmArgs &a, int dtype, int pro, int epi, cudaStream_t st) {
  return dtype == FC_F32 ? launch_gemm_simt_t<float>(a, pro, epi, st)
                         : launch_gemm_simt_t<__nv_bfloat16>(a, pro, epi, st);
}

// ------------------------------------------------------------------------------------ RoPE + K/V write
// One thread per (row, head, pair i): applies the deferred 1/rms factor, rotates q and k heads at
// absolute position kv_len[b] + j (pairs (i, i + hd/2), angle pos * theta^(-2i/hd)), writes q to
// q_out and k, v into the cache at slot kv_len[b] + j (scratch until committed), and clears the
// accumulators it has read.
template <typename T>
__global__ void rope_kv_kernel(RopeArgs a) {
  const int half = a.hd >> 1;
  const int heads = a.hq + 2 * a.hkv;
  const long long total = (long long)a.nb * a.c * heads * half;
  T *q_out = (T *)a.q_out, *kc = (T *)a.kcache, *vc = (T *)a.vcache;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(t % half);
    const int h = (int)((t / half) % heads);
    const int r = (int)(t / ((long long)half * heads));
    const int b = a.seq_map ? a.seq_map[r / a.c] : a.b0 + r / a.c, j = r % a.c;
    const int pos = a.kv_len[b] + j;
    const float s = rsqrtf(a.ss[r] / (float)a.dn + a.eps);
    float *src = a.qkv + (long long)r * a.ldq + (long long)h * a.hd;
    const float v0 = src[i] * s, v1 = src[i + half] * s;
    src[i] = 0.f; src[i + half] = 0.f;
    if (h < a.hq + a.hkv) {
      const float2 rot = a.rope[(long long)pos * half + i];     // host-built table: the device's powf is a few ulp off
      const float cs = rot.x, sn = rot.y;
      const float o0 = v0 * cs - v1 * sn, o1 = v0 * sn + v1 * cs;
      if (h < a.hq) {
        T *dst = q_out + (long long)r * a.hq * a.hd + (long long)h * a.hd;
        dst[i] = from_f32<T>(o0); dst[i + half] = from_f32<T>(o1);
      } else {
        T *dst = kc + (long long)b * a.stride_b + (long long)(h - a.hq) * a.stride_h + (long long)pos * a.hd;
        dst[i] = from_f32<T>(o0); dst[i + half] = from_f32<T>(o1);
      }
    } else {
      T *dst = vc + (long long)b * a.stride_b + (long long)(h - a.hq - a.hkv) * a.stride_h + (long long)pos * a.hd;
      dst[i] = from_f32<T>(v0); dst[i + half] = from_f32<T>(v1);
    }
  }
  zero_side(a.z);
}

cudaError_t launch_rope_kv(const RopeArgs &a, int dtype, cudaStream_t st) {
  int blocks = 148 * 2;
  if (dtype == FC_F32) rope_kv_kernel<float><<<blocks, 256, 0, st>>>(a);
  else rope_kv_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(a);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ window attention
// grid (nsplit, hkv, nb).  A block stages one tile of TK keys/values of one kv head in shared memory
// and evaluates every query that maps to it (group = hq/hkv heads x c window rows): scores with one
// key per lane, tile-local softmax by warp shuffles, then P.V with the head dimension across lanes.
// Row j of sequence b sees keys 0 .. kv_len[b] + j (cache + causal part of the window).  Partial
// (max, sum, out) per split go to scratch; the last block to finish a (b, kv head) merges them.
template <typename T, int HD, int TK>
__global__ void __launch_bounds__(256) attn_window_kernel(AttnArgs a) {
  constexpr int PADK = (sizeof(T) == 2) ? 2 : 1;      // row padding so lanes hit distinct banks
  constexpr int KS = HD + PADK;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T *Ks = (T *)smem_raw;                              // [TK][KS]
  T *Vs = Ks + TK * KS;                               // [TK][HD]
  float *qs = (float *)(Vs + TK * HD);                // [8 warps][HD]
  float *ps = qs + 8 * HD;                            // [8 warps][TK]
  __shared__ unsigned int s_last;

  const int split = blockIdx.x, kvh = blockIdx.y, bl = blockIdx.z;
  const int b = a.seq_map ? a.seq_map[bl] : a.b0 + bl;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int L = a.kv_len[b];
  const int ltot = L + a.c;
  const int k0 = split * TK;
  const int nk = min(TK, ltot - k0);                  // may be <= 0 for surplus splits
  const int group = a.hq / a.hkv;
  const int nq = group * a.c;
  const T *kbase = (const T *)a.kcache + (long long)b * a.stride_b + (long long)kvh * a.stride_h;
  const T *vbase = (const T *)a.vcache + (long long)b * a.stride_b + (long long)kvh * a.stride_h;

  if (nk > 0) {
    for (int e = threadIdx.x; e < nk * HD; e += blockDim.x) {
      int t = e / HD, i = e % HD;
      Ks[t * KS + i] = kbase[(long long)(k0 + t) * HD + i];
      Vs[t * HD + i] = vbase[(long long)(k0 + t) * HD + i];
    }
  }
  __syncthreads();

  const float scale = rsqrtf((float)HD);
  float *qw = qs + warp * HD, *pw = ps + warp * TK;
  for (int qi = warp; qi < nq; qi += 8) {
    const int g = qi / a.c, j = qi % a.c;
    const int h = kvh * group + g;
    const int r = bl * a.c + j;
    const T *qv = (const T *)a.q + (long long)r * a.hq * HD + (long long)h * HD;
    for (int i = lane; i < HD; i += 32) qw[i] = to_f32(qv[i]) * scale;
    __syncwarp();
    const int last_key = L + j;                        // inclusive
    float sc[TK / 32];
    float m = -INFINITY;
#pragma unroll
    for (int t = 0; t < TK / 32; ++t) {
      const int key = t * 32 + lane;
      float s = -INFINITY;
      if (key < nk && k0 + key <= last_key) {
        s = 0.f;
        const T *kr = Ks + key * KS;
#pragma unroll 8
        for (int i = 0; i < HD; ++i) s = fmaf(qw[i], to_f32(kr[i]), s);
      }
      sc[t] = s;
      m = fmaxf(m, s);
    }
    m = warp_max(m);
    float l = 0.f;
#pragma unroll
    for (int t = 0; t < TK / 32; ++t) {
      const float p = (sc[t] == -INFINITY) ? 0.f : expf(sc[t] - m);
      pw[t * 32 + lane] = p;
      l += p;
    }
    l = warp_sum(l);
    __syncwarp();
    float o[HD / 32];
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) o[i] = 0.f;
    const int kend = min(nk, last_key - k0 + 1);
    for (int key = 0; key < kend; ++key) {
      const float p = pw[key];
#pragma unroll
      for (int i = 0; i < HD / 32; ++i) o[i] = fmaf(p, to_f32(Vs[key * HD + i * 32 + lane]), o[i]);
    }
    const long long pidx = ((long long)r * a.hq + h) * a.nsplit + split;
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) a.part_o[pidx * HD + i * 32 + lane] = o[i];
    if (lane == 0) { a.part_ml[pidx * 2] = m; a.part_ml[pidx * 2 + 1] = l; }
    __syncwarp();
  }

  // last block of this (sequence, kv head) merges the splits
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int prev = atomicAdd(&a.counters[b * a.hkv + kvh], 1u);
    s_last = (prev == (unsigned int)a.nsplit - 1u);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    for (int qi = warp; qi < nq; qi += 8) {
      const int g = qi / a.c, j = qi % a.c;
      const int h = kvh * group + g;
      const int r = bl * a.c + j;
      const long long base = ((long long)r * a.hq + h) * a.nsplit;
      float M = -INFINITY;
      for (int s = 0; s < a.nsplit; ++s) M = fmaxf(M, __ldcg(&a.part_ml[(base + s) * 2]));
      float den = 0.f, o[HD / 32];
#pragma unroll
      for (int i = 0; i < HD / 32; ++i) o[i] = 0.f;
      for (int s = 0; s < a.nsplit; ++s) {
        const float ms = __ldcg(&a.part_ml[(base + s) * 2]);
        const float ls = __ldcg(&a.part_ml[(base + s) * 2 + 1]);
        if (ls == 0.f) continue;
        const float wgt = expf(ms - M);
        den = fmaf(ls, wgt, den);
#pragma unroll
        for (int i = 0; i < HD / 32; ++i)
          o[i] = fmaf(wgt, __ldcg(&a.part_o[(base + s) * HD + i * 32 + lane]), o[i]);
      }
      const float inv = 1.0f / den;
#pragma unroll
      for (int i = 0; i < HD / 32; ++i)
        a.out[(long long)r * a.hq * HD + (long long)h * HD + i * 32 + lane] = o[i] * inv;
    }
    if (threadIdx.x == 0) a.counters[b * a.hkv + kvh] = 0u;
  }
  if (blockIdx.y == 0 && blockIdx.z == 0) {
    // side clearing is spread over the blocks of the first (kv head, sequence) only
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long nth = (unsigned long long)gridDim.x * blockDim.x;
    for (int i = 0; i < 4; ++i)
      if (a.z.p[i]) for (unsigned long long e = tid; e < a.z.n[i]; e += nth) a.z.p[i][e] = 0.f;
  }
}

int attn_tile_keys(int dtype, int hd) { return (dtype == FC_F32 && hd == 128) ? 64 : 128; }

template <typename T, int HD, int TK>
static cudaError_t launch_attn_t(const AttnArgs &a, cudaStream_t st) {
  constexpr int PADK = (sizeof(T) == 2) ? 2 : 1;
  size_t smem = sizeof(T) * (size_t)(TK * (HD + PADK) + TK * HD) + sizeof(float) * (8 * HD + 8 * TK);
  static bool attr_done[kMaxDevices] = {false};
  const int dev = current_device_slot();
  if (!attr_done[dev]) {
    cudaError_t e = cudaFuncSetAttribute(attn_window_kernel<T, HD, TK>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  dim3 grid(a.nsplit, a.hkv, a.nb);
  attn_window_kernel<T, HD, TK><<<grid, 256, smem, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_attn(const AttnArgs &a, int dtype, int hd, cudaStream_t st) {
  if (dtype == FC_F32) {
    if (hd == 32) return launch_attn_t<float, 32, 128>(a, st);
    if (hd == 64) return launch_attn_t<float, 64, 128>(a, st);
    if (hd == 128) return launch_attn_t<float, 128, 64>(a, st);
  } else {
    if (hd == 32) return launch_attn_t<__nv_bfloat16, 32, 128>(a, st);
    if (hd == 64) return launch_attn_t<__nv_bfloat16, 64, 128>(a, st);
    if (hd == 128) return launch_attn_t<__nv_bfloat16, 128, 128>(a, st);
  }
  return cudaErrorInvalidValue;
}

// ------------------------------------------------------------------------------------ accept / commit / shift / refill
// One thread per sequence (all integer work; c <= 64).  a[j] = greedy token after window slot j.
// a[0] is always exact; a[j] is exact while every guess w[1..j] matched the exact token before it
// (checked one by one, Eq. 5).  K/V of the accepted rows already sit at their final slots, so the
// commit is kv_len += k.  New window: pending token a[k-1], the unverified outputs a[k..c-1] as next
// guesses, then refill ids for the k-1 positions no forward has predicted yet.
__global__ void accept_kernel(AcceptArgs a) {
  const int bl = blockIdx.x * blockDim.x + threadIdx.x;
  if (bl >= a.nb) return;
  const int b = a.seq_map ? a.seq_map[bl] : a.b0 + bl, c = a.c;
  int32_t *w = a.window + (long long)b * c;
  int32_t arg[64];
  for (int j = 0; j < c; ++j) {
    const int r = bl * c + j;
    if (a.amax) {
      arg[j] = (int32_t)(0xFFFFFFFFu - (unsigned int)(a.amax[r] & 0xFFFFFFFFull));
      if (a.amax_clear) a.amax_clear[r] = 0ull;
    } else {
      arg[j] = a.argmax[r];
    }
  }
  if (a.err_inject && bl == 0) atomicExch(a.err_inject, 1u);
  if (a.done && a.done[b]) { a.accepted_count[b] = 0; return; }
  int k = 1;
  while (k < c && w[k] == arg[k - 1]) ++k;
  // stop rules: cut at max_tokens and just after the first EOS
  const int n0 = a.n_gen[b];
  int kept = 0, finished = 0;
  for (int j = 0; j < k && !finished; ++j) {
    if (a.max_tokens > 0 && n0 + kept >= a.max_tokens) { finished = 1; break; }
    a.accepted_tokens[(long long)b * c + j] = arg[j];
    if (a.out_tokens && n0 + kept < a.out_stride) a.out_tokens[(long long)b * a.out_stride + n0 + kept] = arg[j];
    ++kept;
    if (a.eos_id >= 0 && arg[j] == a.eos_id) finished = 1;
  }
  if (a.max_tokens > 0 && n0 + kept >= a.max_tokens) finished = 1;
  a.accepted_count[b] = kept;
  if (!a.commit) return;
  if (finished && a.done) a.done[b] = 1;
  k = kept;                      // after a cut the remaining state is only reported, never used
  if (k == 0) return;
  a.kv_len[b] += k;
  const int n1 = n0 + k;
  a.n_gen[b] = n1;
  const int P = a.prompt_lens ? a.prompt_lens[b] : 1;
  int32_t nw[64];
  nw[0] = arg[k - 1];
  for (int j = 1; j < c; ++j) {
    if (j <= c - k) nw[j] = arg[k - 1 + j];
    else nw[j] = (a.refill == FC_REFILL_PAD || !a.prompt) ? a.pad_id
                                                          : a.prompt[(long long)b * a.p_stride + (n1 + j - 1) % P];
  }
  for (int j = 0; j < c; ++j) w[j] = nw[j];
}

__global__ void gather_rows_kernel(int32_t *dst, const int32_t *window, const int32_t *seq_map, int nb, int c) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < nb * c) dst[i] = window[(long long)seq_map[i / c] * c + i % c];
}

cudaError_t launch_gather_rows(int32_t *dst, const int32_t *window, const int32_t *seq_map, int nb, int c, cudaStream_t st) {
  gather_rows_kernel<<<(nb * c + 255) / 256, 256, 0, st>>>(dst, window, seq_map, nb, c);
  return cudaGetLastError();
}

cudaError_t launch_accept(const AcceptArgs &a, cudaStream_t st) {
  accept_kernel<<<(a.nb + 31) / 32, 32, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace fc
