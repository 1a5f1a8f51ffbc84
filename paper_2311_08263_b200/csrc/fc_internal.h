// Internal declarations shared by the CUDA sources of the Jacobi-window decode library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fastcot.h"

namespace fc {

// ---- activation transform applied while an fp32 buffer is staged as the GEMM's row operand ----
enum ProOp : int {
  PRO_NONE = 0,      // x
  PRO_GAIN = 1,      // x * gain[k]                (RMSNorm gain; the 1/rms row factor is applied by the consumer)
  PRO_SILU_MUL = 2   // silu(s_r * g) * (s_r * u)  (SwiGLU on gate/up accumulators that still lack 1/rms)
};
enum EpiOp : int {
  EPI_ATOMIC_ADD = 0,  // y[r, n] += acc  (split-K partial sums, or += onto the residual stream)
  EPI_ARGMAX = 1       // logits = s_r * acc + bias; per-row running (max, lowest index) via 64-bit atomicMax
};

constexpr int kMaxMats = 3;

struct GemmArgs {
  // row operand: fp32 [R, K] with leading dimension ldx
  const float *x;
  const float *x2;        // PRO_SILU_MUL: the "up" half (x is the "gate" half)
  int ldx;
  const void *gain;       // PRO_GAIN: [K] in the weight dtype
  const float *ss_in;     // PRO_SILU_MUL: per-row sum of squares of the normalised input; s_r = rsqrt(ss/dn + eps)
  float *ss_out;          // PRO_GAIN: if non-null, sum_k x[r,k]^2 is accumulated here (once per k)
  float eps;
  int dn;                 // width the sums of squares are means over (d_model)
  // weights: up to three matrices [n_rows[m], K], outputs concatenated at column offsets y_off[m]
  const void *w[kMaxMats];
  int ldw;                // row pitch of the weight matrices in elements (0: K) - a column slice of a wider matrix
  int n_rows[kMaxMats];
  int y_off[kMaxMats];
  int n_mats;
  float *y;
  int ldy;
  int R, K;
  // EPI_ARGMAX
  const int32_t *tokens;          // [R] input token of each row (bias lookup)
  const int32_t *perm;            // [vocab] or null
  float beta;
  unsigned long long *amax;       // [R] packed (ordered logit << 32 | ~index)
  float *logits;                  // optional dump [R, vocab]
  int vocab;
  // more than 16 rows: bf16 panel [2][pan_rows][K] (high parts, then low parts) that the launch fills with pro(x) once
  // and streams by TMA; with the argmax epilogue ss_out then holds the row sums of squares the epilogue reads
  void *pan;
  int pan_rows;
  int pan_ready;                  // the panel already holds pro(x), written by the kernel before this launch: no conversion
};

struct ZeroList {       // buffers a kernel clears on the side (fp32 words)
  float *p[4];
  unsigned long long n[4];
};

struct RopeArgs {
  float *qkv;             // [R, ldq] accumulators: q | k | v, unscaled by 1/rms; cleared after reading
  int ldq;
  const float *ss;        // [R] sums of squares for the 1/rms factor
  float eps; int dn;
  const int32_t *kv_len;  // [batch] device
  const int32_t *seq_map; // optional [nb] device: the sequence behind row block i (null: b0 + i)
  int b0, nb, c;          // rows r = i * c + j for row block i
  int hq, hkv, hd;
  const float2 *rope;     // [max_seq][hd/2] (cos, sin) of position * theta^(-2i/hd), built on the host
  void *q_out;            // [R, hq*hd] in the cache dtype
  void *kcache, *vcache;  // layer base; element strides below
  long long stride_b, stride_h;   // per sequence, per kv head (elements); token stride is hd
  ZeroList z;
};

struct AttnArgs {
  const void *q;          // [R, hq*hd] cache dtype, already rotated
  const void *kcache, *vcache;
  long long stride_b, stride_h;
  const int32_t *kv_len;
  const int32_t *seq_map; // optional [nb] device: the sequence behind row block i (null: b0 + i)
  int b0, nb, c, hq, hkv;
  int nsplit;
  float *part_o;          // [R*hq, nsplit, hd]
  float *part_ml;         // [R*hq, nsplit, 2]
  unsigned int *counters; // [batch*hkv], zero on entry, zero on exit
  float *out;             // [R, hq*hd] fp32
  ZeroList z;
};

struct KvTensorMap { alignas(64) unsigned char opaque[128]; };   // storage of one TMA tensor map (CUtensorMap)

struct FusedAttnArgs {   // bf16: rotary embedding + K/V write + window attention in one kernel
  const float *qkv;       // [R, ldq] fp32 accumulators (q | k | v) lacking 1/rms; read only
  int ldq;
  const float *ss;        // [R] sums of squares for 1/rms; read only
  float eps; int dn;
  const float2 *rope;     // [max_seq][hd/2] (cos, sin) of position * theta^(-2i/hd)
  unsigned int c_magic;   // ceil(2^32 / c): q / c == umulhi(q, c_magic) for the small q used here
  void *kcache, *vcache;  // layer base (the window's own rows are stored through these)
  long long stride_b, stride_h;   // per sequence, per kv head (elements); stride_b == hkv * stride_h
  int k_plane0, v_plane0; // plane (= [max_seq][hd] matrix of one sequence and kv head) of sequence 0, kv head 0 in the
                          // K and the V tensor map: cached tiles are fetched by TMA from plane0 + b * hkv + kvh
  const int32_t *kv_len;
  const int32_t *seq_map; // optional [nb] device: the sequence behind row block i (null: b0 + i)
  int b0, nb, c, hq, hkv;
  int nsplit;             // CTAs (one thread-block cluster, <= 8) per (sequence, kv head, query-tile group)
  int qt;                 // 16-row query tiles per CTA: 1, 2 or 4
  int stages;             // K/V ring stages (set by the launcher)
  int pdl;                // launched as a programmatic dependent of the previous kernel
  unsigned int *err;      // device error word, raised when a bounded wait gives up
  float *out;             // [R, hq*hd] fp32
  // instead of `out`: the result as the bf16 pair high + low in the activation panel [2][pan_rows][hq*hd] that the output
  // projection streams by TMA (more than 16 rows per forward), which then needs no conversion pass of its own
  void *out_pan;
  int pan_rows;
  ZeroList z;
};

struct AcceptArgs {
  int32_t *window;                 // [batch, c] in/out
  const unsigned long long *amax;  // packed argmax per row, or null
  unsigned long long *amax_clear;  // cleared after reading (may be null)
  const int32_t *argmax;           // plain argmax per row (used when amax is null)
  int32_t *kv_len, *n_gen, *done;  // [batch]; done may be null
  int32_t *accepted_count, *accepted_tokens;   // [batch], [batch, c]
  const int32_t *prompt, *prompt_lens;
  int32_t *out_tokens;             // [batch, out_stride] or null
  int out_stride;
  int b0, nb, c, p_stride, refill, pad_id;
  const int32_t *seq_map;          // optional [nb] device: the sequence behind row block i (null: b0 + i); rows of the
                                   // forward (amax / argmax) are indexed by row block, sequence state by sequence
  int max_tokens, eos_id;          // max_tokens <= 0: unlimited
  int commit;                      // 0: leave kv_len / n_gen / window untouched (latency measurement)
  unsigned int *err_inject;        // test aid: when non-null the kernel raises this error word (no wait involved)
};

struct EmbedArgs {
  const int32_t *tokens;   // [R]
  const void *emb;         // [vocab, d]
  float *x;                // [R, d]
  int R, d;
  ZeroList z;
};

// Function attributes (dynamic shared memory opt-in, cluster size) are per device: launchers remember what they
// have set per device ordinal.
constexpr int kMaxDevices = 64;
inline int current_device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) dev = 0;
  return dev % kMaxDevices;
}

// ---- launchers (each returns the cudaError_t of the launch) ----
cudaError_t launch_embed(const EmbedArgs &a, int dtype, cudaStream_t st);
cudaError_t launch_gemm_simt(const GemmArgs &a, int dtype, int pro, int epi, cudaStream_t st);
cudaError_t launch_rope_kv(const RopeArgs &a, int dtype, cudaStream_t st);
cudaError_t launch_attn(const AttnArgs &a, int dtype, int hd, cudaStream_t st);
cudaError_t launch_attn_fused(const KvTensorMap &kmap, const KvTensorMap &vmap, const FusedAttnArgs &a, int hd, cudaStream_t st);
// 3-d tensor map (head_dim, max_seq, planes) over bf16 K or V planes laid out [plane][max_seq][head_dim] from `base`.
cudaError_t make_kv_tensor_map(KvTensorMap *out, const void *base, int hd, int max_seq, long long planes);
// Grid of the fused attention kernel: splits per (sequence, kv head, query-tile group) and query tiles per CTA.
void fused_attn_plan(int max_len, int c, int hq, int hkv, int nb, int hd, int n_sms, int &nsplit, int &qt);
int attn_fused_max_rows();   // most window rows per sequence the fused kernel takes in one launch
cudaError_t launch_accept(const AcceptArgs &a, cudaStream_t st);
// dst[i * c + j] = window[seq_map[i] * c + j]: the token rows of a forward over the sequences seq_map[0 .. nb-1]
cudaError_t launch_gather_rows(int32_t *dst, const int32_t *window, const int32_t *seq_map, int nb, int c, cudaStream_t st);
int attn_tile_keys(int dtype, int hd);   // keys per split tile

// Standalone window attention on caller-supplied scratch (shared by the op-level entry points).
size_t window_attention_scratch_bytes(int batch, int c, int hq, int hkv, int hd, int max_len, int dtype);
int run_window_attention(const void *q, const void *kcache, const void *vcache, const int32_t *kv_len, float *out,
                         int batch, int c, int hq, int hkv, int hd, int max_seq, int max_len, int dtype,
                         void *scratch, size_t scratch_bytes, cudaStream_t st);

// tcgen05 path (bf16 only).  `maps` points at prebuilt tensor maps for the weight matrices.
struct UmmaPlan;
UmmaPlan *umma_plan_create(const GemmArgs &a, int pro, int epi, int n_sms, unsigned int *err_word,
                           char *err, int errlen);
void umma_plan_destroy(UmmaPlan *p);
// x/x2/y/ss pointers and R may differ per launch from those the plan was created with.
// claim: one zeroed word per projection of the launch (the work-claim counters).
// zero (optional): buffers the launch clears at its start, once the previous kernel is complete; only for buffers that
// nothing reads before a later kernel or a phase behind a grid barrier of this launch accumulates into them.
// cta_pairs: with 128-row blocks in panel mode and weight matrices of whole 256-row tiles, run as clusters of two
// CTAs that share a tile (tcgen05 cta_group::2).
cudaError_t launch_gemm_umma(const UmmaPlan *p, const GemmArgs &a, unsigned int *claim, unsigned int *bar_b,
                             const ZeroList *zero, int pdl, cudaStream_t st, int cta_pairs = 0);
// Up to four projections in one launch, each consuming the previous one's reduced output; bar: n-1 zeroed words.
// bar_b: n zeroed words (panel-ready barriers), needed when the rows exceed 16 and the plans have panels.
// sync (optional, used up to 16 rows): how each projection is tied to the others, instead of a grid barrier
// after every one.  wait_bar / sig_bar: index of the grid barrier (word of `bar`) the projection waits on before
// its first activation load / arrives on when done, -1 for none.  td_prod: the projection is claimed tile by tile
// and counts finished chunks per 128-column output tile in counter set td_prod (several projections may feed one
// set: partial sums of the same output); td_cons: it is claimed k range by k range and stages a k-block once the
// tile of set td_cons it reads is complete.  tile_done: zeroed words, td_stride per counter set.
// epi_bar: grid barrier the projection's epilogue warps pass before their first reduction into the output (-1: none);
// needed when the output buffer is still being read by a projection that this one does not otherwise wait for.
struct ChainSync { int wait_bar, sig_bar, td_prod, td_cons, epi_bar; };
constexpr int kChainMax = 6;     // projections in one chained launch
cudaError_t launch_gemm_chain(const UmmaPlan *const *plans, const GemmArgs *args, int n, unsigned int *bar,
                              unsigned int *claim, unsigned int *bar_b, const ChainSync *sync, unsigned int *tile_done,
                              int td_stride, const ZeroList *zero, int pdl, cudaStream_t st, int cta_pairs = 0);

}  // namespace fc
