// C ABI of the Jacobi-window decode library: context, workspace carving, the per-step kernel chain.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "fc_internal.h"

using namespace fc;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

constexpr size_t kGuardBytes = 256;       // canary band between two slices of the workspace
constexpr unsigned char kGuardByte = 0xC5;

struct Carver {          // hands out aligned slices of the caller's workspace (or just counts bytes)
  char *base; size_t off;
  std::vector<size_t> *guards;     // offsets of the canary bands (recorded when non-null)
  template <typename T> T *take(size_t n) {
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off = align_up(off + n * sizeof(T));
    return p;
  }
  void guard() {
    if (guards) guards->push_back(off);
    off += kGuardBytes;
  }
};

constexpr int kPrefillRows = 128;         // rows per forward while a prompt is cached (one 128-row accumulator block)


constexpr int kSyncClaim = kChainMax, kSyncPanel = 2 * kChainMax, kSyncTd = 3 * kChainMax;   // offsets in a group

struct Buffers {
  float *x, *qkv, *attn, *gu, *ss_attn, *ss_ffn, *ss_final, *part_o, *part_ml;
  void *pan;
  float2 *rope;
  void *qb;
  unsigned int *counters, *err, *chain_bar;
  unsigned long long *amax;
  int32_t *window, *kv_len, *n_gen, *done, *acc_count, *acc_tokens, *prompt, *prompt_lens, *out_tokens;
  int32_t *row_tokens;     // tokens of a forward that is not a plain decode step (answer-trigger context; the windows of
                           // the live sequences when finished ones are skipped)
  int32_t *seq_map;        // [max_batch] the live sequences of a compacted step
};

struct Dims {
  int rmax;        // rows of a decode step: max_batch * max_c
  int rows_ws;     // rows the activation buffers hold: a decode step or a prefill block, whichever is larger
  int qd, kvd, ldq, nsplit_max, tk, pan_rows, pan_k, sync_words;
  size_t esz;
};

bool shape_ok(const fc_model_shape *s) {
  if (!s) return false;
  if (s->n_layers < 1 || s->d_model < 8 || s->n_heads < 1 || s->n_kv_heads < 1 || s->d_ffn < 8 || s->vocab < 1) return false;
  if (s->dtype != FC_F32 && s->dtype != FC_BF16) return false;
  if (s->head_dim != 32 && s->head_dim != 64 && s->head_dim != 128) return false;
  if (s->n_heads % s->n_kv_heads) return false;
  if (s->d_model % 8 || s->d_ffn % 8) return false;
  if (s->max_batch < 1 || s->max_c < 1 || s->max_c > 64 || s->max_seq < s->max_c + 1) return false;
  return true;
}

Dims dims_of(const fc_model_shape *s) {
  Dims d;
  d.rmax = s->max_batch * s->max_c;
  d.rows_ws = d.rmax > kPrefillRows ? d.rmax : kPrefillRows;
  d.qd = s->n_heads * s->head_dim;
  d.kvd = s->n_kv_heads * s->head_dim;
  d.ldq = d.qd + 2 * d.kvd;
  d.tk = attn_tile_keys(s->dtype, s->head_dim);
  d.nsplit_max = (s->max_seq + d.tk - 1) / d.tk;
  d.esz = s->dtype == FC_F32 ? 4 : 2;
  // beyond 16 rows the tensor-core projections read their activations from a bf16 high/low panel
  d.pan_rows = (d.rows_ws + 127) / 128 * 128;
  d.pan_k = s->d_model > s->d_ffn ? s->d_model : s->d_ffn;
  if (d.qd > d.pan_k) d.pan_k = d.qd;
  // per-layer group of synchronisation words: grid barriers 0..5, work-claim counters 6..11, panel-ready barriers
  // 12..17, then one completion counter per 128-column tile of the O and of the down projection
  d.sync_words = kSyncTd + 2 * ((s->d_model + 127) / 128);
  d.sync_words = (d.sync_words + 3) / 4 * 4;
  return d;
}

size_t carve(const fc_model_shape *s, char *base, Buffers *b, std::vector<size_t> *guards = nullptr) {
  Dims d = dims_of(s);
  Carver c{base, 0, guards};
  Buffers t;
  const size_t R = d.rows_ws, Rs = d.rmax;
  c.guard();
  t.x = c.take<float>(R * s->d_model); c.guard();
  t.qkv = c.take<float>(R * d.ldq); c.guard();
  t.qb = c.take<char>(R * d.qd * d.esz); c.guard();
  t.attn = c.take<float>(R * d.qd); c.guard();
  t.gu = c.take<float>(R * 2 * (size_t)s->d_ffn); c.guard();
  // sums of squares, then one group of synchronisation words per layer plus one for the first QKV and the LM head:
  // adjacent (no canary band in between) so that one pass clears them all
  t.ss_attn = c.take<float>(R);
  t.ss_ffn = c.take<float>(R);
  t.ss_final = c.take<float>(R);
  t.chain_bar = c.take<unsigned int>(((size_t)s->n_layers + 1) * d.sync_words); c.guard();
  t.pan = c.take<char>((size_t)2 * d.pan_rows * d.pan_k * 2); c.guard();
  t.part_o = c.take<float>(R * s->n_heads * (size_t)d.nsplit_max * s->head_dim); c.guard();
  t.part_ml = c.take<float>(R * s->n_heads * (size_t)d.nsplit_max * 2); c.guard();
  t.rope = c.take<float2>((size_t)s->max_seq * (s->head_dim / 2)); c.guard();
  t.counters = c.take<unsigned int>((size_t)s->max_batch * s->n_kv_heads + 1);   // + one grid-wide word
  t.err = c.take<unsigned int>(1);
  t.amax = c.take<unsigned long long>(Rs); c.guard();
  t.window = c.take<int32_t>(Rs);
  t.kv_len = c.take<int32_t>(s->max_batch);
  t.n_gen = c.take<int32_t>(s->max_batch);
  t.done = c.take<int32_t>(s->max_batch);
  t.acc_count = c.take<int32_t>(s->max_batch);
  t.acc_tokens = c.take<int32_t>(Rs); c.guard();
  t.prompt = c.take<int32_t>((size_t)s->max_batch * s->max_seq);
  t.prompt_lens = c.take<int32_t>(s->max_batch);
  t.out_tokens = c.take<int32_t>((size_t)s->max_batch * s->max_seq);
  t.row_tokens = c.take<int32_t>(R);
  t.seq_map = c.take<int32_t>(s->max_batch); c.guard();
  if (b) *b = t;
  return c.off;
}

__global__ void bump_kernel(int32_t *v, int n) { if (threadIdx.x == 0 && blockIdx.x == 0) *v += n; }

}  // namespace

struct fc_ctx {
  fc_model_shape s;
  Dims d;
  Buffers b;
  // weights (host copies of the pointer tables)
  const void *tok_emb, *g_final, *lm_head;
  const int32_t *bias_perm;
  std::vector<const void *> wq, wk, wv, wo, w_gate, w_up, w_down, g_attn, g_ffn;
  char *kv; size_t kv_layer_stride, kv_half_stride;   // bytes
  cudaStream_t st;
  bool use_umma;
  bool pdl;          // chain the tensor-core kernels by programmatic dependent launch
  bool cta_pairs;    // more than 64 rows: projections as clusters of two CTAs per 256-row weight tile
  bool chain;        // run O -> gate/up -> down -> next layer's QKV as one launch with grid barriers
  bool fused_attn;   // bf16 with head_dim 64/128: rotary embedding and K/V write happen inside the attention kernel
  KvTensorMap kv_map; // TMA view of the whole K/V slab: (head_dim, max_seq, layers * 2 * max_batch * kv heads)
  int n_sms;
  std::vector<UmmaPlan *> plan_qkv, plan_o, plan_gu, plan_down;
  std::vector<UmmaPlan *> plan_gu_half[2], plan_down_half[2];   // the FFN in two halves of d_ffn (chained launch, <= 16 rows)
  bool ffn_split = false;
  UmmaPlan *plan_head = nullptr;
  float *dbg_logits = nullptr;
  // sequence state mirrored on the host
  int batch = 0, c = 0, refill = 0, pad_id = 0, p_stride = 0;
  bool ready = false;
  std::vector<int32_t> kv_len_h, n_gen_h, pending_h, done_h;
  std::vector<std::vector<int32_t>> prompt_h;   // host copies of the prompts (refill rule when the window is resized)
  int gen_max_tokens = 0, gen_eos = -1;
  float ms_prefill = 0.f;        // device time of the most recent fc_prefill
  bool inject_timeout = false;   // test aid: the next step's accept kernel raises the device error word
  char *ws_base = nullptr;
  std::vector<size_t> guards;    // offsets of the canary bands inside the workspace
  // pinned staging: [count | tokens | window | err]
  int32_t *pin = nullptr;
  int32_t *pin_map = nullptr;    // pinned [max_batch]: the live sequences of a compacted step
  int64_t launches = 0;
  char cuda_err[256] = {0};
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  // per-launch profiling (fc_profile_step)
  bool prof = false;
  std::vector<cudaEvent_t> prof_ev;
  std::vector<int> prof_cls;
};

#define FC_CK(call)                                                                      \
  do {                                                                                   \
    cudaError_t e_ = (call);                                                             \
    if (e_ != cudaSuccess) {                                                             \
      snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "%s: %s", #call, cudaGetErrorString(e_)); \
      return FC_ERR_CUDA;                                                                \
    }                                                                                    \
  } while (0)

extern "C" size_t fc_kv_bytes(const fc_model_shape *s) {
  if (!shape_ok(s)) return 0;
  Dims d = dims_of(s);
  return (size_t)s->n_layers * 2 * s->max_batch * s->n_kv_heads * (size_t)s->max_seq * s->head_dim * d.esz;
}

extern "C" size_t fc_workspace_bytes(const fc_model_shape *s) {
  if (!shape_ok(s)) return 0;
  return carve(s, nullptr, nullptr);
}

extern "C" const char *fc_strerror(int st) {
  switch (st) {
    case FC_OK: return "ok";
    case FC_ERR_ARG: return "bad argument";
    case FC_ERR_SHAPE: return "unsupported model shape";
    case FC_ERR_CAPACITY: return "capacity exceeded";
    case FC_ERR_TOKEN_RANGE: return "token id out of range";
    case FC_ERR_STATE: return "no prefilled sequences";
    case FC_ERR_BAD_WINDOW: return "window slot 0 is not the pending exact token";
    case FC_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case FC_ERR_CUDA: return "CUDA error";
    default: return "unknown status";
  }
}

extern "C" const char *fc_last_cuda_error(const fc_ctx *ctx) { return ctx ? ctx->cuda_err : ""; }
extern "C" int64_t fc_last_launch_count(const fc_ctx *ctx) { return ctx ? ctx->launches : 0; }

static void destroy_plans(fc_ctx *ctx) {
  for (auto *v : {&ctx->plan_qkv, &ctx->plan_o, &ctx->plan_gu, &ctx->plan_down, &ctx->plan_gu_half[0], &ctx->plan_gu_half[1],
                  &ctx->plan_down_half[0], &ctx->plan_down_half[1]}) {
    for (UmmaPlan *p : *v) umma_plan_destroy(p);
    v->clear();
  }
  umma_plan_destroy(ctx->plan_head);
  ctx->plan_head = nullptr;
}

extern "C" void fc_destroy(fc_ctx *ctx) {
  if (!ctx) return;
  destroy_plans(ctx);
  if (ctx->pin) cudaFreeHost(ctx->pin);
  if (ctx->pin_map) cudaFreeHost(ctx->pin_map);
  if (ctx->ev0) cudaEventDestroy(ctx->ev0);
  if (ctx->ev1) cudaEventDestroy(ctx->ev1);
  delete ctx;
}

// GEMM argument templates for layer l (buffers filled in; R set per forward)
static GemmArgs args_qkv(const fc_ctx *c, int l) {
  GemmArgs a; memset(&a, 0, sizeof(a));
  a.x = c->b.x; a.ldx = c->s.d_model; a.gain = c->g_attn[l]; a.ss_out = c->b.ss_attn;
  a.eps = c->s.rms_eps; a.dn = c->s.d_model;
  a.w[0] = c->wq[l]; a.w[1] = c->wk[l]; a.w[2] = c->wv[l];
  a.n_rows[0] = c->d.qd; a.n_rows[1] = c->d.kvd; a.n_rows[2] = c->d.kvd;
  a.y_off[0] = 0; a.y_off[1] = c->d.qd; a.y_off[2] = c->d.qd + c->d.kvd;
  a.n_mats = 3; a.y = c->b.qkv; a.ldy = c->d.ldq; a.K = c->s.d_model;
  a.pan = c->d.pan_rows ? c->b.pan : nullptr; a.pan_rows = c->d.pan_rows;
  return a;
}
static GemmArgs args_o(const fc_ctx *c, int l) {
  GemmArgs a; memset(&a, 0, sizeof(a));
  a.x = c->b.attn; a.ldx = c->d.qd; a.eps = c->s.rms_eps; a.dn = c->s.d_model;
  a.w[0] = c->wo[l]; a.n_rows[0] = c->s.d_model; a.n_mats = 1;
  a.y = c->b.x; a.ldy = c->s.d_model; a.K = c->d.qd;
  a.pan = c->d.pan_rows ? c->b.pan : nullptr; a.pan_rows = c->d.pan_rows;
  return a;
}
static GemmArgs args_gu(const fc_ctx *c, int l) {
  GemmArgs a; memset(&a, 0, sizeof(a));
  a.x = c->b.x; a.ldx = c->s.d_model; a.gain = c->g_ffn[l]; a.ss_out = c->b.ss_ffn;
  a.eps = c->s.rms_eps; a.dn = c->s.d_model;
  a.w[0] = c->w_gate[l]; a.w[1] = c->w_up[l];
  a.n_rows[0] = c->s.d_ffn; a.n_rows[1] = c->s.d_ffn; a.y_off[0] = 0; a.y_off[1] = c->s.d_ffn;
  a.n_mats = 2; a.y = c->b.gu; a.ldy = 2 * c->s.d_ffn; a.K = c->s.d_model;
  a.pan = c->d.pan_rows ? c->b.pan : nullptr; a.pan_rows = c->d.pan_rows;
  return a;
}
static GemmArgs args_down(const fc_ctx *c, int l) {
  GemmArgs a; memset(&a, 0, sizeof(a));
  a.x = c->b.gu; a.x2 = c->b.gu + c->s.d_ffn; a.ldx = 2 * c->s.d_ffn; a.ss_in = c->b.ss_ffn;
  a.eps = c->s.rms_eps; a.dn = c->s.d_model;
  a.w[0] = c->w_down[l]; a.n_rows[0] = c->s.d_model; a.n_mats = 1;
  a.y = c->b.x; a.ldy = c->s.d_model; a.K = c->s.d_ffn;
  a.pan = c->d.pan_rows ? c->b.pan : nullptr; a.pan_rows = c->d.pan_rows;
  return a;
}
// Half h of the feed-forward block: gate/up rows (= down columns) h * F/2 .. (h + 1) * F/2.  The two down halves are
// partial sums of the same output; only the first gate/up half accumulates the row sums of squares.
static GemmArgs args_gu_half(const fc_ctx *c, int l, int h) {
  GemmArgs a = args_gu(c, l);
  const int F2 = c->s.d_ffn / 2;
  const size_t off = (size_t)h * F2 * c->s.d_model * c->d.esz;
  a.w[0] = (const char *)c->w_gate[l] + off; a.w[1] = (const char *)c->w_up[l] + off;
  a.n_rows[0] = a.n_rows[1] = F2;
  a.y_off[0] = h * F2; a.y_off[1] = c->s.d_ffn + h * F2;
  if (h) a.ss_out = nullptr;
  a.pan = nullptr; a.pan_rows = 0;
  return a;
}
static GemmArgs args_down_half(const fc_ctx *c, int l, int h) {
  GemmArgs a = args_down(c, l);
  const int F2 = c->s.d_ffn / 2;
  a.x = c->b.gu + (size_t)h * F2; a.x2 = c->b.gu + c->s.d_ffn + (size_t)h * F2;
  a.w[0] = (const char *)c->w_down[l] + (size_t)h * F2 * c->d.esz; a.ldw = c->s.d_ffn;
  a.K = F2;
  a.pan = nullptr; a.pan_rows = 0;
  return a;
}
static GemmArgs args_head(const fc_ctx *c) {
  GemmArgs a; memset(&a, 0, sizeof(a));
  a.x = c->b.x; a.ldx = c->s.d_model; a.gain = c->g_final; a.eps = c->s.rms_eps; a.dn = c->s.d_model;
  a.w[0] = c->lm_head; a.n_rows[0] = c->s.vocab; a.n_mats = 1; a.K = c->s.d_model;
  a.tokens = c->b.window; a.perm = c->s.bias_beta != 0.f ? c->bias_perm : nullptr; a.beta = c->s.bias_beta;
  a.amax = c->b.amax; a.logits = c->dbg_logits; a.vocab = c->s.vocab; a.ldy = c->s.vocab;
  a.ss_out = c->b.ss_final;     // panel mode only: the sums of squares of the final norm
  a.pan = c->d.pan_rows ? c->b.pan : nullptr; a.pan_rows = c->d.pan_rows;
  return a;
}

extern "C" int fc_init(fc_ctx **out, const fc_model_shape *shape, const fc_weights *w, void *kv, size_t kv_bytes,
                       void *ws, size_t ws_bytes, void *cuda_stream) {
  if (!out || !shape || !w || !kv || !ws) return FC_ERR_ARG;
  *out = nullptr;
  if (!shape_ok(shape)) return FC_ERR_SHAPE;
  if (kv_bytes < fc_kv_bytes(shape) || ws_bytes < fc_workspace_bytes(shape)) return FC_ERR_CAPACITY;
  if (((uintptr_t)kv | (uintptr_t)ws) % kAlign) return FC_ERR_ARG;
  if (!w->tok_emb || !w->g_final || !w->lm_head || !w->wq || !w->wk || !w->wv || !w->wo || !w->w_gate ||
      !w->w_up || !w->w_down || !w->g_attn || !w->g_ffn) return FC_ERR_ARG;
  fc_ctx *ctx = new (std::nothrow) fc_ctx();
  if (!ctx) return FC_ERR_ARG;
  ctx->s = *shape;
  ctx->d = dims_of(shape);
  carve(shape, (char *)ws, &ctx->b, &ctx->guards);
  ctx->ws_base = (char *)ws;
  ctx->tok_emb = w->tok_emb; ctx->g_final = w->g_final; ctx->lm_head = w->lm_head; ctx->bias_perm = w->bias_perm;
  const int L = shape->n_layers;
  auto copy = [&](std::vector<const void *> &dst, const void *const *src) { dst.assign(src, src + L); };
  copy(ctx->wq, w->wq); copy(ctx->wk, w->wk); copy(ctx->wv, w->wv); copy(ctx->wo, w->wo);
  copy(ctx->w_gate, w->w_gate); copy(ctx->w_up, w->w_up); copy(ctx->w_down, w->w_down);
  copy(ctx->g_attn, w->g_attn); copy(ctx->g_ffn, w->g_ffn);
  for (int l = 0; l < L; ++l)
    if (!ctx->wq[l] || !ctx->wk[l] || !ctx->wv[l] || !ctx->wo[l] || !ctx->w_gate[l] || !ctx->w_up[l] ||
        !ctx->w_down[l] || !ctx->g_attn[l] || !ctx->g_ffn[l]) { delete ctx; return FC_ERR_ARG; }
  ctx->kv = (char *)kv;
  ctx->kv_half_stride = (size_t)shape->max_batch * shape->n_kv_heads * shape->max_seq * shape->head_dim * ctx->d.esz;
  ctx->kv_layer_stride = 2 * ctx->kv_half_stride;
  ctx->st = (cudaStream_t)cuda_stream;
  ctx->use_umma = shape->dtype == FC_BF16 && !(shape->flags & FC_FLAG_SIMT_GEMM);
  ctx->pdl = !(shape->flags & FC_FLAG_NO_PDL);
  ctx->cta_pairs = !(shape->flags & FC_FLAG_NO_CTA_PAIRS);
  ctx->chain = ctx->use_umma && !(shape->flags & FC_FLAG_NO_CHAIN);
  ctx->fused_attn = shape->dtype == FC_BF16 && (shape->head_dim == 64 || shape->head_dim == 128) &&
                    !(shape->flags & FC_FLAG_SIMT_GEMM);

  int rc = FC_OK;
  auto fail = [&](int code) { fc_destroy(ctx); return code; };
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return fail(FC_ERR_CUDA);
  ctx->n_sms = prop.multiProcessorCount;
  if (ctx->use_umma) {
    if (prop.major != 10) return fail(FC_ERR_SHAPE);
    if (shape->d_model < 64 || shape->d_ffn < 64 || ctx->d.qd < 64) return fail(FC_ERR_SHAPE);
    char msg[200];
    // halves of d_ffn must be whole 128-row tiles (and so whole 64-wide k-blocks of the down projection)
    ctx->ffn_split = ctx->chain && shape->d_ffn % 256 == 0 && !(shape->flags & FC_FLAG_NO_FFN_SPLIT);
    for (int l = 0; l < L && rc == FC_OK; ++l) {
      UmmaPlan *p;
      if (!(p = umma_plan_create(args_qkv(ctx, l), PRO_GAIN, EPI_ATOMIC_ADD, ctx->n_sms, ctx->b.err, msg, sizeof msg))) rc = FC_ERR_CUDA; else ctx->plan_qkv.push_back(p);
      if (rc == FC_OK) { if (!(p = umma_plan_create(args_o(ctx, l), PRO_NONE, EPI_ATOMIC_ADD, ctx->n_sms, ctx->b.err, msg, sizeof msg))) rc = FC_ERR_CUDA; else ctx->plan_o.push_back(p); }
      if (rc == FC_OK) { if (!(p = umma_plan_create(args_gu(ctx, l), PRO_GAIN, EPI_ATOMIC_ADD, ctx->n_sms, ctx->b.err, msg, sizeof msg))) rc = FC_ERR_CUDA; else ctx->plan_gu.push_back(p); }
      if (rc == FC_OK) { if (!(p = umma_plan_create(args_down(ctx, l), PRO_SILU_MUL, EPI_ATOMIC_ADD, ctx->n_sms, ctx->b.err, msg, sizeof msg))) rc = FC_ERR_CUDA; else ctx->plan_down.push_back(p); }
      for (int h = 0; h < 2 && rc == FC_OK && ctx->ffn_split; ++h) {
        if (!(p = umma_plan_create(args_gu_half(ctx, l, h), PRO_GAIN, EPI_ATOMIC_ADD, ctx->n_sms, ctx->b.err, msg, sizeof msg))) rc = FC_ERR_CUDA; else ctx->plan_gu_half[h].push_back(p);
        if (rc == FC_OK) { if (!(p = umma_plan_create(args_down_half(ctx, l, h), PRO_SILU_MUL, EPI_ATOMIC_ADD, ctx->n_sms, ctx->b.err, msg, sizeof msg))) rc = FC_ERR_CUDA; else ctx->plan_down_half[h].push_back(p); }
      }
    }
    if (rc == FC_OK && !(ctx->plan_head = umma_plan_create(args_head(ctx), PRO_GAIN, EPI_ARGMAX, ctx->n_sms, ctx->b.err, msg, sizeof msg))) rc = FC_ERR_CUDA;
    if (rc != FC_OK) { fprintf(stderr, "fc_init: %s\n", msg); return fail(rc); }
  }
  if (ctx->fused_attn &&
      make_kv_tensor_map(&ctx->kv_map, kv, shape->head_dim, shape->max_seq,
                         (long long)L * 2 * shape->max_batch * shape->n_kv_heads) != cudaSuccess) {
    fprintf(stderr, "fc_init: tensor map over the K/V slab could not be encoded\n");
    return fail(FC_ERR_CUDA);
  }
  const size_t pin_ints = (size_t)shape->max_batch * (1 + 2 * shape->max_c) + 4;
  if (cudaMallocHost((void **)&ctx->pin, pin_ints * sizeof(int32_t)) != cudaSuccess) return fail(FC_ERR_CUDA);
  if (cudaMallocHost((void **)&ctx->pin_map, (size_t)shape->max_batch * sizeof(int32_t)) != cudaSuccess) return fail(FC_ERR_CUDA);
  if (cudaEventCreate(&ctx->ev0) != cudaSuccess || cudaEventCreate(&ctx->ev1) != cudaSuccess) return fail(FC_ERR_CUDA);
  if (cudaMemsetAsync(ws, 0, fc_workspace_bytes(shape), ctx->st) != cudaSuccess) return fail(FC_ERR_CUDA);
  for (size_t off : ctx->guards)      // canary bands between the slices (checked by fc_debug_check_guards)
    if (cudaMemsetAsync((char *)ws + off, kGuardByte, kGuardBytes, ctx->st) != cudaSuccess) return fail(FC_ERR_CUDA);
  {
    // cos/sin of pos * theta^(-2i/hd), evaluated on the host in fp32 (inverse frequency in fp32, angle in fp32):
    // the device's powf is a few ulp off, and at positions in the thousands an ulp of the frequency is 1e-4 rad
    // of rotation.
    const int half = shape->head_dim / 2;
    std::vector<float2> table((size_t)shape->max_seq * half);
    std::vector<float> inv_freq(half);
    for (int i = 0; i < half; ++i) inv_freq[i] = powf(shape->rope_theta, -2.0f * (float)i / (float)shape->head_dim);
    for (int pos = 0; pos < shape->max_seq; ++pos)
      for (int i = 0; i < half; ++i) {
        const float ang = (float)pos * inv_freq[i];
        table[(size_t)pos * half + i] = make_float2(cosf(ang), sinf(ang));
      }
    if (cudaMemcpyAsync(ctx->b.rope, table.data(), table.size() * sizeof(float2), cudaMemcpyHostToDevice, ctx->st) != cudaSuccess ||
        cudaStreamSynchronize(ctx->st) != cudaSuccess) return fail(FC_ERR_CUDA);
  }
  if (cudaStreamSynchronize(ctx->st) != cudaSuccess) return fail(FC_ERR_CUDA);
  const int B = shape->max_batch;
  ctx->kv_len_h.assign(B, 0); ctx->n_gen_h.assign(B, 0); ctx->pending_h.assign(B, 0); ctx->done_h.assign(B, 0);
  ctx->prompt_h.assign(B, std::vector<int32_t>());
  *out = ctx;
  return FC_OK;
}

static void prof_mark(fc_ctx *ctx, int cls, bool begin) {
  if (!ctx->prof) return;
  cudaEvent_t e;
  if (cudaEventCreate(&e) != cudaSuccess) return;
  cudaEventRecord(e, ctx->st);
  ctx->prof_ev.push_back(e);
  if (begin) ctx->prof_cls.push_back(cls);
}
struct ProfScope {
  fc_ctx *c; int cls;
  ProfScope(fc_ctx *ctx, int k) : c(ctx), cls(k) { prof_mark(c, cls, true); }
  ~ProfScope() { prof_mark(c, cls, false); }
};

// Work-claim counter of a projection (cleared by the embed kernel at the start of every forward).
enum { GEMM_QKV = -1, GEMM_O = 0, GEMM_GU = 1, GEMM_DOWN = 2, GEMM_HEAD = 3 };
static unsigned int *claim_word(fc_ctx *ctx, int l, int which) {
  const int L = ctx->s.n_layers;
  unsigned int *w = ctx->b.chain_bar;
  const size_t G = ctx->d.sync_words;
  if (which == GEMM_HEAD) return w + (size_t)L * G + kSyncClaim + 1;
  if (which == GEMM_QKV) return l == 0 ? w + (size_t)L * G + kSyncClaim : w + (size_t)(l - 1) * G + kSyncClaim + 3;
  return w + (size_t)l * G + kSyncClaim + which;
}

static cudaError_t run_gemm(fc_ctx *ctx, const UmmaPlan *plan, GemmArgs a, int R, int pro, int epi, int cls,
                            unsigned int *claim, const ZeroList *zero = nullptr) {
  ProfScope ps(ctx, cls);
  a.R = R;
  ++ctx->launches;
  if (ctx->use_umma) return launch_gemm_umma(plan, a, claim, claim + (kSyncPanel - kSyncClaim), zero, ctx->pdl && !ctx->prof, ctx->st, ctx->cta_pairs);   // panel-ready word
  return launch_gemm_simt(a, ctx->s.dtype, pro, epi, ctx->st);
}

// One decoder forward over nb sequences (b0 .. b0+nb-1) with `rows` rows each.  tokens: device [nb*rows].
// with_head: LM head + argmax + accept (a decode step); otherwise the rows are committed (prefill chunk).
// seq_map (device, optional): row block i belongs to sequence seq_map[i] instead of b0 + i (finished sequences skipped).
static int forward(fc_ctx *ctx, int b0, int nb, int rows, const int32_t *tokens, bool with_head, int max_len_host,
                   int commit, const int32_t *seq_map = nullptr) {
  const fc_model_shape &s = ctx->s;
  const Dims &d = ctx->d;
  const int R = nb * rows;
  const size_t Rz = R;
  EmbedArgs ea; memset(&ea, 0, sizeof ea);
  ea.tokens = tokens; ea.emb = ctx->tok_emb; ea.x = ctx->b.x; ea.R = R; ea.d = s.d_model;
  ea.z.p[0] = ctx->b.qkv; ea.z.n[0] = Rz * d.ldq;
  ea.z.p[1] = ctx->b.gu; ea.z.n[1] = Rz * 2 * s.d_ffn;
  // sums of squares (both norms) and the grid-barrier words of the chained projections are adjacent
  ea.z.p[2] = ctx->b.ss_attn;
  ea.z.n[2] = (size_t)((char *)(ctx->b.chain_bar + ((size_t)s.n_layers + 1) * d.sync_words) - (char *)ctx->b.ss_attn) / sizeof(float);
  ++ctx->launches;
  { ProfScope ps(ctx, FC_CLS_EMBED); FC_CK(launch_embed(ea, s.dtype, ctx->st)); }

  const int nsplit = (max_len_host + rows + d.tk - 1) / d.tk;
  const long long stride_h = (long long)s.max_seq * s.head_dim;
  const long long stride_b = (long long)s.n_kv_heads * stride_h;
  const bool chained = ctx->chain;
  const bool o_panel = chained && ctx->fused_attn && R > 16 && ctx->d.pan_rows >= R;
  for (int l = 0; l < s.n_layers; ++l) {
    if (!chained || l == 0)
      FC_CK(run_gemm(ctx, ctx->use_umma ? ctx->plan_qkv[l] : nullptr, args_qkv(ctx, l), R, PRO_GAIN, EPI_ATOMIC_ADD, FC_CLS_QKV, claim_word(ctx, l, GEMM_QKV)));
    void *kc = ctx->kv + (size_t)l * ctx->kv_layer_stride;
    void *vc = ctx->kv + (size_t)l * ctx->kv_layer_stride + ctx->kv_half_stride;
    if (ctx->fused_attn) {
      FusedAttnArgs fa; memset(&fa, 0, sizeof fa);
      fa.qkv = ctx->b.qkv; fa.ldq = d.ldq; fa.ss = ctx->b.ss_attn; fa.eps = s.rms_eps; fa.dn = s.d_model;
      fa.rope = ctx->b.rope; fa.c_magic = (unsigned int)((0x100000000ull + (unsigned)rows - 1) / (unsigned)rows);
      fa.kcache = kc; fa.vcache = vc; fa.stride_b = stride_b; fa.stride_h = stride_h;
      fa.k_plane0 = (l * 2) * s.max_batch * s.n_kv_heads; fa.v_plane0 = (l * 2 + 1) * s.max_batch * s.n_kv_heads;
      fa.kv_len = ctx->b.kv_len; fa.b0 = b0; fa.nb = nb; fa.c = rows; fa.hq = s.n_heads; fa.hkv = s.n_kv_heads;
      fa.seq_map = seq_map;
      fused_attn_plan(max_len_host, rows, s.n_heads, s.n_kv_heads, nb, s.head_dim, ctx->n_sms, fa.nsplit, fa.qt);
      fa.err = ctx->b.err;
      fa.out = ctx->b.attn; fa.pdl = ctx->pdl && !ctx->prof;
      // more than 16 rows: the chained launch streams its activations from the bf16 panel; the attention kernel writes
      // its result there directly, which saves the output projection's conversion pass and two grid-wide waits
      if (o_panel) { fa.out_pan = ctx->b.pan; fa.pan_rows = d.pan_rows; }
      fa.z.p[0] = ctx->b.gu; fa.z.n[0] = Rz * 2 * s.d_ffn;
      fa.z.p[1] = ctx->b.ss_ffn; fa.z.n[1] = Rz;
      ++ctx->launches;
      { ProfScope ps(ctx, FC_CLS_ATTN); FC_CK(launch_attn_fused(ctx->kv_map, ctx->kv_map, fa, s.head_dim, ctx->st)); }
    } else {
      RopeArgs ra; memset(&ra, 0, sizeof ra);
      ra.qkv = ctx->b.qkv; ra.ldq = d.ldq; ra.ss = ctx->b.ss_attn; ra.eps = s.rms_eps; ra.dn = s.d_model;
      ra.kv_len = ctx->b.kv_len; ra.b0 = b0; ra.nb = nb; ra.c = rows; ra.seq_map = seq_map;
      ra.hq = s.n_heads; ra.hkv = s.n_kv_heads; ra.hd = s.head_dim; ra.rope = ctx->b.rope;
      ra.q_out = ctx->b.qb; ra.kcache = kc; ra.vcache = vc;
      ra.stride_b = stride_b; ra.stride_h = stride_h;
      ra.z.p[0] = ctx->b.gu; ra.z.n[0] = Rz * 2 * s.d_ffn;
      ra.z.p[1] = ctx->b.ss_ffn; ra.z.n[1] = Rz;
      ++ctx->launches;
      { ProfScope ps(ctx, FC_CLS_ROPE); FC_CK(launch_rope_kv(ra, s.dtype, ctx->st)); }
      AttnArgs aa; memset(&aa, 0, sizeof aa);
      aa.q = ctx->b.qb; aa.kcache = kc; aa.vcache = vc; aa.stride_b = stride_b; aa.stride_h = stride_h;
      aa.kv_len = ctx->b.kv_len; aa.b0 = b0; aa.nb = nb; aa.c = rows; aa.hq = s.n_heads; aa.hkv = s.n_kv_heads;
      aa.seq_map = seq_map;
      aa.nsplit = nsplit; aa.part_o = ctx->b.part_o; aa.part_ml = ctx->b.part_ml; aa.counters = ctx->b.counters;
      aa.out = ctx->b.attn;
      aa.z.p[0] = ctx->b.ss_attn; aa.z.n[0] = Rz;
      ++ctx->launches;
      { ProfScope ps(ctx, FC_CLS_ATTN); FC_CK(launch_attn(aa, s.dtype, s.head_dim, ctx->st)); }
    }
    // The fused attention kernel only reads the QKV accumulators and the sums of squares of the attention norm; the
    // projection launch that follows it clears them (its next-QKV phase, or the next QKV launch, accumulates again).
    ZeroList zl; memset(&zl, 0, sizeof zl);
    zl.p[0] = ctx->b.qkv; zl.n[0] = Rz * d.ldq;
    zl.p[1] = ctx->b.ss_attn; zl.n[1] = Rz;
    const ZeroList *zero = ctx->fused_attn ? &zl : nullptr;
    if (chained) {
      // O projection, gate/up, down and the next layer's QKV: one persistent launch.
      // Up to 16 rows the phases are tied together without a stall where the data allow it (see ChainSync): gate/up
      // (claimed k range by k range) follows the O projection's finished tiles; the feed-forward block runs in two
      // halves of d_ffn, so that a down half waits only for a gate/up half that finished a whole phase earlier; the
      // next layer's QKV follows the finished tiles of the two down halves' sum.
      const UmmaPlan *plans[kChainMax];
      GemmArgs ga[kChainMax];
      ChainSync sy[kChainMax];
      int n = 0;
      const bool split = ctx->ffn_split && R <= 16;
      plans[n] = ctx->plan_o[l]; ga[n] = args_o(ctx, l); ga[n].pan_ready = o_panel ? 1 : 0; sy[n++] = ChainSync{-1, -1, 0, -1, -1};
      if (split) {
        plans[n] = ctx->plan_gu_half[0][l]; ga[n] = args_gu_half(ctx, l, 0); sy[n++] = ChainSync{-1, 0, -1, 0, -1};
        plans[n] = ctx->plan_gu_half[1][l]; ga[n] = args_gu_half(ctx, l, 1); sy[n++] = ChainSync{-1, 1, -1, 0, -1};
        // the first down half adds to the residual that the second gate/up half may still be reading: its epilogue
        // passes that half's barrier (normally long reached) before the first addition
        plans[n] = ctx->plan_down_half[0][l]; ga[n] = args_down_half(ctx, l, 0); sy[n++] = ChainSync{0, -1, 1, -1, 1};
        plans[n] = ctx->plan_down_half[1][l]; ga[n] = args_down_half(ctx, l, 1); sy[n++] = ChainSync{1, -1, 1, -1, -1};
      } else {
        plans[n] = ctx->plan_gu[l]; ga[n] = args_gu(ctx, l); sy[n++] = ChainSync{-1, 0, -1, 0, -1};
        plans[n] = ctx->plan_down[l]; ga[n] = args_down(ctx, l); sy[n++] = ChainSync{0, -1, 1, -1, -1};
      }
      if (l + 1 < s.n_layers) { plans[n] = ctx->plan_qkv[l + 1]; ga[n] = args_qkv(ctx, l + 1); sy[n++] = ChainSync{-1, -1, -1, 1, -1}; }
      for (int i = 0; i < n; ++i) ga[i].R = R;
      ++ctx->launches;
      ProfScope ps(ctx, FC_CLS_CHAIN);
      unsigned int *grp = ctx->b.chain_bar + (size_t)l * d.sync_words;
      FC_CK(launch_gemm_chain(plans, ga, n, grp, grp + kSyncClaim, grp + kSyncPanel, R <= 16 ? sy : nullptr, grp + kSyncTd,
                              (s.d_model + 127) / 128, zero, ctx->pdl && !ctx->prof, ctx->st, ctx->cta_pairs));
    } else {
      FC_CK(run_gemm(ctx, ctx->use_umma ? ctx->plan_o[l] : nullptr, args_o(ctx, l), R, PRO_NONE, EPI_ATOMIC_ADD, FC_CLS_OPROJ, claim_word(ctx, l, GEMM_O), zero));
      FC_CK(run_gemm(ctx, ctx->use_umma ? ctx->plan_gu[l] : nullptr, args_gu(ctx, l), R, PRO_GAIN, EPI_ATOMIC_ADD, FC_CLS_GATEUP, claim_word(ctx, l, GEMM_GU)));
      FC_CK(run_gemm(ctx, ctx->use_umma ? ctx->plan_down[l] : nullptr, args_down(ctx, l), R, PRO_SILU_MUL, EPI_ATOMIC_ADD, FC_CLS_DOWN, claim_word(ctx, l, GEMM_DOWN)));
    }
  }
  if (with_head) {
    GemmArgs ha = args_head(ctx);
    ha.tokens = tokens;
    FC_CK(run_gemm(ctx, ctx->plan_head, ha, R, PRO_GAIN, EPI_ARGMAX, FC_CLS_HEAD, claim_word(ctx, 0, GEMM_HEAD)));
    AcceptArgs ac; memset(&ac, 0, sizeof ac);
    ac.window = ctx->b.window; ac.amax = ctx->b.amax; ac.amax_clear = ctx->b.amax;
    ac.kv_len = ctx->b.kv_len; ac.n_gen = ctx->b.n_gen; ac.done = ctx->b.done;
    ac.accepted_count = ctx->b.acc_count; ac.accepted_tokens = ctx->b.acc_tokens;
    ac.prompt = ctx->b.prompt; ac.prompt_lens = ctx->b.prompt_lens;
    ac.out_tokens = ctx->b.out_tokens; ac.out_stride = s.max_seq;
    ac.b0 = b0; ac.nb = nb; ac.c = rows; ac.p_stride = s.max_seq; ac.refill = ctx->refill; ac.pad_id = ctx->pad_id;
    ac.seq_map = seq_map;
    ac.max_tokens = ctx->gen_max_tokens; ac.eos_id = ctx->gen_eos; ac.commit = commit;
    if (ctx->inject_timeout) { ac.err_inject = ctx->b.err; ctx->inject_timeout = false; }
    ++ctx->launches;
    { ProfScope ps(ctx, FC_CLS_ACCEPT); FC_CK(launch_accept(ac, ctx->st)); }
  } else {
    for (int b = b0; b < b0 + nb; ++b) {
      ++ctx->launches;
      bump_kernel<<<1, 32, 0, ctx->st>>>(ctx->b.kv_len + b, rows);
      FC_CK(cudaGetLastError());
    }
  }
  return FC_OK;
}

// Rows of one forward while tokens are only cached (prompt, answer-trigger context): what the activation buffers
// hold, and no more than the fused attention kernel takes as one window.
static int block_rows(const fc_ctx *ctx) {
  int r = ctx->d.rows_ws;
  if (ctx->fused_attn && r > attn_fused_max_rows()) r = attn_fused_max_rows();
  return r;
}

static int check_device_error(fc_ctx *ctx) {
  unsigned int e = 0;
  FC_CK(cudaMemcpyAsync(&ctx->pin[0], ctx->b.err, sizeof(e), cudaMemcpyDeviceToHost, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));
  e = (unsigned int)ctx->pin[0];
  if (e) {
    cudaMemsetAsync(ctx->b.err, 0, sizeof(e), ctx->st);
    ctx->ready = false;
    return FC_ERR_DEVICE_TIMEOUT;
  }
  return FC_OK;
}

extern "C" int fc_prefill(fc_ctx *ctx, int32_t batch, const int32_t *prompt_ids, int32_t p_stride,
                          const int32_t *prompt_lens, int32_t c, int32_t refill, int32_t pad_id) {
  if (!ctx || !prompt_ids || !prompt_lens || batch < 1 || c < 1 || p_stride < 1) return FC_ERR_ARG;
  if (refill != FC_REFILL_PROMPT_CYCLE && refill != FC_REFILL_PAD) return FC_ERR_ARG;
  const fc_model_shape &s = ctx->s;
  if (batch > s.max_batch || c > s.max_c) return FC_ERR_CAPACITY;
  if (refill == FC_REFILL_PAD && (pad_id < 0 || pad_id >= s.vocab)) return FC_ERR_TOKEN_RANGE;
  for (int b = 0; b < batch; ++b) {
    const int P = prompt_lens[b];
    if (P < 1 || P > p_stride) return FC_ERR_ARG;
    if (P - 1 + c > s.max_seq) return FC_ERR_CAPACITY;
    for (int i = 0; i < P; ++i) {
      const int t = prompt_ids[(size_t)b * p_stride + i];
      if (t < 0 || t >= s.vocab) return FC_ERR_TOKEN_RANGE;
    }
  }
  ctx->ready = false;
  ctx->launches = 0;
  ctx->batch = batch; ctx->c = c; ctx->refill = refill; ctx->pad_id = pad_id;
  ctx->gen_max_tokens = 0; ctx->gen_eos = -1;
  // device copies of the prompts, zeroed sequence state, initial windows
  std::vector<int32_t> win((size_t)batch * c), zeros(batch, 0);
  for (int b = 0; b < batch; ++b) {
    const int P = prompt_lens[b];
    FC_CK(cudaMemcpyAsync(ctx->b.prompt + (size_t)b * s.max_seq, prompt_ids + (size_t)b * p_stride,
                          sizeof(int32_t) * P, cudaMemcpyHostToDevice, ctx->st));
    win[(size_t)b * c] = prompt_ids[(size_t)b * p_stride + P - 1];
    for (int j = 1; j < c; ++j)
      win[(size_t)b * c + j] = refill == FC_REFILL_PAD ? pad_id : prompt_ids[(size_t)b * p_stride + (j - 1) % P];
    ctx->kv_len_h[b] = 0; ctx->n_gen_h[b] = 0; ctx->done_h[b] = 0; ctx->pending_h[b] = win[(size_t)b * c];
    ctx->prompt_h[b].assign(prompt_ids + (size_t)b * p_stride, prompt_ids + (size_t)b * p_stride + P);
  }
  FC_CK(cudaMemcpyAsync(ctx->b.prompt_lens, prompt_lens, sizeof(int32_t) * batch, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.window, win.data(), sizeof(int32_t) * win.size(), cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.kv_len, zeros.data(), sizeof(int32_t) * batch, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.n_gen, zeros.data(), sizeof(int32_t) * batch, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.done, zeros.data(), sizeof(int32_t) * batch, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));   // host vectors above go out of scope
  // K/V of prompt[0 .. P-2]: one sequence at a time, in blocks of as many rows as the activation buffers hold
  // (at least one 128-row accumulator block, so that a prompt of P ids streams the weights ~P / 128 times)
  FC_CK(cudaEventRecord(ctx->ev0, ctx->st));
  for (int b = 0; b < batch; ++b) {
    const int n = prompt_lens[b] - 1;
    const int blk = block_rows(ctx);
    for (int start = 0; start < n; start += blk) {
      const int rows = n - start < blk ? n - start : blk;
      int rc = forward(ctx, b, 1, rows, ctx->b.prompt + (size_t)b * s.max_seq + start, false, start, 1);
      if (rc != FC_OK) return rc;
    }
    ctx->kv_len_h[b] = n;
  }
  FC_CK(cudaEventRecord(ctx->ev1, ctx->st));
  int rc = check_device_error(ctx);
  if (rc != FC_OK) return rc;
  FC_CK(cudaEventElapsedTime(&ctx->ms_prefill, ctx->ev0, ctx->ev1));
  ctx->ready = true;
  return FC_OK;
}

// Copy (count | tokens | window | err) of the finished step to the host and refresh the host mirrors.
static int collect_step(fc_ctx *ctx, int32_t *accepted_count, int32_t *accepted_tokens, int32_t *window_out) {
  const int B = ctx->batch, c = ctx->c;
  int32_t *p_cnt = ctx->pin, *p_tok = p_cnt + B, *p_win = p_tok + (size_t)B * c, *p_err = p_win + (size_t)B * c;
  FC_CK(cudaMemcpyAsync(p_cnt, ctx->b.acc_count, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, ctx->st));
  FC_CK(cudaMemcpyAsync(p_tok, ctx->b.acc_tokens, sizeof(int32_t) * B * c, cudaMemcpyDeviceToHost, ctx->st));
  FC_CK(cudaMemcpyAsync(p_win, ctx->b.window, sizeof(int32_t) * B * c, cudaMemcpyDeviceToHost, ctx->st));
  FC_CK(cudaMemcpyAsync(p_err, ctx->b.err, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));
  if (*p_err) {
    cudaMemsetAsync(ctx->b.err, 0, sizeof(int32_t), ctx->st);
    ctx->ready = false;
    return FC_ERR_DEVICE_TIMEOUT;
  }
  for (int b = 0; b < B; ++b) {
    if (ctx->done_h[b]) p_cnt[b] = 0;         // skipped by the step: the device word is from its last live step
    const int k = p_cnt[b];
    ctx->kv_len_h[b] += k; ctx->n_gen_h[b] += k; ctx->pending_h[b] = p_win[(size_t)b * c];
    if (k > 0) {
      if (ctx->gen_max_tokens > 0 && ctx->n_gen_h[b] >= ctx->gen_max_tokens) ctx->done_h[b] = 1;
      if (ctx->gen_eos >= 0 && p_tok[(size_t)b * c + k - 1] == ctx->gen_eos) ctx->done_h[b] = 2;   // ended for good
    }
  }
  if (accepted_count) memcpy(accepted_count, p_cnt, sizeof(int32_t) * B);
  if (accepted_tokens) memcpy(accepted_tokens, p_tok, sizeof(int32_t) * B * c);
  if (window_out) memcpy(window_out, p_win, sizeof(int32_t) * B * c);
  return FC_OK;
}

static int max_live_len(const fc_ctx *ctx) {
  int m = 0;
  for (int b = 0; b < ctx->batch; ++b) m = ctx->kv_len_h[b] > m ? ctx->kv_len_h[b] : m;
  return m;
}

// One decode forward over the sequences that are not finished (paper, "Time Analysis": a batch member that is done
// otherwise keeps costing rows of every projection and its attention).  With every sequence live this is the plain
// forward over the windows; otherwise the live sequences' windows are gathered into consecutive rows and the kernels
// that touch per-sequence state (attention, accept) go through a map from row block to sequence.
static int decode_forward(fc_ctx *ctx) {
  const int B = ctx->batch, c = ctx->c;
  int n_live = 0, maxlen = 0;
  for (int b = 0; b < B; ++b)
    if (!ctx->done_h[b]) {
      ctx->pin_map[n_live++] = b;
      maxlen = ctx->kv_len_h[b] > maxlen ? ctx->kv_len_h[b] : maxlen;
    }
  if (n_live == B || n_live == 0) return forward(ctx, 0, B, c, ctx->b.window, true, max_live_len(ctx), 1);
  FC_CK(cudaMemcpyAsync(ctx->b.seq_map, ctx->pin_map, sizeof(int32_t) * n_live, cudaMemcpyHostToDevice, ctx->st));
  ++ctx->launches;
  FC_CK(launch_gather_rows(ctx->b.row_tokens, ctx->b.window, ctx->b.seq_map, n_live, c, ctx->st));
  return forward(ctx, 0, n_live, c, ctx->b.row_tokens, true, maxlen, 1, ctx->b.seq_map);
}

extern "C" int fc_jacobi_step(fc_ctx *ctx, const int32_t *window_in, int32_t *accepted_count,
                              int32_t *accepted_tokens, int32_t *window_out) {
  if (!ctx) return FC_ERR_ARG;
  if (!ctx->ready) return FC_ERR_STATE;
  const int B = ctx->batch, c = ctx->c;
  for (int b = 0; b < B; ++b)
    if (ctx->kv_len_h[b] + c > ctx->s.max_seq) return FC_ERR_CAPACITY;
  if (window_in) {
    for (int b = 0; b < B; ++b) {
      if (window_in[(size_t)b * c] != ctx->pending_h[b]) return FC_ERR_BAD_WINDOW;
      for (int j = 0; j < c; ++j) {
        const int t = window_in[(size_t)b * c + j];
        if (t < 0 || t >= ctx->s.vocab) return FC_ERR_TOKEN_RANGE;
      }
    }
    memcpy(ctx->pin, window_in, sizeof(int32_t) * B * c);
    FC_CK(cudaMemcpyAsync(ctx->b.window, ctx->pin, sizeof(int32_t) * B * c, cudaMemcpyHostToDevice, ctx->st));
  }
  ctx->launches = 0;
  int rc = decode_forward(ctx);
  if (rc != FC_OK) return rc;
  return collect_step(ctx, accepted_count, accepted_tokens, window_out);
}

// Resize every sequence's window to c_new rows: slot 0 (the pending exact token) and the guesses that still fit are
// kept; new slots get the refill rule's guess for their generated index.
static int resize_window(fc_ctx *ctx, int c_new) {
  const int B = ctx->batch, c_old = ctx->c;
  if (c_new == c_old) return FC_OK;
  if (c_new < 1) return FC_ERR_ARG;
  if (c_new > ctx->s.max_c) return FC_ERR_CAPACITY;
  for (int b = 0; b < B; ++b)
    if (ctx->kv_len_h[b] + c_new > ctx->s.max_seq) return FC_ERR_CAPACITY;
  std::vector<int32_t> w_old((size_t)B * c_old), w_new((size_t)B * c_new);
  FC_CK(cudaMemcpyAsync(w_old.data(), ctx->b.window, sizeof(int32_t) * w_old.size(), cudaMemcpyDeviceToHost, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));
  for (int b = 0; b < B; ++b) {
    const std::vector<int32_t> &pr = ctx->prompt_h[b];
    for (int j = 0; j < c_new; ++j) {
      int32_t t;
      if (j < c_old) t = w_old[(size_t)b * c_old + j];
      else if (ctx->refill == FC_REFILL_PAD || pr.empty()) t = ctx->pad_id;
      else t = pr[(size_t)(ctx->n_gen_h[b] + j - 1) % pr.size()];
      w_new[(size_t)b * c_new + j] = t;
    }
  }
  FC_CK(cudaMemcpyAsync(ctx->b.window, w_new.data(), sizeof(int32_t) * w_new.size(), cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));
  ctx->c = c_new;
  return FC_OK;
}

extern "C" int fc_set_window(fc_ctx *ctx, int32_t c) {
  if (!ctx) return FC_ERR_ARG;
  if (!ctx->ready) return FC_ERR_STATE;
  return resize_window(ctx, c);
}

extern "C" int fc_generate(fc_ctx *ctx, int32_t max_tokens, int32_t c, int32_t eos_id, int32_t max_iters,
                           int32_t *out_tokens, int32_t *out_lens, fc_stats *stats) {
  if (!ctx || !out_tokens || !out_lens || max_tokens < 1) return FC_ERR_ARG;
  if (!ctx->ready) return FC_ERR_STATE;
  const int B = ctx->batch;
  if (c > 0 && c != ctx->c) {
    int rc = resize_window(ctx, c);
    if (rc != FC_OK) return rc;
  }
  c = ctx->c;
  for (int b = 0; b < B; ++b)
    if (ctx->kv_len_h[b] + (max_tokens - ctx->n_gen_h[b]) + c > ctx->s.max_seq) return FC_ERR_CAPACITY;
  ctx->gen_max_tokens = max_tokens; ctx->gen_eos = eos_id;
  if (stats) { memset(stats, 0, sizeof(*stats)); stats->ms_prefill = ctx->ms_prefill; }
  std::vector<int32_t> cnt(B), tok((size_t)B * c);
  // A sequence is finished when it has max_tokens tokens or ended on eos_id.  A later call with a larger max_tokens
  // continues the sequences that only ran into the earlier limit: the flags are recomputed here and sent to the device.
  for (int b = 0; b < B; ++b) {
    out_lens[b] = 0;
    const bool hit_eos = ctx->done_h[b] == 2;
    ctx->done_h[b] = hit_eos ? 2 : (ctx->n_gen_h[b] >= max_tokens ? 1 : 0);
    ctx->pin[b] = ctx->done_h[b] ? 1 : 0;
  }
  FC_CK(cudaMemcpyAsync(ctx->b.done, ctx->pin, sizeof(int32_t) * B, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));
  int64_t launches = 0;
  int iters = 0;
  FC_CK(cudaEventRecord(ctx->ev0, ctx->st));
  int rc = FC_OK;
  for (;;) {
    bool live = false;
    for (int b = 0; b < B; ++b) live |= !ctx->done_h[b];
    if (!live) break;
    if (max_iters > 0 && iters >= max_iters) break;       // iteration cap ("Iteration Stop Condition", condition 1)
    ctx->launches = 0;
    rc = decode_forward(ctx);
    if (rc != FC_OK) break;
    launches += ctx->launches;
    rc = collect_step(ctx, cnt.data(), tok.data(), nullptr);
    if (rc != FC_OK) break;
    ++iters;
    for (int b = 0; b < B; ++b) {
      const int k = cnt[b];
      for (int j = 0; j < k && out_lens[b] < max_tokens; ++j) out_tokens[(size_t)b * max_tokens + out_lens[b]++] = tok[(size_t)b * c + j];
      if (stats && k > 0) { stats->accept_hist[k > 64 ? 64 : k]++; stats->tokens += k; }
    }
    if (stats) stats->steps++;
  }
  ctx->launches = launches;
  ctx->gen_max_tokens = 0; ctx->gen_eos = -1;
  if (rc != FC_OK) return rc;
  FC_CK(cudaEventRecord(ctx->ev1, ctx->st));
  FC_CK(cudaEventSynchronize(ctx->ev1));
  if (stats) FC_CK(cudaEventElapsedTime(&stats->ms_steps, ctx->ev0, ctx->ev1));
  return FC_OK;
}

extern "C" int fc_finish_with_trigger(fc_ctx *ctx, const int32_t *trigger_ids, int32_t n_trigger, int32_t max_answer_tokens,
                                      int32_t eos_id, int32_t *answer_tokens, int32_t *answer_lens) {
  if (!ctx || n_trigger < 0 || (n_trigger > 0 && !trigger_ids) || max_answer_tokens < 0 || !answer_lens ||
      (max_answer_tokens > 0 && !answer_tokens)) return FC_ERR_ARG;
  if (!ctx->ready) return FC_ERR_STATE;
  const fc_model_shape &s = ctx->s;
  const int B = ctx->batch, c = ctx->c;
  for (int j = 0; j < n_trigger; ++j)
    if (trigger_ids[j] < 0 || trigger_ids[j] >= s.vocab) return FC_ERR_TOKEN_RANGE;
  const int n_ctx = c + n_trigger;           // rows per sequence: the window (pending exact token + approximate tokens), then the trigger
  for (int b = 0; b < B; ++b)
    if (ctx->kv_len_h[b] + n_ctx + max_answer_tokens > s.max_seq) return FC_ERR_CAPACITY;
  ctx->launches = 0;
  int64_t launches = 0;
  // context rows of every sequence: [window | trigger]
  std::vector<int32_t> win((size_t)B * c), rows_h((size_t)B * n_ctx);
  FC_CK(cudaMemcpyAsync(win.data(), ctx->b.window, sizeof(int32_t) * win.size(), cudaMemcpyDeviceToHost, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));
  for (int b = 0; b < B; ++b) {
    for (int j = 0; j < c; ++j) rows_h[(size_t)b * n_ctx + j] = win[(size_t)b * c + j];
    for (int j = 0; j < n_trigger; ++j) rows_h[(size_t)b * n_ctx + c + j] = trigger_ids[j];
  }
  ctx->ready = false;                        // from here on the Jacobi state is consumed
  // (1) commit K/V of every context row but the last, in blocks of rows; sequences one at a time (ragged lengths)
  const int n_commit = n_ctx - 1;
  for (int b = 0; b < B && n_commit > 0; ++b) {
    const int blk = block_rows(ctx);
    for (int start = 0; start < n_commit; start += blk) {
      const int rows = n_commit - start < blk ? n_commit - start : blk;
      FC_CK(cudaMemcpyAsync(ctx->b.row_tokens, rows_h.data() + (size_t)b * n_ctx + start, sizeof(int32_t) * rows,
                            cudaMemcpyHostToDevice, ctx->st));
      int rc = forward(ctx, b, 1, rows, ctx->b.row_tokens, false, ctx->kv_len_h[b] + start, 1);
      if (rc != FC_OK) return rc;
      FC_CK(cudaStreamSynchronize(ctx->st));   // rows_h / row_tokens are reused by the next block
    }
    ctx->kv_len_h[b] += n_commit;
  }
  launches += ctx->launches;
  // (2) plain greedy decoding (Eq. 1) from the last context row: steps with one row per sequence
  std::vector<int32_t> pend(B), zeros(B, 0);
  for (int b = 0; b < B; ++b) { pend[b] = rows_h[(size_t)b * n_ctx + n_ctx - 1]; answer_lens[b] = 0; }
  FC_CK(cudaMemcpyAsync(ctx->b.window, pend.data(), sizeof(int32_t) * B, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.done, zeros.data(), sizeof(int32_t) * B, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));
  ctx->c = 1; ctx->gen_max_tokens = 0; ctx->gen_eos = -1;
  std::vector<int32_t> cnt(B), tok(B);
  std::vector<char> ended(B, 0);
  for (int i = 0; i < max_answer_tokens; ++i) {
    bool live = false;
    for (int b = 0; b < B; ++b) live |= !ended[b];
    if (!live) break;
    ctx->launches = 0;
    int rc = forward(ctx, 0, B, 1, ctx->b.window, true, max_live_len(ctx), 1);
    if (rc != FC_OK) return rc;
    launches += ctx->launches;
    rc = collect_step(ctx, cnt.data(), tok.data(), nullptr);
    if (rc != FC_OK) return rc;
    for (int b = 0; b < B; ++b) {
      if (ended[b]) continue;
      answer_tokens[(size_t)b * max_answer_tokens + answer_lens[b]++] = tok[b];
      if (eos_id >= 0 && tok[b] == eos_id) ended[b] = 1;
    }
  }
  ctx->launches = launches;
  return check_device_error(ctx);
}

extern "C" int fc_debug_inject_timeout(fc_ctx *ctx) {
  if (!ctx) return FC_ERR_ARG;
  ctx->inject_timeout = true;
  return FC_OK;
}

extern "C" int fc_debug_check_guards(fc_ctx *ctx, int32_t *n_damaged) {
  if (!ctx || !n_damaged) return FC_ERR_ARG;
  *n_damaged = 0;
  std::vector<unsigned char> band(kGuardBytes);
  for (size_t off : ctx->guards) {
    FC_CK(cudaMemcpyAsync(band.data(), ctx->ws_base + off, kGuardBytes, cudaMemcpyDeviceToHost, ctx->st));
    FC_CK(cudaStreamSynchronize(ctx->st));
    for (unsigned char v : band)
      if (v != kGuardByte) { ++*n_damaged; break; }
  }
  return FC_OK;
}

extern "C" int fc_debug_set_state(fc_ctx *ctx, int32_t batch, const int32_t *kv_lens, const int32_t *pending,
                                  int32_t c, int32_t pad_id) {
  if (!ctx || !kv_lens || !pending || batch < 1 || c < 1) return FC_ERR_ARG;
  const fc_model_shape &s = ctx->s;
  if (batch > s.max_batch || c > s.max_c) return FC_ERR_CAPACITY;
  if (pad_id < 0 || pad_id >= s.vocab) return FC_ERR_TOKEN_RANGE;
  for (int b = 0; b < batch; ++b) {
    if (kv_lens[b] < 0 || kv_lens[b] + c > s.max_seq) return FC_ERR_CAPACITY;
    if (pending[b] < 0 || pending[b] >= s.vocab) return FC_ERR_TOKEN_RANGE;
  }
  ctx->ready = false;
  ctx->batch = batch; ctx->c = c; ctx->refill = FC_REFILL_PAD; ctx->pad_id = pad_id;
  ctx->gen_max_tokens = 0; ctx->gen_eos = -1;
  std::vector<int32_t> win((size_t)batch * c, pad_id), zeros(batch, 0), ones(batch, 1);
  for (int b = 0; b < batch; ++b) {
    win[(size_t)b * c] = pending[b];
    ctx->kv_len_h[b] = kv_lens[b]; ctx->n_gen_h[b] = 0; ctx->done_h[b] = 0; ctx->pending_h[b] = pending[b];
  }
  FC_CK(cudaMemcpyAsync(ctx->b.window, win.data(), sizeof(int32_t) * win.size(), cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.kv_len, kv_lens, sizeof(int32_t) * batch, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.n_gen, zeros.data(), sizeof(int32_t) * batch, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.done, zeros.data(), sizeof(int32_t) * batch, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaMemcpyAsync(ctx->b.prompt_lens, ones.data(), sizeof(int32_t) * batch, cudaMemcpyHostToDevice, ctx->st));
  FC_CK(cudaStreamSynchronize(ctx->st));
  ctx->ready = true;
  return FC_OK;
}

extern "C" int fc_debug_logits(fc_ctx *ctx, float *dev_logits) {
  if (!ctx) return FC_ERR_ARG;
  ctx->dbg_logits = dev_logits;
  return FC_OK;
}

extern "C" int fc_get_state(fc_ctx *ctx, int32_t *kv_lens, int32_t *n_gen) {
  if (!ctx) return FC_ERR_ARG;
  if (!ctx->ready) return FC_ERR_STATE;
  for (int b = 0; b < ctx->batch; ++b) {
    if (kv_lens) kv_lens[b] = ctx->kv_len_h[b];
    if (n_gen) n_gen[b] = ctx->n_gen_h[b];
  }
  return FC_OK;
}

extern "C" int fc_bench_steps(fc_ctx *ctx, int32_t n_steps, int32_t commit, float *ms_total, int64_t *tokens_out) {
  if (!ctx || n_steps < 1 || !ms_total) return FC_ERR_ARG;
  if (!ctx->ready) return FC_ERR_STATE;
  const int B = ctx->batch, c = ctx->c;
  const int growth = commit ? n_steps * c : c;
  for (int b = 0; b < B; ++b)
    if (ctx->kv_len_h[b] + growth > ctx->s.max_seq) return FC_ERR_CAPACITY;
  ctx->launches = 0;
  int maxlen = max_live_len(ctx);
  int32_t *p_kv = ctx->pin;
  FC_CK(cudaEventRecord(ctx->ev0, ctx->st));
  for (int i = 0, since = 0; i < n_steps; ++i, ++since) {
    // Committed steps grow each cache by at most c tokens.  The host needs an upper bound on kv_len to size
    // the attention grid, so the bound grows by c per enqueued step and is refreshed from the device every
    // eighth step (one small copy; the steps in between are enqueued without any host round trip).
    if (commit && since == 8) {
      FC_CK(cudaMemcpyAsync(p_kv, ctx->b.kv_len, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, ctx->st));
      FC_CK(cudaStreamSynchronize(ctx->st));
      maxlen = 0;
      for (int b = 0; b < B; ++b) maxlen = p_kv[b] > maxlen ? p_kv[b] : maxlen;
      since = 0;
    }
    int rc = forward(ctx, 0, B, c, ctx->b.window, true, commit ? maxlen + since * c : maxlen, commit ? 1 : 0);
    if (rc != FC_OK) return rc;
  }
  FC_CK(cudaEventRecord(ctx->ev1, ctx->st));
  FC_CK(cudaEventSynchronize(ctx->ev1));
  FC_CK(cudaEventElapsedTime(ms_total, ctx->ev0, ctx->ev1));
  if (tokens_out) *tokens_out = 0;
  if (commit) {
    int32_t *p_ng = p_kv + B, *p_win = p_ng + B;   // pin holds B * (1 + 2c) + 4 ints
    FC_CK(cudaMemcpyAsync(p_kv, ctx->b.kv_len, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, ctx->st));
    FC_CK(cudaMemcpyAsync(p_ng, ctx->b.n_gen, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, ctx->st));
    FC_CK(cudaMemcpyAsync(p_win, ctx->b.window, sizeof(int32_t) * B * c, cudaMemcpyDeviceToHost, ctx->st));
    FC_CK(cudaStreamSynchronize(ctx->st));
    for (int b = 0; b < B; ++b) {
      if (tokens_out) *tokens_out += p_ng[b] - ctx->n_gen_h[b];
      ctx->kv_len_h[b] = p_kv[b]; ctx->n_gen_h[b] = p_ng[b]; ctx->pending_h[b] = p_win[(size_t)b * c];
    }
  }
  return check_device_error(ctx);
}

extern "C" int fc_profile_step(fc_ctx *ctx, float *ms_by_class, int32_t *launches_by_class) {
  if (!ctx || !ms_by_class || !launches_by_class) return FC_ERR_ARG;
  if (!ctx->ready) return FC_ERR_STATE;
  for (int b = 0; b < ctx->batch; ++b)
    if (ctx->kv_len_h[b] + ctx->c > ctx->s.max_seq) return FC_ERR_CAPACITY;
  for (int i = 0; i < FC_N_CLASSES; ++i) { ms_by_class[i] = 0.f; launches_by_class[i] = 0; }
  ctx->prof = true; ctx->prof_ev.clear(); ctx->prof_cls.clear();
  ctx->launches = 0;
  int rc = forward(ctx, 0, ctx->batch, ctx->c, ctx->b.window, true, max_live_len(ctx), 0);
  ctx->prof = false;
  cudaError_t e = cudaStreamSynchronize(ctx->st);
  if (rc == FC_OK && e == cudaSuccess) {
    for (size_t i = 0; i < ctx->prof_cls.size() && 2 * i + 1 < ctx->prof_ev.size(); ++i) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]) == cudaSuccess) {
        ms_by_class[ctx->prof_cls[i]] += ms;
        launches_by_class[ctx->prof_cls[i]] += 1;
      }
    }
  }
  for (cudaEvent_t ev : ctx->prof_ev) cudaEventDestroy(ev);
  ctx->prof_ev.clear(); ctx->prof_cls.clear();
  if (rc != FC_OK) return rc;
  if (e != cudaSuccess) { snprintf(ctx->cuda_err, sizeof ctx->cuda_err, "%s", cudaGetErrorString(e)); return FC_ERR_CUDA; }
  return check_device_error(ctx);
}

// ------------------------------------------------------------------------------------ single operations
static __device__ unsigned int g_op_err[2];   // error word, work-claim counter of fc_op_linear

extern "C" int fc_op_linear(const float *x, const void *w, float *y, int32_t R, int32_t N, int32_t K, int32_t dtype,
                            int32_t use_tensor_cores, void *cuda_stream) {
  if (!x || !w || !y || R < 1 || N < 1 || K < 8 || K % 8) return FC_ERR_ARG;
  if (dtype != FC_F32 && dtype != FC_BF16) return FC_ERR_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  GemmArgs a; memset(&a, 0, sizeof a);
  a.x = x; a.ldx = K; a.w[0] = w; a.n_rows[0] = N; a.n_mats = 1; a.y = y; a.ldy = N; a.R = R; a.K = K;
  a.eps = 1e-5f; a.dn = K;
  if (!use_tensor_cores) {
    if (launch_gemm_simt(a, dtype, PRO_NONE, EPI_ATOMIC_ADD, st) != cudaSuccess) return FC_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? FC_OK : FC_ERR_CUDA;
  }
  if (dtype != FC_BF16 || K < 64 || N % 4 || ((uintptr_t)y % 16)) return FC_ERR_SHAPE;   // 16-byte reductions into y
  int dev = 0, sms = 0;
  unsigned int *err_word = nullptr;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaGetSymbolAddress((void **)&err_word, g_op_err) != cudaSuccess) return FC_ERR_CUDA;
  if (cudaMemsetAsync(err_word, 0, 2 * sizeof(unsigned int), st) != cudaSuccess) return FC_ERR_CUDA;
  char msg[200];
  UmmaPlan *pl = umma_plan_create(a, PRO_NONE, EPI_ATOMIC_ADD, sms, err_word, msg, sizeof msg);
  if (!pl) { fprintf(stderr, "fc_op_linear: %s\n", msg); return FC_ERR_CUDA; }
  cudaError_t e = launch_gemm_umma(pl, a, err_word + 1, nullptr, nullptr, 0, st);
  unsigned int herr = 0;
  if (e == cudaSuccess) e = cudaMemcpyAsync(&herr, err_word, sizeof herr, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  umma_plan_destroy(pl);
  if (e != cudaSuccess) { fprintf(stderr, "fc_op_linear: %s\n", cudaGetErrorString(e)); return FC_ERR_CUDA; }
  return herr ? FC_ERR_DEVICE_TIMEOUT : FC_OK;
}

extern "C" int fc_op_accept(int32_t *window, const int32_t *argmax, int32_t *kv_len, int32_t *n_gen,
                            int32_t *accepted_count, int32_t *accepted_tokens, const int32_t *prompt,
                            const int32_t *prompt_lens, int32_t batch, int32_t c, int32_t p_stride, int32_t refill,
                            int32_t pad_id, void *cuda_stream) {
  if (!window || !argmax || !kv_len || !n_gen || !accepted_count || !accepted_tokens) return FC_ERR_ARG;
  if (batch < 1 || c < 1 || c > 64) return FC_ERR_ARG;
  if (refill == FC_REFILL_PROMPT_CYCLE && (!prompt || !prompt_lens || p_stride < 1)) return FC_ERR_ARG;
  AcceptArgs ac; memset(&ac, 0, sizeof ac);
  ac.window = window; ac.argmax = argmax; ac.kv_len = kv_len; ac.n_gen = n_gen;
  ac.accepted_count = accepted_count; ac.accepted_tokens = accepted_tokens; ac.prompt = prompt; ac.prompt_lens = prompt_lens;
  ac.nb = batch; ac.c = c; ac.p_stride = p_stride; ac.refill = refill; ac.pad_id = pad_id; ac.eos_id = -1; ac.commit = 1;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (launch_accept(ac, st) != cudaSuccess) return FC_ERR_CUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? FC_OK : FC_ERR_CUDA;
}

// ------------------------------------------------------------------------------------ window attention op
namespace fc {
static bool attn_shape_ok(int batch, int c, int hq, int hkv, int hd, int max_len, int dtype) {
  return batch >= 1 && c >= 1 && hq >= 1 && hkv >= 1 && hq % hkv == 0 && (hd == 32 || hd == 64 || hd == 128) &&
         max_len >= 0 && (dtype == FC_F32 || dtype == FC_BF16);
}

size_t window_attention_scratch_bytes(int batch, int c, int hq, int hkv, int hd, int max_len, int dtype) {
  if (!attn_shape_ok(batch, c, hq, hkv, hd, max_len, dtype)) return 0;
  const size_t nsplit = (size_t)(max_len + c + attn_tile_keys(dtype, hd) - 1) / attn_tile_keys(dtype, hd);
  const size_t rows = (size_t)batch * c * hq;
  return align_up(rows * nsplit * hd * sizeof(float)) + align_up(rows * nsplit * 2 * sizeof(float)) +
         align_up((size_t)batch * hkv * sizeof(unsigned int));
}

int run_window_attention(const void *q, const void *kcache, const void *vcache, const int32_t *kv_len, float *out,
                         int batch, int c, int hq, int hkv, int hd, int max_seq, int max_len, int dtype,
                         void *scratch, size_t scratch_bytes, cudaStream_t st) {
  if (!q || !kcache || !vcache || !kv_len || !out || !scratch) return FC_ERR_ARG;
  if (!attn_shape_ok(batch, c, hq, hkv, hd, max_len, dtype)) return FC_ERR_ARG;
  if (max_len + c > max_seq) return FC_ERR_CAPACITY;
  if ((uintptr_t)scratch % kAlign) return FC_ERR_ARG;
  if (scratch_bytes < window_attention_scratch_bytes(batch, c, hq, hkv, hd, max_len, dtype)) return FC_ERR_CAPACITY;
  const int tk = attn_tile_keys(dtype, hd);
  const size_t nsplit = (size_t)(max_len + c + tk - 1) / tk;
  const size_t rows = (size_t)batch * c * hq;
  char *p = (char *)scratch;
  AttnArgs aa; memset(&aa, 0, sizeof aa);
  aa.part_o = (float *)p; p += align_up(rows * nsplit * hd * sizeof(float));
  aa.part_ml = (float *)p; p += align_up(rows * nsplit * 2 * sizeof(float));
  aa.counters = (unsigned int *)p;
  // the arrival counters must start at zero; the partial results are fully overwritten
  if (cudaMemsetAsync(aa.counters, 0, (size_t)batch * hkv * sizeof(unsigned int), st) != cudaSuccess) return FC_ERR_CUDA;
  aa.q = q; aa.kcache = kcache; aa.vcache = vcache;
  aa.stride_h = (long long)max_seq * hd; aa.stride_b = (long long)hkv * aa.stride_h;
  aa.kv_len = kv_len; aa.b0 = 0; aa.nb = batch; aa.c = c; aa.hq = hq; aa.hkv = hkv;
  aa.nsplit = (int)nsplit; aa.out = out;
  if (launch_attn(aa, dtype, hd, st) != cudaSuccess) return FC_ERR_CUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? FC_OK : FC_ERR_CUDA;
}

// ---- the fused kernel of the bf16 step (1/rms + rotary embedding + K/V write + window attention) as one operation
static bool fused_shape_ok(int batch, int c, int hq, int hkv, int hd, int max_seq, int max_len) {
  return batch >= 1 && c >= 1 && c <= attn_fused_max_rows() && hq >= 1 && hkv >= 1 && hq % hkv == 0 &&
         (hd == 64 || hd == 128) && max_len >= 0 && max_seq >= 1;
}
static void fused_layout(int hd, int max_seq, size_t off[3]) {
  off[0] = 0;                                                                   // rope table
  off[1] = off[0] + align_up((size_t)max_seq * (hd / 2) * sizeof(float2));      // error word
  off[2] = off[1] + align_up(sizeof(unsigned int));                             // end
}
}  // namespace fc

extern "C" size_t fc_op_fused_window_attention_scratch_bytes(int32_t batch, int32_t c, int32_t n_heads, int32_t n_kv_heads,
                                                             int32_t head_dim, int32_t max_seq, int32_t max_len) {
  if (!fused_shape_ok(batch, c, n_heads, n_kv_heads, head_dim, max_seq, max_len)) return 0;
  size_t off[3];
  fused_layout(head_dim, max_seq, off);
  return off[2];
}

extern "C" int fc_op_fused_window_attention(float *qkv_acc, float *sumsq, float rms_eps, int32_t d_norm, float rope_theta,
                                            void *kcache, void *vcache, const int32_t *kv_len, float *out, int32_t batch,
                                            int32_t c, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                                            int32_t max_seq, int32_t max_len, int32_t n_splits, int32_t q_tiles,
                                            void *scratch, size_t scratch_bytes, void *cuda_stream) {
  if (!qkv_acc || !sumsq || !kcache || !vcache || !kv_len || !out || !scratch || d_norm < 1 || n_splits < 0 || n_splits > 8) return FC_ERR_ARG;
  if (q_tiles != 0 && q_tiles != 1 && q_tiles != 2 && q_tiles != 4) return FC_ERR_ARG;
  if (!fused_shape_ok(batch, c, n_heads, n_kv_heads, head_dim, max_seq, max_len)) return FC_ERR_ARG;
  if (max_len + c > max_seq) return FC_ERR_CAPACITY;
  if ((uintptr_t)scratch % kAlign || ((uintptr_t)kcache | (uintptr_t)vcache) % 16) return FC_ERR_ARG;
  size_t off[3];
  fused_layout(head_dim, max_seq, off);
  if (scratch_bytes < off[2]) return FC_ERR_CAPACITY;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char *base = (char *)scratch;
  // rotary table exactly as fc_init builds it
  const int half = head_dim / 2;
  std::vector<float2> table((size_t)max_seq * half);
  for (int i = 0; i < half; ++i) {
    const float inv_freq = powf(rope_theta, -2.0f * (float)i / (float)head_dim);
    for (int pos = 0; pos < max_seq; ++pos) {
      const float ang = (float)pos * inv_freq;
      table[(size_t)pos * half + i] = make_float2(cosf(ang), sinf(ang));
    }
  }
  if (cudaMemcpyAsync(base + off[0], table.data(), table.size() * sizeof(float2), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemsetAsync(base + off[1], 0, off[2] - off[1], st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return FC_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return FC_ERR_CUDA;
  KvTensorMap kmap, vmap;
  const long long planes = (long long)batch * n_kv_heads;
  if (make_kv_tensor_map(&kmap, kcache, head_dim, max_seq, planes) != cudaSuccess ||
      make_kv_tensor_map(&vmap, vcache, head_dim, max_seq, planes) != cudaSuccess) return FC_ERR_CUDA;
  FusedAttnArgs fa; memset(&fa, 0, sizeof fa);
  fa.qkv = qkv_acc; fa.ldq = (n_heads + 2 * n_kv_heads) * head_dim; fa.ss = sumsq; fa.eps = rms_eps; fa.dn = d_norm;
  fa.rope = (const float2 *)(base + off[0]);
  fa.c_magic = (unsigned int)((0x100000000ull + (unsigned)c - 1) / (unsigned)c);
  fa.kcache = kcache; fa.vcache = vcache;
  fa.stride_h = (long long)max_seq * head_dim; fa.stride_b = (long long)n_kv_heads * fa.stride_h;
  fa.k_plane0 = 0; fa.v_plane0 = 0;
  fa.kv_len = kv_len; fa.b0 = 0; fa.nb = batch; fa.c = c; fa.hq = n_heads; fa.hkv = n_kv_heads;
  fused_attn_plan(max_len, c, n_heads, n_kv_heads, batch, head_dim, sms, fa.nsplit, fa.qt);
  if (n_splits > 0) fa.nsplit = n_splits;
  if (q_tiles > 0) fa.qt = q_tiles;
  fa.err = (unsigned int *)(base + off[1]);
  fa.out = out; fa.pdl = 0;
  if (launch_attn_fused(kmap, vmap, fa, head_dim, st) != cudaSuccess) return FC_ERR_CUDA;
  // inside a step the projection launch that follows clears the accumulators; here the call does it
  unsigned int herr = 0;
  if (cudaMemsetAsync(qkv_acc, 0, (size_t)batch * c * fa.ldq * sizeof(float), st) != cudaSuccess ||
      cudaMemsetAsync(sumsq, 0, (size_t)batch * c * sizeof(float), st) != cudaSuccess ||
      cudaMemcpyAsync(&herr, fa.err, sizeof herr, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) return FC_ERR_CUDA;
  return herr ? FC_ERR_DEVICE_TIMEOUT : FC_OK;
}

extern "C" size_t fc_op_window_attention_scratch_bytes(int32_t batch, int32_t c, int32_t n_heads, int32_t n_kv_heads,
                                                       int32_t head_dim, int32_t max_len, int32_t dtype) {
  return window_attention_scratch_bytes(batch, c, n_heads, n_kv_heads, head_dim, max_len, dtype);
}

extern "C" int fc_op_window_attention(const void *q, const void *kcache, const void *vcache, const int32_t *kv_len,
                                      float *out, int32_t batch, int32_t c, int32_t n_heads, int32_t n_kv_heads,
                                      int32_t head_dim, int32_t max_seq, int32_t max_len, int32_t dtype,
                                      void *scratch, size_t scratch_bytes, void *cuda_stream) {
  return run_window_attention(q, kcache, vcache, kv_len, out, batch, c, n_heads, n_kv_heads, head_dim, max_seq,
                              max_len, dtype, scratch, scratch_bytes, (cudaStream_t)cuda_stream);
}
