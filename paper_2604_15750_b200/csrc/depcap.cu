// C ABI and step scheduler of the DepCap block-step library.
//
// The scheduler turns one dc_step into a fixed sequence of kernel launches on the context's
// stream; it never synchronises (except in dc_step_profiled) and never touches the outputs on
// an argument error.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <string>
#include <vector>

#include "kernels.h"
#include "tc.h"

using namespace dc;

namespace {

thread_local std::string g_create_error = "";

struct Profiler : dc::StageHook {
  bool on = false;
  struct Span { int stage; cudaEvent_t a, b; };
  std::vector<Span> spans;
  std::vector<cudaEvent_t> pool;
  size_t used = 0;
  int launches[DC_STAGE_COUNT] = {};
  cudaStream_t s = nullptr;
  cudaEvent_t get() {
    if (used == pool.size()) {
      cudaEvent_t e;
      cudaEventCreate(&e);
      pool.push_back(e);
    }
    return pool[used++];
  }
  void begin(int stage, int n_launch) override {
    launches[stage] += n_launch;
    if (!on) return;
    Span sp{stage, get(), get()};
    cudaEventRecord(sp.a, s);
    spans.push_back(sp);
  }
  void end() override {
    if (!on) return;
    cudaEventRecord(spans.back().b, s);
  }
  void reset(bool enable, cudaStream_t st) {
    on = enable; s = st; used = 0; spans.clear();
    memset(launches, 0, sizeof(launches));
  }
  ~Profiler() { for (auto e : pool) cudaEventDestroy(e); }
};

}  // namespace

void dc::set_thread_error(const char* msg) { g_create_error = msg ? msg : ""; }

struct dc_ctx {
  dc_config cfg{};
  Hyper hp{};
  cudaStream_t stream = nullptr;
  int device = 0;
  bool bf16 = false;
  bool use_tc = false;  // tensor-core kernels for the transformer layers
  bool tc_lm = false;   // tensor-core LM head fused with the streaming softmax statistics
  const void *embed = nullptr, *final_norm = nullptr, *lm_head = nullptr;
  std::vector<const void*> wq, wk, wv, wo, w_gate, w_up, w_down, norm1, norm2;
  std::vector<const void*> bq, bk, bv;   // q / k / v projection biases (cfg.qkv_bias), else empty
  // capacities
  int R_cap_max = 0, M_max = 0, Mlm_max = 0;
  // workspace (device)
  std::vector<void*> allocs;
  float* x = nullptr;        // residual stream [M, d] fp32
  void* a = nullptr;         // normed activations [M, d]
  void* q = nullptr;         // [M, nq*hd] rotated
  void* k = nullptr;         // [M, nkv*hd] rotated
  void* v = nullptr;         // [M, nkv*hd]
  void* o = nullptr;         // attention output [M, nq*hd]
  void* act = nullptr;       // SwiGLU output [M, F]
  float* tmp = nullptr;      // fp32 GEMM outputs of the CUDA-core path
  void* h = nullptr;         // LM-head input [M_lm, d]
  float* logits = nullptr;   // [M_lm, V] fp32, CUDA-core LM head only
  float* cos_sin = nullptr;  // RoPE table [max_batch * R_cap_max + 1, hd] (last row: angle step)
  int32_t* ws_pred = nullptr;
  float *ws_conf = nullptr, *ws_ent = nullptr, *ws_infl = nullptr, *ws_lse = nullptr;
  TcState* tc = nullptr;
  // workspace of dc_generate: window / last-block ids, step and selection outputs, counters
  int32_t *g_win = nullptr, *g_last = nullptr, *g_pred = nullptr, *g_blk = nullptr, *g_cnt = nullptr,
          *g_idx = nullptr, *g_rem = nullptr, *g_status = nullptr;
  float *g_conf = nullptr, *g_xlogp = nullptr;
  char *g_hout = nullptr, *g_carry = nullptr;   // LM-head rows of a boundary step / kept for the next one
  uint8_t* g_mask = nullptr;
  int32_t* g_host = nullptr;   // pinned: what a generation step reads back (block_len, remaining, status, window ids)
  SeqMeta last_meta{};
  bool have_logits = false;
  Profiler prof;
  std::string err;
};

namespace {

int fail(dc_ctx* c, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  if (c) c->err = buf; else g_create_error = buf;
  return code;
}

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

template <typename T>
T* ws_alloc(dc_ctx* c, size_t n, bool* ok) {
  void* p = nullptr;
  if (n == 0) n = 1;
  if (cudaMalloc(&p, n * sizeof(T)) != cudaSuccess) {
    *ok = false;
    cudaGetLastError();
    return nullptr;
  }
  c->allocs.push_back(p);
  return reinterpret_cast<T*>(p);
}

int build_meta(dc_ctx* c, int batch, int flags, const int32_t* ctx_len, const int32_t* last_len,
               const int32_t* win_len, const int32_t* remain_len, SeqMeta* m,
               bool no_window = false) {
  const dc_config& g = c->cfg;
  if (batch < 1 || batch > g.max_batch)
    return fail(c, DC_ERR_SHAPE, "batch %d outside [1, max_batch=%d]", batch, g.max_batch);
  memset(m, 0, sizeof(*m));
  m->batch = batch;
  m->nv = (flags & DC_STEP_INFLUENCE) ? 2 : 1;
  int maxR = 0, maxW = 0;
  for (int b = 0; b < batch; ++b) {
    const int P = ctx_len ? ctx_len[b] : 0, Lb = last_len ? last_len[b] : 0;
    const int W = no_window ? 0 : win_len[b];
    if (P < 0 || P > g.max_ctx)
      return fail(c, DC_ERR_SHAPE, "ctx_len[%d]=%d outside [0, max_ctx=%d]", b, P, g.max_ctx);
    if (Lb < 0 || Lb > g.max_last)
      return fail(c, DC_ERR_SHAPE, "last_len[%d]=%d outside [0, max_last=%d]", b, Lb, g.max_last);
    if (!no_window && (W < 1 || W > g.max_window))
      return fail(c, DC_ERR_SHAPE, "win_len[%d]=%d outside [1, max_window=%d]", b, W,
                  g.max_window);
    m->ctx_len[b] = P; m->last_len[b] = Lb; m->win_len[b] = W;
    m->pos0[b] = P;   // active rows sit right behind the cached context
    m->remain[b] = remain_len ? remain_len[b] : W;
    m->have_prev[b] = (m->nv == 2 && Lb > 0) ? 1 : 0;
    maxR = maxR > Lb + W ? maxR : Lb + W;
    maxW = maxW > W ? maxW : W;
  }
  m->R_cap = round_up(maxR, 16);
  m->W_cap = round_up(maxW, 16);
  const int npos = batch * m->W_cap;
  const int gmax = 128 / m->nv;  // an LM-head group is [G curr rows ; G prev rows] <= 128 rows
  m->G = npos < gmax ? npos : gmax;
  if (m->G < 1) m->G = 1;   // no window rows (prefill): the LM head does not run
  m->npos_pad = round_up(npos, m->G);
  return DC_OK;
}

// The meta the LM-head stage sees when p_prev is carried in: two variants of LM rows over a stack
// that ran one.
SeqMeta carried_meta(const SeqMeta& m, const int32_t* prev_len) {
  SeqMeta ml = m;
  ml.nv = 2;
  const int npos = m.batch * m.W_cap, gmax = 64;
  ml.G = npos < gmax ? npos : gmax;
  if (ml.G < 1) ml.G = 1;
  ml.npos_pad = round_up(npos, ml.G);
  for (int b = 0; b < m.batch; ++b) ml.have_prev[b] = prev_len[b] > 0 ? 1 : 0;
  return ml;
}

#define DC_CHECK_LAUNCH(c)                                                                   \
  do {                                                                                       \
    cudaError_t e_ = cudaGetLastError();                                                     \
    if (e_ != cudaSuccess)                                                                   \
      return fail(c, DC_ERR_CUDA, "CUDA error after launch (%s:%d): %s", __FILE__, __LINE__, \
                  cudaGetErrorString(e_));                                                   \
  } while (0)

template <typename T>
int run_step(dc_ctx* c, const dc_step_in* in, const dc_step_out* out, const SeqMeta& m,
             const bool kv_only = false) {
  const dc_config& g = c->cfg;
  cudaStream_t s = c->stream;
  Profiler& pf = c->prof;
  const int d = g.d_model, nq = g.n_q_heads, nkv = g.n_kv_heads, hd = g.head_dim, F = g.d_ff;
  const int M = m.nv * m.batch * m.R_cap;
  const bool carried = (in->flags & DC_STEP_CARRIED_PREV) != 0;
  const SeqMeta ml = carried ? carried_meta(m, in->prev_len) : m;   // what the LM-head stage sees
  const int Mlm = ml.nv * ml.npos_pad;
  const int nqkv = (nq + 2 * nkv) * hd;
  T* a = (T*)c->a; T* q = (T*)c->q; T* k = (T*)c->k; T* v = (T*)c->v; T* o = (T*)c->o;
  T* act = (T*)c->act; T* h = (T*)c->h;
  const size_t k_layer = (size_t)g.max_batch * nkv * g.max_ctx * hd;

  cudaMemsetAsync(out->status, 0, sizeof(int32_t) * m.batch, s);
  pf.begin(DC_STAGE_EMBED, 2);
  launch_embed<T>((const T*)c->embed, in->last_ids, in->win_ids, g.max_last, g.max_window,
                  g.mask_id, g.vocab, d, m, c->x, out->status, s);
  launch_rope_table(m, hd, g.rope_theta, c->cos_sin, s);
  pf.end();
  DC_CHECK_LAUNCH(c);

  // split-K partial sums produced by the previous residual GEMM, folded in by the next norm
  const float* part = nullptr;
  int nsplit = 0;
  size_t part_stride = 0;

  const bool export_kv = (in->flags & DC_STEP_EXPORT_KV) != 0;
  const bool chain = c->use_tc && tc_chain_ok(c->tc, m);
  if (c->use_tc) tc_step_begin(c->tc);
  if (chain) {
    // persistent dense chain: norm1 + QKV of layer 0, then per layer attention and one launch
    // that runs O projection .. QKV of the next layer
    const int L = g.n_layers;
    pf.begin(DC_STAGE_DENSE, 1);
    int rc = tc_chain(c->tc, 0, 0, CH_NORM1, CH_END, m, c->x, (const __nv_bfloat16*)a, c->cos_sin,
                      nullptr, (const __nv_bfloat16*)c->norm1[0], 0, &part, &nsplit, &part_stride);
    pf.end();
    if (rc != DC_OK) return fail(c, rc, "dense chain failed: %s", tc_error(c->tc));
    for (int l = 0; l < L; ++l) {
      if (export_kv) tc_export_kv(c->tc, l, m, (__nv_bfloat16*)in->k_cache, (__nv_bfloat16*)in->v_cache);
      if (kv_only && l + 1 == L) break;   // prefill: nothing after the last layer's K / V is used
      pf.begin(DC_STAGE_ATTN, 1);
      rc = tc_attention(c->tc, l, m, (const __nv_bfloat16*)in->k_cache,
                        (const __nv_bfloat16*)in->v_cache);
      pf.end();
      if (rc != DC_OK) return fail(c, rc, "attention failed: %s", tc_error(c->tc));
      const bool last = l + 1 == L;
      pf.begin(DC_STAGE_DENSE, 1);
      rc = tc_chain(c->tc, l, l + 1, CH_OPROJ, last ? CH_NORM1 : CH_END, m, c->x,
                    (const __nv_bfloat16*)a, c->cos_sin, (const __nv_bfloat16*)c->norm2[l],
                    last ? nullptr : (const __nv_bfloat16*)c->norm1[l + 1], nsplit, &part, &nsplit,
                    &part_stride);
      pf.end();
      if (rc != DC_OK) return fail(c, rc, "dense chain failed: %s", tc_error(c->tc));
    }
    DC_CHECK_LAUNCH(c);
  }

  for (int l = 0; l < g.n_layers && !chain; ++l) {
    pf.begin(DC_STAGE_NORM, 1);
    launch_rmsnorm<T>(c->x, part, nsplit, part_stride, (const T*)c->norm1[l], g.rms_eps, M, d, a, s);
    pf.end();
    part = nullptr; nsplit = 0;
    const T* kc = in->k_cache ? (const T*)in->k_cache + (size_t)l * k_layer : nullptr;
    const T* vc = in->v_cache ? (const T*)in->v_cache + (size_t)l * k_layer : nullptr;
    if (c->use_tc) {
      int rc = tc_layer(c->tc, l, m, c->x, (const __nv_bfloat16*)a,
                        (const __nv_bfloat16*)in->k_cache, (const __nv_bfloat16*)in->v_cache,
                        c->cos_sin, (const __nv_bfloat16*)c->norm2[l],
                        &part, &nsplit, &part_stride, pf, export_kv, kv_only && l + 1 == g.n_layers);
      if (rc != DC_OK) return fail(c, rc, "tensor-core layer %d failed: %s", l, tc_error(c->tc));
      continue;
    }
    pf.begin(DC_STAGE_QKV, 4);
    launch_gemm_simt<T>(a, (const T*)c->wq[l], c->tmp, M, nq * hd, d, nqkv, EPI_STORE_F32, s);
    launch_gemm_simt<T>(a, (const T*)c->wk[l], c->tmp + nq * hd, M, nkv * hd, d, nqkv,
                        EPI_STORE_F32, s);
    launch_gemm_simt<T>(a, (const T*)c->wv[l], c->tmp + (nq + nkv) * hd, M, nkv * hd, d, nqkv,
                        EPI_STORE_F32, s);
    launch_rope_store<T>(c->tmp, c->cos_sin, m, nq, nkv, hd,
                         c->bq.empty() ? nullptr : (const T*)c->bq[l], c->bq.empty() ? nullptr : (const T*)c->bk[l],
                         c->bq.empty() ? nullptr : (const T*)c->bv[l], q, k, v, s);
    pf.end();
    if (export_kv)
      launch_export_kv<T>(k, v, 0, m, nkv, hd, g.max_ctx, (T*)in->k_cache + (size_t)l * k_layer,
                          (T*)in->v_cache + (size_t)l * k_layer, s);
    if (kv_only && l + 1 == g.n_layers) break;
    pf.begin(DC_STAGE_ATTN, 1);
    launch_attn_simt<T>(q, k, v, kc, vc, g.max_ctx, m, nq, nkv, hd, o, s);
    pf.end();
    pf.begin(DC_STAGE_OPROJ, 1);
    launch_gemm_simt<T>(o, (const T*)c->wo[l], c->x, M, d, nq * hd, d, EPI_ADD_F32, s);
    pf.end();
    pf.begin(DC_STAGE_NORM, 1);
    launch_rmsnorm<T>(c->x, nullptr, 0, 0, (const T*)c->norm2[l], g.rms_eps, M, d, a, s);
    pf.end();
    pf.begin(DC_STAGE_GATEUP, 3);
    launch_gemm_simt<T>(a, (const T*)c->w_gate[l], c->tmp, M, F, d, 2 * F, EPI_STORE_F32, s);
    launch_gemm_simt<T>(a, (const T*)c->w_up[l], c->tmp + F, M, F, d, 2 * F, EPI_STORE_F32, s);
    launch_swiglu<T>(c->tmp, M, F, act, s);
    pf.end();
    pf.begin(DC_STAGE_DOWN, 1);
    launch_gemm_simt<T>(act, (const T*)c->w_down[l], c->x, M, d, F, d, EPI_ADD_F32, s);
    pf.end();
    DC_CHECK_LAUNCH(c);
  }

  if (kv_only) {
    if (c->use_tc) tc_flush_status(c->tc, out->status, m.batch);
    DC_CHECK_LAUNCH(c);
    return DC_OK;
  }
  pf.begin(DC_STAGE_NORM, in->h_final_in ? 2 : 1);
  launch_final_norm<T>(c->x, part, nsplit, part_stride, (const T*)c->final_norm, g.rms_eps, d, ml,
                       h, s, m.nv);
  if (carried || out->h_out) {
    PrevLen pl{};
    if (carried) for (int b = 0; b < m.batch; ++b) pl.n[b] = in->prev_len[b];
    launch_carry<T>(carried ? (const T*)in->h_prev_in : nullptr, pl, (T*)out->h_out, g.max_window, d,
                    ml, h, s);
  }
  if (in->h_final_in) launch_h_override<T>((const T*)in->h_final_in, g.max_window, d, ml, h, s);
  pf.end();

  SignalOut so{out->pred_id, out->conf, out->entropy, out->influence, out->lse, g.max_window};
  if (c->tc_lm) {
    pf.begin(DC_STAGE_LMHEAD, 2);
    int rc = tc_lmhead(c->tc, ml, (const __nv_bfloat16*)h, g.mask_id, g.forbid_mask_pred,
                       c->ws_pred, c->ws_conf, c->ws_ent, c->ws_infl, c->ws_lse, so, out->status);
    pf.end();
    if (rc != DC_OK) return fail(c, rc, "tensor-core LM head failed: %s", tc_error(c->tc));
    c->have_logits = false;
  } else {
    pf.begin(DC_STAGE_LMHEAD, 2);
    launch_gemm_simt<T>(h, (const T*)c->lm_head, c->logits, Mlm, g.vocab, d, g.vocab,
                        EPI_STORE_F32, s);
    launch_signals_from_logits(c->logits, g.vocab, g.mask_id, g.forbid_mask_pred, ml, c->ws_pred,
                               c->ws_conf, c->ws_ent, c->ws_infl, c->ws_lse, so, out->status, s);
    pf.end();
    c->have_logits = true;
  }
  if (out->xlogp) {
    pf.begin(DC_STAGE_XLOGP, 1);
    launch_xlogp<T>(h, (const T*)c->lm_head, c->ws_pred, c->ws_lse, d, g.vocab, ml, g.max_window,
                    out->xlogp, s);
    pf.end();
  }
  if ((in->flags & DC_STEP_BOUNDARY) && out->block_len) {
    pf.begin(DC_STAGE_BOUNDARY, 1);
    launch_boundary(c->ws_infl, c->ws_ent, ml.W_cap, ml, c->hp, g.max_window, out->score,
                    out->cum_influence, out->cum_score, out->block_len, s);
    pf.end();
  }
  if (c->use_tc) tc_flush_status(c->tc, out->status, m.batch);
  DC_CHECK_LAUNCH(c);
  c->last_meta = ml;
  return DC_OK;
}

int validate_step(dc_ctx* c, const dc_step_in* in, const dc_step_out* out, SeqMeta* m) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!in || !out) return fail(c, DC_ERR_INVALID_ARG, "null in/out");
  if (!out->status) return fail(c, DC_ERR_INVALID_ARG, "out->status is required");
  if (!in->win_ids || !in->win_len) return fail(c, DC_ERR_INVALID_ARG, "win_ids/win_len null");
  if (in->flags & ~(DC_STEP_INFLUENCE | DC_STEP_BOUNDARY | DC_STEP_EXPORT_KV | DC_STEP_CARRIED_PREV))
    return fail(c, DC_ERR_INVALID_ARG, "unknown flag bits 0x%x", in->flags);
  if (in->flags & DC_STEP_CARRIED_PREV) {
    if (in->flags & DC_STEP_INFLUENCE)
      return fail(c, DC_ERR_INVALID_ARG, "DC_STEP_CARRIED_PREV and DC_STEP_INFLUENCE exclude each other");
    if (!in->h_prev_in || !in->prev_len)
      return fail(c, DC_ERR_INVALID_ARG, "DC_STEP_CARRIED_PREV needs h_prev_in and prev_len");
    for (int b = 0; b < in->batch && b < c->cfg.max_batch; ++b)
      if (in->prev_len[b] < 0 || in->prev_len[b] > in->win_len[b])
        return fail(c, DC_ERR_SHAPE, "prev_len[%d]=%d outside [0, win_len=%d]", b, in->prev_len[b],
                    in->win_len[b]);
  }
  int rc = build_meta(c, in->batch, in->flags, in->ctx_len, in->last_len, in->win_len,
                      in->remain_len, m);
  if (rc != DC_OK) return rc;
  if (in->pos0)
    for (int b = 0; b < m->batch; ++b) {
      if (in->pos0[b] < 0) return fail(c, DC_ERR_INVALID_ARG, "pos0[%d] negative", b);
      m->pos0[b] = in->pos0[b];
    }
  bool any_ctx = false, any_last = false;
  for (int b = 0; b < m->batch; ++b) {
    any_ctx |= m->ctx_len[b] > 0;
    any_last |= m->last_len[b] > 0;
  }
  if (any_ctx && (!in->k_cache || !in->v_cache))
    return fail(c, DC_ERR_INVALID_ARG, "ctx_len > 0 but k_cache/v_cache null");
  if (any_last && !in->last_ids) return fail(c, DC_ERR_INVALID_ARG, "last_len > 0 but last_ids null");
  if ((in->flags & DC_STEP_EXPORT_KV) && any_last) {
    if (!in->k_cache || !in->v_cache)
      return fail(c, DC_ERR_INVALID_ARG, "DC_STEP_EXPORT_KV needs k_cache / v_cache");
    for (int b = 0; b < m->batch; ++b)
      if (m->ctx_len[b] + m->last_len[b] > c->cfg.max_ctx)
        return fail(c, DC_ERR_SHAPE, "ctx_len[%d] + last_len[%d] = %d exceeds max_ctx=%d", b, b,
                    m->ctx_len[b] + m->last_len[b], c->cfg.max_ctx);
  }
  return DC_OK;
}

int do_step(dc_ctx* c, const dc_step_in* in, const dc_step_out* out, bool profile,
            float* stage_ms, int32_t* stage_launches) {
  SeqMeta m;
  int rc = validate_step(c, in, out, &m);
  if (rc != DC_OK) return rc;
  int dev = -1;
  cudaGetDevice(&dev);
  if (dev != c->device) cudaSetDevice(c->device);
  c->prof.reset(profile, c->stream);
  rc = c->bf16 ? run_step<__nv_bfloat16>(c, in, out, m) : run_step<float>(c, in, out, m);
  if (profile) {
    cudaError_t e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess && rc == DC_OK)
      rc = fail(c, DC_ERR_CUDA, "stream sync failed: %s", cudaGetErrorString(e));
    for (int i = 0; i < DC_STAGE_COUNT; ++i) {
      stage_ms[i] = 0.f;
      if (stage_launches) stage_launches[i] = c->prof.launches[i];
    }
    if (e == cudaSuccess)
      for (auto& sp : c->prof.spans) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, sp.a, sp.b);
        stage_ms[sp.stage] += ms;
      }
    c->prof.on = false;
  }
  if (dev != c->device && dev >= 0) cudaSetDevice(dev);
  return rc;
}

}  // namespace

extern "C" {

int dc_create(const dc_config* cfg, const dc_weights* w, void* cuda_stream, dc_ctx** out) {
  if (!cfg || !w || !out) return fail(nullptr, DC_ERR_INVALID_ARG, "null argument");
  *out = nullptr;
  const dc_config& g = *cfg;
  if (g.n_layers < 0 || g.d_model < 1 || g.n_q_heads < 1 || g.n_kv_heads < 1 || g.head_dim < 2 ||
      g.d_ff < 1 || g.vocab < 2)
    return fail(nullptr, DC_ERR_INVALID_ARG, "non-positive model dimension");
  if (g.head_dim % 2) return fail(nullptr, DC_ERR_INVALID_ARG, "head_dim must be even");
  if (g.d_model % 4) return fail(nullptr, DC_ERR_UNSUPPORTED, "d_model must be a multiple of 4");
  if (g.n_q_heads % g.n_kv_heads)
    return fail(nullptr, DC_ERR_INVALID_ARG, "n_q_heads must be a multiple of n_kv_heads");
  if (g.mask_id < 0 || g.mask_id >= g.vocab)
    return fail(nullptr, DC_ERR_INVALID_ARG, "mask_id outside the vocabulary");
  if (g.dtype != DC_F32 && g.dtype != DC_BF16) return fail(nullptr, DC_ERR_INVALID_ARG, "dtype");
  if (g.max_batch < 1 || g.max_batch > DC_MAX_BATCH)
    return fail(nullptr, DC_ERR_INVALID_ARG, "max_batch outside [1, %d]", DC_MAX_BATCH);
  if (g.max_window < 16 || g.max_window > DC_MAX_WINDOW || g.max_window % 16)
    return fail(nullptr, DC_ERR_INVALID_ARG, "max_window must be a multiple of 16 in [16, %d]",
                DC_MAX_WINDOW);
  if (g.max_ctx < 0 || g.max_ctx % 64)
    return fail(nullptr, DC_ERR_INVALID_ARG, "max_ctx must be a non-negative multiple of 64");
  if (g.max_last < 0) return fail(nullptr, DC_ERR_INVALID_ARG, "max_last negative");
  if (g.L_min < 1 || g.L_max < 1 || g.smooth_radius < 0 || g.smooth_radius > 8)
    return fail(nullptr, DC_ERR_INVALID_ARG, "L_min/L_max/smooth_radius out of range");
  if (g.norm_mode < 0 || g.norm_mode > 2 || g.boundary_mode < 0 || g.boundary_mode > 1 ||
      g.cap_mode < 0 || g.cap_mode > 1 || g.impl < 0 || g.impl > 1)
    return fail(nullptr, DC_ERR_INVALID_ARG, "bad mode selector");
  if (!w->embed || !w->final_norm || !w->lm_head)
    return fail(nullptr, DC_ERR_INVALID_ARG, "null embed/final_norm/lm_head");
  if (g.n_layers > 0 && (!w->wq || !w->wk || !w->wv || !w->wo || !w->w_gate || !w->w_up ||
                         !w->w_down || !w->norm1 || !w->norm2))
    return fail(nullptr, DC_ERR_INVALID_ARG, "null per-layer weight array");
  if (g.qkv_bias != 0 && g.qkv_bias != 1) return fail(nullptr, DC_ERR_INVALID_ARG, "qkv_bias must be 0 or 1");
  if (g.qkv_bias && g.n_layers > 0) {
    if (!w->bq || !w->bk || !w->bv) return fail(nullptr, DC_ERR_INVALID_ARG, "qkv_bias set but bq / bk / bv null");
    for (int l = 0; l < g.n_layers; ++l)
      if (!w->bq[l] || !w->bk[l] || !w->bv[l])
        return fail(nullptr, DC_ERR_INVALID_ARG, "null bias pointer in layer %d", l);
  }
  for (int l = 0; l < g.n_layers; ++l)
    if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->w_gate[l] || !w->w_up[l] ||
        !w->w_down[l] || !w->norm1[l] || !w->norm2[l])
      return fail(nullptr, DC_ERR_INVALID_ARG, "null weight pointer in layer %d", l);

  dc_ctx* c = new dc_ctx();
  c->cfg = g;
  c->hp = Hyper{g.lambda, g.L_min, g.L_max, g.tau_low, g.tau_high, g.gamma,
                g.smooth_radius, g.norm_mode, g.boundary_mode, g.cap_mode};
  c->stream = (cudaStream_t)cuda_stream;
  if (cudaGetDevice(&c->device) != cudaSuccess) {
    delete c;
    cudaGetLastError();
    return fail(nullptr, DC_ERR_CUDA, "no current CUDA device");
  }
  c->bf16 = g.dtype == DC_BF16;
  c->embed = w->embed; c->final_norm = w->final_norm; c->lm_head = w->lm_head;
  auto cp = [&](std::vector<const void*>& dst, const void* const* src) {
    dst.assign(src, src + g.n_layers);
  };
  if (g.n_layers > 0) {
    cp(c->wq, w->wq); cp(c->wk, w->wk); cp(c->wv, w->wv); cp(c->wo, w->wo);
    cp(c->w_gate, w->w_gate); cp(c->w_up, w->w_up); cp(c->w_down, w->w_down);
    cp(c->norm1, w->norm1); cp(c->norm2, w->norm2);
    if (g.qkv_bias) { cp(c->bq, w->bq); cp(c->bk, w->bk); cp(c->bv, w->bv); }
  }
  c->use_tc = g.impl == DC_IMPL_AUTO && tc_supported(g);
  c->tc_lm = c->use_tc && tc_has_lmhead(g);
  const size_t es = c->bf16 ? 2 : 4;
  c->R_cap_max = round_up(g.max_last + g.max_window, 16);
  c->M_max = 2 * g.max_batch * c->R_cap_max;
  const int npos_max = round_up(g.max_batch * g.max_window, 128);
  c->Mlm_max = 2 * npos_max;
  const size_t M = c->M_max;
  const int nq = g.n_q_heads, nkv = g.n_kv_heads, hd = g.head_dim;
  bool ok = true;
  c->x = ws_alloc<float>(c, M * g.d_model, &ok);
  c->a = ws_alloc<char>(c, M * g.d_model * es, &ok);
  c->h = ws_alloc<char>(c, (size_t)c->Mlm_max * g.d_model * es, &ok);
  c->cos_sin = ws_alloc<float>(c, ((size_t)g.max_batch * c->R_cap_max + 1) * hd, &ok);
  const size_t nw = (size_t)g.max_batch * g.max_window;
  c->ws_pred = ws_alloc<int32_t>(c, nw, &ok);
  c->ws_conf = ws_alloc<float>(c, nw, &ok);
  c->ws_ent = ws_alloc<float>(c, nw, &ok);
  c->ws_infl = ws_alloc<float>(c, nw, &ok);
  c->ws_lse = ws_alloc<float>(c, nw, &ok);
  {
    const size_t nww = nw * g.max_window;
    c->g_win = ws_alloc<int32_t>(c, nw, &ok);
    c->g_last = ws_alloc<int32_t>(c, (size_t)g.max_batch * (g.max_last > 0 ? g.max_last : 1), &ok);
    c->g_pred = ws_alloc<int32_t>(c, nw, &ok);
    c->g_conf = ws_alloc<float>(c, nw, &ok);
    c->g_xlogp = ws_alloc<float>(c, nww, &ok);
    c->g_mask = ws_alloc<uint8_t>(c, nw, &ok);
    c->g_idx = ws_alloc<int32_t>(c, nw, &ok);
    c->g_blk = ws_alloc<int32_t>(c, g.max_batch, &ok);
    c->g_cnt = ws_alloc<int32_t>(c, g.max_batch, &ok);
    c->g_rem = ws_alloc<int32_t>(c, g.max_batch, &ok);
    c->g_status = ws_alloc<int32_t>(c, g.max_batch, &ok);
    const size_t hbytes = nw * g.d_model * (g.dtype == DC_BF16 ? 2 : 4);
    c->g_hout = ws_alloc<char>(c, hbytes, &ok);
    c->g_carry = ws_alloc<char>(c, hbytes, &ok);
  }
  if (c->use_tc) {
    int rc = tc_create(g, c->stream, c->M_max, c->Mlm_max, c->wq, c->wk, c->wv, c->wo, c->w_gate,
                       c->w_up, c->w_down, c->lm_head, (const __nv_bfloat16*)c->h, &c->tc);
    if (rc != DC_OK) {
      std::string why = c->tc ? tc_error(c->tc) : "tensor-core state allocation failed";
      dc_destroy(c);
      return fail(nullptr, rc, "%s", why.c_str());
    }
    if (g.qkv_bias) tc_set_qkv_bias(c->tc, c->bq, c->bk, c->bv);
  } else {
    c->q = ws_alloc<char>(c, M * nq * hd * es, &ok);
    c->k = ws_alloc<char>(c, M * nkv * hd * es, &ok);
    c->v = ws_alloc<char>(c, M * nkv * hd * es, &ok);
    c->o = ws_alloc<char>(c, M * nq * hd * es, &ok);
    c->act = ws_alloc<char>(c, M * g.d_ff * es, &ok);
    const size_t tmp_cols = (size_t)((nq + 2 * nkv) * hd > 2 * g.d_ff ? (nq + 2 * nkv) * hd
                                                                      : 2 * g.d_ff);
    c->tmp = ws_alloc<float>(c, M * tmp_cols, &ok);
  }
  if (!c->tc_lm) c->logits = ws_alloc<float>(c, (size_t)c->Mlm_max * g.vocab, &ok);
  if (!ok) {
    dc_destroy(c);
    return fail(nullptr, DC_ERR_NOMEM, "workspace allocation failed");
  }
  *out = c;
  return DC_OK;
}

int dc_step(dc_ctx* c, const dc_step_in* in, const dc_step_out* out) {
  return do_step(c, in, out, false, nullptr, nullptr);
}

int dc_step_profiled(dc_ctx* c, const dc_step_in* in, const dc_step_out* out, float* stage_ms,
                     int32_t* stage_launches) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!stage_ms) return fail(c, DC_ERR_INVALID_ARG, "stage_ms null");
  return do_step(c, in, out, true, stage_ms, stage_launches);
}

int dc_boundary(dc_ctx* c, const dc_boundary_in* in, const dc_boundary_out* out) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!in || !out || !in->influence || !in->entropy || !in->win_len || !out->block_len)
    return fail(c, DC_ERR_INVALID_ARG, "null argument");
  SeqMeta m;
  int rc = build_meta(c, in->batch, 0, nullptr, nullptr, in->win_len, in->remain_len, &m);
  if (rc != DC_OK) return rc;
  for (int b = 0; b < m.batch; ++b) m.have_prev[b] = in->have_prev ? (in->have_prev[b] != 0) : 1;
  launch_boundary(in->influence, in->entropy, c->cfg.max_window, m, c->hp, c->cfg.max_window,
                  out->score, out->cum_influence, out->cum_score, out->block_len, c->stream);
  DC_CHECK_LAUNCH(c);
  return DC_OK;
}

int dc_select(dc_ctx* c, const dc_select_in* in, const dc_select_out* out) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!in || !out || !in->conf || !in->win_ids || !in->xlogp || !in->block_len || !in->win_len)
    return fail(c, DC_ERR_INVALID_ARG, "null argument");
  if (!out->sel_mask && !out->sel_idx && !out->sel_count)
    return fail(c, DC_ERR_INVALID_ARG, "no output requested");
  SeqMeta m;
  int rc = build_meta(c, in->batch, 0, nullptr, nullptr, in->win_len, nullptr, &m);
  if (rc != DC_OK) return rc;
  Hyper hp = c->hp;
  if (in->override_thresholds) {
    hp.tau_low = in->tau_low; hp.tau_high = in->tau_high; hp.gamma = in->gamma;
  }
  launch_select(in->conf, in->win_ids, in->xlogp, in->block_len, m, hp, c->cfg.mask_id,
                c->cfg.max_window, out->sel_mask, out->sel_idx, out->sel_count, c->stream);
  DC_CHECK_LAUNCH(c);
  return DC_OK;
}

int dc_boundary_batched(dc_ctx* c, int32_t batch, const float* influence, const float* entropy,
                        const int32_t* win_len, const int32_t* remain_len, const int32_t* have_prev,
                        const dc_boundary_out* out) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!influence || !entropy || !win_len || !remain_len || !out || !out->block_len || batch < 1)
    return fail(c, DC_ERR_INVALID_ARG, "null argument or batch < 1");
  DevLens dl;
  dl.win_len = win_len; dl.remain = remain_len; dl.have_prev = have_prev;
  if (!have_prev) {   // all 1: any non-zero array of the right length serves; win_len >= 1 everywhere
    dl.have_prev = win_len;
  }
  launch_boundary_dev(influence, entropy, c->cfg.max_window, batch, dl, c->hp, c->cfg.max_window,
                      out->score, out->cum_influence, out->cum_score, out->block_len, c->stream);
  DC_CHECK_LAUNCH(c);
  return DC_OK;
}

int dc_select_batched(dc_ctx* c, int32_t batch, const float* conf, const int32_t* win_ids,
                      const float* xlogp, const int32_t* block_len, const int32_t* win_len,
                      const dc_select_out* out) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!conf || !win_ids || !xlogp || !block_len || !win_len || !out || batch < 1)
    return fail(c, DC_ERR_INVALID_ARG, "null argument or batch < 1");
  if (!out->sel_mask && !out->sel_idx && !out->sel_count)
    return fail(c, DC_ERR_INVALID_ARG, "no output requested");
  DevLens dl;
  dl.win_len = win_len;
  launch_select_dev(conf, win_ids, xlogp, block_len, batch, dl, c->hp, c->cfg.mask_id, c->cfg.max_window,
                    out->sel_mask, out->sel_idx, out->sel_count, c->stream);
  DC_CHECK_LAUNCH(c);
  return DC_OK;
}

int dc_prefill(dc_ctx* c, const dc_prefill_in* in, const dc_prefill_out* out) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!in || !out || !in->ids || !in->n_ids || !in->k_cache || !in->v_cache || !out->status)
    return fail(c, DC_ERR_INVALID_ARG, "null argument");
  SeqMeta m;
  int rc = build_meta(c, in->batch, 0, in->ctx_len, in->n_ids, nullptr, nullptr, &m, true);
  if (rc != DC_OK) return rc;
  for (int b = 0; b < m.batch; ++b) {
    if (m.last_len[b] < 1) return fail(c, DC_ERR_SHAPE, "n_ids[%d] must be positive", b);
    if (m.ctx_len[b] + m.last_len[b] > c->cfg.max_ctx)
      return fail(c, DC_ERR_SHAPE, "ctx_len[%d] + n_ids[%d] = %d exceeds max_ctx=%d", b, b,
                  m.ctx_len[b] + m.last_len[b], c->cfg.max_ctx);
  }
  if (in->pos0)   // the tokens' positions are not the cache slots (suffix rows of a dual cache)
    for (int b = 0; b < m.batch; ++b) {
      if (in->pos0[b] < 0) return fail(c, DC_ERR_INVALID_ARG, "pos0[%d] negative", b);
      m.pos0[b] = in->pos0[b];
    }
  dc_step_in si{};
  si.batch = in->batch; si.flags = DC_STEP_EXPORT_KV;
  si.k_cache = in->k_cache; si.v_cache = in->v_cache; si.ctx_len = in->ctx_len;
  si.last_ids = in->ids; si.last_len = in->n_ids;
  si.win_ids = c->g_win;       // never read: no sequence has window rows
  dc_step_out so{};
  so.status = out->status;
  int dev = -1;
  cudaGetDevice(&dev);
  if (dev != c->device) cudaSetDevice(c->device);
  c->prof.reset(false, c->stream);
  rc = c->bf16 ? run_step<__nv_bfloat16>(c, &si, &so, m, true) : run_step<float>(c, &si, &so, m, true);
  if (dev != c->device && dev >= 0) cudaSetDevice(dev);
  return rc;
}

int dc_commit(dc_ctx* c, const dc_commit_in* in, const dc_commit_out* out) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!in || !in->win_ids || !in->pred_id || !in->sel_mask || !in->block_len || !in->win_len)
    return fail(c, DC_ERR_INVALID_ARG, "null argument");
  SeqMeta m;
  int rc = build_meta(c, in->batch, 0, nullptr, nullptr, in->win_len, nullptr, &m);
  if (rc != DC_OK) return rc;
  launch_commit(in->win_ids, in->pred_id, in->sel_mask, in->block_len, m, c->cfg.mask_id,
                c->cfg.max_window, out ? out->remaining : nullptr, c->stream);
  DC_CHECK_LAUNCH(c);
  return DC_OK;
}

int dc_generate(dc_ctx* c, const dc_generate_in* in, const dc_generate_out* out) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!in || !out || !in->ctx_len || !out->tokens || !out->nfe)
    return fail(c, DC_ERR_INVALID_ARG, "null argument");
  const dc_config& g = c->cfg;
  const int B = in->batch, N = in->gen_len, MW = g.max_window;
  if (B < 1 || B > g.max_batch) return fail(c, DC_ERR_SHAPE, "batch %d outside [1, max_batch=%d]", B, g.max_batch);
  if (N < 1) return fail(c, DC_ERR_INVALID_ARG, "gen_len must be positive");
  const int Lw_cap = g.L_max < MW ? g.L_max : MW;       // window positions a boundary step looks at
  if (g.max_last < Lw_cap) return fail(c, DC_ERR_SHAPE, "max_last=%d cannot hold a block of %d", g.max_last, Lw_cap);
  for (int b = 0; b < B; ++b) {
    if (in->ctx_len[b] < 0 || in->ctx_len[b] + N > g.max_ctx)
      return fail(c, DC_ERR_SHAPE, "ctx_len[%d] + gen_len = %d exceeds max_ctx=%d", b, in->ctx_len[b] + N, g.max_ctx);
  }
  if ((!in->k_cache || !in->v_cache)) return fail(c, DC_ERR_INVALID_ARG, "k_cache / v_cache null");
  const int max_steps = in->max_steps > 0 ? in->max_steps : 4 * N;

  struct Seq { int cache, done, blk, last_len, nblocks, carry; };   // cache: keys in the cache; done: tokens decoded; carry: rows kept for p_prev
  const bool carried = in->carried_prev != 0;
  const size_t row_bytes = (size_t)g.d_model * (c->bf16 ? 2 : 4);
  std::vector<int32_t> h_prevlen(B);
  std::vector<Seq> sq(B);
  std::vector<int32_t> h_ctx(B), h_lastlen(B), h_winlen(B), h_remain(B);
  std::vector<int32_t> h_win((size_t)B * MW), h_last((size_t)B * (g.max_last > 0 ? g.max_last : 1));
  if (!c->g_host && cudaMallocHost(reinterpret_cast<void**>(&c->g_host),
                                   sizeof(int32_t) * (size_t)g.max_batch * (3 + MW)) != cudaSuccess) {
    cudaGetLastError();
    c->g_host = nullptr;
    return fail(c, DC_ERR_NOMEM, "pinned staging buffer of dc_generate");
  }
  // one read-back per forward: [block_len | remaining | status | window ids], then one wait
  int32_t *h_blk = c->g_host, *h_rem = h_blk + g.max_batch, *h_status = h_rem + g.max_batch,
          *h_ids = h_status + g.max_batch;
  for (int b = 0; b < B; ++b) sq[b] = Seq{in->ctx_len[b], 0, 0, 0, 0, 0};
  if (out->block_lens) memset(out->block_lens, 0, sizeof(int32_t) * (size_t)B * N);
  cudaStream_t s = c->stream;
  int nfe = 0;
  // device time of the forwards (optional): one pair of events, read after each forward's wait
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  double dev_ms = 0.0;
  if (out->device_ms && (cudaEventCreate(&ev0) != cudaSuccess || cudaEventCreate(&ev1) != cudaSuccess)) {
    if (ev0) cudaEventDestroy(ev0);
    return fail(c, DC_ERR_CUDA, "event creation failed in dc_generate");
  }
  struct EvGuard { cudaEvent_t &a, &b; ~EvGuard() { if (a) cudaEventDestroy(a); if (b) cudaEventDestroy(b); } } ev_guard{ev0, ev1};
  while (true) {
    bool any_open = false, any_boundary = false;
    for (int b = 0; b < B; ++b) {
      any_open |= sq[b].done < N;
      any_boundary |= sq[b].done < N && sq[b].blk == 0;
    }
    if (!any_open) break;
    if (nfe >= max_steps) { *out->nfe = nfe; return fail(c, DC_ERR_TIMEOUT, "max_steps=%d reached", max_steps); }
    if (ev0) cudaEventRecord(ev0, s);
    // ---- inputs of this step
    for (int b = 0; b < B; ++b) {
      Seq& q = sq[b];
      h_ctx[b] = q.cache;
      h_remain[b] = N - q.done > 0 ? N - q.done : 1;
      if (q.done >= N) {                       // finished: a dummy window of one masked position
        h_lastlen[b] = 0; h_winlen[b] = 1; h_win[(size_t)b * MW] = g.mask_id;
      } else if (q.blk == 0) {                 // boundary step: all of the look-ahead window masked
        const int W = (N - q.done) < Lw_cap ? (N - q.done) : Lw_cap;
        h_lastlen[b] = q.last_len; h_winlen[b] = W;
        h_prevlen[b] = q.carry < W ? q.carry : W;
        for (int i = 0; i < W; ++i) h_win[(size_t)b * MW + i] = g.mask_id;
      } else {                                 // denoising step inside the block: ids live on the device
        h_lastlen[b] = 0; h_winlen[b] = q.blk;
      }
    }
    for (int b = 0; b < B; ++b)
      if (sq[b].done >= N || sq[b].blk == 0)
        cudaMemcpyAsync(c->g_win + (size_t)b * MW, h_win.data() + (size_t)b * MW, sizeof(int32_t) * h_winlen[b],
                        cudaMemcpyHostToDevice, s);
    if (any_boundary)
      cudaMemcpyAsync(c->g_last, h_last.data(), sizeof(int32_t) * h_last.size(), cudaMemcpyHostToDevice, s);
    dc_step_in si{};
    si.batch = B;
    si.flags = any_boundary ? ((carried ? DC_STEP_CARRIED_PREV : DC_STEP_INFLUENCE) | DC_STEP_BOUNDARY |
                               DC_STEP_EXPORT_KV) : 0;
    if (any_boundary && carried) {
      for (int b = 0; b < B; ++b)
        if (!(sq[b].done < N && sq[b].blk == 0)) h_prevlen[b] = 0;
      si.h_prev_in = c->g_carry; si.prev_len = h_prevlen.data();
    }
    si.k_cache = in->k_cache; si.v_cache = in->v_cache; si.ctx_len = h_ctx.data();
    si.last_ids = c->g_last; si.last_len = h_lastlen.data();
    si.win_ids = c->g_win; si.win_len = h_winlen.data(); si.remain_len = h_remain.data();
    dc_step_out so{};
    so.pred_id = c->g_pred; so.conf = c->g_conf; so.xlogp = c->g_xlogp; so.status = c->g_status;
    so.block_len = any_boundary ? c->g_blk : nullptr;
    so.h_out = (any_boundary && carried) ? c->g_hout : nullptr;
    int rc = dc_step(c, &si, &so);
    if (rc != DC_OK) return rc;
    ++nfe;
    // sequences inside a block keep their block length; the boundary rule wrote the others'
    {
      PrevLen keep{};
      bool any_keep = false;
      for (int b = 0; b < B; ++b) {
        const bool at_boundary = sq[b].done < N && sq[b].blk == 0;
        keep.n[b] = at_boundary ? -1 : (sq[b].done >= N ? 1 : sq[b].blk);
        any_keep |= !at_boundary;
      }
      if (any_keep) launch_keep_block_len(c->g_blk, keep, B, s);
    }
    dc_select_in se{};
    se.batch = B; se.conf = c->g_conf; se.win_ids = c->g_win; se.xlogp = c->g_xlogp;
    se.block_len = c->g_blk; se.win_len = h_winlen.data();
    dc_select_out seo{c->g_mask, c->g_idx, c->g_cnt};
    rc = dc_select(c, &se, &seo);
    if (rc != DC_OK) return rc;
    dc_commit_in ci{B, c->g_win, c->g_pred, c->g_mask, c->g_blk, h_winlen.data()};
    dc_commit_out co{c->g_rem};
    rc = dc_commit(c, &ci, &co);
    if (rc != DC_OK) return rc;
    cudaMemcpyAsync(h_blk, c->g_blk, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, s);
    cudaMemcpyAsync(h_rem, c->g_rem, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, s);
    cudaMemcpyAsync(h_status, c->g_status, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, s);
    cudaMemcpyAsync(h_ids, c->g_win, sizeof(int32_t) * (size_t)B * MW, cudaMemcpyDeviceToHost, s);
    if (ev1) cudaEventRecord(ev1, s);
    if (cudaStreamSynchronize(s) != cudaSuccess) return fail(c, DC_ERR_CUDA, "stream sync failed in dc_generate");
    if (ev1) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, ev0, ev1) == cudaSuccess) dev_ms += ms;
    }
    for (int b = 0; b < B; ++b)
      if (h_status[b] != DC_OK) return fail(c, h_status[b], "device-side status %d in sequence %d", h_status[b], b);
    // ---- state update
    for (int b = 0; b < B; ++b) {
      Seq& q = sq[b];
      if (q.done >= N) continue;
      if (q.blk == 0) {                        // this was the boundary step
        q.cache += q.last_len;                 // the last block now lives in the cache
        q.last_len = 0;
        q.blk = h_blk[b];
        if (out->block_lens) out->block_lens[(size_t)b * N + q.nblocks] = q.blk;
        ++q.nblocks;
        if (carried) {   // rows blk .. W of this window are rows 0 .. of the next one
          q.carry = h_winlen[b] - q.blk;
          if (q.carry > 0)
            cudaMemcpyAsync(c->g_carry + (size_t)b * MW * row_bytes,
                            c->g_hout + ((size_t)b * MW + q.blk) * row_bytes, (size_t)q.carry * row_bytes,
                            cudaMemcpyDeviceToDevice, s);
        }
      }
      if (h_rem[b] == 0) {                     // block complete: its ids came back with the counters
        memcpy(out->tokens + (size_t)b * N + q.done, h_ids + (size_t)b * MW, sizeof(int32_t) * q.blk);
        memcpy(h_last.data() + (size_t)b * g.max_last, h_ids + (size_t)b * MW, sizeof(int32_t) * q.blk);
        q.last_len = q.blk;
        q.done += q.blk;
        q.blk = 0;
      }
    }
  }
  *out->nfe = nfe;
  if (out->device_ms) *out->device_ms = (float)dev_ms;
  return DC_OK;
}

int dc_set_option(dc_ctx* c, int32_t option, int32_t value) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (option == DC_OPT_COOPERATIVE) {
    if (c->tc) tc_set_cooperative(c->tc, value != 0);
    return DC_OK;
  }
  if (option == DC_OPT_WAIT_LIMIT_US) {
    if (value < 1000 || value > 60000000) return fail(c, DC_ERR_INVALID_ARG, "wait limit outside [1000, 60000000] us");
    if (!c->tc) return DC_OK;   // the CUDA-core kernels have no device-side waits
    const int rc = tc_set_wait_limit_us(c->tc, value);
    return rc == DC_OK ? DC_OK : fail(c, rc, "%s", tc_error(c->tc));
  }
  if (option == DC_OPT_TEST_STALL_LMHEAD) {
    if (c->tc) tc_set_stall_lmhead(c->tc, value != 0);
    return DC_OK;
  }
  return fail(c, DC_ERR_INVALID_ARG, "unknown option %d", option);
}

int dc_debug_logits(dc_ctx* c, int32_t variant, float* outp) {
  if (!c) return DC_ERR_INVALID_ARG;
  if (!outp || variant < 0 || variant > 1) return fail(c, DC_ERR_INVALID_ARG, "bad argument");
  if (!c->have_logits || !c->logits)
    return fail(c, DC_ERR_UNSUPPORTED, "logits exist only after a CUDA-core LM head step");
  const SeqMeta& m = c->last_meta;
  if (variant >= m.nv) return fail(c, DC_ERR_INVALID_ARG, "the last step ran no prev variant");
  const int V = c->cfg.vocab;
  for (int b = 0; b < m.batch; ++b)
    for (int k = 0; k < m.win_len[b]; ++k) {
      const float* src = c->logits + (size_t)lm_row(m, variant, b * m.W_cap + k) * V;
      float* dst = outp + ((size_t)b * c->cfg.max_window + k) * V;
      if (cudaMemcpyAsync(dst, src, sizeof(float) * V, cudaMemcpyDeviceToDevice, c->stream) !=
          cudaSuccess)
        return fail(c, DC_ERR_CUDA, "logit copy failed");
    }
  return DC_OK;
}

int dc_destroy(dc_ctx* c) {
  if (!c) return DC_OK;
  if (c->tc) tc_destroy(c->tc);
  for (void* p : c->allocs) cudaFree(p);
  if (c->g_host) cudaFreeHost(c->g_host);
  delete c;
  return DC_OK;
}

const char* dc_last_error(const dc_ctx* c) {
  return c ? c->err.c_str() : g_create_error.c_str();
}

}  // extern "C"
