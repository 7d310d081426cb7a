// Host side of the tensor-core path: tensor maps, workspace, launch configuration.
#include "tc.h"

#include <cuda.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <string>

#include "tc_attn.cuh"
#include "tc_chain.cuh"
#include "tc_gemm.cuh"
#include "tc_lmhead.cuh"

namespace dc {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
            cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D bf16 row-major [rows, cols] tensor, box = 64 columns (128 bytes) x box_rows rows,
// 128-byte swizzle, zero fill outside the tensor
bool make_map_2d(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D bf16 tensor [n2][n1][n0] (n0 contiguous), box = 64 x box1 x 1, 128-byte swizzle
bool make_map_3d(CUtensorMap* m, const void* base, uint64_t n0, uint64_t n1, uint64_t n2,
                 uint32_t box1) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[3] = {n0, n1, n2};
  cuuint64_t strides[2] = {n0 * 2, n0 * n1 * 2};
  cuuint32_t box[3] = {64, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kSmemBudget = 232448 - 1024;  // opt-in shared memory per CTA, minus alignment slack
constexpr int kStaticQkv = 128 * 33 * 4 + 512;  // static shared memory of the kernels (upper bounds)
constexpr int kStaticOther = 512;

}  // namespace

struct LayerMaps {
  CUtensorMap wq, wk, wv, wo, w_gate, w_up, w_down;
};

struct ActMaps {
  CUtensorMap a, o, act;
};

constexpr int kFlagWords = 512;    // per-tile hand-over counters of the balanced QKV phase

struct TcState {
  dc_config g{};
  cudaStream_t s = nullptr;
  int M_max = 0;
  std::vector<LayerMaps> layers;
  std::vector<const void*> bq, bk, bv;   // per-layer q / k / v projection biases (empty: none)
  std::map<int, ActMaps> act_maps;  // keyed by BN
  std::vector<void*> allocs;
  __nv_bfloat16 *a_buf = nullptr;  // borrowed: the normed activations of the scheduler
  __nv_bfloat16 *q = nullptr, *k = nullptr, *v = nullptr, *o = nullptr, *act = nullptr;
  float* part = nullptr;
  size_t part_stride = 0;
  int max_split = 4;
  int32_t* status = nullptr;
  int ldv = 0;  // row pitch of the transposed active V
  CUtensorMap map_q, map_k, map_vt, map_kc, map_vc;
  const void *kc_base = nullptr, *vc_base = nullptr;
  CUtensorMap map_h, map_lm;
  float* lm_part = nullptr;
  int n_sm = 148, lm_stages = 6;
  unsigned int* grid_bar = nullptr;  // arrival counter of the dense chain's grid barrier, then kFlagWords tile flags
  unsigned int qkv_launches = 0;     // chain launches of this step that ran a QKV phase
  unsigned int bar_count = 0;        // arrivals the launches of this step have used up so far
  int chain_grid = 0;                // CTAs of the dense chain (0 = unavailable)
  bool stall_lmhead = false;         // test hook (DC_OPT_TEST_STALL_LMHEAD)
  bool coop_supported = false;       // the device can launch cooperatively
  bool chain_coop = false;           // the dense chain is launched cooperatively (co-residency guaranteed)
  std::string err;
  bool attrs_set = false;
};

namespace {

int tfail(TcState* t, int code, const char* fmt, ...) {
  char buf[400];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  t->err = buf;
  return code;
}

template <typename T>
T* talloc(TcState* t, size_t n, bool* ok) {
  void* p = nullptr;
  if (cudaMalloc(&p, (n ? n : 1) * sizeof(T)) != cudaSuccess) {
    cudaGetLastError();
    *ok = false;
    return nullptr;
  }
  t->allocs.push_back(p);
  return reinterpret_cast<T*>(p);
}

int pick_bn(int M) {
  const int nblk = (M + 255) / 256;
  const int bn = ((M + nblk - 1) / nblk + 15) / 16 * 16;
  return bn;
}

}  // namespace

bool tc_supported(const dc_config& g) {
  return g.dtype == DC_BF16 && g.head_dim == 128 && g.d_model % 128 == 0 && g.d_ff % 128 == 0 &&
         g.n_layers > 0 && get_encode() != nullptr;
}

const char* tc_error(const TcState* t) { return t ? t->err.c_str() : ""; }

void tc_destroy(TcState* t) {
  if (!t) return;
  for (void* p : t->allocs) cudaFree(p);
  delete t;
}

int tc_create(const dc_config& g, cudaStream_t s, int M_max, int Mlm_max,
              const std::vector<const void*>& wq, const std::vector<const void*>& wk,
              const std::vector<const void*>& wv, const std::vector<const void*>& wo,
              const std::vector<const void*>& w_gate, const std::vector<const void*>& w_up,
              const std::vector<const void*>& w_down, const void* lm_head,
              const __nv_bfloat16* h_buf, TcState** out) {
  TcState* t = new TcState();
  *out = t;
  t->g = g; t->s = s; t->M_max = M_max;
  const uint64_t d = g.d_model, hq = (uint64_t)g.n_q_heads * g.head_dim,
                 hkv = (uint64_t)g.n_kv_heads * g.head_dim, F = g.d_ff;
  t->layers.resize(g.n_layers);
  for (int l = 0; l < g.n_layers; ++l) {
    LayerMaps& L = t->layers[l];
    bool ok = make_map_2d(&L.wq, wq[l], hq, d, 128) && make_map_2d(&L.wk, wk[l], hkv, d, 128) &&
              make_map_2d(&L.wv, wv[l], hkv, d, 128) && make_map_2d(&L.wo, wo[l], d, hq, 128) &&
              make_map_2d(&L.w_gate, w_gate[l], F, d, 128) &&
              make_map_2d(&L.w_up, w_up[l], F, d, 128) && make_map_2d(&L.w_down, w_down[l], d, F, 128);
    if (!ok) return tfail(t, DC_ERR_CUDA, "tensor map encoding failed for layer %d (weights must be 16-byte aligned)", l);
  }
  bool ok = true;
  const size_t M = M_max;
  t->q = talloc<__nv_bfloat16>(t, M * hq, &ok);
  t->k = talloc<__nv_bfloat16>(t, M * hkv, &ok);
  t->ldv = (M_max + 63) / 64 * 64;
  t->v = talloc<__nv_bfloat16>(t, (size_t)t->ldv * hkv, &ok);
  t->o = talloc<__nv_bfloat16>(t, M * hq, &ok);
  t->act = talloc<__nv_bfloat16>(t, M * F, &ok);
  t->part_stride = M * d;
  t->part = talloc<float>(t, (size_t)t->max_split * t->part_stride, &ok);
  t->status = talloc<int32_t>(t, 4, &ok);
  if (!ok) return tfail(t, DC_ERR_NOMEM, "tensor-core workspace allocation failed");
  cudaMemsetAsync(t->status, 0, 4 * sizeof(int32_t), s);
  // active rows beyond the step's M are read by the attention tiles (and masked): keep them finite
  cudaMemsetAsync(t->q, 0, M * hq * 2, s);
  cudaMemsetAsync(t->k, 0, M * hkv * 2, s);
  cudaMemsetAsync(t->v, 0, (size_t)t->ldv * hkv * 2, s);
  cudaMemsetAsync(t->o, 0, M * hq * 2, s);
  if (!(make_map_2d(&t->map_q, t->q, M, hq, 64) && make_map_2d(&t->map_k, t->k, M, hkv, 128) &&
        make_map_2d(&t->map_vt, t->v, hkv, t->ldv, 128)))
    return tfail(t, DC_ERR_CUDA, "attention tensor map encoding failed");
  t->map_kc = t->map_k; t->map_vc = t->map_vt;  // placeholders until a cache is supplied
  {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&t->n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (t->n_sm < 1) t->n_sm = 148;
    const size_t groups_max = ((size_t)g.max_batch * g.max_window + 63) / 64 + 1;
    t->lm_part = talloc<float>(t, groups_max * t->n_sm * 128 * 8, &ok);
    if (!ok) return tfail(t, DC_ERR_NOMEM, "LM-head workspace allocation failed");
    if (!(make_map_2d(&t->map_h, h_buf, Mlm_max, d, 128) &&
          make_map_2d(&t->map_lm, lm_head, g.vocab, d, 128)))
      return tfail(t, DC_ERR_CUDA, "LM-head tensor map encoding failed");
    const int lm_static = 2 * 64 * 33 * 4 + 512;
    t->lm_stages = (kSmemBudget - lm_static) / kLmStageBytes;
    if (t->lm_stages > 8) t->lm_stages = 8;
    if (cudaFuncSetAttribute(k_lmhead_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             t->lm_stages * kLmStageBytes + 1024) != cudaSuccess) {
      cudaGetLastError();
      return tfail(t, DC_ERR_CUDA, "cannot opt in to shared memory for the LM head");
    }
  }
  if (cudaFuncSetAttribute(k_attn_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmem) !=
      cudaSuccess) {
    cudaGetLastError();
    return tfail(t, DC_ERR_CUDA, "cannot opt in to %d bytes of shared memory", kAttnSmem);
  }
  cudaError_t e1 = cudaFuncSetAttribute(k_gemm_tc<GEMM_EPI_QKV, false>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        kSmemBudget + 1024 - kStaticQkv);
  cudaError_t e2 = cudaFuncSetAttribute(k_gemm_tc<GEMM_EPI_PARTIAL, false>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        kSmemBudget + 1024 - kStaticOther);
  cudaError_t e3 = cudaFuncSetAttribute(k_gemm_tc<GEMM_EPI_SWIGLU, false>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        kSmemBudget + 1024 - kStaticOther);
  if (e1 == cudaSuccess) e1 = cudaFuncSetAttribute(k_gemm_tc<GEMM_EPI_QKV, true>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   kSmemBudget + 1024 - kStaticQkv);
  if (e2 == cudaSuccess) e2 = cudaFuncSetAttribute(k_gemm_tc<GEMM_EPI_PARTIAL, true>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   kSmemBudget + 1024 - kStaticOther);
  if (e3 == cudaSuccess) e3 = cudaFuncSetAttribute(k_gemm_tc<GEMM_EPI_SWIGLU, true>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   kSmemBudget + 1024 - kStaticOther);
  if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess) {
    cudaGetLastError();
    return tfail(t, DC_ERR_CUDA, "cannot opt in to %d bytes of shared memory", kSmemBudget);
  }
  // the persistent dense chain needs every CTA resident at once (cooperative launch)
  {
    t->grid_bar = talloc<unsigned int>(t, 2 + kFlagWords, &ok);
    if (!ok) return tfail(t, DC_ERR_NOMEM, "dense-chain workspace allocation failed");
    cudaMemsetAsync(t->grid_bar, 0, (2 + kFlagWords) * sizeof(unsigned int), s);
    int dev = 0, coop = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    if (cudaFuncSetAttribute(k_dense_chain, cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmem) ==
        cudaSuccess) {
      // one CTA per SM in clusters of two: all of them must be resident at once
      cudaLaunchConfig_t cfg{};
      const int grid = t->n_sm & ~1;
      cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kChainThreads); cfg.dynamicSmemBytes = kChainSmem;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
      cfg.attrs = &attr; cfg.numAttrs = 1;
      int n_clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&n_clusters, k_dense_chain, &cfg) == cudaSuccess &&
          2 * n_clusters >= grid && grid >= 2) {
        t->chain_grid = grid;
        t->coop_supported = coop != 0;
        t->chain_coop = t->coop_supported;
      }
    }
    cudaGetLastError();
  }
  return DC_OK;
}

static int get_act_maps(TcState* t, const __nv_bfloat16* a, int BN, ActMaps** out) {
  auto it = t->act_maps.find(BN);
  if (it == t->act_maps.end() || t->a_buf != a) {
    const dc_config& g = t->g;
    ActMaps am;
    const uint64_t hq = (uint64_t)g.n_q_heads * g.head_dim;
    bool ok = make_map_2d(&am.a, a, t->M_max, g.d_model, BN) &&
              make_map_2d(&am.o, t->o, t->M_max, hq, BN) &&
              make_map_2d(&am.act, t->act, t->M_max, g.d_ff, BN);
    if (!ok) return tfail(t, DC_ERR_CUDA, "activation tensor map encoding failed");
    if (t->a_buf != a) t->act_maps.clear();
    t->a_buf = const_cast<__nv_bfloat16*>(a);
    it = t->act_maps.insert_or_assign(BN, am).first;
  }
  *out = &it->second;
  return DC_OK;
}

// ma: activation map with a box of BN rows; ma_half: with BN / 2 rows (CTA pairs), or null
template <int EPI>
static int launch_gemm(TcState* t, const CUtensorMap& w0, const CUtensorMap& w1,
                       const CUtensorMap& w2, const CUtensorMap& ma, const CUtensorMap* ma_half,
                       GemmParams p, int tiles, int static_smem) {
  const int nw = (EPI == GEMM_EPI_SWIGLU) ? 2 : 1;
  const int n_cblk = (p.M + p.BN - 1) / p.BN;
  // CTA pairs (each CTA stages half of the activation block) when the shapes allow it and there
  // is more than one column block: below that the fused chain is the path that matters
  const bool pair = ma_half != nullptr && tiles % 2 == 0 && p.BN % 32 == 0 &&
                    p.BN >= 64 && n_cblk > 1 && t->n_sm >= 2;
  const int sb = gemm_stage_bytes(nw, pair ? p.BN / 2 : p.BN);
  int stages = (kSmemBudget - static_smem) / sb;
  if (stages > 8) stages = 8;
  if (stages < 2) return tfail(t, DC_ERR_UNSUPPORTED, "activation block too large for the smem ring");
  const size_t smem = (size_t)stages * sb + 1024;
  // persistent: one CTA (pair) per SM (pair) works through the units; with more units than
  // workers the accumulators of consecutive units alternate between two TMEM sets
  const int n_units = (pair ? tiles / 2 : tiles) * n_cblk * p.nsplit;
  const int workers_max = pair ? t->n_sm / 2 : t->n_sm;
  const int workers = n_units < workers_max ? n_units : workers_max;
  p.tiles = tiles;
  // gate / up keep both TMEM sets for one unit (column blocks of 256 rows: with 128-row blocks
  // every weight tile is pulled from L2 twice as often, which cost more than the overlap gained)
  p.pingpong = (n_units > workers && nw == 1) ? 1 : 0;
  p.status = t->status;
  cudaError_t e;
  if (pair) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * workers); cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = smem; cfg.stream = t->s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, k_gemm_tc<EPI, true>, w0, w1, w2, *ma_half, p, stages);
  } else {
    k_gemm_tc<EPI, false><<<workers, kGemmThreads, smem, t->s>>>(w0, w1, w2, ma, p, stages);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    return tfail(t, DC_ERR_CUDA, "GEMM launch failed: %s", cudaGetErrorString(e));
  }
  return DC_OK;
}

static int pick_split(int tiles, int KB, int max_split) {
  // enough CTAs to cover the SMs, at least 8 k-blocks each; `tiles` counts every CTA of one
  // split (weight tiles x activation column blocks)
  int s = 148 / tiles;
  if (s < 1) s = 1;
  if (s > max_split) s = max_split;
  while (s > 1 && KB / s < 8) --s;
  return s;
}

// K splits of a split-K projection on the per-op path.  With few units (one column block) the
// splits fill the SMs (pick_split).  With many, units come in rounds over the workers (SMs, or SM
// pairs) and the last round is partly empty - 160 pair-units on 74 pairs are 3 rounds for 2.16
// rounds of work; splitting K makes the rounds finer at the price of one more fp32 partial array
// written and read back per split.  Rough model: GEMM at 1 PFLOP/s, partials at 5 TB/s.
static int pick_split_rounds(const TcState* t, int tiles, int M, int BN, int N, int K, int max_split) {
  const int n_cblk = (M + BN - 1) / BN;
  if (n_cblk <= 1) return pick_split(tiles * n_cblk, K / kTileK, max_split);
  const bool pair = tiles % 2 == 0 && BN % 32 == 0 && BN >= 64 && t->n_sm >= 2;
  const int units = (pair ? tiles / 2 : tiles) * n_cblk, workers = pair ? t->n_sm / 2 : t->n_sm;
  const double t1 = 2.0 * M * N * K / 1e15, work_rounds = (double)units / workers;
  const double per_split = 2.0 * M * N * 4.0 / 5e12;
  int best = 1;
  double best_t = 1e30;
  for (int s = 1; s <= max_split && (K / kTileK) / s >= 8; ++s) {
    const double rounds = (double)((units * s + workers - 1) / workers) / s;
    const double est = t1 * rounds / work_rounds + (s - 1) * per_split;
    if (est < best_t - 1e-9) { best_t = est; best = s; }
  }
  return best;
}

int tc_attention(TcState* t, int layer, const SeqMeta& m, const __nv_bfloat16* k_cache,
                 const __nv_bfloat16* v_cache) {
  const dc_config& g = t->g;
  const int nq = g.n_q_heads, nkv = g.n_kv_heads, hd = g.head_dim;
  bool any_ctx = false;
  for (int b = 0; b < m.batch; ++b) any_ctx |= m.ctx_len[b] > 0;
  if (any_ctx && (t->kc_base != k_cache || t->vc_base != v_cache)) {
    const uint64_t heads = (uint64_t)g.max_batch * nkv;
    if (!(make_map_3d(&t->map_kc, k_cache, 128, heads * g.max_ctx, g.n_layers, 128) &&
          make_map_3d(&t->map_vc, v_cache, g.max_ctx, heads * 128, g.n_layers, 128)))
      return tfail(t, DC_ERR_CUDA, "cache tensor map encoding failed (caches must be 16-byte aligned)");
    t->kc_base = k_cache; t->vc_base = v_cache;
  }
  AttnParams ap;
  ap.m = m; ap.nq = nq; ap.nkv = nkv; ap.max_ctx = g.max_ctx; ap.layer = layer;
  ap.scale_log2 = 1.4426950408889634f / sqrtf((float)hd);
  ap.o = t->o; ap.status = t->status;
  const int nqt = (m.R_cap + 127) / 128;
  // one CTA per query tile: (row tile, variant) with two variants in the pass (a row tile with 64
  // rows or fewer packs both variants into the curr CTA, the prev CTA returns at once)
  dim3 grid(m.nv == 2 ? 2 * nqt : nqt, nq, m.batch);
  k_attn_tc<<<grid, kAttnThreads, kAttnSmem, t->s>>>(t->map_q, t->map_k, t->map_vt, t->map_kc,
                                                     t->map_vc, ap);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tfail(t, DC_ERR_CUDA, "attention launch failed: %s", cudaGetErrorString(e));
  return DC_OK;
}

void tc_export_kv(TcState* t, int layer, const SeqMeta& m, __nv_bfloat16* k_cache, __nv_bfloat16* v_cache) {
  const dc_config& g = t->g;
  const size_t per_layer = (size_t)g.max_batch * g.n_kv_heads * g.max_ctx * g.head_dim;
  launch_export_kv<__nv_bfloat16>(t->k, t->v, t->ldv, m, g.n_kv_heads, g.head_dim, g.max_ctx,
                                  k_cache + (size_t)layer * per_layer, v_cache + (size_t)layer * per_layer, t->s);
}

void tc_set_qkv_bias(TcState* t, const std::vector<const void*>& bq, const std::vector<const void*>& bk,
                     const std::vector<const void*>& bv) {
  t->bq = bq; t->bk = bk; t->bv = bv;
}

void tc_set_stall_lmhead(TcState* t, bool on) { t->stall_lmhead = on; }

int tc_set_wait_limit_us(TcState* t, long long us) {
  const unsigned long long ns = (unsigned long long)us * 1000ull;
  if (cudaMemcpyToSymbolAsync(ptx::g_wait_limit_ns, &ns, sizeof(ns), 0, cudaMemcpyHostToDevice, t->s) != cudaSuccess ||
      cudaStreamSynchronize(t->s) != cudaSuccess) {
    cudaGetLastError();
    return tfail(t, DC_ERR_CUDA, "setting the wait limit failed");
  }
  return DC_OK;
}

void tc_set_cooperative(TcState* t, bool on) { t->chain_coop = on && t->coop_supported; }

bool tc_chain_ok(const TcState* t, const SeqMeta& m) {
  const dc_config& g = t->g;
  const int M = m.nv * m.batch * m.R_cap;
  // One column block of at most 256 activation rows.  The norm phases reuse the TMA ring as
  // staging space, which needs at most one GEMM unit per CTA and phase, and both rows of a norm
  // step (x plus the split-K partial sums) inside the ring.
  const int units_qkv = g.n_q_heads + 2 * g.n_kv_heads, units_f = g.d_ff / kChainTile;
  const int units_d = (g.d_model / kChainTile) * t->max_split;
  const size_t norm_bytes = (size_t)2 * (1 + t->max_split) * g.d_model * sizeof(float) + g.d_model * 2;
  const bool even = g.n_q_heads % 2 == 0 && g.n_kv_heads % 2 == 0 && (g.d_model / kChainTile) % 2 == 0 &&
                    (g.d_ff / kChainTile) % 2 == 0;   // a CTA pair takes two adjacent tiles of one matrix
  return t->chain_grid > 0 && even && M >= 32 && M <= 256 && units_qkv <= t->chain_grid && units_f <= t->chain_grid &&
         units_d <= t->chain_grid && norm_bytes <= (size_t)kChainRing;
}

void tc_step_begin(TcState* t) {
  // a step that gave up inside a grid barrier leaves the arrival count behind
  cudaMemsetAsync(t->grid_bar, 0, (2 + kFlagWords) * sizeof(unsigned int), t->s);
  t->bar_count = 0;
  t->qkv_launches = 0;
}

int tc_chain(TcState* t, int layer, int qkv_layer, int phase_begin, int phase_end, const SeqMeta& m,
             float* x, const __nv_bfloat16* a, const float* cos_sin, const __nv_bfloat16* g2,
             const __nv_bfloat16* g1, int fold_norm1, const float** part, int* nsplit,
             size_t* part_stride) {
  const dc_config& g = t->g;
  const int d = g.d_model, nq = g.n_q_heads, nkv = g.n_kv_heads, F = g.d_ff;
  const int M = m.nv * m.batch * m.R_cap;
  const int BN = (M + 15) / 16 * 16;
  ActMaps* am = nullptr;
  int rc = get_act_maps(t, a, BN / 2, &am);  // every CTA of a pair stages half of the rows
  if (rc != DC_OK) return rc;
  ChainMaps maps;
  const LayerMaps& L = t->layers[layer];
  const LayerMaps& Lq = t->layers[qkv_layer < g.n_layers ? qkv_layer : layer];
  maps.wo = L.wo; maps.wg = L.w_gate; maps.wu = L.w_up; maps.wd = L.w_down;
  maps.wq = Lq.wq; maps.wk = Lq.wk; maps.wv = Lq.wv;
  maps.wo_n = Lq.wo;
  maps.a = am->a; maps.o = am->o; maps.act = am->act;
  ChainParams p{};
  p.M = M; p.BN = BN; p.d = d; p.F = F; p.nq = nq; p.nkv = nkv;
  p.phase_begin = phase_begin; p.phase_end = phase_end;
  p.split_o = pick_split(d / kChainTile, nq * g.head_dim / kChainTileK, t->max_split);
  p.split_down = pick_split(d / kChainTile, F / kChainTileK, t->max_split);
  p.fold_norm1 = fold_norm1;
  p.x = x; p.a = const_cast<__nv_bfloat16*>(a); p.act = t->act;
  p.part = t->part; p.part_stride = t->part_stride;
  p.g2 = g2; p.g1 = g1; p.eps = g.rms_eps;
  p.cos_sin = cos_sin; p.rows_per_variant = m.batch * m.R_cap;
  p.q = t->q; p.k = t->k; p.v = t->v; p.ldv = t->ldv;
  if (!t->bq.empty()) {
    const int lq = qkv_layer < g.n_layers ? qkv_layer : layer;
    p.bq = (const __nv_bfloat16*)t->bq[lq]; p.bk = (const __nv_bfloat16*)t->bk[lq]; p.bv = (const __nv_bfloat16*)t->bv[lq];
  }
  p.bar = t->grid_bar; p.status = t->status;
  // QKV has nq + 2 nkv tiles; when that is fewer than the grid has CTAs, the CTA pairs left over
  // take a share of every tile's k-blocks
  p.bal_h = 0;
  p.tile_flags = t->grid_bar + 2;
  if (phase_end > CH_QKV) {
    const int tp = (nq + 2 * nkv) / 2, n_help = t->chain_grid / 2 - tp, KB = d / kChainTileK;
    if (n_help > 0 && tp <= 2 * n_help && nq + 2 * nkv <= kFlagWords && KB >= 4 &&
        (size_t)(nq + 2 * nkv) * BN * kChainTile <= (size_t)t->max_split * t->part_stride) {
      // An owner waits for its helper's sums before its own epilogue, so a helper should be done
      // (loop and hand-over) when the owner's loop ends.  Both loops run at the rate an SM takes
      // data in: a k-block is one weight tile (two for a helper pair that serves two tile pairs)
      // plus this CTA's half of the activations; handing a tile's sums over costs about as long
      // as taking in 1.8 times their bytes (measured: 5.4 us for two tiles of 96 KB).
      const double wb = kChainTile * kChainTileK * 2.0, ab = (BN / 2) * kChainTileK * 2.0;
      const int nt = tp > n_help ? 2 : 1;
      const double hand = 1.8 * nt * BN * kChainTile * 4.0;
      const double hf = (KB * (wb + ab) - hand) / ((nt + 1) * wb + 2.0 * ab);
      int h = (int)(hf + 0.5);
      if (h < 1) h = 1;
      if (h > KB - 1) h = KB - 1;
      p.bal_h = h;
    }
    p.flag_target = (unsigned int)(kChainThreads / 32) * ++t->qkv_launches;
  }
  p.bar_base = t->bar_count;
  t->bar_count += (unsigned int)(phase_end - phase_begin - 1) * (unsigned int)t->chain_grid;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(t->chain_grid); cfg.blockDim = dim3(kChainThreads);
  cfg.dynamicSmemBytes = kChainSmem; cfg.stream = t->s;
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeClusterDimension;
  attrs[0].val.clusterDim.x = 2; attrs[0].val.clusterDim.y = 1; attrs[0].val.clusterDim.z = 1;
  attrs[1].id = cudaLaunchAttributeCooperative;
  attrs[1].val.cooperative = 1;
  cfg.attrs = attrs; cfg.numAttrs = t->chain_coop ? 2 : 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, k_dense_chain, maps, p);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return tfail(t, DC_ERR_CUDA, "dense chain launch failed: %s", cudaGetErrorString(e));
  }
  *part = t->part; *nsplit = p.split_down; *part_stride = t->part_stride;
  return DC_OK;
}

int tc_layer(TcState* t, int layer, const SeqMeta& m, float* x, const __nv_bfloat16* a,
             const __nv_bfloat16* k_cache, const __nv_bfloat16* v_cache, const float* cos_sin,
             const __nv_bfloat16* norm2, const float** part, int* nsplit, size_t* part_stride,
             StageHook& hook, bool export_kv, bool kv_only) {
  const dc_config& g = t->g;
  const int d = g.d_model, nq = g.n_q_heads, nkv = g.n_kv_heads, hd = g.head_dim, F = g.d_ff;
  const int M = m.nv * m.batch * m.R_cap;
  const int BN = pick_bn(M);
  ActMaps *am = nullptr, *amh = nullptr;
  int rc = get_act_maps(t, a, BN, &am);
  if (rc != DC_OK) return rc;
  if (BN % 32 == 0 && BN >= 64 && M > BN) {
    rc = get_act_maps(t, a, BN / 2, &amh);
    if (rc != DC_OK) return rc;
    rc = get_act_maps(t, a, BN, &am);   // (the cache may have been rebuilt)
    if (rc != DC_OK) return rc;
  }
  const LayerMaps& L = t->layers[layer];
  GemmParams p{};
  p.M = M; p.BN = BN; p.nq = nq; p.nkv = nkv; p.hd = hd;
  p.cos_sin = cos_sin; p.rows_per_variant = m.batch * m.R_cap;
  p.q = t->q; p.k = t->k; p.v = t->v; p.ldv = t->ldv; p.act = t->act;
  if (!t->bq.empty()) {
    p.bq = (const __nv_bfloat16*)t->bq[layer]; p.bk = (const __nv_bfloat16*)t->bk[layer]; p.bv = (const __nv_bfloat16*)t->bv[layer];
  }
  p.part = t->part; p.part_stride = t->part_stride;

  hook.begin(DC_STAGE_QKV, 1);
  p.N = (nq + 2 * nkv) * hd; p.K = d; p.nsplit = 1;
  rc = launch_gemm<GEMM_EPI_QKV>(t, L.wq, L.wk, L.wv, am->a, amh ? &amh->a : nullptr, p, nq + 2 * nkv, kStaticQkv);
  hook.end();
  if (rc != DC_OK) return rc;

  if (export_kv)
    tc_export_kv(t, layer, m, const_cast<__nv_bfloat16*>(k_cache), const_cast<__nv_bfloat16*>(v_cache));
  if (kv_only) return DC_OK;   // prefill, last layer: only its K / V were wanted
  hook.begin(DC_STAGE_ATTN, 1);
  rc = tc_attention(t, layer, m, k_cache, v_cache);
  hook.end();
  if (rc != DC_OK) return rc;

  hook.begin(DC_STAGE_OPROJ, 1);
  p.N = d; p.K = nq * hd; p.nsplit = pick_split_rounds(t, d / kTileN, M, BN, p.N, p.K, t->max_split);
  rc = launch_gemm<GEMM_EPI_PARTIAL>(t, L.wo, L.wo, L.wo, am->o, amh ? &amh->o : nullptr, p, d / kTileN, kStaticOther);
  hook.end();
  if (rc != DC_OK) return rc;

  hook.begin(DC_STAGE_NORM, 1);
  launch_rmsnorm<__nv_bfloat16>(x, t->part, p.nsplit, t->part_stride, norm2, g.rms_eps, M, d,
                                const_cast<__nv_bfloat16*>(a), t->s);
  hook.end();

  hook.begin(DC_STAGE_GATEUP, 1);
  p.N = F; p.K = d; p.nsplit = 1;
  rc = launch_gemm<GEMM_EPI_SWIGLU>(t, L.w_gate, L.w_up, L.w_up, am->a, amh ? &amh->a : nullptr, p, F / kTileN, kStaticOther);
  hook.end();
  if (rc != DC_OK) return rc;

  hook.begin(DC_STAGE_DOWN, 1);
  p.N = d; p.K = F; p.nsplit = pick_split_rounds(t, d / kTileN, M, BN, p.N, p.K, t->max_split);
  rc = launch_gemm<GEMM_EPI_PARTIAL>(t, L.w_down, L.w_down, L.w_down, am->act, amh ? &amh->act : nullptr, p, d / kTileN, kStaticOther);
  hook.end();
  if (rc != DC_OK) return rc;

  *part = t->part; *nsplit = p.nsplit; *part_stride = t->part_stride;
  return DC_OK;
}

int tc_lmhead(TcState* t, const SeqMeta& m, const __nv_bfloat16* h, int mask_id, int forbid,
              int32_t* ws_pred, float* ws_conf, float* ws_ent, float* ws_infl, float* ws_lse,
              SignalOut out, int32_t* status) {
  (void)h;  // the tensor map was built over the scheduler's LM-head input buffer
  const dc_config& g = t->g;
  LmParams p;
  p.m = m; p.V = g.vocab; p.K = g.d_model; p.mask_id = forbid ? mask_id : -1;
  p.part = t->lm_part; p.status = t->status; p.stall = t->stall_lmhead ? 1 : 0;
  const int ntiles = (g.vocab + 127) / 128;
  const int groups = m.npos_pad / m.G;
  int nctas = t->n_sm / groups;             // vocabulary slices: one resident CTA per (group, slice)
  if (nctas < 1) nctas = 1;
  if (nctas > ntiles) nctas = ntiles;
  p.ngroups = groups;
  k_lmhead_tc<<<groups * nctas, kLmThreads, t->lm_stages * kLmStageBytes + 1024, t->s>>>(t->map_h, t->map_lm,
                                                                                      p, t->lm_stages);
  const int npos = m.batch * m.W_cap;
  k_lm_combine<<<(npos + 3) / 4, 128, 0, t->s>>>(t->lm_part, nctas, m, g.vocab, mask_id, status, 1, ws_pred,
                                                 ws_conf, ws_ent, ws_infl, ws_lse, out);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tfail(t, DC_ERR_CUDA, "LM-head launch failed: %s", cudaGetErrorString(e));
  return DC_OK;
}

bool tc_has_lmhead(const dc_config& g) { return tc_supported(g); }

__global__ void k_flush_status(int32_t* tc_status, int32_t* status, int batch) {
  if (*tc_status != 0) {
    for (int b = threadIdx.x; b < batch; b += blockDim.x) status[b] = *tc_status;
    __syncthreads();
    if (threadIdx.x == 0) *tc_status = 0;
  }
}

void tc_flush_status(TcState* t, int32_t* status, int batch) {
  k_flush_status<<<1, 32, 0, t->s>>>(t->status, status, batch);
}

}  // namespace dc

// ---- dc_signals_static: the LM-head stage with its scratch data in the library image ------------
namespace {

// Scratch of dc_signals_static.  In host code this name is only a handle for
// cudaGetSymbolAddress; the device address is looked up once per device.
static __device__ __align__(256) unsigned char g_static_scratch[DC_STATIC_SCRATCH_BYTES];

constexpr size_t kStaticHBytes = (size_t)2 * DC_STATIC_MAX_POS * DC_STATIC_MAX_D * 2;
constexpr size_t kStaticPartBytes = (size_t)2 * 160 * 128 * 8 * 4;

struct StaticDev {
  bool ready = false;
  unsigned char* base = nullptr;
  int n_sm = 0, lm_stages = 0;
};
StaticDev g_static_dev[64];

// LM-head input rows [batch][2][max_window][d] -> the LM head's row order (groups of G positions,
// curr rows then prev rows); rows of pad positions are zero.
__global__ void k_static_rows(const __nv_bfloat16* __restrict__ h_in, int max_window, int d,
                              dc::SeqMeta m, __nv_bfloat16* __restrict__ h) {
  const int lrow = blockIdx.x;
  const int grp = lrow / (m.nv * m.G), in = lrow % (m.nv * m.G);
  const int v = in / m.G, p = grp * m.G + in % m.G;
  const int b = p / m.W_cap, k = p % m.W_cap;
  uint4* dst = reinterpret_cast<uint4*>(h + (size_t)lrow * d);
  if (b >= m.batch || k >= m.win_len[b]) {
    for (int i = threadIdx.x; i < d / 8; i += blockDim.x) dst[i] = make_uint4(0, 0, 0, 0);
    return;
  }
  const uint4* src = reinterpret_cast<const uint4*>(h_in + (((size_t)b * 2 + v) * max_window + k) * d);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x) dst[i] = src[i];
}

__global__ void k_static_status(const int32_t* word, int32_t* status, int batch) {
  for (int b = threadIdx.x; b < batch; b += blockDim.x) status[b] = *word;
}

int sfail(int code, const char* msg) {
  dc::set_thread_error(msg);  // read back with dc_last_error(NULL)
  return code;
}

}  // namespace

extern "C" int dc_signals_static(const dc_signals_in* in, const dc_signals_out* out, void* cuda_stream) {
  using namespace dc;
  if (!in || !out || !in->lm_head || !in->h || !in->win_len || !out->status)
    return sfail(DC_ERR_INVALID_ARG, "null argument");
  if (in->d_model < 128 || in->d_model % 128 || in->d_model > DC_STATIC_MAX_D)
    return sfail(DC_ERR_UNSUPPORTED, "d_model must be a multiple of 128, at most DC_STATIC_MAX_D");
  if (in->vocab < 2 || in->mask_id < 0 || in->mask_id >= in->vocab)
    return sfail(DC_ERR_INVALID_ARG, "bad vocab / mask_id");
  if (in->batch < 1 || in->batch > DC_MAX_BATCH || in->max_window < 16 || in->max_window % 16 ||
      in->max_window > DC_MAX_WINDOW)
    return sfail(DC_ERR_SHAPE, "batch or max_window out of range");
  SeqMeta m{};
  m.batch = in->batch; m.nv = 2;
  int maxW = 0;
  for (int b = 0; b < in->batch; ++b) {
    const int W = in->win_len[b];
    if (W < 1 || W > in->max_window) return sfail(DC_ERR_SHAPE, "win_len outside [1, max_window]");
    m.win_len[b] = W;
    m.have_prev[b] = in->have_prev ? (in->have_prev[b] != 0) : 1;
    maxW = maxW > W ? maxW : W;
  }
  m.W_cap = (maxW + 15) / 16 * 16;
  m.R_cap = m.W_cap;
  const int npos = in->batch * m.W_cap;
  if (npos > DC_STATIC_MAX_POS)
    return sfail(DC_ERR_SHAPE, "more than DC_STATIC_MAX_POS window positions: the fixed scratch array cannot hold them");
  m.G = npos < 64 ? npos : 64;
  m.npos_pad = (npos + m.G - 1) / m.G * m.G;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
    return sfail(DC_ERR_CUDA, "no current CUDA device");
  StaticDev& sd = g_static_dev[dev];
  if (!sd.ready) {
    // once per device, with that device current: the device address of the scratch array, the
    // kernel's shared-memory opt-in, the SM count.  Nothing here allocates.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return sfail(DC_ERR_CUDA, "cudaGetSymbolAddress failed for the scratch array");
    }
    sd.base = static_cast<unsigned char*>(p);
    cudaDeviceGetAttribute(&sd.n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (sd.n_sm < 1) return sfail(DC_ERR_CUDA, "cannot read the SM count");
    if (sd.n_sm > 160) sd.n_sm = 160;  // the partial-record region is sized for 160 CTAs
    const int lm_static = 2 * 64 * 33 * 4 + 512;
    sd.lm_stages = (kSmemBudget - lm_static) / kLmStageBytes;
    if (sd.lm_stages > 8) sd.lm_stages = 8;
    if (cudaFuncSetAttribute(k_lmhead_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             sd.lm_stages * kLmStageBytes + 1024) != cudaSuccess) {
      cudaGetLastError();
      return sfail(DC_ERR_CUDA, "cannot opt in to shared memory for the LM head");
    }
    if (!get_encode()) return sfail(DC_ERR_CUDA, "cuTensorMapEncodeTiled unavailable");
    sd.ready = true;
  }
  cudaStream_t s = (cudaStream_t)cuda_stream;
  __nv_bfloat16* h_rows = reinterpret_cast<__nv_bfloat16*>(sd.base);
  float* part = reinterpret_cast<float*>(sd.base + kStaticHBytes);
  unsigned char* tail = sd.base + kStaticHBytes + kStaticPartBytes;
  int32_t* ws_pred = reinterpret_cast<int32_t*>(tail);
  float* ws_conf = reinterpret_cast<float*>(tail + 512);
  float* ws_ent = reinterpret_cast<float*>(tail + 1024);
  float* ws_infl = reinterpret_cast<float*>(tail + 1536);
  float* ws_lse = reinterpret_cast<float*>(tail + 2048);
  int32_t* word = reinterpret_cast<int32_t*>(tail + 2560);

  const int Mlm = m.nv * m.npos_pad;
  CUtensorMap map_h, map_lm;
  if (!(make_map_2d(&map_h, h_rows, 2 * DC_STATIC_MAX_POS, in->d_model, 128) &&
        make_map_2d(&map_lm, in->lm_head, in->vocab, in->d_model, 128)))
    return sfail(DC_ERR_CUDA, "tensor map encoding failed (lm_head must be 16-byte aligned)");

  // the status word is the only part of the array that must start at zero; every row and record
  // the kernels read below is rewritten by this call first
  cudaMemsetAsync(word, 0, sizeof(int32_t), s);
  k_static_rows<<<Mlm, 128, 0, s>>>((const __nv_bfloat16*)in->h, in->max_window, in->d_model, m, h_rows);
  LmParams p;
  p.m = m; p.V = in->vocab; p.K = in->d_model; p.mask_id = in->forbid_mask_pred ? in->mask_id : -1;
  p.part = part; p.status = word; p.stall = 0;
  const int ntiles = (in->vocab + 127) / 128;
  const int groups = m.npos_pad / m.G;
  int nctas = sd.n_sm / groups;
  if (nctas < 1) nctas = 1;
  if (nctas > ntiles) nctas = ntiles;
  p.ngroups = groups;
  k_lmhead_tc<<<groups * nctas, kLmThreads, sd.lm_stages * kLmStageBytes + 1024, s>>>(map_h, map_lm, p, sd.lm_stages);
  SignalOut so{out->pred_id, out->conf, out->entropy, out->influence, out->lse, in->max_window};
  k_lm_combine<<<(npos + 3) / 4, 128, 0, s>>>(part, nctas, m, in->vocab, in->mask_id, word, 0, ws_pred, ws_conf,
                                              ws_ent, ws_infl, ws_lse, so);
  k_static_status<<<1, 32, 0, s>>>(word, out->status, in->batch);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return sfail(DC_ERR_CUDA, cudaGetErrorString(e));
  return DC_OK;
}

