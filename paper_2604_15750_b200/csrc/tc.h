// Tensor-core (tcgen05 + TMA) half of the block-step: dense layers, attention, LM head.
#pragma once
#include <vector>

#include "kernels.h"

namespace dc {

// Stage bracket used for per-stage timing; a no-op unless profiling.
struct StageHook {
  virtual void begin(int stage, int n_launch) = 0;
  virtual void end() = 0;
  virtual ~StageHook() {}
};

struct TcState;

// phases of the persistent dense chain, in execution order
enum { CH_OPROJ = 0, CH_NORM2 = 1, CH_GATEUP = 2, CH_DOWN = 3, CH_NORM1 = 4, CH_QKV = 5, CH_END = 6 };

// true if the tensor-core kernels take this model shape
bool tc_supported(const dc_config& g);
// true if the fused tensor-core LM head takes this model shape
bool tc_has_lmhead(const dc_config& g);
// copies a device-side timeout raised by a tensor-core kernel into status[0..batch) and clears it
void tc_flush_status(TcState* t, int32_t* status, int batch);

int tc_create(const dc_config& g, cudaStream_t s, int M_max, int Mlm_max,
              const std::vector<const void*>& wq, const std::vector<const void*>& wk,
              const std::vector<const void*>& wv, const std::vector<const void*>& wo,
              const std::vector<const void*>& w_gate, const std::vector<const void*>& w_up,
              const std::vector<const void*>& w_down, const void* lm_head,
              const __nv_bfloat16* h_buf, TcState** out);
// per-layer biases of the q / k / v projections (all three or none)
void tc_set_qkv_bias(TcState* t, const std::vector<const void*>& bq, const std::vector<const void*>& bk,
                     const std::vector<const void*>& bv);
void tc_destroy(TcState* t);
const char* tc_error(const TcState* t);

// One transformer layer after the first RMSNorm: a = norm1(x) is given; on return the
// attention and MLP residual updates are applied to x except for the split-K partial sums of
// the last GEMM, which are handed back (part / nsplit / part_stride) for the next norm to fold.
// k_cache / v_cache are the BASE pointers of the whole caches (all layers).
int tc_layer(TcState* t, int layer, const SeqMeta& m, float* x, const __nv_bfloat16* a,
             const __nv_bfloat16* k_cache, const __nv_bfloat16* v_cache, const float* cos_sin,
             const __nv_bfloat16* norm2, const float** part, int* nsplit, size_t* part_stride,
             StageHook& hook, bool export_kv = false, bool kv_only = false);

// Attention of one layer alone (reads the rotated q / k / transposed v the QKV epilogue wrote).
int tc_attention(TcState* t, int layer, const SeqMeta& m, const __nv_bfloat16* k_cache,
                 const __nv_bfloat16* v_cache);

// Launch the dense chain with (default) or without the cooperative attribute; see DC_OPT_COOPERATIVE.
void tc_set_cooperative(TcState* t, bool on);
// Bound of every device-side wait of the tensor-core kernels, microseconds (device-wide).
int tc_set_wait_limit_us(TcState* t, long long us);
// Test hook: the LM-head kernel issues no loads, so that its bounded waits run out.
void tc_set_stall_lmhead(TcState* t, bool on);
// true if the persistent dense chain takes this step (all activation rows in one column block)
bool tc_chain_ok(const TcState* t, const SeqMeta& m);
// resets the chain's grid barrier; call once at the start of a step
void tc_step_begin(TcState* t);
// Phases [phase_begin, phase_end) of the dense chain (CH_* in tc_chain.cuh): O projection,
// residual + norm2 (gain g2), gate/up, down projection of `layer`; residual + norm1 (gain g1,
// folding fold_norm1 partial sums) and the rotated QKV of `qkv_layer`.  The partial sums of the
// last GEMM that ran are handed back like tc_layer does.
int tc_chain(TcState* t, int layer, int qkv_layer, int phase_begin, int phase_end, const SeqMeta& m,
             float* x, const __nv_bfloat16* a, const float* cos_sin, const __nv_bfloat16* g2,
             const __nv_bfloat16* g1, int fold_norm1, const float** part, int* nsplit,
             size_t* part_stride);

// Appends the curr variant's K / V of the last-block rows of `layer` (as the QKV epilogue left
// them) to the caller's caches (base pointers of the whole caches).
void tc_export_kv(TcState* t, int layer, const SeqMeta& m, __nv_bfloat16* k_cache, __nv_bfloat16* v_cache);

// LM head fused with the streaming softmax statistics; fills the workspace signal arrays and
// the caller's outputs.  Never writes logits.
int tc_lmhead(TcState* t, const SeqMeta& m, const __nv_bfloat16* h, int mask_id, int forbid,
              int32_t* ws_pred, float* ws_conf, float* ws_ent, float* ws_infl, float* ws_lse,
              SignalOut out, int32_t* status);

}  // namespace dc
