// Internal launcher interface between the step scheduler and the kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/depcap.h"

namespace dc {

// reason of the last failed call that had no context (what dc_last_error(NULL) returns)
void set_thread_error(const char* msg);

// Per-step sequence description, passed by value to kernels (baked into a captured graph).
struct SeqMeta {
  int ctx_len[DC_MAX_BATCH];
  int last_len[DC_MAX_BATCH];
  int win_len[DC_MAX_BATCH];
  int remain[DC_MAX_BATCH];
  int have_prev[DC_MAX_BATCH];
  int pos0[DC_MAX_BATCH];   // absolute position of active row 0 (ctx_len unless a prefill says otherwise)
  int batch;     // B
  int nv;        // variants in the pass: 1 (curr) or 2 (curr, prev)
  int R_cap;     // active rows per (variant, sequence), multiple of 16: [last ; window ; pad]
  int W_cap;     // window rows per sequence, multiple of 16
  int G;         // LM-head group: positions per group (<= 128)
  int npos_pad;  // B * W_cap rounded up to a multiple of G
};

// active row index of (variant v, sequence b, row r)
__host__ __device__ inline int act_row(const SeqMeta& m, int v, int b, int r) {
  return (v * m.batch + b) * m.R_cap + r;
}
// LM-head row of (variant v, flattened position p = b * W_cap + k): groups of G positions,
// inside a group the curr rows come first, then the prev rows.
__host__ __device__ inline int lm_row(const SeqMeta& m, int v, int p) {
  return (p / m.G) * (m.nv * m.G) + v * m.G + (p % m.G);
}

struct Hyper {
  float lambda;
  int L_min, L_max;
  float tau_low, tau_high, gamma;
  int smooth_radius, norm_mode, boundary_mode, cap_mode;
};

// ---- CUDA-core kernels (any shape, fp32 or bf16 storage) -------------------------------------
template <typename T>
void launch_embed(const T* embed, const int32_t* last_ids, const int32_t* win_ids, int max_last,
                  int max_window, int mask_id, int vocab, int d, const SeqMeta& m, float* x,
                  int32_t* status, cudaStream_t s);

// x += sum of nsplit partials (if part != null), then out = T(rmsnorm(x) * g).  rows of x: M.
template <typename T>
void launch_rmsnorm(float* x, const float* part, int nsplit, size_t part_stride, const T* g,
                    float eps, int M, int d, T* out, cudaStream_t s);

// final norm of the window rows into the LM-head row order (pad rows are zeroed)
template <typename T>
void launch_final_norm(float* x, const float* part, int nsplit, size_t part_stride, const T* g,
                       float eps, int d, const SeqMeta& m, T* h, cudaStream_t s, int nv_x = -1);
// LM rows carried between steps: h_out[b][k] <- curr row (if h_out); prev rows <- h_prev_in[b][k]
// for k < prev_len.n[b], else the curr row of the same position (if h_prev_in); m.nv must be 2 then
struct PrevLen { int n[DC_MAX_BATCH]; };
template <typename T>
void launch_carry(const T* h_prev_in, const PrevLen& pl, T* h_out, int max_window, int d,
                  const SeqMeta& m, T* h, cudaStream_t s);

// copy caller-supplied LM-head input [B][2][max_window][d] into the LM-head row order
template <typename T>
void launch_h_override(const T* h_in, int max_window, int d, const SeqMeta& m, T* h,
                       cudaStream_t s);

enum { EPI_STORE_F32 = 0, EPI_ADD_F32 = 1 };
// C[M,N] (fp32, ldc) (=|+=) A[M,K] * W[N,K]^T
template <typename T>
void launch_gemm_simt(const T* A, const T* W, float* C, int M, int N, int K, int ldc, int epi,
                      cudaStream_t s);

void launch_rope_table(const SeqMeta& m, int head_dim, float theta, float* cos_sin,
                       cudaStream_t s);

// q,k: (+ bias) rotate + store as T; v: (+ bias) store as T.  tmp layout [M, (nq + 2 nkv) * hd]
// fp32; bq / bk / bv: projection biases or null.
template <typename T>
void launch_rope_store(const float* tmp, const float* cos_sin, const SeqMeta& m, int nq, int nkv,
                       int hd, const T* bq, const T* bk, const T* bv, T* q, T* k, T* v, cudaStream_t s);

template <typename T>
void launch_swiglu(const float* gate_up, int M, int F, T* act, cudaStream_t s);

// k_cache [.. max_ctx][hd], v_cache [.. hd][max_ctx] of one layer: [max_batch][nkv][...]
template <typename T>
void launch_attn_simt(const T* q, const T* k, const T* v, const T* k_cache, const T* v_cache,
                      int max_ctx, const SeqMeta& m, int nq, int nkv, int hd, T* o,
                      cudaStream_t s);

struct SignalOut {
  int32_t* pred_id;
  float *conf, *entropy, *influence, *lse;
  int max_window;
};
// logits [M_lm, V] fp32 in LM-head row order -> per-position signals (into ws arrays, always
// non-null, laid out [B][W_cap]) and optionally the caller's arrays.
void launch_signals_from_logits(const float* logits, int V, int mask_id, int forbid,
                                const SeqMeta& m, int32_t* ws_pred, float* ws_conf,
                                float* ws_ent, float* ws_infl, float* ws_lse, SignalOut out,
                                int32_t* status, cudaStream_t s);

template <typename T>
void launch_xlogp(const T* h, const T* lm_head, const int32_t* ws_pred, const float* ws_lse,
                  int d, int V, const SeqMeta& m, int max_window, float* xlogp, cudaStream_t s);

// appends the curr variant's K / V of the last-block rows to one layer's context cache
// (k_cache / v_cache: that layer's slice); v_ld != 0: v is transposed with that row pitch
template <typename T>
void launch_export_kv(const T* k, const T* v, int v_ld, const SeqMeta& m, int nkv, int hd,
                      int max_ctx, T* k_cache, T* v_cache, cudaStream_t s);

// ---- decision kernels --------------------------------------------------------------------------
// per-sequence lengths in device memory (all null: the lengths inside SeqMeta are used)
struct DevLens {
  const int32_t* win_len = nullptr;
  const int32_t* remain = nullptr;
  const int32_t* have_prev = nullptr;
};
// influence/entropy rows have stride `ld`; outputs have stride max_window.
void launch_boundary(const float* influence, const float* entropy, int ld, const SeqMeta& m,
                     const Hyper& hp, int max_window, float* score, float* cum_i, float* cum_s,
                     int32_t* block_len, cudaStream_t s);

// the same kernel over `batch` sequences (any number) whose lengths are arrays in device memory
void launch_boundary_dev(const float* influence, const float* entropy, int ld, int batch, const DevLens& dl,
                         const Hyper& hp, int max_window, float* score, float* cum_i, float* cum_s,
                         int32_t* block_len, cudaStream_t s);
void launch_select_dev(const float* conf, const int32_t* win_ids, const float* xlogp,
                       const int32_t* block_len, int batch, const DevLens& dl, const Hyper& hp, int mask_id,
                       int max_window, uint8_t* sel_mask, int32_t* sel_idx, int32_t* sel_count,
                       cudaStream_t s);

void launch_select(const float* conf, const int32_t* win_ids, const float* xlogp,
                   const int32_t* block_len, const SeqMeta& m, const Hyper& hp, int mask_id,
                   int max_window, uint8_t* sel_mask, int32_t* sel_idx, int32_t* sel_count,
                   cudaStream_t s);

// Eq. (2): win_ids[i] <- pred_id[i] where selected and still masked, inside [0, block_len);
// remaining[b] = masked positions left in the block (may be null)
void launch_commit(int32_t* win_ids, const int32_t* pred_id, const uint8_t* sel_mask,
                   const int32_t* block_len, const SeqMeta& m, int mask_id, int max_window,
                   int32_t* remaining, cudaStream_t s);

// block_len[b] = keep.n[b] for every sequence with keep.n[b] >= 0 (the others keep what the
// boundary rule wrote)
void launch_keep_block_len(int32_t* block_len, const PrevLen& keep, int batch, cudaStream_t s);

}  // namespace dc
