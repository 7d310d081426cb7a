// Decision kernels: the DepGA-Block boundary scan (Section 4.2, cumulative form Section 4.4)
// and CAP-Decoding (Section 4.3, Algorithm 1).  One thread block per sequence.
//
// Every floating-point step that decides an integer is written with explicit round-to-nearest
// intrinsics (no contraction into FMA) and a fixed operation order, so the decisions are a
// function of the input bits alone; running sums use 2^40 fixed point, which is order-free.
#include <math.h>

#include "kernels.h"

namespace dc {

constexpr int kMaxW = DC_MAX_WINDOW;  // 256
constexpr int kThreads = 256;         // one thread per window position
constexpr double kFxScale = 1099511627776.0;          // 2^40
constexpr double kFxInv = 1.0 / 1099511627776.0;

__device__ __forceinline__ float smooth_at(const float* x, int k, int n, int radius) {
  const int lo = max(0, k - radius), hi = min(n - 1, k + radius);
  float acc = x[lo];
  for (int j = lo + 1; j <= hi; ++j) acc = __fadd_rn(acc, x[j]);
  return __fdiv_rn(acc, (float)(hi - lo + 1));
}

// block-wide max / min over one value per thread (exact, order-free)
__device__ __forceinline__ float block_max(float v, float* red) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = red[0];
  for (int i = 1; i < (int)(blockDim.x >> 5); ++i) t = fmaxf(t, red[i]);
  return t;
}
__device__ __forceinline__ int block_min_int(int v, int* red) {
  for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  int t = red[0];
  for (int i = 1; i < (int)(blockDim.x >> 5); ++i) t = min(t, red[i]);
  return t;
}

// inclusive prefix sum of one int64 per thread: shuffle scan inside each warp, then the
// warp totals are scanned by every thread (8 values)
__device__ __forceinline__ long long block_scan(long long v, long long* wtot) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  __syncthreads();
  if (lane == 31) wtot[w] = v;
  __syncthreads();
  long long base = 0;
  for (int i = 0; i < w; ++i) base += wtot[i];
  return v + base;
}

__device__ __forceinline__ float normalise(float x, float hi, float lo, int mode) {
  if (mode == DC_NORM_NONE) return x;
  if (mode == DC_NORM_MAX) return __fdiv_rn(x, fmaxf(hi, 1e-8f));
  return __fdiv_rn(__fsub_rn(x, lo), fmaxf(__fsub_rn(hi, lo), 1e-8f));
}

// Lengths of the sequences of a call: by value inside SeqMeta (a step: at most DC_MAX_BATCH
// sequences), or - when the pointers are set - arrays in device memory, for calls over any number
// of sequences.
__device__ __forceinline__ int len_of(const int32_t* dev, const int* by_value, int b) {
  return dev != nullptr ? dev[b] : by_value[b];
}

__global__ void __launch_bounds__(kThreads) k_boundary(
    const float* __restrict__ influence, const float* __restrict__ entropy, int ld, SeqMeta m,
    DevLens dl, Hyper hp, int max_window, float* __restrict__ score, float* __restrict__ cum_i,
    float* __restrict__ cum_s, int32_t* __restrict__ block_len) {
  __shared__ float sI[kMaxW], sH[kMaxW];
  __shared__ float redf[kThreads / 32];
  __shared__ int redi[kThreads / 32];
  __shared__ long long wtot[kThreads / 32];
  const int b = blockIdx.x, k = threadIdx.x;
  const int Lw = max(0, min(min(hp.L_max, len_of(dl.remain, m.remain, b)), len_of(dl.win_len, m.win_len, b)));
  const size_t o = (size_t)b * max_window + k;
  if (!len_of(dl.have_prev, m.have_prev, b)) {  // cold start: the first block uses L_min
    if (k < Lw) {
      if (score) score[o] = 0.f;
      if (cum_i) cum_i[o] = 0.f;
      if (cum_s) cum_s[o] = 0.f;
    }
    if (k == 0) block_len[b] = min(hp.L_min, Lw);
    return;
  }
  const bool in = k < Lw;
  sI[k] = in ? influence[(size_t)b * ld + k] : 0.f;
  sH[k] = in ? entropy[(size_t)b * ld + k] : 0.f;
  __syncthreads();
  const float rawI = sI[k];
  float Is = in ? smooth_at(sI, k, Lw, hp.smooth_radius) : 0.f;
  float Hs = in ? smooth_at(sH, k, Lw, hp.smooth_radius) : 0.f;
  if (hp.norm_mode != DC_NORM_NONE) {
    const float hiI = block_max(in ? Is : -INFINITY, redf);
    const float hiH = block_max(in ? Hs : -INFINITY, redf);
    float loI = 0.f, loH = 0.f;
    if (hp.norm_mode == DC_NORM_MINMAX) {
      loI = -block_max(in ? -Is : -INFINITY, redf);
      loH = -block_max(in ? -Hs : -INFINITY, redf);
    }
    Is = normalise(Is, hiI, loI, hp.norm_mode);
    Hs = normalise(Hs, hiH, loH, hp.norm_mode);
  }
  const float S = in ? __fsub_rn(Is, __fmul_rn(hp.lambda, Hs)) : 0.f;
  const long long fxS = in ? __double2ll_rn((double)S * kFxScale) : 0;
  const long long fxI = in ? __double2ll_rn((double)rawI * kFxScale) : 0;
  const long long accS = block_scan(fxS, wtot);
  const long long accI = block_scan(fxI, wtot);
  const bool neg = in && ((hp.boundary_mode == DC_BOUNDARY_CUMULATIVE) ? (accS < 0) : (S < 0.f));
  const int kstar = block_min_int(neg ? k : Lw, redi);
  if (in) {
    if (score) score[o] = S;
    if (cum_i) cum_i[o] = __double2float_rn(__ll2double_rn(accI) * kFxInv);
    if (cum_s) cum_s[o] = __double2float_rn(__ll2double_rn(accS) * kFxInv);
  }
  if (k == 0) block_len[b] = min(max(kstar, hp.L_min), Lw);
}

// one thread per window position, in whole warps (the block-wide reductions and scans cost a
// barrier pair per warp-count step, so a window of 128 runs on 4 warps, not 8)
static int boundary_threads(int max_window) {
  const int t = (max_window + 31) / 32 * 32;
  return t < 32 ? 32 : (t > kThreads ? kThreads : t);
}

void launch_boundary(const float* influence, const float* entropy, int ld, const SeqMeta& m,
                     const Hyper& hp, int max_window, float* score, float* cum_i, float* cum_s,
                     int32_t* block_len, cudaStream_t s) {
  k_boundary<<<m.batch, boundary_threads(max_window), 0, s>>>(influence, entropy, ld, m, DevLens{}, hp, max_window, score,
                                          cum_i, cum_s, block_len);
}

void launch_boundary_dev(const float* influence, const float* entropy, int ld, int batch, const DevLens& dl,
                         const Hyper& hp, int max_window, float* score, float* cum_i, float* cum_s,
                         int32_t* block_len, cudaStream_t s) {
  k_boundary<<<batch, boundary_threads(max_window), 0, s>>>(influence, entropy, ld, SeqMeta{}, dl, hp, max_window, score,
                                        cum_i, cum_s, block_len);
}

// ---- CAP-Decoding ------------------------------------------------------------------------------
// Bit sets over the window: kMaxW / 32 words.
constexpr int kWords = kMaxW / 32;

__device__ __forceinline__ bool before(float ci, int i, float cj, int j) {
  return ci > cj || (ci == cj && i < j);  // descending confidence, ties: lower position first
}

// Greedy pass over the members of `cand` in confidence order: take a candidate unless an
// earlier taken one conflicts with it.  Run by warp 0; rank[] holds the visiting order.
__device__ void greedy_pass(const uint32_t* cand, const int* order, int n_order,
                            const uint32_t (*confl)[kWords], uint32_t* sel, uint32_t* alive) {
  // all lanes of warp 0 execute the same scalar walk; lane l owns word l of the bit sets
  const int lane = threadIdx.x & 31;
  uint32_t a = (lane < kWords) ? cand[lane] : 0u;
  uint32_t s = 0u;
  for (int t = 0; t < n_order; ++t) {
    const int i = order[t];
    const uint32_t word = __shfl_sync(0xffffffffu, a, i >> 5);
    if (!((word >> (i & 31)) & 1u)) continue;
    if (lane == (i >> 5)) s |= 1u << (i & 31);
    if (lane < kWords) a &= ~confl[i][lane];
    if (lane == (i >> 5)) a &= ~(1u << (i & 31));
  }
  if (lane < kWords) { sel[lane] |= s; alive[lane] = a; }
}

__global__ void __launch_bounds__(kThreads) k_select(
    const float* __restrict__ conf, const int32_t* __restrict__ win_ids,
    const float* __restrict__ xlogp, const int32_t* __restrict__ block_len, SeqMeta m, DevLens dl,
    Hyper hp, int mask_id, int max_window, uint8_t* __restrict__ sel_mask,
    int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_count) {
  __shared__ float sc[kMaxW];
  __shared__ uint32_t s_block[kWords], s_pool[kWords], s_hi[kWords], s_sel[kWords],
      s_cand[kWords], s_alive[kWords];
  __shared__ uint32_t s_confl[kMaxW][kWords];
  __shared__ int s_order[kMaxW];
  __shared__ int s_n;
  const int b = blockIdx.x, i = threadIdx.x;
  const int W = len_of(dl.win_len, m.win_len, b);
  const int L = min(max(block_len[b], 0), W);
  const bool in_block = i < L && win_ids[(size_t)b * max_window + i] == mask_id;  // M^t ∩ B^t
  const float c = (i < W) ? conf[(size_t)b * max_window + i] : 0.f;
  const bool in_pool = in_block && c >= hp.tau_low;  // Eq. (5)
  const bool is_hi = in_pool && c >= hp.tau_high;
  sc[i] = c;
  if (i < kWords) { s_sel[i] = 0u; s_alive[i] = 0u; }
  const uint32_t bb = __ballot_sync(0xffffffffu, in_block);
  const uint32_t bp = __ballot_sync(0xffffffffu, in_pool);
  const uint32_t bh = __ballot_sync(0xffffffffu, is_hi);
  if ((i & 31) == 0) { s_block[i >> 5] = bb; s_pool[i >> 5] = bp; s_hi[i >> 5] = bh; }
  __syncthreads();
  // conflict rows of pool members: bit j set iff D_ij = xlogp[i,j] + xlogp[j,i] > gamma (Eq. 6)
  {
    uint32_t row[kWords];
#pragma unroll
    for (int w = 0; w < kWords; ++w) row[w] = 0u;
    if (in_pool) {
      const float* xb = xlogp + (size_t)b * max_window * max_window;
      for (int j = 0; j < L; ++j) {
        if (j == i || !((s_pool[j >> 5] >> (j & 31)) & 1u)) continue;
        const float D = __fadd_rn(xb[(size_t)i * max_window + j], xb[(size_t)j * max_window + i]);
        if (D > hp.gamma) row[j >> 5] |= 1u << (j & 31);
      }
    }
#pragma unroll
    for (int w = 0; w < kWords; ++w) s_confl[i][w] = row[w];
  }
  __syncthreads();

  auto make_order = [&](const uint32_t* set) {
    // position of i among the members of `set` in (confidence desc, position asc) order
    const bool member = (set[i >> 5] >> (i & 31)) & 1u;
    if (i == 0) s_n = 0;
    __syncthreads();
    if (member) {
      int rank = 0;
      for (int j = 0; j < L; ++j)
        if (j != i && ((set[j >> 5] >> (j & 31)) & 1u) && before(sc[j], j, c, i)) ++rank;
      s_order[rank] = i;
      atomicAdd(&s_n, 1);
    }
    __syncthreads();
  };

  if (hp.cap_mode == DC_CAP_STRICT) {
    // phase 1 with conflict checks: greedy over the high-confidence members
    if (i < kWords) s_cand[i] = s_hi[i];
    __syncthreads();
    make_order(s_cand);
    if (i < 32) greedy_pass(s_cand, s_order, s_n, s_confl, s_sel, s_alive);
  } else {
    // phase 1 as printed: every c_i >= tau_high enters S
    if (i < kWords) s_sel[i] = s_hi[i];
  }
  __syncthreads();
  // remove S and everything that conflicts with a member of S from the pool
  {
    bool keep = in_pool && !((s_sel[i >> 5] >> (i & 31)) & 1u);
    if (keep) {
      for (int w = 0; w < kWords; ++w)
        if (s_confl[i][w] & s_sel[w]) { keep = false; break; }
    }
    const uint32_t bk = __ballot_sync(0xffffffffu, keep);
    __syncthreads();
    if ((i & 31) == 0) s_cand[i >> 5] = bk;
  }
  __syncthreads();
  // phase 2: greedy completion in descending confidence
  make_order(s_cand);
  if (i < 32) greedy_pass(s_cand, s_order, s_n, s_confl, s_sel, s_alive);
  __syncthreads();
  // fallback: the most confident masked position of the block
  bool any = false;
  for (int w = 0; w < kWords; ++w) any |= (s_sel[w] != 0u);
  if (!any) {
    bool best = in_block;
    if (best)
      for (int j = 0; j < L; ++j)
        if (j != i && ((s_block[j >> 5] >> (j & 31)) & 1u) && before(sc[j], j, c, i)) {
          best = false;
          break;
        }
    __syncthreads();
    if (best) s_sel[i >> 5] = 1u << (i & 31);
    __syncthreads();
  }
  // outputs: mask, ascending index list, count
  const bool selected = (s_sel[i >> 5] >> (i & 31)) & 1u;
  int below = 0, total = 0;
  for (int w = 0; w < kWords; ++w) {
    const uint32_t word = s_sel[w];
    total += __popc(word);
    if (w < (i >> 5)) below += __popc(word);
    else if (w == (i >> 5)) below += __popc(word & ((1u << (i & 31)) - 1u));
  }
  if (i < W) {
    if (sel_mask) sel_mask[(size_t)b * max_window + i] = selected ? 1 : 0;
    if (sel_idx && selected) sel_idx[(size_t)b * max_window + below] = i;
  }
  if (i == 0 && sel_count) sel_count[b] = total;
}

void launch_select(const float* conf, const int32_t* win_ids, const float* xlogp,
                   const int32_t* block_len, const SeqMeta& m, const Hyper& hp, int mask_id,
                   int max_window, uint8_t* sel_mask, int32_t* sel_idx, int32_t* sel_count,
                   cudaStream_t s) {
  k_select<<<m.batch, kThreads, 0, s>>>(conf, win_ids, xlogp, block_len, m, DevLens{}, hp, mask_id,
                                        max_window, sel_mask, sel_idx, sel_count);
}

void launch_select_dev(const float* conf, const int32_t* win_ids, const float* xlogp,
                       const int32_t* block_len, int batch, const DevLens& dl, const Hyper& hp, int mask_id,
                       int max_window, uint8_t* sel_mask, int32_t* sel_idx, int32_t* sel_count,
                       cudaStream_t s) {
  k_select<<<batch, kThreads, 0, s>>>(conf, win_ids, xlogp, block_len, SeqMeta{}, dl, hp, mask_id,
                                      max_window, sel_mask, sel_idx, sel_count);
}

// ---- commit (Eq. 2): y_i <- yhat_i for the selected positions; masked positions left in the block --
__global__ void __launch_bounds__(kThreads) k_commit(int32_t* __restrict__ win_ids,
                                                    const int32_t* __restrict__ pred_id,
                                                    const uint8_t* __restrict__ sel_mask,
                                                    const int32_t* __restrict__ block_len, SeqMeta m,
                                                    int mask_id, int max_window,
                                                    int32_t* __restrict__ remaining) {
  __shared__ int red[kThreads / 32];
  const int b = blockIdx.x, i = threadIdx.x;
  const int W = m.win_len[b];
  const int L = min(max(block_len[b], 0), W);
  int left = 0;
  if (i < W) {
    const size_t o = (size_t)b * max_window + i;
    int id = win_ids[o];
    if (i < L && id == mask_id && sel_mask[o]) { id = pred_id[o]; win_ids[o] = id; }
    left = (i < L && id == mask_id) ? 1 : 0;
  }
  for (int o = 16; o > 0; o >>= 1) left += __shfl_xor_sync(0xffffffffu, left, o);
  if ((i & 31) == 0) red[i >> 5] = left;
  __syncthreads();
  if (i == 0 && remaining) {
    int t = 0;
    for (int w = 0; w < kThreads / 32; ++w) t += red[w];
    remaining[b] = t;
  }
}

__global__ void k_keep_block_len(int32_t* block_len, const PrevLen keep, int batch) {
  const int b = threadIdx.x;
  if (b < batch && keep.n[b] >= 0) block_len[b] = keep.n[b];
}

void launch_keep_block_len(int32_t* block_len, const PrevLen& keep, int batch, cudaStream_t s) {
  k_keep_block_len<<<1, DC_MAX_BATCH, 0, s>>>(block_len, keep, batch);
}

void launch_commit(int32_t* win_ids, const int32_t* pred_id, const uint8_t* sel_mask,
                   const int32_t* block_len, const SeqMeta& m, int mask_id, int max_window,
                   int32_t* remaining, cudaStream_t s) {
  k_commit<<<m.batch, kThreads, 0, s>>>(win_ids, pred_id, sel_mask, block_len, m, mask_id, max_window,
                                        remaining);
}

}  // namespace dc
