// CUDA-core kernels of the block-step: any shape, fp32 or bf16 storage, fp32 arithmetic.
// They are the whole path for fp32 models and for shapes the tensor-core kernels do not take,
// and the small glue kernels (embedding gather, norms, RoPE, SwiGLU, signals, cross log-probs)
// of the tensor-core path.
#include <math.h>

#include "kernels.h"

namespace dc {

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

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
// block-wide sum for blockDim.x <= 1024 (multiple of 32); red: >= 32 floats of shared memory
__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = (l < nw) ? red[l] : 0.f;
  t = warp_sum(t);
  return t;
}

// ---- 4-element vector loads / stores ------------------------------------------------------------
template <typename T> __device__ __forceinline__ void store4(T* dst, const float (&v)[4]);
template <> __device__ __forceinline__ void store4<float>(float* dst, const float (&v)[4]) {
  *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* dst,
                                                                   const float (&v)[4]) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  *reinterpret_cast<uint2*>(dst) =
      make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
}
template <typename T> __device__ __forceinline__ void load4(const T* src, float (&v)[4]);
template <> __device__ __forceinline__ void load4<float>(const float* src, float (&v)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(src);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* src,
                                                                  float (&v)[4]) {
  const uint2 t = *reinterpret_cast<const uint2*>(src);
  const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&t.x);
  const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&t.y);
  v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b);
}

// ---- embedding gather: x[row] = E[token of row] -----------------------------------------------
// Variant 0 (curr): [last block ; window]; variant 1 (prev): the last block's ids replaced by
// the mask id, everything else fixed, which makes p_prev = p(Z_k | c) (Section 4.4).
template <typename T>
__global__ void k_embed(const T* __restrict__ embed, const int32_t* __restrict__ last_ids,
                        const int32_t* __restrict__ win_ids, int max_last, int max_window,
                        int mask_id, int vocab, int d, SeqMeta m, float* __restrict__ x,
                        int32_t* __restrict__ status) {
  const int row = blockIdx.x;
  const int r = row % m.R_cap;
  const int vb = row / m.R_cap;
  const int b = vb % m.batch, v = vb / m.batch;
  const int Lb = m.last_len[b], W = m.win_len[b];
  int tok = mask_id;
  if (r < Lb) tok = (v == 0) ? last_ids[b * max_last + r] : mask_id;
  else if (r < Lb + W) tok = win_ids[b * max_window + (r - Lb)];
  if (tok < 0 || tok >= vocab) {
    if (threadIdx.x == 0) status[b] = DC_ERR_INDEX;
    tok = mask_id;
  }
  const T* e = embed + (size_t)tok * d;
  float* xr = x + (size_t)row * d;
  // d is a multiple of 4: four elements per thread and step
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    float v[4];
    load4<T>(e + i, v);
    *reinterpret_cast<float4*>(xr + i) = make_float4(v[0], v[1], v[2], v[3]);
  }
}

template <typename T>
void launch_embed(const T* embed, const int32_t* last_ids, const int32_t* win_ids, int max_last,
                  int max_window, int mask_id, int vocab, int d, const SeqMeta& m, float* x,
                  int32_t* status, cudaStream_t s) {
  const int M = m.nv * m.batch * m.R_cap;
  k_embed<T><<<M, 128, 0, s>>>(embed, last_ids, win_ids, max_last, max_window, mask_id, vocab, d,
                               m, x, status);
}

// ---- RMSNorm (with the split-K partial sums of the preceding GEMM folded into x) --------------
// One row per block; d is a multiple of 4.  The row (with the partial sums folded in, in split
// order, so the result does not depend on the launch shape) is written back to x and normed.
template <typename T>
__device__ __forceinline__ void rmsnorm_row(float* __restrict__ xr, const float* __restrict__ part,
                                            int nsplit, size_t part_stride, const T* __restrict__ g,
                                            float eps, int d, T* __restrict__ outr, float* red) {
  float ss = 0.f;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(xr + i);
    if (part) {
      for (int sidx = 0; sidx < nsplit; ++sidx) {
        const float4 pv = *reinterpret_cast<const float4*>(part + sidx * part_stride + i);
        v.x += pv.x; v.y += pv.y; v.z += pv.z; v.w += pv.w;
      }
      *reinterpret_cast<float4*>(xr + i) = v;
    }
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum(ss, red);
  const float inv = rsqrtf(ss / (float)d + eps);
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(xr + i);
    float gv[4];
    load4<T>(g + i, gv);
    const float o[4] = {v.x * inv * gv[0], v.y * inv * gv[1], v.z * inv * gv[2], v.w * inv * gv[3]};
    store4<T>(outr + i, o);
  }
}

template <typename T>
__global__ void __launch_bounds__(256) k_rmsnorm(float* __restrict__ x,
                                                 const float* __restrict__ part, int nsplit,
                                                 size_t part_stride, const T* __restrict__ g,
                                                 float eps, int d, T* __restrict__ out) {
  __shared__ float red[32];
  const size_t off = (size_t)blockIdx.x * d;
  rmsnorm_row<T>(x + off, part ? part + off : nullptr, nsplit, part_stride, g, eps, d, out + off,
                 red);
}

template <typename T>
void launch_rmsnorm(float* x, const float* part, int nsplit, size_t part_stride, const T* g,
                    float eps, int M, int d, T* out, cudaStream_t s) {
  k_rmsnorm<T><<<M, 256, 0, s>>>(x, part, nsplit, part_stride, g, eps, d, out);
}

template <typename T>
__global__ void k_final_norm(float* __restrict__ x, const float* __restrict__ part, int nsplit,
                             size_t part_stride, const T* __restrict__ g, float eps, int d,
                             SeqMeta m, T* __restrict__ h, int nv_x) {
  __shared__ float red[32];
  // grid: nv * npos_pad LM rows
  const int lrow = blockIdx.x;
  const int grp = lrow / (m.nv * m.G), in = lrow % (m.nv * m.G);
  const int v = in / m.G, p = grp * m.G + in % m.G;
  if (v >= nv_x) return;   // x holds fewer variants than the LM head sees: those rows are carried in
  T* hr = h + (size_t)lrow * d;
  const int b = p / m.W_cap, k = p % m.W_cap;
  if (b >= m.batch || k >= m.win_len[b]) {
    for (int i = threadIdx.x; i < d; i += blockDim.x) hr[i] = from_f<T>(0.f);
    return;
  }
  const size_t off = (size_t)act_row(m, v, b, m.last_len[b] + k) * d;
  rmsnorm_row<T>(x + off, part ? part + off : nullptr, nsplit, part_stride, g, eps, d, hr, red);
}

template <typename T>
void launch_final_norm(float* x, const float* part, int nsplit, size_t part_stride, const T* g,
                       float eps, int d, const SeqMeta& m, T* h, cudaStream_t s, int nv_x) {
  k_final_norm<T><<<m.nv * m.npos_pad, 256, 0, s>>>(x, part, nsplit, part_stride, g, eps, d, m, h,
                                                    nv_x < 0 ? m.nv : nv_x);
}

template <typename T>
__global__ void k_carry(const T* __restrict__ h_prev_in, PrevLen pl, T* __restrict__ h_out,
                        int max_window, int d, SeqMeta m, T* __restrict__ h) {
  const int lrow = blockIdx.x;
  const int grp = lrow / (m.nv * m.G), in = lrow % (m.nv * m.G);
  const int v = in / m.G, p = grp * m.G + in % m.G;
  const int b = p / m.W_cap, k = p % m.W_cap;
  const bool live = b < m.batch && k < m.win_len[b];
  T* row = h + (size_t)lrow * d;
  if (v == 0) {
    if (!live || !h_out) return;
    T* dst = h_out + ((size_t)b * max_window + k) * d;
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
      float v4[4];
      load4<T>(row + i, v4);
      store4<T>(dst + i, v4);
    }
    return;
  }
  if (!h_prev_in) return;
  // prev row: the carried row, or (no earlier prediction for this position) the curr row itself,
  // which makes the two distributions equal and I_k = 0; pad rows are zero
  const T* src = !live ? nullptr
               : (k < pl.n[b]) ? h_prev_in + ((size_t)b * max_window + k) * d
                               : h + (size_t)lm_row(m, 0, p) * d;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    float v4[4] = {0.f, 0.f, 0.f, 0.f};
    if (src) load4<T>(src + i, v4);
    store4<T>(row + i, v4);
  }
}

template <typename T>
void launch_carry(const T* h_prev_in, const PrevLen& pl, T* h_out, int max_window, int d,
                  const SeqMeta& m, T* h, cudaStream_t s) {
  k_carry<T><<<m.nv * m.npos_pad, 128, 0, s>>>(h_prev_in, pl, h_out, max_window, d, m, h);
}
template void launch_carry<float>(const float*, const PrevLen&, float*, int, int, const SeqMeta&, float*, cudaStream_t);
template void launch_carry<__nv_bfloat16>(const __nv_bfloat16*, const PrevLen&, __nv_bfloat16*, int, int,
                                          const SeqMeta&, __nv_bfloat16*, cudaStream_t);

template <typename T>
__global__ void k_h_override(const T* __restrict__ h_in, int max_window, int d, SeqMeta m,
                             T* __restrict__ h) {
  const int lrow = blockIdx.x;
  const int grp = lrow / (m.nv * m.G), in = lrow % (m.nv * m.G);
  const int v = in / m.G, p = grp * m.G + in % m.G;
  const int b = p / m.W_cap, k = p % m.W_cap;
  if (b >= m.batch || k >= m.win_len[b]) return;  // pad rows were zeroed by the final norm
  const T* src = h_in + (((size_t)b * 2 + v) * max_window + k) * d;
  T* dst = h + (size_t)lrow * d;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    float v4[4];
    load4<T>(src + i, v4);
    store4<T>(dst + i, v4);
  }
}

template <typename T>
void launch_h_override(const T* h_in, int max_window, int d, const SeqMeta& m, T* h,
                       cudaStream_t s) {
  k_h_override<T><<<m.nv * m.npos_pad, 128, 0, s>>>(h_in, max_window, d, m, h);
}

// ---- plain tiled GEMM: C[M,N] (=|+=) A[M,K] W[N,K]^T, fp32 accumulate -------------------------
template <typename T>
__global__ void __launch_bounds__(256) k_gemm_simt(const T* __restrict__ A,
                                                   const T* __restrict__ W, float* __restrict__ C,
                                                   int M, int N, int K, int ldc, int epi) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += BK) {
    for (int i = threadIdx.x; i < BM * BK; i += 256) {
      const int r = i / BK, c = i % BK;
      const int gm = m0 + r, gk = k0 + c;
      As[c][r] = (gm < M && gk < K) ? to_f<T>(A[(size_t)gm * K + gk]) : 0.f;
      const int gn = n0 + r;
      Ws[c][r] = (gn < N && gk < K) ? to_f<T>(W[(size_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] = Ws[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      float* c = C + (size_t)gm * ldc + gn;
      *c = (epi == EPI_ADD_F32) ? (*c + acc[i][j]) : acc[i][j];
    }
  }
}

template <typename T>
void launch_gemm_simt(const T* A, const T* W, float* C, int M, int N, int K, int ldc, int epi,
                      cudaStream_t s) {
  dim3 grid((N + 63) / 64, (M + 63) / 64);
  k_gemm_simt<T><<<grid, 256, 0, s>>>(A, W, C, M, N, K, ldc, epi);
}

// ---- RoPE ----------------------------------------------------------------------------------------
// cos_sin[(b * R_cap + r) * hd + i] = cos(angle), [.. + hd/2 + i] = sin(angle),
// angle = (pos0[b] + r) * theta^(-2i/hd), evaluated in double precision.  Row batch * R_cap
// holds cos / sin of theta^(-2i/hd) itself, the angle step between consecutive rows.
__global__ void k_rope_table(SeqMeta m, int hd, float theta, float* __restrict__ cos_sin) {
  const int half = hd / 2;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  const int rows = m.batch * m.R_cap;
  const int total = (rows + 1) * half;   // one extra row: cos / sin of the per-row angle step
  if (idx >= total) return;
  const int i = idx % half, br = idx / half;
  const int r = br % m.R_cap, b = br / m.R_cap;
  const double inv_freq = pow((double)theta, -2.0 * (double)i / (double)hd);
  const double ang = (br < rows) ? (double)(m.pos0[b] + r) * inv_freq : inv_freq;
  double sn, cs;
  sincos(ang, &sn, &cs);
  cos_sin[(size_t)br * hd + i] = (float)cs;
  cos_sin[(size_t)br * hd + half + i] = (float)sn;
}

void launch_rope_table(const SeqMeta& m, int head_dim, float theta, float* cos_sin,
                       cudaStream_t s) {
  const int total = (m.batch * m.R_cap + 1) * (head_dim / 2);
  k_rope_table<<<(total + 255) / 256, 256, 0, s>>>(m, head_dim, theta, cos_sin);
}

template <typename T>
__global__ void k_rope_store(const float* __restrict__ tmp, const float* __restrict__ cos_sin,
                             SeqMeta m, int nq, int nkv, int hd, const T* __restrict__ bq,
                             const T* __restrict__ bk, const T* __restrict__ bv, T* __restrict__ q,
                             T* __restrict__ k, T* __restrict__ v) {
  const int row = blockIdx.x;
  const int br = row % (m.batch * m.R_cap);  // (b, r): the table is shared by both variants
  const int half = hd / 2;
  const int ntot = (nq + 2 * nkv) * hd;
  const float* t = tmp + (size_t)row * ntot;
  const float* cs = cos_sin + (size_t)br * hd;
  // rotated heads: q then k; one thread per (head, i < half)
  for (int idx = threadIdx.x; idx < (nq + nkv) * half; idx += blockDim.x) {
    const int h = idx / half, i = idx % half;
    float x1 = t[h * hd + i], x2 = t[h * hd + half + i];
    if (bq != nullptr) {   // projection bias, before the rotation
      const T* bb = h < nq ? bq + h * hd : bk + (h - nq) * hd;
      x1 += to_f<T>(bb[i]); x2 += to_f<T>(bb[half + i]);
    }
    const float c = cs[i], sn = cs[half + i];
    const float y1 = x1 * c - x2 * sn, y2 = x2 * c + x1 * sn;
    if (h < nq) {
      q[(size_t)row * nq * hd + h * hd + i] = from_f<T>(y1);
      q[(size_t)row * nq * hd + h * hd + half + i] = from_f<T>(y2);
    } else {
      const int hk = h - nq;
      k[(size_t)row * nkv * hd + hk * hd + i] = from_f<T>(y1);
      k[(size_t)row * nkv * hd + hk * hd + half + i] = from_f<T>(y2);
    }
  }
  for (int idx = threadIdx.x; idx < nkv * hd; idx += blockDim.x)
    v[(size_t)row * nkv * hd + idx] = from_f<T>(t[(nq + nkv) * hd + idx] + (bv != nullptr ? to_f<T>(bv[idx]) : 0.f));
}

template <typename T>
void launch_rope_store(const float* tmp, const float* cos_sin, const SeqMeta& m, int nq, int nkv,
                       int hd, const T* bq, const T* bk, const T* bv, T* q, T* k, T* v, cudaStream_t s) {
  const int M = m.nv * m.batch * m.R_cap;
  k_rope_store<T><<<M, 256, 0, s>>>(tmp, cos_sin, m, nq, nkv, hd, bq, bk, bv, q, k, v);
}

// ---- SwiGLU: act = silu(gate) * up; gate_up is [M, 2F] (gate columns first) ----------------------
template <typename T>
__global__ void k_swiglu(const float* __restrict__ gate_up, int M, int F, T* __restrict__ act) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)M * F) return;
  const size_t r = idx / F, c = idx % F;
  const float g = gate_up[r * 2 * F + c], u = gate_up[r * 2 * F + F + c];
  act[idx] = from_f<T>(g / (1.f + expf(-g)) * u);
}

template <typename T>
void launch_swiglu(const float* gate_up, int M, int F, T* act, cudaStream_t s) {
  const size_t n = (size_t)M * F;
  k_swiglu<T><<<(unsigned)((n + 255) / 256), 256, 0, s>>>(gate_up, M, F, act);
}

// ---- bidirectional attention, one warp per query row -----------------------------------------
// Keys of query (v, b, r): the ctx_len[b] cached rows, then the last_len[b] + win_len[b] active
// rows of the same variant.  No causal mask.
template <typename T>
__global__ void __launch_bounds__(128) k_attn_simt(
    const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
    const T* __restrict__ k_cache, const T* __restrict__ v_cache, int max_ctx, SeqMeta m, int nq,
    int nkv, int hd, T* __restrict__ o, int score_stride) {
  extern __shared__ float smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y;
  const int vb = blockIdx.z;
  const int b = vb % m.batch, vv = vb / m.batch;
  const int g = h / (nq / nkv);
  const int P = m.ctx_len[b], R = m.last_len[b] + m.win_len[b];
  const int nkeys = P + R;
  float* sc = smem + (size_t)warp * score_stride;  // scores of this warp's row
  float* qs = sc + (score_stride - hd);            // the query row, tail of the warp's slice
  const float scale = rsqrtf((float)hd);
  const T* kc = k_cache ? k_cache + ((size_t)b * nkv + g) * (size_t)max_ctx * hd : nullptr;
  const T* vc = v_cache ? v_cache + ((size_t)b * nkv + g) * (size_t)hd * max_ctx : nullptr;
  const int row0 = act_row(m, vv, b, 0);
  for (int r = blockIdx.x * 4 + warp; r < R; r += gridDim.x * 4) {
    const size_t qoff = (size_t)(row0 + r) * nq * hd + (size_t)h * hd;
    for (int e = lane; e < hd; e += 32) qs[e] = to_f<T>(q[qoff + e]);
    __syncwarp();
    float mx = -INFINITY;
    for (int j = lane; j < nkeys; j += 32) {
      const T* kr = (j < P) ? kc + (size_t)j * hd
                            : k + (size_t)(row0 + j - P) * nkv * hd + (size_t)g * hd;
      float acc = 0.f;
      for (int e = 0; e < hd; ++e) acc = fmaf(qs[e], to_f<T>(kr[e]), acc);
      acc *= scale;
      sc[j] = acc;
      mx = fmaxf(mx, acc);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int j = lane; j < nkeys; j += 32) {
      const float p = expf(sc[j] - mx);
      sc[j] = p;
      sum += p;
    }
    sum = warp_sum(sum);
    __syncwarp();
    const float inv = 1.f / sum;
    for (int e = lane; e < hd; e += 32) {
      float acc = 0.f;
      if (P > 0) {
        const T* vr = vc + (size_t)e * max_ctx;
        for (int j = 0; j < P; ++j) acc = fmaf(sc[j], to_f<T>(vr[j]), acc);
      }
      for (int j = 0; j < R; ++j)
        acc = fmaf(sc[P + j], to_f<T>(v[(size_t)(row0 + j) * nkv * hd + (size_t)g * hd + e]), acc);
      o[qoff + e] = from_f<T>(acc * inv);
    }
    __syncwarp();
  }
}

template <typename T>
void launch_attn_simt(const T* q, const T* k, const T* v, const T* k_cache, const T* v_cache,
                      int max_ctx, const SeqMeta& m, int nq, int nkv, int hd, T* o,
                      cudaStream_t s) {
  int max_keys = 0;
  for (int b = 0; b < m.batch; ++b)
    max_keys = max(max_keys, m.ctx_len[b] + m.last_len[b] + m.win_len[b]);
  const int score_stride = ((max_keys + 31) / 32) * 32 + hd;
  const size_t smem = (size_t)4 * score_stride * sizeof(float);
  static size_t configured = 0;
  if (smem > 48 * 1024 && smem > configured) {
    cudaFuncSetAttribute(k_attn_simt<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    configured = smem;
  }
  dim3 grid((m.R_cap + 3) / 4, nq, m.nv * m.batch);
  k_attn_simt<T><<<grid, 128, smem, s>>>(q, k, v, k_cache, v_cache, max_ctx, m, nq, nkv, hd, o,
                                          score_stride);
}

// ---- per-position signals from full logits (CUDA-core LM head only) ------------------------------
// One block per window position.  c = max_v p(v), yhat = argmax (lowest id on ties),
// H = lse - sum p z, I = sum p [(z - lse) - (z' - lse')] clamped at 0 (Eq. 3).
__global__ void __launch_bounds__(256) k_signals(const float* __restrict__ logits, int V,
                                                 int mask_id, int forbid, SeqMeta m,
                                                 int32_t* __restrict__ ws_pred,
                                                 float* __restrict__ ws_conf,
                                                 float* __restrict__ ws_ent,
                                                 float* __restrict__ ws_infl,
                                                 float* __restrict__ ws_lse, SignalOut out,
                                                 int32_t* __restrict__ status) {
  __shared__ float red[32];
  __shared__ float s_m[8], s_m2[8];
  __shared__ int s_i[8];
  const int p = blockIdx.x;
  const int b = p / m.W_cap, k = p % m.W_cap;
  if (b >= m.batch || k >= m.win_len[b]) return;
  const bool prev = (m.nv == 2);
  const float* z = logits + (size_t)lm_row(m, 0, p) * V;
  const float* z2 = prev ? logits + (size_t)lm_row(m, 1, p) * V : nullptr;
  const int skip = forbid ? mask_id : -1;
  float mx = -INFINITY, mx2 = -INFINITY;
  int am = 0x7fffffff;
  for (int v = threadIdx.x; v < V; v += blockDim.x) {
    if (v == skip) continue;
    const float a = z[v];
    if (a > mx) { mx = a; am = v; }  // strided ascending: the first maximum kept per thread
    if (prev) mx2 = fmaxf(mx2, z2[v]);
  }
  // reduce (max, lowest index) across the block
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, mx, o);
    const int oi = __shfl_xor_sync(0xffffffffu, am, o);
    if (om > mx || (om == mx && oi < am)) { mx = om; am = oi; }
    mx2 = fmaxf(mx2, __shfl_xor_sync(0xffffffffu, mx2, o));
  }
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) { s_m[w] = mx; s_i[w] = am; s_m2[w] = mx2; }
  __syncthreads();
  mx = s_m[0]; am = s_i[0]; mx2 = s_m2[0];
  for (int i = 1; i < 8; ++i) {
    if (s_m[i] > mx || (s_m[i] == mx && s_i[i] < am)) { mx = s_m[i]; am = s_i[i]; }
    mx2 = fmaxf(mx2, s_m2[i]);
  }
  float S = 0.f, Az = 0.f, Ad = 0.f, S2 = 0.f;
  for (int v = threadIdx.x; v < V; v += blockDim.x) {
    if (v == skip) continue;
    const float a = z[v];
    const float e = expf(a - mx);
    S += e;
    if (e > 0.f) {
      Az = fmaf(e, a, Az);
      if (prev) Ad = fmaf(e, a - z2[v], Ad);
    }
    if (prev) S2 += expf(z2[v] - mx2);
  }
  S = block_sum(S, red);
  Az = block_sum(Az, red);
  Ad = block_sum(Ad, red);
  S2 = block_sum(S2, red);
  if (threadIdx.x == 0) {
    const float lse = mx + logf(S);
    const float conf = 1.f / S;
    const float ent = lse - Az / S;
    float infl = 0.f;
    if (prev && m.have_prev[b]) {
      const float lse2 = mx2 + logf(S2);
      infl = fmaxf(Ad / S - lse + lse2, 0.f);
    }
    // no finite admissible logit (a NaN / inf hidden row): the argmax sentinel must not reach
    // the kernels that index the vocabulary matrix with the id
    if (am < 0 || am >= V || !isfinite(lse)) {
      am = mask_id;
      if (status) atomicMax(status + b, (int)DC_ERR_NUMERIC);
    }
    const int wi = b * m.W_cap + k;
    ws_pred[wi] = am; ws_conf[wi] = conf; ws_ent[wi] = ent; ws_infl[wi] = infl; ws_lse[wi] = lse;
    const int oi = b * out.max_window + k;
    if (out.pred_id) out.pred_id[oi] = am;
    if (out.conf) out.conf[oi] = conf;
    if (out.entropy) out.entropy[oi] = ent;
    if (out.influence) out.influence[oi] = infl;
    if (out.lse) out.lse[oi] = lse;
  }
}

void launch_signals_from_logits(const float* logits, int V, int mask_id, int forbid,
                                const SeqMeta& m, int32_t* ws_pred, float* ws_conf,
                                float* ws_ent, float* ws_infl, float* ws_lse, SignalOut out,
                                int32_t* status, cudaStream_t s) {
  k_signals<<<m.batch * m.W_cap, 256, 0, s>>>(logits, V, mask_id, forbid, m, ws_pred, ws_conf,
                                              ws_ent, ws_infl, ws_lse, out, status);
}

// ---- cross log-probabilities: xlogp[b,i,j] = h_i . W_lm[yhat_j] - lse_i  (Eq. 6 halves) ---------
template <typename T>
__global__ void __launch_bounds__(256) k_xlogp(const T* __restrict__ h,
                                               const T* __restrict__ lm_head,
                                               const int32_t* __restrict__ ws_pred,
                                               const float* __restrict__ ws_lse, int d, int V,
                                               SeqMeta m, int max_window,
                                               float* __restrict__ xlogp) {
  extern __shared__ __align__(16) float wrow[];  // W_lm[yhat_j] as fp32
  const int b = blockIdx.y, j = blockIdx.x;
  const int W = m.win_len[b];
  if (j >= W) return;
  const int tok = ws_pred[b * m.W_cap + j];
  if (tok < 0 || tok >= V) {   // never index the vocabulary matrix with an id outside it
    for (int i = blockIdx.z * (blockDim.x >> 5) + (threadIdx.x >> 5); i < W; i += gridDim.z * (blockDim.x >> 5))
      if ((threadIdx.x & 31) == 0) xlogp[((size_t)b * max_window + i) * max_window + j] = -INFINITY;
    return;
  }
  const T* wr = lm_head + (size_t)tok * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) wrow[i] = to_f<T>(wr[i]);
  __syncthreads();
  // one window position per warp: blockIdx.z picks the group of positions, so that a step's W * W
  // dot products are spread over W * W / 8 CTAs instead of W (the kernel is bound by the latency
  // of a row load, not by bytes: 37 -> 8 us at W = 64)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int i = blockIdx.z * nw + warp; i < W; i += gridDim.z * nw) {
    const T* hr = h + (size_t)lm_row(m, 0, b * m.W_cap + i) * d;
    float acc = 0.f;
    // d is a multiple of 4: four elements per lane and step (8- or 16-byte loads), eight steps
    // in flight at a time (the loop is bound by the latency of the h loads otherwise)
    int e = lane * 4;
    for (; e + 7 * 128 < d; e += 8 * 128) {
      float hv[8][4];
#pragma unroll
      for (int u = 0; u < 8; ++u) load4<T>(hr + e + u * 128, hv[u]);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float4 wv = *reinterpret_cast<const float4*>(wrow + e + u * 128);
        acc = fmaf(hv[u][0], wv.x, acc); acc = fmaf(hv[u][1], wv.y, acc);
        acc = fmaf(hv[u][2], wv.z, acc); acc = fmaf(hv[u][3], wv.w, acc);
      }
    }
    for (; e < d; e += 128) {
      float hv[4];
      load4<T>(hr + e, hv);
      const float4 wv = *reinterpret_cast<const float4*>(wrow + e);
      acc = fmaf(hv[0], wv.x, acc); acc = fmaf(hv[1], wv.y, acc);
      acc = fmaf(hv[2], wv.z, acc); acc = fmaf(hv[3], wv.w, acc);
    }
    acc = warp_sum(acc);
    if (lane == 0)
      xlogp[((size_t)b * max_window + i) * max_window + j] = acc - ws_lse[b * m.W_cap + i];
  }
}

template <typename T>
void launch_xlogp(const T* h, const T* lm_head, const int32_t* ws_pred, const float* ws_lse, int d,
                  int V, const SeqMeta& m, int max_window, float* xlogp, cudaStream_t s) {
  dim3 grid(m.W_cap, m.batch, (m.W_cap + 7) / 8);
  k_xlogp<T><<<grid, 256, d * sizeof(float), s>>>(h, lm_head, ws_pred, ws_lse, d, V, m, max_window,
                                                  xlogp);
}

// ---- export of the last decoded block's K / V into the context cache -----------------------------
// The curr variant's rotated K and V of rows [0, last_len[b]) (the last decoded block, all of its
// tokens clean) are appended to the cache of one layer at keys ctx_len[b] + r.  k: [M, nkv*hd];
// v: row-major [M, nkv*hd] (v_ld = 0) or transposed [nkv*hd, v_ld].
template <typename T>
__global__ void k_export_kv(const T* __restrict__ k, const T* __restrict__ v, int v_ld, SeqMeta m,
                            int nkv, int hd, int max_ctx, T* __restrict__ k_cache,
                            T* __restrict__ v_cache) {
  const int b = blockIdx.y, r = blockIdx.x;
  if (r >= m.last_len[b]) return;
  const int row = act_row(m, 0, b, r);
  const int key = m.ctx_len[b] + r;
  for (int i = threadIdx.x; i < nkv * hd; i += blockDim.x) {
    const int g = i / hd, e = i % hd;
    k_cache[(((size_t)b * nkv + g) * max_ctx + key) * hd + e] = k[(size_t)row * nkv * hd + i];
    const T vv = v_ld ? v[(size_t)i * v_ld + row] : v[(size_t)row * nkv * hd + i];
    v_cache[(((size_t)b * nkv + g) * hd + e) * max_ctx + key] = vv;
  }
}

template <typename T>
void launch_export_kv(const T* k, const T* v, int v_ld, const SeqMeta& m, int nkv, int hd,
                      int max_ctx, T* k_cache, T* v_cache, cudaStream_t s) {
  int maxl = 0;
  for (int b = 0; b < m.batch; ++b) maxl = max(maxl, m.last_len[b]);
  if (maxl == 0) return;
  dim3 grid(maxl, m.batch);
  k_export_kv<T><<<grid, 256, 0, s>>>(k, v, v_ld, m, nkv, hd, max_ctx, k_cache, v_cache);
}
template void launch_export_kv<float>(const float*, const float*, int, const SeqMeta&, int, int, int,
                                      float*, float*, cudaStream_t);
template void launch_export_kv<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, int,
                                              const SeqMeta&, int, int, int, __nv_bfloat16*,
                                              __nv_bfloat16*, cudaStream_t);

// explicit instantiations
#define DC_INST(T)                                                                              \
  template void launch_embed<T>(const T*, const int32_t*, const int32_t*, int, int, int, int,   \
                                int, const SeqMeta&, float*, int32_t*, cudaStream_t);           \
  template void launch_rmsnorm<T>(float*, const float*, int, size_t, const T*, float, int, int, \
                                  T*, cudaStream_t);                                            \
  template void launch_final_norm<T>(float*, const float*, int, size_t, const T*, float, int,   \
                                     const SeqMeta&, T*, cudaStream_t, int);                         \
  template void launch_h_override<T>(const T*, int, int, const SeqMeta&, T*, cudaStream_t);     \
  template void launch_gemm_simt<T>(const T*, const T*, float*, int, int, int, int, int,        \
                                    cudaStream_t);                                              \
  template void launch_rope_store<T>(const float*, const float*, const SeqMeta&, int, int, int, \
                                     const T*, const T*, const T*, T*, T*, T*, cudaStream_t);                                 \
  template void launch_swiglu<T>(const float*, int, int, T*, cudaStream_t);                     \
  template void launch_attn_simt<T>(const T*, const T*, const T*, const T*, const T*, int,      \
                                    const SeqMeta&, int, int, int, T*, cudaStream_t);           \
  template void launch_xlogp<T>(const T*, const T*, const int32_t*, const float*, int, int,     \
                                const SeqMeta&, int, float*, cudaStream_t);
DC_INST(float)
DC_INST(__nv_bfloat16)

}  // namespace dc
