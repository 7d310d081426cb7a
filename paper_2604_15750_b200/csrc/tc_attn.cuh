// Bidirectional block attention on tcgen05: every active query row of one (variant, sequence,
// head) attends all cached context keys of the sequence and all active keys of its own variant
// (no causal mask), streaming K / V^T tiles of 128 keys through shared memory with TMA.
//
// One CTA = one (query tile of 128 rows, query head, variant * sequence).  Per key tile:
//   S = Q K^T        tcgen05.mma, fp32 in TMEM (two buffers)
//   P = exp2(S - m)  softmax warps: thread <-> query row; S is read from TMEM once and held in
//                    registers; P is rounded to bf16 into shared memory (two buffers) in the
//                    swizzled K-major layout
//   O += P V         tcgen05.mma accumulating in TMEM over all tiles (V is kept transposed, keys
//                    contiguous)
// The running maximum m is only raised when a tile exceeds it by more than 2^8 (P stays within
// bf16 / fp32 range either way); only then is O rescaled, in TMEM, by the row's own thread.  So
// the common path of a tile never reads O, and the softmax of tile t+1 overlaps P V of tile t.
// Keys beyond the valid length are masked to -inf in S, and the V^T columns of cached keys
// beyond ctx_len are zeroed in shared memory (the cache may hold anything there).
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = softmax / output.
#pragma once
#include "kernels.h"
#include "tc_ptx.cuh"

namespace dc {

struct AttnParams {
  SeqMeta m;
  int nq, nkv;
  int max_ctx;
  int layer;
  float scale_log2;        // log2(e) / sqrt(head_dim)
  __nv_bfloat16* o;        // [M, nq * 128]
  int32_t* status;
};

constexpr int kAttnThreads = 192;
constexpr int kHd = 128;
constexpr int kBK = 128;                       // keys per tile
constexpr int kSub = 128 * 128;                // bytes of one [128 rows x 64 bf16] sub-tile
constexpr int kAttnSmem = 2 * kSub /*Q*/ + 2 * 4 * kSub /*2 stages of K and V^T*/ + 2 * 2 * kSub /*2 x P*/ + 1024;
constexpr float kRescaleGap = 8.f;             // log2 units the tile maximum may exceed m before m moves

__device__ __forceinline__ float attn_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kAttnThreads, 1)
k_attn_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
          const __grid_constant__ CUtensorMap map_vt, const __grid_constant__ CUtensorMap map_kc,
          const __grid_constant__ CUtensorMap map_vc, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t q_full, kv_full[2], kv_empty[2], s_full[2], s_empty[2], p_full[2], pv_done;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* Qs = smem;
  uint8_t* KVs = smem + 2 * kSub;          // stage s: K at KVs + s*4*kSub, V^T at + 2*kSub
  uint8_t* Ps = smem + 2 * kSub + 8 * kSub;  // buffer s at Ps + s*2*kSub

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, h = blockIdx.y, vb = blockIdx.z;
  const int b = vb % p.m.batch, vv = vb / p.m.batch;
  const int g = h / (p.nq / p.nkv);
  const int P = p.m.ctx_len[b], R = p.m.last_len[b] + p.m.win_len[b];
  const int row0 = act_row(p.m, vv, b, 0);
  const int Tc = (P + kBK - 1) / kBK, Ta = (R + kBK - 1) / kBK;
  const int T = Tc + Ta;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(&q_full, 1);
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&kv_full[i], 1); ptx::mbar_init(&kv_empty[i], 1);
      ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&s_empty[i], 128);
      ptx::mbar_init(&p_full[i], 128);
    }
    ptx::mbar_init(&pv_done, 1);
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tmem_base_s, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;

  if (warp == 0) {
    if (lane == 0) {
      ptx::mbar_expect_tx(&q_full, 2 * kSub);
      ptx::tma_load_2d(Qs, &map_q, &q_full, h * kHd, row0 + qt * 128);
      ptx::tma_load_2d(Qs + kSub, &map_q, &q_full, h * kHd + 64, row0 + qt * 128);
      for (int t = 0; t < T; ++t) {
        const int s = t & 1;
        if (!ptx::mbar_wait(&kv_empty[s], (((uint32_t)t >> 1) & 1u) ^ 1u, &abort_flag)) break;
        uint8_t* Ks = KVs + (size_t)s * 4 * kSub;
        uint8_t* Vs = Ks + 2 * kSub;
        ptx::mbar_expect_tx(&kv_full[s], 4 * kSub);
        if (t < Tc) {
          const int j0 = t * kBK;
          const int krow = (b * p.nkv + g) * p.max_ctx + j0;
          ptx::tma_load_3d(Ks, &map_kc, &kv_full[s], 0, krow, p.layer);
          ptx::tma_load_3d(Ks + kSub, &map_kc, &kv_full[s], 64, krow, p.layer);
          const int vrow = (b * p.nkv + g) * kHd;
          ptx::tma_load_3d(Vs, &map_vc, &kv_full[s], j0, vrow, p.layer);
          ptx::tma_load_3d(Vs + kSub, &map_vc, &kv_full[s], j0 + 64, vrow, p.layer);
        } else {
          const int j0 = (t - Tc) * kBK;
          ptx::tma_load_2d(Ks, &map_k, &kv_full[s], g * kHd, row0 + j0);
          ptx::tma_load_2d(Ks + kSub, &map_k, &kv_full[s], g * kHd + 64, row0 + j0);
          ptx::tma_load_2d(Vs, &map_vt, &kv_full[s], row0 + j0, g * kHd);
          ptx::tma_load_2d(Vs + kSub, &map_vt, &kv_full[s], row0 + j0 + 64, g * kHd);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = ptx::idesc_bf16(128, 128);
      const uint32_t q_addr = ptx::smem_u32(Qs);
      bool ok = ptx::mbar_wait(&q_full, 0, &abort_flag);
      auto issue_qk = [&](int t) {
        const int s = t & 1;
        const uint32_t ph = ((uint32_t)t >> 1) & 1u;
        if (!ptx::mbar_wait(&kv_full[s], ph, &abort_flag)) return false;
        if (!ptx::mbar_wait(&s_empty[s], ph ^ 1u, &abort_flag)) return false;
        ptx::tc_fence_after();
        const uint32_t k_addr = ptx::smem_u32(KVs + (size_t)s * 4 * kSub);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t off = (kk >> 2) * kSub + (kk & 3) * 32;
          ptx::umma_bf16(tmem_base + s * 128, ptx::smem_desc_sw128(q_addr + off),
                         ptx::smem_desc_sw128(k_addr + off), idesc, kk > 0 ? 1u : 0u);
        }
        ptx::umma_commit(&s_full[s]);
        return true;
      };
      auto issue_pv = [&](int t) {
        const int s = t & 1;
        if (!ptx::mbar_wait(&p_full[s], ((uint32_t)t >> 1) & 1u, &abort_flag)) return false;
        ptx::tc_fence_after();
        const uint32_t p_addr = ptx::smem_u32(Ps + (size_t)s * 2 * kSub);
        const uint32_t v_addr = ptx::smem_u32(KVs + (size_t)s * 4 * kSub + 2 * kSub);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t off = (kk >> 2) * kSub + (kk & 3) * 32;
          ptx::umma_bf16(tmem_base + 256, ptx::smem_desc_sw128(p_addr + off),
                         ptx::smem_desc_sw128(v_addr + off), idesc, (t > 0 || kk > 0) ? 1u : 0u);
        }
        ptx::umma_commit(&pv_done);
        ptx::umma_commit(&kv_empty[s]);
        return true;
      };
      if (ok && T > 0) ok = issue_qk(0);
      for (int t = 0; t < T && ok; ++t) {
        if (t + 1 < T) ok = issue_qk(t + 1);
        if (ok) ok = issue_pv(t);
      }
    }
  } else {
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;  // query row inside the tile = TMEM lane; also V^T row
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int t = 0; t < T && ok; ++t) {
      const int s = t & 1;
      const uint32_t ph = ((uint32_t)t >> 1) & 1u;
      const bool is_ctx = t < Tc;
      const int valid = is_ctx ? min(kBK, P - t * kBK) : min(kBK, R - (t - Tc) * kBK);
      ok = ptx::mbar_wait(&s_full[s], ph, &abort_flag);
      if (!ok) break;
      ptx::tc_fence_after();
      // the whole score row into registers, then the TMEM buffer is free for Q K^T of tile t+2
      float sv[128];
#pragma unroll
      for (int c = 0; c < 4; ++c)
        ptx::tmem_ld_32x32(t_lane + s * 128 + c * 32, *reinterpret_cast<float(*)[32]>(&sv[c * 32]));
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      ptx::mbar_arrive(&s_empty[s]);
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 128; ++j)
        if (j < valid) mx = fmaxf(mx, sv[j]);
      const float m_tile = mx * p.scale_log2;
      // raise the running maximum only when the tile exceeds it by more than the gap
      const bool raise = m_tile > m_run + kRescaleGap;   // true on the first tile (m_run = -inf)
      const float m_new = raise ? m_tile : m_run;
      const float alpha = raise ? attn_ex2(m_run - m_new) : 1.f;  // 0 on the first tile
      float l_tile = 0.f;
      uint8_t* pbuf = Ps + (size_t)s * 2 * kSub;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t packed[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          const int k0 = c * 32 + j;
          const float p0 = (k0 < valid) ? attn_ex2(fmaf(sv[k0], p.scale_log2, -m_new)) : 0.f;
          const float p1 = (k0 + 1 < valid) ? attn_ex2(fmaf(sv[k0 + 1], p.scale_log2, -m_new)) : 0.f;
          l_tile += p0 + p1;
          __nv_bfloat162 pr = __floats2bfloat162_rn(p0, p1);
          packed[j >> 1] = *reinterpret_cast<uint32_t*>(&pr);
        }
        // keys [c*32, c*32+32) = 4 chunks of 8 keys; sub-tile c/2, chunk index (c%2)*4 + q
        uint8_t* prow = pbuf + (c >> 1) * kSub + r * 128;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const int chunk = ((c & 1) * 4 + q4) ^ (r & 7);
          *reinterpret_cast<uint4*>(prow + (chunk << 4)) =
              make_uint4(packed[q4 * 4], packed[q4 * 4 + 1], packed[q4 * 4 + 2], packed[q4 * 4 + 3]);
        }
      }
      l_run = l_run * alpha + l_tile;
      m_run = m_new;
      if (is_ctx && valid < kBK) {
        // cached keys beyond ctx_len: zero the V^T columns so that 0 * garbage cannot make NaN
        ok = ptx::mbar_wait(&kv_full[s], ph, &abort_flag);
        uint8_t* vrow_base = KVs + (size_t)s * 4 * kSub + 2 * kSub;
        for (int cidx = valid; cidx < kBK; ++cidx) {
          const int cc = cidx & 63;
          uint8_t* a = vrow_base + (cidx >> 6) * kSub + r * 128 + (((cc >> 3) ^ (r & 7)) << 4) + (cc & 7) * 2;
          *reinterpret_cast<uint16_t*>(a) = 0;
        }
      }
      if (t > 0) {
        // P V of the previous tile is complete: O may be rescaled, and the P buffer this thread
        // writes next (tile t+1) is no longer read
        ok = ok && ptx::mbar_wait(&pv_done, (uint32_t)(t - 1) & 1u, &abort_flag);
        if (!ok) break;
        if (__any_sync(0xffffffffu, raise)) {
          ptx::tc_fence_after();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            float ov[32];
            ptx::tmem_ld_32x32(t_lane + 256 + c * 32, ov);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] *= alpha;
            ptx::tmem_st_32x32(t_lane + 256 + c * 32, ov);
          }
          ptx::tmem_st_wait();
          ptx::tc_fence_before();
        }
      }
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(&p_full[s]);
    }
    if (ok && T > 0) ok = ptx::mbar_wait(&pv_done, (uint32_t)(T - 1) & 1u, &abort_flag);
    const int rq = qt * 128 + r;
    if (ok && T > 0) {
      ptx::tc_fence_after();
      const float inv = 1.f / l_run;
      __nv_bfloat16* dst = p.o + (size_t)(row0 + rq) * p.nq * kHd + (size_t)h * kHd;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float ov[32];
        ptx::tmem_ld_32x32(t_lane + 256 + c * 32, ov);
        ptx::tmem_ld_wait();
        if (rq < p.m.R_cap) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              __nv_bfloat162 pr = __floats2bfloat162_rn(ov[i + 2 * j] * inv, ov[i + 2 * j + 1] * inv);
              w[j] = *reinterpret_cast<uint32_t*>(&pr);
            }
            *reinterpret_cast<uint4*>(dst + c * 32 + i) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && abort_flag && p.status) atomicExch(p.status, DC_ERR_TIMEOUT);
}

}  // namespace dc
