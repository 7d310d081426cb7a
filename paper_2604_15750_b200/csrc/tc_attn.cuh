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
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..9 = softmax / output: two threads per query row (TMEM lane quarter = warp % 4), one
// for each half of the tile's 128 keys (and of O's 128 columns); they meet once per tile to
// agree on the row maximum and once at the end to add their row sums.
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

constexpr int kAttnThreads = 320;
constexpr int kHd = 128;
constexpr int kBK = 128;                       // keys per tile
constexpr int kSub = 128 * 128;                // bytes of one [128 rows x 64 bf16] sub-tile
constexpr int kAttnSmem = 2 * kSub /*Q*/ + 2 * 4 * kSub /*2 stages of K and V^T*/ + 2 * 2 * kSub /*2 x P*/ + 1024;
constexpr int kAttnPrefetch = 4;               // context tiles the L2 prefetch runs ahead of the ring
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
  __shared__ uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], s_empty[2], p_full[2], pv_done;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float xchg[2][128];   // row maximum / row sum of each key half
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
      ptx::mbar_init(&k_full[i], 1); ptx::mbar_init(&k_empty[i], 1);
      ptx::mbar_init(&v_full[i], 1); ptx::mbar_init(&v_empty[i], 1);
      ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&s_empty[i], 256);
      ptx::mbar_init(&p_full[i], 256);
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
    // Two producer lanes with a ring of their own each: a K slot is free again as soon as
    // S = Q K^T of its tile has been computed, a V^T slot only after P V, a softmax later.  With
    // one ring for both, the load of tile t+2 could not start before P V of tile t and its
    // latency sat in the loop (2 us per tile); now K runs ahead of V.
    // Context tiles are also prefetched into L2 kAttnPrefetch tiles ahead (the active tiles were
    // just written: L2-resident).
    if (lane == 0) {
      ptx::mbar_expect_tx(&q_full, 2 * kSub);
      ptx::tma_load_2d(Qs, &map_q, &q_full, h * kHd, row0 + qt * 128);
      ptx::tma_load_2d(Qs + kSub, &map_q, &q_full, h * kHd + 64, row0 + qt * 128);
      auto prefetch_k = [&](int t) {
        if (t < Tc) {
          const int krow = (b * p.nkv + g) * p.max_ctx + t * kBK;
          ptx::tma_prefetch_l2_3d(&map_kc, 0, krow, p.layer);
          ptx::tma_prefetch_l2_3d(&map_kc, 64, krow, p.layer);
        }
      };
      for (int t = 2; t < 2 + kAttnPrefetch; ++t) prefetch_k(t);
      for (int t = 0; t < T; ++t) {
        const int s = t & 1;
        prefetch_k(t + 2 + kAttnPrefetch);
        if (!ptx::mbar_wait(&k_empty[s], (((uint32_t)t >> 1) & 1u) ^ 1u, &abort_flag)) break;
        uint8_t* Ks = KVs + (size_t)s * 4 * kSub;
        ptx::mbar_expect_tx(&k_full[s], 2 * kSub);
        if (t < Tc) {
          const int krow = (b * p.nkv + g) * p.max_ctx + t * kBK;
          ptx::tma_load_3d(Ks, &map_kc, &k_full[s], 0, krow, p.layer);
          ptx::tma_load_3d(Ks + kSub, &map_kc, &k_full[s], 64, krow, p.layer);
        } else {
          const int j0 = (t - Tc) * kBK;
          ptx::tma_load_2d(Ks, &map_k, &k_full[s], g * kHd, row0 + j0);
          ptx::tma_load_2d(Ks + kSub, &map_k, &k_full[s], g * kHd + 64, row0 + j0);
        }
      }
    } else if (lane == 1) {
      auto prefetch_v = [&](int t) {
        if (t < Tc) {
          const int j0 = t * kBK, vrow = (b * p.nkv + g) * kHd;
          ptx::tma_prefetch_l2_3d(&map_vc, j0, vrow, p.layer);
          ptx::tma_prefetch_l2_3d(&map_vc, j0 + 64, vrow, p.layer);
        }
      };
      for (int t = 2; t < 2 + kAttnPrefetch; ++t) prefetch_v(t);
      for (int t = 0; t < T; ++t) {
        const int s = t & 1;
        prefetch_v(t + 2 + kAttnPrefetch);
        if (!ptx::mbar_wait(&v_empty[s], (((uint32_t)t >> 1) & 1u) ^ 1u, &abort_flag)) break;
        uint8_t* Vs = KVs + (size_t)s * 4 * kSub + 2 * kSub;
        ptx::mbar_expect_tx(&v_full[s], 2 * kSub);
        if (t < Tc) {
          const int j0 = t * kBK, vrow = (b * p.nkv + g) * kHd;
          ptx::tma_load_3d(Vs, &map_vc, &v_full[s], j0, vrow, p.layer);
          ptx::tma_load_3d(Vs + kSub, &map_vc, &v_full[s], j0 + 64, vrow, p.layer);
        } else {
          const int j0 = (t - Tc) * kBK;
          ptx::tma_load_2d(Vs, &map_vt, &v_full[s], row0 + j0, g * kHd);
          ptx::tma_load_2d(Vs + kSub, &map_vt, &v_full[s], row0 + j0 + 64, g * kHd);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // lean issue path: this one thread issues 16 MMAs per key tile, so its own instruction
      // stream is the critical path; descriptors are built once and advanced by additions
      const uint32_t idesc = ptx::idesc_bf16(128, 128);
      const uint64_t hi = ptx::smem_desc_sw128_hi();
      const uint64_t dq = hi | (uint64_t)(ptx::smem_u32(Qs) >> 4);
      const uint64_t dk0 = hi | (uint64_t)(ptx::smem_u32(KVs) >> 4);                 // stage 0; stage 1 = + 4*kSub
      const uint64_t dv0 = dk0 + (2 * kSub >> 4);
      const uint64_t dp0 = hi | (uint64_t)(ptx::smem_u32(Ps) >> 4);                  // buffer 0; buffer 1 = + 2*kSub
      const uint32_t b_k_full = ptx::smem_u32(&k_full[0]), b_k_empty = ptx::smem_u32(&k_empty[0]);
      const uint32_t b_v_full = ptx::smem_u32(&v_full[0]), b_v_empty = ptx::smem_u32(&v_empty[0]);
      const uint32_t b_s_full = ptx::smem_u32(&s_full[0]), b_s_empty = ptx::smem_u32(&s_empty[0]);
      const uint32_t b_p_full = ptx::smem_u32(&p_full[0]), b_pv_done = ptx::smem_u32(&pv_done);
      constexpr uint64_t kSubU = kSub >> 4;   // one 64-column sub-tile in descriptor units
      bool ok = ptx::mbar_wait(&q_full, 0, &abort_flag);
      auto issue_qk = [&](int t) {
        const uint32_t s = (uint32_t)t & 1u;
        const uint32_t ph = ((uint32_t)t >> 1) & 1u;
        if (!ptx::mbar_wait_a(b_k_full + 8u * s, ph, &abort_flag)) return false;
        if (!ptx::mbar_wait_a(b_s_empty + 8u * s, ph ^ 1u, &abort_flag)) return false;
        ptx::tc_fence_after();
        const uint64_t dk = dk0 + s * (4 * kSubU);
        const uint32_t d = tmem_base + s * 128;
        ptx::umma_bf16(d, dq, dk, idesc, 0u);
#pragma unroll
        for (int kk = 1; kk < 8; ++kk) {
          const uint64_t off = (uint64_t)(kk >> 2) * kSubU + (uint64_t)(kk & 3) * 2;
          ptx::umma_bf16_acc(d, dq + off, dk + off, idesc);
        }
        ptx::umma_commit_a(b_s_full + 8u * s);
        ptx::umma_commit_a(b_k_empty + 8u * s);   // the K slot is free once S is there
        return true;
      };
      auto issue_pv = [&](int t) {
        const uint32_t s = (uint32_t)t & 1u;
        if (!ptx::mbar_wait_a(b_v_full + 8u * s, ((uint32_t)t >> 1) & 1u, &abort_flag)) return false;
        if (!ptx::mbar_wait_a(b_p_full + 8u * s, ((uint32_t)t >> 1) & 1u, &abort_flag)) return false;
        ptx::tc_fence_after();
        const uint64_t dp = dp0 + s * (2 * kSubU);
        const uint64_t dv = dv0 + s * (4 * kSubU);
        const uint32_t d = tmem_base + 256;
        ptx::umma_bf16(d, dp, dv, idesc, t > 0 ? 1u : 0u);
#pragma unroll
        for (int kk = 1; kk < 8; ++kk) {
          const uint64_t off = (uint64_t)(kk >> 2) * kSubU + (uint64_t)(kk & 3) * 2;
          ptx::umma_bf16_acc(d, dp + off, dv + off, idesc);
        }
        ptx::umma_commit_a(b_pv_done);
        ptx::umma_commit_a(b_v_empty + 8u * s);
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
    const int half = (warp - 2) >> 2;   // which 64 keys of a tile / which 64 columns of O
    const int r = quarter * 32 + lane;  // query row inside the tile = TMEM lane; also V^T row
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int kbase = half * 64;
    float m_run = -INFINITY, l_run = 0.f;   // l_run: this thread's keys only
    bool ok = true;
    // the two threads of a row meet on the named barrier of their lane quarter (64 threads)
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(quarter + 1) : "memory"); };
    // Every iteration executes both pair barriers whatever happened (a wait that gave up makes
    // `ok` false for the whole warp and the work is skipped), so that a failure cannot leave the
    // partner warp waiting on a barrier.
    for (int t = 0; t < T; ++t) {
      const int s = t & 1;
      const uint32_t ph = ((uint32_t)t >> 1) & 1u;
      const bool is_ctx = t < Tc;
      const int valid = is_ctx ? min(kBK, P - t * kBK) : min(kBK, R - (t - Tc) * kBK);
      const int vloc = max(0, min(64, valid - kbase));   // valid keys inside this thread's half
      if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[s], ph, &abort_flag));
      float sv[64];
      float mx = -INFINITY;
      if (ok) {
        ptx::tc_fence_after();
        // this half of the score row into registers, then the TMEM buffer is free for tile t+2
        ptx::tmem_ld_32x32(t_lane + s * 128 + kbase, *reinterpret_cast<float(*)[32]>(&sv[0]));
        ptx::tmem_ld_32x32(t_lane + s * 128 + kbase + 32, *reinterpret_cast<float(*)[32]>(&sv[32]));
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        ptx::mbar_arrive(&s_empty[s]);
        // The softmax warps are bound by instruction issue (85% of the issue slots of their
        // schedulers), so the per-element work is kept to max, fma, ex2, add and half a convert:
        // keys beyond the valid length are set to -inf once (only the last tile of a kind has
        // any; whatever the cache holds there, NaN included, is overwritten), after which they
        // need no further test (ex2(-inf) = 0); maxima and sums run in four independent chains.
        if (vloc < 64) {
#pragma unroll
          for (int j = 0; j < 64; ++j)
            if (j >= vloc) sv[j] = -INFINITY;
        }
        float m0 = sv[0], m1 = sv[1], m2 = sv[2], m3 = sv[3];
#pragma unroll
        for (int j = 4; j < 64; j += 4) {
          m0 = fmaxf(m0, sv[j]); m1 = fmaxf(m1, sv[j + 1]);
          m2 = fmaxf(m2, sv[j + 2]); m3 = fmaxf(m3, sv[j + 3]);
        }
        mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
      }
      xchg[half][r] = mx;
      pair_sync();
      mx = fmaxf(mx, xchg[half ^ 1][r]);
      pair_sync();   // the partner has read before the next tile overwrites
      if (!ok) continue;
      const float m_tile = mx * p.scale_log2;
      // raise the running maximum only when the tile exceeds it by more than the gap
      const bool raise = m_tile > m_run + kRescaleGap;   // true on the first tile (m_run = -inf)
      const float m_new = raise ? m_tile : m_run;
      const float alpha = raise ? attn_ex2(m_run - m_new) : 1.f;  // 0 on the first tile
      float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
      const float scale = p.scale_log2, neg_m = -m_new;
      // keys [kbase, kbase+64) are sub-tile `half` of the P buffer: 8 chunks of 8 keys per row
      uint8_t* prow = Ps + (size_t)s * 2 * kSub + half * kSub + r * 128;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t packed[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          const int k0 = c * 32 + j;
          const float p0 = attn_ex2(fmaf(sv[k0], scale, neg_m));
          const float p1 = attn_ex2(fmaf(sv[k0 + 1], scale, neg_m));
          if ((j & 6) == 0) l0 += p0 + p1;
          else if ((j & 6) == 2) l1 += p0 + p1;
          else if ((j & 6) == 4) l2 += p0 + p1;
          else l3 += p0 + p1;
          __nv_bfloat162 pr = __floats2bfloat162_rn(p0, p1);
          packed[j >> 1] = *reinterpret_cast<uint32_t*>(&pr);
        }
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const int chunk = (c * 4 + q4) ^ (r & 7);
          *reinterpret_cast<uint4*>(prow + (chunk << 4)) =
              make_uint4(packed[q4 * 4], packed[q4 * 4 + 1], packed[q4 * 4 + 2], packed[q4 * 4 + 3]);
        }
      }
      l_run = l_run * alpha + ((l0 + l1) + (l2 + l3));
      m_run = m_new;
      if (is_ctx && valid < kBK) {
        // cached keys beyond ctx_len: zero the V^T columns so that 0 * garbage cannot make NaN
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&v_full[s], ph, &abort_flag));
        if (ok) {
          uint8_t* vrow = KVs + (size_t)s * 4 * kSub + 2 * kSub + half * kSub + r * 128;
          for (int cc = vloc; cc < 64; ++cc)
            *reinterpret_cast<uint16_t*>(vrow + (((cc >> 3) ^ (r & 7)) << 4) + (cc & 7) * 2) = 0;
        }
      }
      if (ok && t > 0) {
        // P V of the previous tile is complete: O may be rescaled, and the P buffer this thread
        // writes next (tile t+1) is no longer read
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&pv_done, (uint32_t)(t - 1) & 1u, &abort_flag));
        if (ok && __any_sync(0xffffffffu, raise)) {
          ptx::tc_fence_after();
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            float ov[32];
            ptx::tmem_ld_32x32(t_lane + 256 + kbase + c * 32, ov);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] *= alpha;
            ptx::tmem_st_32x32(t_lane + 256 + kbase + c * 32, ov);
          }
          ptx::tmem_st_wait();
          ptx::tc_fence_before();
        }
      }
      if (ok) {
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(&p_full[s]);
      }
    }
    if (ok && T > 0) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&pv_done, (uint32_t)(T - 1) & 1u, &abort_flag));
    // row sum = the two halves' sums
    xchg[half][r] = l_run;
    pair_sync();
    const float l_all = l_run + xchg[half ^ 1][r];
    const int rq = qt * 128 + r;
    if (ok && T > 0) {
      ptx::tc_fence_after();
      const float inv = 1.f / l_all;
      __nv_bfloat16* dst = p.o + (size_t)(row0 + rq) * p.nq * kHd + (size_t)h * kHd + kbase;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float ov[32];
        ptx::tmem_ld_32x32(t_lane + 256 + kbase + c * 32, ov);
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
