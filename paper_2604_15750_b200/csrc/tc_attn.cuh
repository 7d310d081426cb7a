// Bidirectional block attention on tcgen05: every active query row attends all cached context
// keys of its sequence and all active keys of its own variant (no causal mask), streaming K / V^T
// tiles of 128 keys through shared memory with TMA.
//
// One CTA = one query tile of 128 rows of one (sequence, query head): 128 rows of one variant, or -
// when a variant has 64 rows or fewer left in this row tile - the rows of BOTH variants packed into
// one tile (curr rows in lanes 0..63, prev rows in lanes 64..127), which then shares every staged
// context tile between the variants and masks, per row, the active keys of the other variant.
//
// Per key tile:
//   S = Q K^T        tcgen05.mma, fp32 in TMEM (three buffers of 128 columns)
//   P = exp2(S - m)  softmax warps: thread <-> (row, quarter of the keys); the scores are read from
//                    TMEM once, the probabilities go back into TMEM as packed bf16 over the
//                    thread's own score columns
//   O += P V         tcgen05.mma with the A operand in TMEM, accumulating over all tiles
// S has three buffers and runs two tiles ahead, so the softmax never waits for the scores: with
// two buffers S of tile t + 2 could only start after P V of tile t, i.e. after the softmax of tile
// t, and the period was half of (softmax + issue of both MMA groups) plus the load waits.  The
// running maximum m only moves when a tile exceeds it by more than 2^8 (then the row's own
// threads rescale O in TMEM).  Keys beyond the valid length are masked to -inf in S, and the V^T
// columns of cached keys beyond ctx_len are zeroed in shared memory (the cache may hold anything
// there).
//
// Warp roles (640 threads): warp 0 = TMA producer for Q and K, warp 1 = TMEM owner + issuer of the
// score MMAs (Q K^T), warp 2 = TMA producer for V^T, warp 3 = issuer of the output MMAs (P V; all
// its lanes first clear the V^T columns beyond ctx_len in the one tile that has any), warps 4..19 =
// softmax / output: four threads per row (TMEM lane quarter = warp % 4), one for each quarter of a
// tile's keys and of O's columns.  Two issuing threads because one was the bottleneck: with its
// four barrier waits and two commits per tile it needed about 2270 clocks per tile for MMAs that
// keep the tensor pipe busy for 1024.
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

constexpr int kAttnThreads = 640;
constexpr int kHd = 128;
constexpr int kBK = 128;                       // keys per tile
constexpr int kSub = 128 * 128;                // bytes of one [128 rows x 64 bf16] sub-tile
constexpr int kAttnStagesK = 3, kAttnStagesV = 2;   // ring slots of K and of V^T
constexpr int kAttnSmem = 2 * kSub /*Q*/ + kAttnStagesK * 2 * kSub + kAttnStagesV * 2 * kSub + 1024;
constexpr int kAttnPrefetch = 0;               // context tiles the L2 prefetch runs ahead of the tile after the ring
                                               // (measured: 0 -> 1.36 ms, 4 -> 1.41 ms, 8 -> 1.46 ms on 4 x 4096 keys x 8 layers)
constexpr float kRescaleGap = 8.f;             // log2 units the tile maximum may exceed m before m moves

__device__ __forceinline__ float attn_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 32 lanes x 16 consecutive 32-bit columns, registers -> TMEM
__device__ __forceinline__ void attn_tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),
        "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]),
        "r"(r[14]), "r"(r[15])
      : "memory");
}

// What a CTA works on: its query tile and its sequence of key tiles.  blockIdx.x = 2 * row tile +
// variant with two variants in the pass, = row tile with one.
struct AttnUnit {
  int packed;        // both variants' rows of this row tile in one query tile
  int Tc, Ta, T;     // context tiles, active tiles per variant, all tiles of this CTA
  int P, R;
  // row half hh (tile rows 64 hh .. 64 hh + 63): variant, first row, valid rows
  int v[2], q[2], n[2];
};
struct AttnTile { int is_ctx, kv, u, valid; };

__device__ __forceinline__ bool attn_unit(const SeqMeta& m, int b, int u, AttnUnit& a) {
  const int P = m.ctx_len[b], R = m.last_len[b] + m.win_len[b];
  const int nqt = (R + 127) / 128;
  a.P = P; a.R = R;
  a.Tc = (P + kBK - 1) / kBK; a.Ta = nqt;
  const int t = m.nv == 2 ? (u >> 1) : u, var = m.nv == 2 ? (u & 1) : 0;
  if (t >= nqt) return false;
  const int rows = min(128, R - 128 * t);
  a.packed = (m.nv == 2 && rows <= 64) ? 1 : 0;
  if (a.packed) {
    if (var != 0) return false;          // the curr CTA of this row tile carries both variants
    a.v[0] = 0; a.v[1] = 1; a.q[0] = a.q[1] = 128 * t; a.n[0] = a.n[1] = rows;
    a.T = a.Tc + 2 * a.Ta;
  } else {
    a.v[0] = a.v[1] = var; a.q[0] = 128 * t; a.q[1] = 128 * t + 64;
    a.n[0] = min(64, rows); a.n[1] = max(0, rows - 64);
    a.T = a.Tc + a.Ta;
  }
  return true;
}

__device__ __forceinline__ AttnTile attn_tile(const AttnUnit& a, int j) {
  AttnTile t;
  if (j < a.Tc) {
    t.is_ctx = 1; t.kv = 0; t.u = j; t.valid = min(kBK, a.P - j * kBK);
    return t;
  }
  const int jj = j - a.Tc;
  t.is_ctx = 0;
  if (a.packed) { t.kv = jj & 1; t.u = jj >> 1; }       // the active tiles of both variants
  else { t.kv = a.v[0]; t.u = jj; }
  t.valid = min(kBK, a.R - t.u * kBK);
  return t;
}

__global__ void __launch_bounds__(kAttnThreads, 1)
k_attn_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
          const __grid_constant__ CUtensorMap map_vt, const __grid_constant__ CUtensorMap map_kc,
          const __grid_constant__ CUtensorMap map_vc, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t q_full, k_full[kAttnStagesK], k_empty[kAttnStagesK], v_loc[kAttnStagesV],
      s_full[3], p_full[3], pv_done[3], o_done;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float xchg[2][4][128];   // [tile parity][key quarter][row]: row maximum / row sum of each quarter

  const int b = blockIdx.z, h = blockIdx.y;
  AttnUnit un;
  if (!attn_unit(p.m, b, blockIdx.x, un)) return;   // nothing of this sequence in this unit (uniform)

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* Qs = smem;
  uint8_t* Ks = smem + 2 * kSub;                       // slot s at Ks + s * 2 * kSub
  uint8_t* Vs = Ks + kAttnStagesK * 2 * kSub;          // slot s at Vs + s * 2 * kSub

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = h / (p.nq / p.nkv);
  const int T = un.T;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(&q_full, 1);
    for (int i = 0; i < kAttnStagesK; ++i) { ptx::mbar_init(&k_full[i], 1); ptx::mbar_init(&k_empty[i], 1); }
    for (int i = 0; i < kAttnStagesV; ++i) ptx::mbar_init(&v_loc[i], 1);
    for (int i = 0; i < 3; ++i) {
      ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&p_full[i], 16); ptx::mbar_init(&pv_done[i], 1);
    }
    ptx::mbar_init(&o_done, 1);
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
  // TMEM columns: S / P of tile j in buffer j % 3 (columns 0..127, 128..255, 256..383), O 384..511

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- Q, then the K ring ----------------
      ptx::mbar_expect_tx(&q_full, 2 * kSub);
      for (int hh = 0; hh < 2; ++hh) {
        const int row = act_row(p.m, un.v[hh], b, un.q[hh]);
        ptx::tma_load_2d(Qs + hh * 8192, &map_q, &q_full, h * kHd, row);
        ptx::tma_load_2d(Qs + kSub + hh * 8192, &map_q, &q_full, h * kHd + 64, row);
      }
      auto prefetch_k = [&](int t) {
        if (t < un.Tc) {
          const int krow = (b * p.nkv + g) * p.max_ctx + t * kBK;
          ptx::tma_prefetch_l2_3d(&map_kc, 0, krow, p.layer);
          ptx::tma_prefetch_l2_3d(&map_kc, 64, krow, p.layer);
        }
      };
      for (int t = kAttnStagesK; t < kAttnStagesK + kAttnPrefetch; ++t) prefetch_k(t);
      for (int j = 0; j < T; ++j) {
        const int s = j % kAttnStagesK;
        const AttnTile t = attn_tile(un, j);
        prefetch_k(j + kAttnStagesK + kAttnPrefetch);
        if (!ptx::mbar_wait(&k_empty[s], (((uint32_t)(j / kAttnStagesK)) & 1u) ^ 1u, &abort_flag)) break;
        uint8_t* dst = Ks + (size_t)s * 2 * kSub;
        ptx::mbar_expect_tx(&k_full[s], 2 * kSub);
        if (t.is_ctx) {
          const int krow = (b * p.nkv + g) * p.max_ctx + t.u * kBK;
          ptx::tma_load_3d(dst, &map_kc, &k_full[s], 0, krow, p.layer);
          ptx::tma_load_3d(dst + kSub, &map_kc, &k_full[s], 64, krow, p.layer);
        } else {
          const int row = act_row(p.m, t.kv, b, t.u * kBK);
          ptx::tma_load_2d(dst, &map_k, &k_full[s], g * kHd, row);
          ptx::tma_load_2d(dst + kSub, &map_k, &k_full[s], g * kHd + 64, row);
        }
      }
    }
  } else if (warp == 2) {
    if (lane == 0) {
      // ---------------- the V^T ring ----------------
      auto prefetch_v = [&](int t) {
        if (t < un.Tc) {
          const int j0 = t * kBK, vrow = (b * p.nkv + g) * kHd;
          ptx::tma_prefetch_l2_3d(&map_vc, j0, vrow, p.layer);
          ptx::tma_prefetch_l2_3d(&map_vc, j0 + 64, vrow, p.layer);
        }
      };
      for (int t = kAttnStagesV; t < kAttnStagesV + kAttnPrefetch; ++t) prefetch_v(t);
      for (int j = 0; j < T; ++j) {
        const int s = j % kAttnStagesV;
        const AttnTile t = attn_tile(un, j);
        prefetch_v(j + kAttnStagesV + kAttnPrefetch);
        // the slot held tile j - 2: free once its P V has completed
        if (j >= kAttnStagesV &&
            !ptx::mbar_wait(&pv_done[(j - 2) % 3], ((uint32_t)(j - 2) / 3u) & 1u, &abort_flag)) break;
        uint8_t* dst = Vs + (size_t)s * 2 * kSub;
        ptx::mbar_expect_tx(&v_loc[s], 2 * kSub);
        if (t.is_ctx) {
          const int j0 = t.u * kBK, vrow = (b * p.nkv + g) * kHd;
          ptx::tma_load_3d(dst, &map_vc, &v_loc[s], j0, vrow, p.layer);
          ptx::tma_load_3d(dst + kSub, &map_vc, &v_loc[s], j0 + 64, vrow, p.layer);
        } else {
          const int col = act_row(p.m, t.kv, b, t.u * kBK);
          ptx::tma_load_2d(dst, &map_vt, &v_loc[s], col, g * kHd);
          ptx::tma_load_2d(dst + kSub, &map_vt, &v_loc[s], col + 64, g * kHd);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- issuer of S = Q K^T ----------------
      // Lean issue path (the issuing thread does not run ahead of the tensor core): descriptor low
      // words are kept in registers and advanced by 32-bit additions of constants.
      const uint32_t idesc = ptx::idesc_bf16(128, 128);
      const uint32_t hi32 = ptx::smem_desc_hi32();
      const uint32_t q_lo = ptx::smem_desc_lo(ptx::smem_u32(Qs));
      const uint32_t k_lo = ptx::smem_desc_lo(ptx::smem_u32(Ks));
      constexpr uint32_t kSub16 = kSub >> 4;
      const uint32_t b_k_full = ptx::smem_u32(&k_full[0]), b_s_full = ptx::smem_u32(&s_full[0]);
      const uint32_t b_pv_done = ptx::smem_u32(&pv_done[0]);
      bool ok = ptx::mbar_wait(&q_full, 0, &abort_flag);
      for (int j = 0; j < T && ok; ++j) {
        const uint32_t s = (uint32_t)(j % kAttnStagesK), sb = (uint32_t)j % 3u;
        // score buffer j % 3 last held P of tile j - 3: its P V (issued by another thread) must be done
        if (j >= 3 && !ptx::mbar_wait_a(b_pv_done + 8u * sb, ((uint32_t)(j - 3) / 3u) & 1u, &abort_flag)) break;
        if (!ptx::mbar_wait_a(b_k_full + 8u * s, ((uint32_t)(j / kAttnStagesK)) & 1u, &abort_flag)) break;
        ptx::tc_fence_after();
        const uint32_t d = tmem_base + sb * 128u, bk = k_lo + s * (2 * kSub16);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t off = (uint32_t)(kk >> 2) * kSub16 + (uint32_t)(kk & 3) * 2u;
          ptx::umma_bf16_lo(d, q_lo + off, bk + off, hi32, idesc, kk > 0 ? 1u : 0u);
        }
        // (the K slot is handed back by a softmax thread that has seen S)
        ptx::umma_commit_a(b_s_full + 8u * sb);
      }
    }
  } else if (warp == 3) {
    // ---------------- issuer of O (+)= P V ----------------
    // P sits in the score columns of its threads: keys 32 q + 2 c, + 1 in column 32 q + c.
    static_assert(kAttnStagesV == 2, "the slot of tile j is the slot of tile j - 2");
    const uint32_t idesc = ptx::idesc_bf16(128, 128);
    const uint32_t hi32 = ptx::smem_desc_hi32();
    const uint32_t v_lo = ptx::smem_desc_lo(ptx::smem_u32(Vs));
    constexpr uint32_t kSub16 = kSub >> 4;
    const uint32_t b_v_loc = ptx::smem_u32(&v_loc[0]), b_p_full = ptx::smem_u32(&p_full[0]);
    const uint32_t b_pv_done = ptx::smem_u32(&pv_done[0]);
    bool ok = true;
    for (int j = 0; j < T && ok; ++j) {
      const uint32_t s = (uint32_t)(j % kAttnStagesV), ph = ((uint32_t)(j / kAttnStagesV)) & 1u;
      const uint32_t sb = (uint32_t)j % 3u;
      const AttnTile t = attn_tile(un, j);
      if (t.is_ctx && t.valid < kBK) {
        // The one context tile with cached keys beyond ctx_len: all lanes zero those V^T columns
        // (0 * whatever the cache holds there, NaN included, must not reach O).
        ok = __all_sync(0xffffffffu, ptx::mbar_wait_a(b_v_loc + 8u * s, ph, &abort_flag));
        if (!ok) break;
        uint8_t* base = Vs + (size_t)s * 2 * kSub;
        for (int rr = lane; rr < 128; rr += 32)
          for (int cc = t.valid; cc < kBK; ++cc) {
            const int c6 = cc & 63;
            *reinterpret_cast<uint16_t*>(base + (cc >> 6) * kSub + rr * 128 + (((c6 >> 3) ^ (rr & 7)) << 4) + (c6 & 7) * 2) = 0;
          }
        ptx::fence_proxy_async_smem();
        __syncwarp();
      }
      if (lane == 0) {
        ok = ptx::mbar_wait_a(b_p_full + 8u * sb, ((uint32_t)j / 3u) & 1u, &abort_flag) &&
             ptx::mbar_wait_a(b_v_loc + 8u * s, ph, &abort_flag);
        if (ok) {
          ptx::tc_fence_after();
          const uint32_t d = tmem_base + 384u, a = tmem_base + sb * 128u, bv = v_lo + s * (2 * kSub16);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (uint32_t)(kk >> 2) * kSub16 + (uint32_t)(kk & 3) * 2u;
            ptx::umma_bf16_ts_lo(d, a + (uint32_t)(kk >> 1) * 32u + (uint32_t)(kk & 1) * 8u, bv + off, hi32, idesc,
                                 (kk > 0 || j > 0) ? 1u : 0u);
          }
          // also tells the V^T producer that the slot is free, the score issuer that the buffer
          // is, and the softmax warps that O may be rescaled
          ptx::umma_commit_a(b_pv_done + 8u * sb);
        }
      }
      // the other lanes wait here (not spinning) while lane 0 issues
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    }
    if (ok && lane == 0) ptx::umma_commit(&o_done);
  } else {
    // ---------------- softmax / output warps ----------------
    const int gw = warp - 4;
    const int quarter = gw & 3;         // = warp % 4: the TMEM lanes this warp can reach
    const int kq = gw >> 2;             // which 32 keys of a tile / which 32 columns of O
    const int r = quarter * 32 + lane;  // query row inside the tile = TMEM lane
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t o_addr = t_lane + 384u + (uint32_t)kq * 32u;
    const int kbase = kq * 32;
    const int my_variant = un.v[r >> 6];
    float m_run = -INFINITY, l_run = 0.f;   // l_run: this thread's keys only
    bool ok = true;
    // the four threads of a row meet on the named barrier of their lane quarter (128 threads)
    auto row_sync = [&]() { asm volatile("bar.sync %0, 128;" ::"r"(1 + quarter) : "memory"); };
    // Every tile executes both row barriers whatever happened (a wait that gave up makes `ok`
    // false for the whole warp and the work is skipped), so that a failure cannot leave the
    // partner warps waiting on a barrier.
    for (int j = 0; j < T; ++j) {
      const AttnTile t = attn_tile(un, j);
      const uint32_t sb = (uint32_t)j % 3u;
      const uint32_t s_addr = t_lane + sb * 128u + (uint32_t)kq * 32u;   // this thread's score columns
      // packed unit: an active key tile of the other variant contributes nothing to this warp's rows
      const bool other = un.packed && !t.is_ctx && t.kv != my_variant;
      const int nc = other ? 0 : max(0, min(32, t.valid - kbase));   // valid keys inside this thread's quarter
      if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[sb], ((uint32_t)j / 3u) & 1u, &abort_flag));
      // S of this tile is complete, so its K slot has been read: hand it back to the producer
      if (ok && gw == 0 && lane == 0) ptx::mbar_arrive(&k_empty[j % kAttnStagesK]);
      float sv[32];
      if (ok && nc > 0) {
        ptx::tc_fence_after();
        ptx::tmem_ld_32x32(s_addr, sv);
        ptx::tmem_ld_wait();
      }
      // keys beyond the valid length (only the last tile of a kind has any; whatever the cache holds
      // there, NaN included) are set to -inf once; ex2(-inf) = 0, so they need no further test
      if (nc < 32) {
#pragma unroll
        for (int jj = 0; jj < 32; ++jj)
          if (jj >= nc) sv[jj] = -INFINITY;
      }
      float m0 = sv[0], m1 = sv[1], m2 = sv[2], m3 = sv[3];
#pragma unroll
      for (int jj = 4; jj < 32; jj += 4) {
        m0 = fmaxf(m0, sv[jj]); m1 = fmaxf(m1, sv[jj + 1]);
        m2 = fmaxf(m2, sv[jj + 2]); m3 = fmaxf(m3, sv[jj + 3]);
      }
      float mx = ok ? fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) : -INFINITY;
      // (two exchange buffers: the partners have passed the barrier of tile j + 1, hence read tile
      // j's values, before anyone writes tile j + 2's)
      float (*xc)[128] = xchg[j & 1];
      xc[kq][r] = mx;
      row_sync();
      mx = fmaxf(fmaxf(xc[0][r], xc[1][r]), fmaxf(xc[2][r], xc[3][r]));
      if (!ok) continue;
      const float m_tile = mx * p.scale_log2;
      // raise the running maximum only when the tile exceeds it by more than the gap
      const bool raise = m_tile > m_run + kRescaleGap;   // true on the first tile with a valid key
      const float m_new = raise ? m_tile : m_run;
      const float alpha = raise ? attn_ex2(m_run - m_new) : 1.f;  // 0 when m_run was -inf
      const float scale = p.scale_log2, neg_m = m_new == -INFINITY ? 0.f : -m_new;
      float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
      uint32_t packed[16];
#pragma unroll
      for (int jj = 0; jj < 32; jj += 2) {
        const float p0 = attn_ex2(fmaf(sv[jj], scale, neg_m));
        const float p1 = attn_ex2(fmaf(sv[jj + 1], scale, neg_m));
        if ((jj & 6) == 0) l0 += p0 + p1;
        else if ((jj & 6) == 2) l1 += p0 + p1;
        else if ((jj & 6) == 4) l2 += p0 + p1;
        else l3 += p0 + p1;
        __nv_bfloat162 pr = __floats2bfloat162_rn(p0, p1);
        packed[jj >> 1] = *reinterpret_cast<uint32_t*>(&pr);
      }
      // P over the thread's own score columns (the first 16 of its 32)
      attn_tmem_st16(s_addr, packed);
      l_run = l_run * alpha + ((l0 + l1) + (l2 + l3));
      m_run = m_new;
      if (j > 0 && __any_sync(0xffffffffu, raise)) {
        // O may be rescaled once P V of the tile before has completed
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&pv_done[(j - 1) % 3], ((uint32_t)(j - 1) / 3u) & 1u, &abort_flag));
        if (ok) {
          ptx::tc_fence_after();
          float ov[32];
          ptx::tmem_ld_32x32(o_addr, ov);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) ov[jj] *= alpha;
          ptx::tmem_st_32x32(o_addr, ov);
        }
      }
      ptx::tmem_st_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (ok && lane == 0) ptx::mbar_arrive(&p_full[sb]);
    }
    if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&o_done, 0, &abort_flag));
    // row sum = the four quarters' sums
    float (*xl)[128] = xchg[T & 1];
    xl[kq][r] = l_run;
    row_sync();
    const float l_all = (xl[0][r] + xl[1][r]) + (xl[2][r] + xl[3][r]);
    const int hh = r >> 6, ri = r & 63;
    if (ok) {   // (the TMEM load is warp-wide: every lane takes part, valid row or not)
      ptx::tc_fence_after();
      float ov[32];
      ptx::tmem_ld_32x32(o_addr, ov);
      ptx::tmem_ld_wait();
      if (ri < un.n[hh]) {
        const float inv = 1.f / l_all;
        const int row = act_row(p.m, un.v[hh], b, un.q[hh] + ri);
        __nv_bfloat16* dst = p.o + (size_t)row * p.nq * kHd + (size_t)h * kHd + kbase;
#pragma unroll
        for (int i8 = 0; i8 < 32; i8 += 8) {
          uint32_t w[4];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            __nv_bfloat162 pr = __floats2bfloat162_rn(ov[i8 + 2 * jj] * inv, ov[i8 + 2 * jj + 1] * inv);
            w[jj] = *reinterpret_cast<uint32_t*>(&pr);
          }
          *reinterpret_cast<uint4*>(dst + i8) = make_uint4(w[0], w[1], w[2], w[3]);
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
