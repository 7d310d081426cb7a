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
//   S = Q K^T         tcgen05.mma, fp32 in TMEM (three buffers of 128 columns, up to three tiles ahead)
//   P = exp2(S - m0)  one softmax thread per row and tile; the probabilities go back into TMEM as
//                     packed bf16 over the first half of the tile's score columns
//   O += P V          tcgen05.mma with the A operand in TMEM, accumulating over all tiles
//
// The reference point m0 of a row is fixed for the whole pass: the row's maximum over the first
// 32 keys of the first tile (0 if none of them is valid for the row).  Floating point does not care how far
// the later scores lie from it as long as 2^(s - m0) stays in range; a pass in which some row's
// running maximum ends more than 2^100 above its m0 is run again with m0 = that maximum (a CTA-wide
// decision at the end of the pass; at most once).  With m0 fixed the tiles of a row are
// independent, so consecutive tiles go to DIFFERENT warps: softmax warp (quarter q, slot s) owns
// rows 32 q .. 32 q + 31 of every tile t with t % 3 == s (and score buffer s).  The three warps of
// a scheduler therefore work on three tiles at once and cover each other's latencies (TMEM loads
// and stores, the special-function unit).  An earlier arrangement with four threads per row (32
// keys each) exchanged the row maximum through shared memory every tile, which kept the four
// warps of a scheduler in lockstep: 1900 clocks per tile of which the special-function unit was
// busy 770.  Keys beyond the valid length are masked to -inf in S, and the V^T columns of cached
// keys beyond ctx_len are zeroed in shared memory (the cache may hold anything there).
//
// Warp roles (512 threads): warp 0 = TMA producer for Q and K, warp 1 = TMEM owner + issuer of the
// score MMAs (Q K^T), warp 2 = TMA producer for V^T, warp 3 = issuer of the output MMAs (P V; all
// its lanes first clear the V^T columns beyond ctx_len in the one tile that has any), warps 4..15 =
// softmax / output (TMEM lane quarter = warp % 4, slot = (warp - 4) / 4).  Two issuing threads
// because one was the bottleneck: with its four barrier waits and two commits per tile it needed
// about 2270 clocks per tile for MMAs that keep the tensor pipe busy for 1024.
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

constexpr int kAttnThreads = 512;
constexpr int kHd = 128;
constexpr int kBK = 128;                       // keys per tile
constexpr int kSub = 128 * 128;                // bytes of one [128 rows x 64 bf16] sub-tile
constexpr int kAttnStagesK = 3, kAttnStagesV = 2;   // ring slots of K and of V^T
constexpr int kAttnSmem = 2 * kSub /*Q*/ + kAttnStagesK * 2 * kSub + kAttnStagesV * 2 * kSub + 1024;
constexpr int kAttnPrefetch = 0;               // context tiles the L2 prefetch runs ahead of the tile after the ring
                                               // (measured: 0 -> 1.36 ms, 4 -> 1.41 ms, 8 -> 1.46 ms on 4 x 4096 keys x 8 layers)
constexpr float kAttnRange = 100.f;            // log2 units a row's maximum may end above its m0 before the pass is run again

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
      s_full[3], p_full[3], pv_done[3], o_done, m_ready;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag, again_flag;
  __shared__ float m_row[128];     // the rows' reference points of the first pass
  __shared__ float xl[3][128];     // [slot][row]: sum of the probabilities of the slot's tiles
  __shared__ float xm[3][128];     // [slot][row]: maximum raw score of the slot's tiles

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
    abort_flag = 0; again_flag = 0;
    ptx::mbar_init(&q_full, 1);
    for (int i = 0; i < kAttnStagesK; ++i) { ptx::mbar_init(&k_full[i], 1); ptx::mbar_init(&k_empty[i], 1); }
    for (int i = 0; i < kAttnStagesV; ++i) ptx::mbar_init(&v_loc[i], 1);
    for (int i = 0; i < 3; ++i) {
      ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&p_full[i], 4); ptx::mbar_init(&pv_done[i], 1);
    }
    ptx::mbar_init(&o_done, 1);
    ptx::mbar_init(&m_ready, 4);
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
  // TMEM columns: S / P of tile J in buffer J % 3 (columns 0..127, 128..255, 256..383), O 384..511

  // softmax threads: row, slot and per-pass state (other warps carry the variables along)
  const int gw = warp - 4;
  const int quarter = warp & 3;       // = the TMEM lanes this warp can reach
  const int slot = gw >> 2;           // which tiles (and which score buffer) this warp owns
  const int r = quarter * 32 + lane;  // query row inside the tile = TMEM lane
  float m0 = 0.f;                     // reference point of the row, in log2 units (softmax threads)
  float run_max = -INFINITY;          // maximum raw score the thread has seen
  bool sm_ok = true;                  // no wait of this warp has given up
  float l_all = 0.f;                  // the row's sum of probabilities over all tiles

  // A pass = all T key tiles.  Tiles are counted through both passes (J = pass * T + j), so that
  // ring slots, score buffers and barrier parities simply go on in the second pass.
  for (int pass = 0; pass < 2; ++pass) {
    const int J0 = pass * T;
    if (warp == 0) {
      if (lane == 0) {
        // ---------------- Q (once), then the K ring ----------------
        if (pass == 0) {
          ptx::mbar_expect_tx(&q_full, 2 * kSub);
          for (int hh = 0; hh < 2; ++hh) {
            const int row = act_row(p.m, un.v[hh], b, un.q[hh]);
            ptx::tma_load_2d(Qs + hh * 8192, &map_q, &q_full, h * kHd, row);
            ptx::tma_load_2d(Qs + kSub + hh * 8192, &map_q, &q_full, h * kHd + 64, row);
          }
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
          const int J = J0 + j, s = J % kAttnStagesK;
          const AttnTile t = attn_tile(un, j);
          prefetch_k(j + kAttnStagesK + kAttnPrefetch);
          if (!ptx::mbar_wait(&k_empty[s], (((uint32_t)(J / kAttnStagesK)) & 1u) ^ 1u, &abort_flag)) break;
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
          const int J = J0 + j, s = J % kAttnStagesV;
          const AttnTile t = attn_tile(un, j);
          prefetch_v(j + kAttnStagesV + kAttnPrefetch);
          // the slot held tile J - 2: free once its P V has completed
          if (J >= kAttnStagesV &&
              !ptx::mbar_wait(&pv_done[(J - 2) % 3], ((uint32_t)(J - 2) / 3u) & 1u, &abort_flag)) break;
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
          const int J = J0 + j;
          const uint32_t s = (uint32_t)(J % kAttnStagesK), sb = (uint32_t)J % 3u;
          // score buffer J % 3 last held P of tile J - 3: its P V (issued by another thread) must be done
          if (J >= 3 && !ptx::mbar_wait_a(b_pv_done + 8u * sb, ((uint32_t)(J - 3) / 3u) & 1u, &abort_flag)) break;
          if (!ptx::mbar_wait_a(b_k_full + 8u * s, ((uint32_t)(J / kAttnStagesK)) & 1u, &abort_flag)) break;
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
      // P sits in the first half of the tile's score columns: keys 32 c + 2 i, + 1 in column 32 c + i.
      static_assert(kAttnStagesV == 2, "the slot of tile J is the slot of tile J - 2");
      const uint32_t idesc = ptx::idesc_bf16(128, 128);
      const uint32_t hi32 = ptx::smem_desc_hi32();
      const uint32_t v_lo = ptx::smem_desc_lo(ptx::smem_u32(Vs));
      constexpr uint32_t kSub16 = kSub >> 4;
      const uint32_t b_v_loc = ptx::smem_u32(&v_loc[0]), b_p_full = ptx::smem_u32(&p_full[0]);
      const uint32_t b_pv_done = ptx::smem_u32(&pv_done[0]);
      bool ok = true;
      for (int j = 0; j < T && ok; ++j) {
        const int J = J0 + j;
        const uint32_t s = (uint32_t)(J % kAttnStagesV), ph = ((uint32_t)(J / kAttnStagesV)) & 1u;
        const uint32_t sb = (uint32_t)J % 3u;
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
          ok = ptx::mbar_wait_a(b_p_full + 8u * sb, ((uint32_t)J / 3u) & 1u, &abort_flag) &&
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
            // also tells the V^T producer that the slot is free and the score issuer that the
            // buffer is
            ptx::umma_commit_a(b_pv_done + 8u * sb);
          }
        }
        // the other lanes wait here (not spinning) while lane 0 issues
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      }
      if (ok && lane == 0) ptx::umma_commit(&o_done);
    } else {
      // ---------------- softmax warps ----------------
      const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
      const uint32_t s_addr = t_lane + (uint32_t)slot * 128u;   // this warp's score buffer (= J % 3)
      const int my_variant = un.v[r >> 6];
      const float scale = p.scale_log2;
      bool have_m0 = pass > 0;   // second pass: m0 was set at the end of the first
      float l_run = 0.f;         // the thread's tiles only
      sm_ok = true;
      for (int J = J0 + (slot + 3 - J0 % 3) % 3; J < J0 + T; J += 3) {
        const int j = J - J0;
        const AttnTile t = attn_tile(un, j);
        // packed unit: an active key tile of the other variant contributes nothing to this warp's rows
        const bool other = un.packed && !t.is_ctx && t.kv != my_variant;
        if (sm_ok) sm_ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[slot], ((uint32_t)J / 3u) & 1u, &abort_flag));
        // S of this tile is complete, so its K slot has been read: hand it back to the producer
        if (sm_ok && quarter == 0 && lane == 0) ptx::mbar_arrive(&k_empty[J % kAttnStagesK]);
        const int nvalid = (other || !sm_ok) ? 0 : t.valid;   // warp-uniform
        if (sm_ok) ptx::tc_fence_after();
        float sv[2][32];
        if (nvalid > 0) ptx::tmem_ld_32x32(s_addr, sv[0]);   // the first 32 keys of the tile
        if (!have_m0) {
          if (J == 0) {
            // this warp owns the first tile: the rows' maxima over its first 32 keys are the rows'
            // reference points (any score of the row would do)
            ptx::tmem_ld_wait();
            const int nc = max(0, min(32, nvalid));
            float mx = -INFINITY;
#pragma unroll
            for (int jj = 0; jj < 32; ++jj) mx = fmaxf(mx, jj < nc ? sv[0][jj] : -INFINITY);
            m0 = mx == -INFINITY ? 0.f : mx * scale;
            m_row[r] = m0;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&m_ready);
          } else {
            if (sm_ok) sm_ok = __all_sync(0xffffffffu, ptx::mbar_wait(&m_ready, 0, &abort_flag));
            m0 = m_row[r];
          }
          have_m0 = true;
        }
        // (two keys per instruction where the pipe has one: packed fma / add, three-input max)
        const ptx::f32x2 scale2 = ptx::f2_pack(scale, scale), negm2 = ptx::f2_pack(-m0, -m0);
        ptx::f32x2 la = ptx::f2_pack(0.f, 0.f), lb = la;
        float x0 = run_max, x1 = -INFINITY, x2 = -INFINITY, x3 = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float (&v)[32] = sv[c & 1];
          ptx::tmem_ld_wait();                                  // chunk c is in registers
          if (c < 3 && nvalid > 32 * (c + 1)) ptx::tmem_ld_32x32(s_addr + 32u * (c + 1), sv[(c + 1) & 1]);
          // keys beyond the valid length (whatever the cache holds there, NaN included) are set to
          // -inf once; ex2(-inf) = 0, so they need no further test
          const int nc = max(0, min(32, nvalid - 32 * c));
          if (nc < 32) {
#pragma unroll
            for (int jj = 0; jj < 32; ++jj)
              if (jj >= nc) v[jj] = -INFINITY;
          }
          uint32_t packed[16];
#pragma unroll
          for (int jj = 0; jj < 32; jj += 2) {
            float xa, xb;
            ptx::f2_unpack(ptx::f2_fma(ptx::f2_pack(v[jj], v[jj + 1]), scale2, negm2), xa, xb);
            const float p0 = attn_ex2(xa), p1 = attn_ex2(xb);
            if (jj & 2) lb = ptx::f2_add(lb, ptx::f2_pack(p0, p1));
            else la = ptx::f2_add(la, ptx::f2_pack(p0, p1));
            if ((jj & 6) == 0) x0 = ptx::fmax3(x0, v[jj], v[jj + 1]);
            else if ((jj & 6) == 2) x1 = ptx::fmax3(x1, v[jj], v[jj + 1]);
            else if ((jj & 6) == 4) x2 = ptx::fmax3(x2, v[jj], v[jj + 1]);
            else x3 = ptx::fmax3(x3, v[jj], v[jj + 1]);
            __nv_bfloat162 pr = __floats2bfloat162_rn(p0, p1);
            packed[jj >> 1] = *reinterpret_cast<uint32_t*>(&pr);
          }
          // P of these 32 keys over the first 16 of their 32 score columns
          attn_tmem_st16(s_addr + 32u * c, packed);
        }
        {
          float a0, a1, b0, b1;
          ptx::f2_unpack(la, a0, a1);
          ptx::f2_unpack(lb, b0, b1);
          l_run += (a0 + a1) + (b0 + b1);
        }
        run_max = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (sm_ok && lane == 0) ptx::mbar_arrive(&p_full[slot]);
      }
      // every P V of the pass has completed
      if (sm_ok) sm_ok = __all_sync(0xffffffffu, ptx::mbar_wait(&o_done, (uint32_t)pass & 1u, &abort_flag));
      // the three threads of a row (one per slot) meet on the named barrier of their lane quarter
      xl[slot][r] = l_run;
      xm[slot][r] = run_max;
      asm volatile("bar.sync %0, 96;" ::"r"(1 + quarter) : "memory");
      l_all = (xl[0][r] + xl[1][r]) + xl[2][r];
      if (pass == 0 && slot == 0) {
        const float top = fmaxf(fmaxf(xm[0][r], xm[1][r]), xm[2][r]) * scale;
        // (with one tile only the other slots never read m_row: this warp has m0 in any case)
        const bool far = sm_ok && (top - m0 > kAttnRange);
        m_row[r] = top;          // the reference points of a second pass
        if (__any_sync(0xffffffffu, far) && lane == 0) again_flag = 1;
      }
    }
    // ---------------- end of the pass: once more, or write the output ----------------
    __syncthreads();
    const bool again = pass == 0 && again_flag != 0 && abort_flag == 0;
    if (again) {
      if (warp >= 4) m0 = m_row[r];
      continue;
    }
    if (warp >= 4 && sm_ok) {   // (the TMEM loads are warp-wide: every lane takes part, valid row or not)
      ptx::tc_fence_after();
      const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
      const int hh = r >> 6, ri = r & 63;
      const float inv = 1.f / l_all;
      for (int ch = slot; ch < 4; ch += 3) {   // 32 output columns each; slot 0 takes chunks 0 and 3
        float ov[32];
        ptx::tmem_ld_32x32(t_lane + 384u + 32u * (uint32_t)ch, ov);
        ptx::tmem_ld_wait();
        if (ri < un.n[hh]) {
          const int row = act_row(p.m, un.v[hh], b, un.q[hh] + ri);
          __nv_bfloat16* dst = p.o + (size_t)row * p.nq * kHd + (size_t)h * kHd + ch * 32;
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
        __syncwarp();
      }
    }
    break;
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
