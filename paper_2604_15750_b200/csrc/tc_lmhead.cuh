// LM head on tcgen05 fused with the streaming vocabulary softmax statistics.
//
// For each window position the curr-variant row h and the prev-variant row h' are multiplied
// with the vocabulary matrix tile by tile; the logits z, z' live only in TMEM and registers.
// Per position the kernel keeps, online over the vocabulary (Section 4.2 / 4.3 signals):
//   curr: m = max z, yhat = argmax (lowest id on ties), S = sum e^(z-m), A = sum e^(z-m) z,
//         D = sum e^(z-m) (z - z')
//   prev: m' = max z', S' = sum e^(z'-m')
// from which   c = 1/S,  lse = m + ln S,  H = lse - A/S,  I = D/S - lse + lse'   (Eq. 3).
//
// Orientation: the 128 TMEM lanes are LM rows of one group ([G curr rows ; G prev rows]), the
// TMEM columns are 128 vocabulary entries, so each thread scans its own row serially; the only
// exchange is z' from the prev row's thread to the curr row's thread, through shared memory.
// CTAs are persistent over vocabulary tiles (tile = blockIdx.x, += gridDim.x), two tiles at a
// time: the MMAs of a pair alternate between two TMEM accumulators (both MMAs of a k-step share
// the h operand; the issue rate is set by the instructions between two MMAs of the issuing
// thread, not by the accumulator dependence: a lean loop reaches the tensor core's own 64 clk per
// 128 x 128 x 16 MMA with one accumulator as with two), and two such pairs of accumulators exist, so that the
// statistics of one pair overlap the MMAs of the next.  Each CTA writes one partial record per
// row; k_lm_combine merges the records of all CTAs.
#pragma once
#include "kernels.h"
#include "tc_ptx.cuh"

namespace dc {

struct LmParams {
  SeqMeta m;
  int V, K;          // vocabulary size, d_model
  int mask_id;       // skipped when >= 0
  int ngroups;       // groups of LM rows; gridDim.x = ngroups * vocabulary slices
  float* part;       // [groups][slices][128][8]
  int32_t* status;
  int stall;         // test hook: the producer issues no load, so every wait of the kernel runs out
};

constexpr int kLmThreads = 192;
constexpr int kLmStageBytes = 3 * 128 * 64 * 2;  // h tile + W tiles of the two vocabulary tiles of a pair
constexpr float kLog2e = 1.4426950408889634f;

__global__ void __launch_bounds__(kLmThreads, 1)
k_lmhead_tc(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
            const LmParams p, const int stages) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bar_full[8], bar_empty[8], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float xch[2][64 * 33];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // CTA -> (group of LM rows, vocabulary slice), groups fastest: the CTAs that stream the same
  // vocabulary tiles for different groups run at the same time, so a tile crosses HBM once and is
  // served to the other groups from L2
  const int grp = (int)blockIdx.x % p.ngroups;
  const int slice = (int)blockIdx.x / p.ngroups, nslices = (int)gridDim.x / p.ngroups;
  const int KB = p.K / 64;
  const int ntiles = (p.V + 127) / 128;
  const int my_tiles = (ntiles - slice + nslices - 1) / nslices;
  const int my_pairs = (my_tiles + 1) / 2;
  const int G = p.m.G, nv = p.m.nv;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < stages; ++i) { ptx::mbar_init(&bar_full[i], 1); ptx::mbar_init(&bar_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 128); }
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&map_h);
    ptx::prefetch_tmap(&map_w);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tmem_base_s, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;

  // (lean single-thread loops: addresses and descriptors advance by additions only)
  if (warp == 0) {
    if (lane == 0) {
      const uint32_t ring0 = ptx::smem_u32(smem);
      const uint32_t full0 = ptx::smem_u32(&bar_full[0]), empty0 = ptx::smem_u32(&bar_empty[0]);
      const uint64_t pol_w = ptx::l2_policy_evict_first();
      uint32_t s = 0, ph = 0, slot = ring0;
      bool ok = true;
      for (int q = 0; q < my_pairs && ok && !p.stall; ++q) {
        // second tile of the pair may lie beyond the vocabulary: the load is zero-filled there
        // and the epilogue skips ids >= V
        const int vrow0 = (slice + (2 * q) * nslices) * 128;
        const int vrow1 = (slice + (2 * q + 1) * nslices) * 128;
        const bool two = 2 * q + 1 < my_tiles;
        for (int kb = 0; kb < KB; ++kb) {
          ok = ptx::mbar_wait_a(empty0 + 8u * s, ph ^ 1u, &abort_flag);
          if (!ok) break;
          const uint32_t bar = full0 + 8u * s;
          ptx::mbar_expect_tx_a(bar, two ? (uint32_t)kLmStageBytes : (uint32_t)(2 * 128 * 64 * 2));
          ptx::tma_load_2d_a(slot, &map_h, bar, kb * 64, grp * nv * G);
          ptx::tma_load_2d_hint_a(slot + 128 * 64 * 2, &map_w, bar, kb * 64, vrow0, pol_w);
          if (two) ptx::tma_load_2d_hint_a(slot + 2 * 128 * 64 * 2, &map_w, bar, kb * 64, vrow1, pol_w);
          if (++s == (uint32_t)stages) { s = 0; ph ^= 1u; slot = ring0; } else slot += (uint32_t)kLmStageBytes;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = ptx::idesc_bf16(128, 128);
      const uint32_t ring0 = ptx::smem_u32(smem);
      const uint32_t full0 = ptx::smem_u32(&bar_full[0]), empty0 = ptx::smem_u32(&bar_empty[0]);
      const uint64_t hi = ptx::smem_desc_sw128_hi();
      uint32_t s = 0, ph = 0, slot = ring0;
      bool ok = true;
      for (int q = 0; q < my_pairs && ok; ++q) {
        const int buf = q & 1;
        const bool two = 2 * q + 1 < my_tiles;
        ok = ptx::mbar_wait(&acc_empty[buf], (((uint32_t)q >> 1) & 1u) ^ 1u, &abort_flag);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d0 = tmem_base + buf * 256, d1 = d0 + 128;
        uint32_t acc_first = 0;
        for (int kb = 0; kb < KB; ++kb) {
          ok = ptx::mbar_wait_a(full0 + 8u * s, ph, &abort_flag);
          if (!ok) break;
          const uint64_t dh = hi | (uint64_t)(slot >> 4);
          const uint64_t dw0 = dh + (128 * 64 * 2 >> 4), dw1 = dh + (2 * 128 * 64 * 2 >> 4);
          if (two) {
            ptx::umma_bf16(d0, dh, dw0, idesc, acc_first);
            ptx::umma_bf16(d1, dh, dw1, idesc, acc_first);
#pragma unroll
            for (int kk = 1; kk < 4; ++kk) {
              ptx::umma_bf16_acc(d0, dh + 2 * kk, dw0 + 2 * kk, idesc);
              ptx::umma_bf16_acc(d1, dh + 2 * kk, dw1 + 2 * kk, idesc);
            }
          } else {
            ptx::umma_bf16(d0, dh, dw0, idesc, acc_first);
#pragma unroll
            for (int kk = 1; kk < 4; ++kk) ptx::umma_bf16_acc(d0, dh + 2 * kk, dw0 + 2 * kk, idesc);
          }
          acc_first = 1;
          ptx::umma_commit_a(empty0 + 8u * s);
          if (++s == (uint32_t)stages) { s = 0; ph ^= 1u; slot = ring0; } else slot += (uint32_t)kLmStageBytes;
        }
        if (ok) ptx::umma_commit(&acc_full[buf]);
      }
    }
  } else {
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;          // LM row inside the group = TMEM lane
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const bool is_curr = row < G;
    const bool is_prev = nv == 2 && row >= G && row < 2 * G;
    // running statistics in the base-2 domain: t = z * log2(e)
    float mt = -INFINITY, S = 0.f, A = 0.f, D = 0.f;
    int idx = 0x7fffffff;
    bool ok = true;
    // Every iteration executes its named barriers whatever happened: a wait that gave up makes
    // `ok` false for the whole warp and the work is skipped, so that no warp is left waiting on
    // a barrier the others never reach.
    for (int q = 0; q < my_pairs; ++q) {
      const int buf = q & 1;
      if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&acc_full[buf], ((uint32_t)q >> 1) & 1u, &abort_flag));
      if (ok) ptx::tc_fence_after();
      const int n_in_pair = (2 * q + 1 < my_tiles) ? 2 : 1;
      for (int w = 0; w < n_in_pair; ++w) {
      const int v0 = (slice + (2 * q + w) * nslices) * 128;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float z[32];
        if (ok) {
          ptx::tmem_ld_32x32(t_lane + buf * 256 + w * 128 + c * 32, z);
          ptx::tmem_ld_wait();
        }
        float* xb = xch[c & 1];
        if (ok && is_prev) {
#pragma unroll
          for (int i = 0; i < 32; ++i) xb[(row - G) * 33 + i] = z[i];
        }
        if (nv == 2) asm volatile("bar.sync 1, 128;" ::: "memory");
        const int vbase = v0 + c * 32;
        if (ok && (is_curr || is_prev)) {
          // chunk maximum over the admissible vocabulary entries
          float cm = -INFINITY;
          int ci = 0x7fffffff;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int v = vbase + i;
            const bool adm = v < p.V && v != p.mask_id;
            if (adm && z[i] > cm) { cm = z[i]; ci = v; }
          }
          const float cmt = cm * kLog2e;
          if (cmt > mt) {
            const float sc = exp2f(mt - cmt);
            S *= sc; A *= sc; D *= sc;
            mt = cmt;
            idx = ci;   // tiles and chunks arrive in ascending id order: first maximum kept
          }
          if (cm > -INFINITY) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int v = vbase + i;
              const bool adm = v < p.V && v != p.mask_id;
              if (adm) {
                const float e = exp2f(fmaf(z[i], kLog2e, -mt));
                S += e;
                if (is_curr) {
                  A = fmaf(e, z[i], A);
                  if (nv == 2) D = fmaf(e, z[i] - xb[row * 33 + i], D);
                }
              }
            }
          }
        }
      }
      }
      if (ok) {
        ptx::tc_fence_before();
        ptx::mbar_arrive(&acc_empty[buf]);
      }
    }
    float* rec = p.part + (((size_t)grp * nslices + slice) * 128 + row) * 8;
    rec[0] = mt; rec[1] = __int_as_float(idx); rec[2] = S; rec[3] = A; rec[4] = D;
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && abort_flag && p.status) atomicExch(p.status, DC_ERR_TIMEOUT);
}

// Merge the per-CTA records of one window position; one warp per position.
// A position without any finite admissible logit (a NaN / inf hidden row, or every vocabulary slice
// gave up in a bounded wait) keeps the argmax sentinel: it is reported as DC_ERR_NUMERIC in
// status[b * status_stride] and its id is replaced by fallback_id, so that nothing downstream
// indexes the vocabulary matrix with it.
__global__ void k_lm_combine(const float* __restrict__ part, int nctas, SeqMeta m, int V,
                             int fallback_id, int32_t* __restrict__ status, int status_stride,
                             int32_t* __restrict__ ws_pred, float* __restrict__ ws_conf,
                             float* __restrict__ ws_ent, float* __restrict__ ws_infl,
                             float* __restrict__ ws_lse, SignalOut out) {
  const int pos = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (pos >= m.batch * m.W_cap) return;
  const int b = pos / m.W_cap, k = pos % m.W_cap;
  if (k >= m.win_len[b]) return;
  const int grp = pos / m.G, r = pos % m.G;
  float mt = -INFINITY, S = 0.f, A = 0.f, D = 0.f, mt2 = -INFINITY, S2 = 0.f;
  int idx = 0x7fffffff;
  for (int c = lane; c < nctas; c += 32) {
    const float* rc = part + (((size_t)grp * nctas + c) * 128 + r) * 8;
    const float cm = rc[0];
    const int ci = __float_as_int(rc[1]);
    if (cm > mt || (cm == mt && ci < idx)) {
      const float sc = exp2f(mt - cm);
      S = S * sc + rc[2]; A = A * sc + rc[3]; D = D * sc + rc[4];
      if (cm > mt || ci < idx) idx = ci;
      mt = cm;
    } else if (cm > -INFINITY) {
      const float sc = exp2f(cm - mt);
      S += rc[2] * sc; A += rc[3] * sc; D += rc[4] * sc;
    }
    if (m.nv == 2) {
      const float* rp = rc + (size_t)m.G * 8;
      const float pm = rp[0];
      if (pm > mt2) { S2 = S2 * exp2f(mt2 - pm) + rp[2]; mt2 = pm; }
      else if (pm > -INFINITY) S2 += rp[2] * exp2f(pm - mt2);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, mt, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    const float oS = __shfl_xor_sync(0xffffffffu, S, o);
    const float oA = __shfl_xor_sync(0xffffffffu, A, o);
    const float oD = __shfl_xor_sync(0xffffffffu, D, o);
    const float nm = fmaxf(mt, om);
    if (nm > -INFINITY) {
      const float s0 = exp2f(mt - nm), s1 = exp2f(om - nm);
      S = S * s0 + oS * s1; A = A * s0 + oA * s1; D = D * s0 + oD * s1;
    }
    if (om > mt || (om == mt && oi < idx)) idx = oi;
    mt = nm;
    const float om2 = __shfl_xor_sync(0xffffffffu, mt2, o);
    const float oS2 = __shfl_xor_sync(0xffffffffu, S2, o);
    const float nm2 = fmaxf(mt2, om2);
    if (nm2 > -INFINITY) S2 = S2 * exp2f(mt2 - nm2) + oS2 * exp2f(om2 - nm2);
    mt2 = nm2;
  }
  if (lane == 0) {
    const float ln2 = 0.6931471805599453f;
    const float lse = mt * ln2 + logf(S);
    const float conf = 1.f / S;
    const float ent = lse - A / S;
    float infl = 0.f;
    if (m.nv == 2 && m.have_prev[b]) {
      const float lse2 = mt2 * ln2 + logf(S2);
      infl = fmaxf(D / S - lse + lse2, 0.f);
    }
    if (idx < 0 || idx >= V || !isfinite(lse)) {
      idx = fallback_id;
      if (status) atomicMax(status + b * status_stride, (int)DC_ERR_NUMERIC);
    }
    const int wi = b * m.W_cap + k;
    ws_pred[wi] = idx; ws_conf[wi] = conf; ws_ent[wi] = ent; ws_infl[wi] = infl; ws_lse[wi] = lse;
    const int oi = b * out.max_window + k;
    if (out.pred_id) out.pred_id[oi] = idx;
    if (out.conf) out.conf[oi] = conf;
    if (out.entropy) out.entropy[oi] = ent;
    if (out.influence) out.influence[oi] = infl;
    if (out.lse) out.lse[oi] = lse;
  }
}

}  // namespace dc
