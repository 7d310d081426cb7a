// Weight-streaming bf16 GEMM on tcgen05 for the dense layers of the block-step.
//
// out[m, n] = sum_k A[m, k] * W[n, k]        A: activations [M, K], W: weights [N, K]
//
// The step has few activation rows (M = 2 * batch * rows, 192 for one sequence) and very many
// weight rows, so the roles of the MMA operands are swapped: a CTA owns 128 weight rows (the MMA
// "M" side, one TMEM lane per output feature) and a block of up to 256 activation rows (the MMA
// "N" side, one TMEM column per row).  Every weight byte is read from HBM exactly once per
// column block; the activation tile is re-read from L2.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = epilogue (TMEM -> registers -> global).  Shared memory is a ring of kStages
// slots, each {NW weight tiles 128 x 64, one activation tile BN x 64}, all in the 128-byte
// swizzled K-major layout that both TMA and tcgen05.mma understand.
//
// A CTA works through the units (weight tile, column block, K split) blockIdx.x, + gridDim.x, ...
// With more units than CTAs (`pingpong`) the accumulators of consecutive units alternate
// between two TMEM sets, the producer and the MMA issuer run on into the next unit, and the
// epilogue of a unit - which took 25..60% of a unit's time when every unit was a CTA of its own -
// runs under the MMAs of the next.  A set is one accumulator of up to 256 columns (at N = 256 a
// single chain of MMAs already runs at the tensor core's rate).  Without `pingpong` (one unit per
// CTA, or gate / up, which need both sets for one unit) both sets serve a unit - even / odd
// k-steps, because small N needs two independent chains, or gate / up - and a CTA's next unit
// starts when the epilogue has drained them.
#pragma once
#include "kernels.h"
#include "tc_ptx.cuh"

namespace dc {

enum GemmEpi {
  GEMM_EPI_QKV = 0,      // rotate q/k heads (RoPE), round to bf16, store q, k, v
  GEMM_EPI_PARTIAL = 1,  // fp32 split-K partial sums [split][M][N]
  GEMM_EPI_SWIGLU = 2    // two accumulators (gate, up): bf16 silu(gate) * up
};

struct GemmParams {
  int M;          // valid activation rows
  int N;          // weight rows of one matrix (output features)
  int K;          // reduction length
  int BN;         // activation rows per column block (multiple of 16, <= 256)
  int nsplit;     // split-K factor
  int tiles;      // weight tiles (over all matrices of the call)
  int pingpong;   // more units than CTAs: one accumulator set per unit, sets alternate
  // QKV epilogue
  int nq, nkv, hd;          // tiles [0,nq) are q heads, [nq,nq+nkv) k heads, rest v heads
  const float* cos_sin;     // RoPE table [(b, r)][hd]
  int rows_per_variant;     // batch * R_cap: the table is shared by the variants
  const __nv_bfloat16 *bq, *bk, *bv;  // projection biases [nq*hd], [nkv*hd], [nkv*hd], or null
  __nv_bfloat16 *q, *k, *v; // outputs q [M, nq*hd], k [M, nkv*hd], v TRANSPOSED [nkv*hd, ldv]
  int ldv;                  // row pitch of the transposed v (elements, multiple of 8)
  // PARTIAL epilogue
  float* part;              // [nsplit][M_ld][N]
  size_t part_stride;       // elements between splits
  // SWIGLU epilogue
  __nv_bfloat16* act;       // [M, N]
  int32_t* status;          // device status word(s); DC_ERR_TIMEOUT on an expired wait
};

constexpr int kGemmThreads = 192;
constexpr int kTileN = 128;  // weight rows per CTA tile
constexpr int kTileK = 64;   // bf16 elements per k-block (one 128-byte swizzle row)

__host__ __device__ inline int gemm_stage_bytes(int nw, int BN) {
  return nw * kTileN * kTileK * 2 + BN * kTileK * 2;
}

// PAIR: the launch uses clusters of two CTAs and every MMA is a pair MMA (cta_group::2, M = 256):
// the two CTAs own adjacent weight tiles and each stages only half of the activation block, so a
// k-block is 16 KB of weights plus 16 KB of activations per CTA instead of 16 + 32 - the main
// loops of these GEMMs are bound by what an SM takes in from L2.  The even CTA issues the MMAs;
// TMA loads of both CTAs report to its full barrier, tcgen05.commit releases ring slots and
// signals the accumulators in both; the odd CTA's epilogue warps report the drained accumulators
// to the even CTA's barrier.  No load is multicast.
template <int EPI, bool PAIR>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
          const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_a,
          const GemmParams p, const int stages) {
  constexpr int NW = (EPI == GEMM_EPI_SWIGLU) ? 2 : 1;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bar_full[8], bar_empty[8], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float xch[(EPI == GEMM_EPI_QKV) ? 128 * 33 : 1];

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Column blocks of one weight tile sit next to each other in the unit order, so that the
  // CTAs that share a weight tile run together and all but one read it from L2.
  const int n_cblk = (p.M + p.BN - 1) / p.BN;
  const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;
  const int cta = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // worker index: CTA or CTA pair
  const int n_cta = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int a_rows = PAIR ? p.BN / 2 : p.BN;                             // activation rows this CTA stages
  const int per_split = (PAIR ? p.tiles / 2 : p.tiles) * n_cblk;
  const int n_units = per_split * p.nsplit;
  const int stage_bytes = gemm_stage_bytes(NW, a_rows);
  const int KB = p.K / kTileK;
  const bool pp = p.pingpong != 0;
  const uint32_t up_off = pp ? 128u : 256u;   // second accumulator of a set (gate / up), or the odd k-steps' one
  const uint32_t tmem_cols = 512u;

  struct Unit { int tile, cblk, split, kb0, nkb, wrow; const CUtensorMap* map_w; };
  auto unit_of = [&](int u) {
    Unit w;
    w.split = u / per_split;
    const int rem = u - w.split * per_split;
    w.tile = rem / n_cblk;
    w.cblk = rem - w.tile * n_cblk;
    if (PAIR) w.tile = 2 * w.tile + (int)rank;
    w.kb0 = (int)(((long long)w.split * KB) / p.nsplit);
    w.nkb = (int)(((long long)(w.split + 1) * KB) / p.nsplit) - w.kb0;
    // which weight matrix and which row of it this tile starts at
    w.map_w = &map_w0;
    w.wrow = w.tile * kTileN;
    if (EPI == GEMM_EPI_QKV) {
      if (w.tile >= p.nq + p.nkv) { w.map_w = &map_w2; w.wrow = (w.tile - p.nq - p.nkv) * kTileN; }
      else if (w.tile >= p.nq) { w.map_w = &map_w1; w.wrow = (w.tile - p.nq) * kTileN; }
    }
    return w;
  };

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < stages; ++i) { ptx::mbar_init(&bar_full[i], 1); ptx::mbar_init(&bar_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], PAIR ? 256 : 128); }
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&map_w0);
    ptx::prefetch_tmap(&map_a);
    if (NW == 2 || EPI == GEMM_EPI_QKV) ptx::prefetch_tmap(&map_w1);
    if (EPI == GEMM_EPI_QKV) ptx::prefetch_tmap(&map_w2);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tmem_base_s, tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  if (PAIR) {
    // both CTAs hold all 512 columns, so the pair MMA's accumulator address names the same columns
    // in both; the partner's barriers are initialised before any load can report to them
    if (threadIdx.x == 0 && tmem_base != 0) abort_flag = 1;
    ptx::cluster_sync();
  }

  // One thread issues every TMA load and one every MMA, so their own instruction streams are on
  // the critical path: slot indices, addresses and descriptors advance by additions only.
  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      const uint32_t ring0 = ptx::smem_u32(smem);
      const uint32_t full0 = ptx::smem_u32(&bar_full[0]), empty0 = ptx::smem_u32(&bar_empty[0]);
      uint32_t s = 0, ph = 0, slot = ring0;
      bool ok = true;
      const uint32_t full_r0 = (PAIR && rank != 0) ? ptx::mapa_shared(full0, 0) : full0;   // the even CTA's
      for (int u = cta; u < n_units && ok; u += n_cta) {
        const Unit w = unit_of(u);
        const int arow = w.cblk * p.BN + (int)rank * a_rows;
        for (int i = 0; i < w.nkb; ++i) {
          if (!ptx::mbar_wait_a(empty0 + 8u * s, ph ^ 1u, &abort_flag)) { ok = false; break; }
          const int kc = (w.kb0 + i) * kTileK;
          if (PAIR) {
            if (rank == 0) ptx::mbar_expect_tx_a(full0 + 8u * s, 2u * (uint32_t)stage_bytes);
            const uint32_t bar = full_r0 + 8u * s;
            ptx::tma_load_2d_pair_a(slot, w.map_w, bar, kc, w.wrow);
            if (NW == 2) ptx::tma_load_2d_pair_a(slot + kTileN * kTileK * 2, &map_w1, bar, kc, w.wrow);
            ptx::tma_load_2d_pair_a(slot + NW * kTileN * kTileK * 2, &map_a, bar, kc, arow);
          } else {
            ptx::mbar_expect_tx_a(full0 + 8u * s, (uint32_t)stage_bytes);
            ptx::tma_load_2d_a(slot, w.map_w, full0 + 8u * s, kc, w.wrow);
            if (NW == 2) ptx::tma_load_2d_a(slot + kTileN * kTileK * 2, &map_w1, full0 + 8u * s, kc, w.wrow);
            ptx::tma_load_2d_a(slot + NW * kTileN * kTileK * 2, &map_a, full0 + 8u * s, kc, arow);
          }
          if (++s == (uint32_t)stages) { s = 0; ph ^= 1u; slot = ring0; } else slot += (uint32_t)stage_bytes;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = ptx::idesc_bf16(PAIR ? 2 * kTileN : kTileN, p.BN);
      const uint32_t ring0 = ptx::smem_u32(smem);
      const uint32_t full0 = ptx::smem_u32(&bar_full[0]), empty0 = ptx::smem_u32(&bar_empty[0]);
      const uint64_t hi = ptx::smem_desc_sw128_hi();
      uint32_t s = 0, ph = 0, slot = ring0;
      bool ok = true;
      int j = 0;   // units of this CTA so far
      for (int u = cta; u < n_units && ok; u += n_cta, ++j) {
        const Unit w = unit_of(u);
        const uint32_t set = pp ? (uint32_t)(j & 1) : 0u;
        // the epilogue has drained this set (its use before the last one)
        if (j >= (pp ? 2 : 1)) {
          const uint32_t uses = pp ? (uint32_t)(j >> 1) : (uint32_t)j;   // completed uses of the set
          if (!ptx::mbar_wait(&acc_empty[set], (uses - 1) & 1u, &abort_flag)) { ok = false; break; }
        }
        ptx::tc_fence_after();
        const uint32_t acc0 = tmem_base + set * 256u, acc1 = acc0 + up_off;
        uint32_t acc_first = 0;
        for (int i = 0; i < w.nkb; ++i) {
          if (!ptx::mbar_wait_a(full0 + 8u * s, ph, &abort_flag)) { ok = false; break; }
          const uint64_t dw0 = hi | (uint64_t)(slot >> 4);
          const uint64_t dw1 = dw0 + (kTileN * kTileK * 2 >> 4);
          const uint64_t da = dw0 + (NW * kTileN * kTileK * 2 >> 4);
          if (PAIR) {
            if (NW == 2) {
              ptx::umma_bf16_pair(acc0, dw0, da, idesc, acc_first);
              ptx::umma_bf16_pair(acc1, dw1, da, idesc, acc_first);
#pragma unroll
              for (int kk = 1; kk < kTileK / 16; ++kk) {
                ptx::umma_bf16_pair_acc(acc0, dw0 + 2 * kk, da + 2 * kk, idesc);
                ptx::umma_bf16_pair_acc(acc1, dw1 + 2 * kk, da + 2 * kk, idesc);
              }
            } else if (pp) {
              ptx::umma_bf16_pair(acc0, dw0, da, idesc, acc_first);
              ptx::umma_bf16_pair_acc(acc0, dw0 + 2, da + 2, idesc);
              ptx::umma_bf16_pair_acc(acc0, dw0 + 4, da + 4, idesc);
              ptx::umma_bf16_pair_acc(acc0, dw0 + 6, da + 6, idesc);
            } else {
              ptx::umma_bf16_pair(acc0, dw0, da, idesc, acc_first);
              ptx::umma_bf16_pair(acc1, dw0 + 2, da + 2, idesc, acc_first);
              ptx::umma_bf16_pair_acc(acc0, dw0 + 4, da + 4, idesc);
              ptx::umma_bf16_pair_acc(acc1, dw0 + 6, da + 6, idesc);
            }
            acc_first = 1;
            ptx::umma_commit_pair_a(empty0 + 8u * s);   // frees the slot in both CTAs
          } else {
          if (NW == 2) {
            ptx::umma_bf16(acc0, dw0, da, idesc, acc_first);
            ptx::umma_bf16(acc1, dw1, da, idesc, acc_first);
#pragma unroll
            for (int kk = 1; kk < kTileK / 16; ++kk) {
              ptx::umma_bf16_acc(acc0, dw0 + 2 * kk, da + 2 * kk, idesc);
              ptx::umma_bf16_acc(acc1, dw1 + 2 * kk, da + 2 * kk, idesc);
            }
          } else if (pp) {
            ptx::umma_bf16(acc0, dw0, da, idesc, acc_first);
            ptx::umma_bf16_acc(acc0, dw0 + 2, da + 2, idesc);
            ptx::umma_bf16_acc(acc0, dw0 + 4, da + 4, idesc);
            ptx::umma_bf16_acc(acc0, dw0 + 6, da + 6, idesc);
          } else {
            ptx::umma_bf16(acc0, dw0, da, idesc, acc_first);
            ptx::umma_bf16(acc1, dw0 + 2, da + 2, idesc, acc_first);
            ptx::umma_bf16_acc(acc0, dw0 + 4, da + 4, idesc);
            ptx::umma_bf16_acc(acc1, dw0 + 6, da + 6, idesc);
          }
          acc_first = 1;
          ptx::umma_commit_a(empty0 + 8u * s);  // slot free once these MMAs have read it
          }
          if (++s == (uint32_t)stages) { s = 0; ph ^= 1u; slot = ring0; } else slot += (uint32_t)stage_bytes;
        }
        if (ok) {   // this unit's accumulators are complete (in both CTAs of a pair)
          if (PAIR) ptx::umma_commit_pair(&acc_full[set]);
          else ptx::umma_commit(&acc_full[set]);
        }
      }
    }
  } else {
    // ---------------- epilogue: warps 2..5, TMEM lane quarter = warp % 4 ----------------
    const int quarter = warp & 3;
    const int f = quarter * 32 + lane;  // feature (weight row) inside the tile = TMEM lane
    bool ok = true;
    int j = 0;
    const uint32_t acc_empty_r0 = (PAIR && rank != 0) ? ptx::mapa_shared(ptx::smem_u32(&acc_empty[0]), 0) : 0u;
    for (int u = cta; u < n_units && ok; u += n_cta, ++j) {
      const Unit w = unit_of(u);
      const int tile = w.tile, split = w.split;
      const uint32_t set = pp ? (uint32_t)(j & 1) : 0u;
      const uint32_t uses = pp ? (uint32_t)(j >> 1) : (uint32_t)j;
      ok = ptx::mbar_wait(&acc_full[set], uses & 1u, &abort_flag);
      ptx::tc_fence_after();
      if (!ok) break;
      if (w.nkb > 0) {
      const uint32_t t_lane = tmem_base + set * 256u + ((uint32_t)(quarter * 32) << 16);
      const int m_base = w.cblk * p.BN;
      float bias_f = 0.f;   // bias of this thread's output feature (q / k / v projections)
      if (EPI == GEMM_EPI_QKV && p.bq != nullptr) {
        const __nv_bfloat16* bb = tile >= p.nq + p.nkv ? p.bv + (tile - p.nq - p.nkv) * p.hd
                                  : tile >= p.nq ? p.bk + (tile - p.nq) * p.hd : p.bq + tile * p.hd;
        bias_f = __bfloat162float(bb[f]);
      }
      for (int c0 = 0; c0 < p.BN; c0 += 32) {
        float acc[32];
        // BN is a multiple of 16: the last chunk may be 16 wide
        const int width = (p.BN - c0 >= 32) ? 32 : 16;
        if (width == 32) ptx::tmem_ld_32x32(t_lane + c0, acc);
        else {
          float a16[16];
          ptx::tmem_ld_32x16(t_lane + c0, a16);
#pragma unroll
          for (int j2 = 0; j2 < 16; ++j2) { acc[j2] = a16[j2]; acc[16 + j2] = 0.f; }
        }
        ptx::tmem_ld_wait();
        if (EPI != GEMM_EPI_SWIGLU && !pp) {
          // odd k-steps went to the second accumulator
          float odd[32];
          if (width == 32) ptx::tmem_ld_32x32(t_lane + up_off + c0, odd);
          else {
            float a16[16];
            ptx::tmem_ld_32x16(t_lane + up_off + c0, a16);
#pragma unroll
            for (int j2 = 0; j2 < 16; ++j2) { odd[j2] = a16[j2]; odd[16 + j2] = 0.f; }
          }
          ptx::tmem_ld_wait();
#pragma unroll
          for (int j2 = 0; j2 < 32; ++j2) acc[j2] += odd[j2];
        }
        if (EPI == GEMM_EPI_PARTIAL) {
          float* dst = p.part + (size_t)split * p.part_stride + (size_t)(tile * kTileN + f);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int m = m_base + c0 + j;
            if (j < width && m < p.M) dst[(size_t)m * p.N] = acc[j];
          }
        } else if (EPI == GEMM_EPI_SWIGLU) {
          float up[32];
          if (width == 32) ptx::tmem_ld_32x32(t_lane + up_off + c0, up);
          else {
            float a16[16];
            ptx::tmem_ld_32x16(t_lane + up_off + c0, a16);
#pragma unroll
            for (int j = 0; j < 16; ++j) { up[j] = a16[j]; up[16 + j] = 0.f; }
          }
          ptx::tmem_ld_wait();
          __nv_bfloat16* dst = p.act + (size_t)(tile * kTileN + f);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int m = m_base + c0 + j;
            if (j < width && m < p.M) {
              // silu(g) = g * (0.5 + 0.5 * tanh(g / 2)): one special-function instruction (as in
              // the fused chain's epilogue; tanh.approx is good to 2^-11, the result goes to bf16)
              const float g = acc[j];
              float th;
              asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(0.5f * g));
              dst[(size_t)m * p.N] = __float2bfloat16_rn(g * fmaf(0.5f, th, 0.5f) * up[j]);
            }
          }
        } else {  // GEMM_EPI_QKV
#pragma unroll
          for (int j = 0; j < 32; ++j) acc[j] += bias_f;
          const bool is_v = tile >= p.nq + p.nkv;
          if (is_v) {
            // V is stored transposed (keys contiguous): this thread's 32 columns are 32
            // consecutive keys of feature row f
            __nv_bfloat16* dst = p.v + (size_t)((tile - p.nq - p.nkv) * p.hd + f) * p.ldv + m_base + c0;
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              if (j < width && m_base + c0 + j < p.M) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  __nv_bfloat162 pr = __floats2bfloat162_rn(acc[j + 2 * e], acc[j + 2 * e + 1]);
                  w[e] = *reinterpret_cast<uint32_t*>(&pr);
                }
                *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
              }
            }
          } else {
            // rotate-half RoPE: feature i < hd/2 pairs with i + hd/2, held by the warp two
            // quarters away; exchange the chunk through shared memory
#pragma unroll
            for (int j = 0; j < 32; ++j) xch[f * 33 + j] = acc[j];
            asm volatile("bar.sync 1, 128;" ::: "memory");
            const int half = p.hd / 2;
            const int i = f % half;
            const bool lo = f < half;
            const bool is_k = tile >= p.nq;
            __nv_bfloat16* dst = is_k ? p.k + (size_t)((tile - p.nq) * p.hd + f)
                                      : p.q + (size_t)(tile * p.hd + f);
            const int ld = is_k ? p.nkv * p.hd : p.nq * p.hd;
            // all table reads of the chunk first (independent loads), then the rotation
            float cv[32], sv[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              int m = m_base + c0 + j;
              if (m >= p.rows_per_variant) m -= p.rows_per_variant;  // prev variant: same table
              const bool in = j < width && m_base + c0 + j < p.M;
              const float* cs = p.cos_sin + (size_t)(in ? m : 0) * p.hd;
              cv[j] = __ldg(cs + i);
              sv[j] = __ldg(cs + half + i);
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int m = m_base + c0 + j;
              if (j < width && m < p.M) {
                const float other = xch[(f ^ half) * 33 + j];
                const float y = lo ? (acc[j] * cv[j] - other * sv[j]) : (acc[j] * cv[j] + other * sv[j]);
                dst[(size_t)m * ld] = __float2bfloat16_rn(y);
              }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
          }
        }
      }
      }
      // the set may be overwritten by the unit after the next; the even CTA's MMA issuer waits
      // for the epilogue warps of both CTAs
      ptx::tc_fence_before();
      if (PAIR && rank != 0) ptx::mbar_arrive_remote(acc_empty_r0 + 8u * set);
      else ptx::mbar_arrive(&acc_empty[set]);
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  // neither CTA of a pair leaves while the other may still read its shared memory or signal its
  // barriers
  if (PAIR) ptx::cluster_sync();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, tmem_cols);
  }
  if (threadIdx.x == 0 && abort_flag && p.status) atomicExch(p.status, DC_ERR_TIMEOUT);
}

}  // namespace dc
