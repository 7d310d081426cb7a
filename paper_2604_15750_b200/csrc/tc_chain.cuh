// Persistent dense chain: everything of a transformer layer between two attention calls, in one
// cooperative launch with one CTA per SM.
//
//   phase 0  O projection        split-K partial sums of  o . Wo^T                (tcgen05)
//   phase 1  residual + norm2    x += sum of partials;  a = bf16(rmsnorm(x) * g2)
//   phase 2  gate / up           act = bf16(silu(a . Wg^T) * (a . Wu^T))          (tcgen05)
//   phase 3  down projection     split-K partial sums of  act . Wd^T              (tcgen05)
//   phase 4  residual + norm1    x += sum of partials;  a = bf16(rmsnorm(x) * g1') (next layer)
//   phase 5  QKV of the next layer, rotated (RoPE), q / k row-major, v transposed  (tcgen05)
//
// A launch runs the phases [phase_begin, phase_end); CTAs meet at a grid-wide barrier between
// phases.  The first layer starts with a launch of phases 4..5, the last layer ends after phase 3
// (the final norm folds its partial sums).
//
// Why one kernel: at 192 activation rows a layer is 436 MB of weights (67 us of HBM time) cut
// into four GEMMs of 5..30 us each; as separate launches every one of them pays its own launch,
// pipeline ramp, and an epilogue that nothing overlaps.  Here the weight stream of the next phase
// is already on its way into L2 (cp.async.bulk.prefetch) while the current phase drains, and the
// only cost between phases is the barrier.
//
// GEMM orientation (as in tc_gemm.cuh): a CTA owns 128 weight rows (MMA M, one TMEM lane per
// output feature) and all activation rows (MMA N <= 256, one TMEM column per row).  Every unit
// keeps two accumulators: gate / up use one each, the other GEMMs send even k-steps to the first
// and odd k-steps to the second and add them in the epilogue.  (The split is not what sets the
// issue rate: a lean issue loop reaches the tensor core's own N / 2 clocks per pair MMA with one
// accumulator chain as with two; what costs is every instruction the issuing thread executes
// between two MMAs.  These GEMMs wait for their weights, not for the issue.)
//
// CTA pairs: the launch uses clusters of two CTAs and every MMA is a pair MMA (cta_group::2,
// M = 256): each CTA streams its own 128 weight rows but only HALF of the activation rows, the
// tensor cores of both SMs read the two halves from both shared memories.  What an SM can take in
// from L2 (about 100 GB/s, measured) bounds these GEMMs, and the activation tile is the part of
// that traffic that carries no new information; halving it is worth 15..30% per phase.  The even
// CTA of a pair issues the MMAs; TMA loads of both CTAs report to the even CTA's full barrier,
// tcgen05.commit releases the ring slot in both CTAs.  No load is multicast.
//
// Warp roles (512 threads): warp 0 lane 0 = TMA producer, warp 1 lane 0 = MMA issuer (warp 1
// owns the TMEM allocation).  All sixteen warps run the epilogue: warp w reads the TMEM lanes
// 32 * (w % 4) .. +31 (the only ones it can reach) and the column part w / 4, so four warps share
// every lane quarter.  The RoPE epilogue is a chain of dependent shared-memory exchanges and
// barriers: with four warps per scheduler instead of two it takes 7.2 k instead of 12.2 k clocks.
// All warps run the norm phases.
#pragma once
#include "kernels.h"
#include "tc.h"
#include "tc_ptx.cuh"

namespace dc {

struct ChainMaps {
  CUtensorMap wo, wg, wu, wd;   // this layer: [d, hq], [F, d], [F, d], [d, F]
  CUtensorMap wq, wk, wv;       // the layer whose QKV phase 5 computes
  CUtensorMap wo_n;             // that layer's O projection: what phase 5 prefetches into L2
  CUtensorMap a, o, act;        // activation operands, box = BN/2 rows x 64 columns (one CTA's half)
};

struct ChainParams {
  int M, BN;                    // valid activation rows; rows per MMA (multiple of 16, <= 256)
  int d, F, nq, nkv;            // model width, MLP width, query / kv heads (head_dim 128)
  int phase_begin, phase_end;
  int split_o, split_down;      // split-K factors of the two projections back to d
  int fold_norm1;               // partial sums phase 4 folds (0 when the launch starts there)
  float* x;                     // residual stream [M, d] fp32
  __nv_bfloat16* a;             // normed activations [M, d]
  __nv_bfloat16* act;           // SwiGLU output [M, F]
  float* part;                  // split-K partial sums [split][M][d]
  size_t part_stride;
  const __nv_bfloat16* g2;      // norm2 gain of this layer
  const __nv_bfloat16* g1;      // norm1 gain of the layer phase 5 belongs to
  float eps;
  const float* cos_sin;         // RoPE table [(b, r)][128]; row rows_per_variant: angle step
  int rows_per_variant;
  const __nv_bfloat16 *bq, *bk, *bv;  // biases of the q / k / v projections phase 5 computes, or null
  __nv_bfloat16 *q, *k, *v;     // q [M, nq*128], k [M, nkv*128], v transposed [nkv*128, ldv]
  int ldv;
  // QKV has fewer tiles than the grid has CTAs: the CTA pairs beyond the tiles take the last
  // bal_h k-blocks of the tiles off the others' hands (0: off) and hand the sums over in `part`
  // (BN * 128 floats per tile); tile_flags[tile] counts the warps that have done so (16 per
  // launch, counting up over a step), flag_target is the count that means "this launch's"
  int bal_h;
  unsigned int* tile_flags;
  unsigned int flag_target;
  unsigned int* bar;            // grid barrier arrival counter (counts up over a step)
  unsigned int bar_base;        // its value when this launch starts
  int32_t* status;              // DC_ERR_TIMEOUT lands here; non-zero on entry = do nothing
};

constexpr int kChainThreads = 512;
constexpr int kChainParts = kChainThreads / 128;  // warps per TMEM lane quarter = column parts of the epilogue
constexpr int kChainRing = 184 * 1024;          // TMA ring
constexpr int kXchRow = 20;                     // floats per thread in a RoPE exchange buffer (16 + padding, 16-byte rows)
constexpr int kChainXch = kChainParts * 128 * kXchRow * 4;  // RoPE exchange buffers of the QKV epilogue (one per column part)
constexpr int kChainSmem = kChainRing + kChainXch + 1024;
constexpr int kChainTile = 128;                 // weight rows per unit
constexpr int kChainTileK = 64;
// k-blocks of its next unit that a CTA prefetches into L2 when its own loads are issued (measured:
// 8 / 12 / 24 k-blocks cost +0.03 / +0.04 / +0.25 ms per step against 4)
constexpr int kPfGateUp = 4, kPfDown = 4, kPfQkv = 4;

struct ChainCtx {
  uint8_t* ring;
  float* xch;
  uint64_t *full, *empty, *acc_full, *acc_empty, *norm_bar;
  volatile int* abort_flag;
  uint32_t tmem_base;
  uint32_t fill_bits;   // producer: parity of the next fill of each slot
  uint32_t use_bits;    // MMA issuer: parity of the next use of each slot
  uint32_t units_done;  // units whose accumulators this thread has drained (epilogue role)
  uint32_t mma_units;   // units whose MMAs this thread has issued (MMA issuer only)
  uint32_t norm_uses;   // completed phases of norm_bar
  int warp, lane;
  uint32_t rank;        // 0 / 1 inside the CTA pair
};

struct GemmPhase {
  const CUtensorMap *w0, *w1, *w2;  // weight maps (QKV: q, k, v;  gate/up: gate, up)
  const CUtensorMap* amap;          // activation operand
  int tiles;                        // 128-row weight tiles (over all matrices of the phase)
  int nsplit;                       // K splits
  int KB;                           // k-blocks of 64
  int N;                            // output features (row pitch of the output)
  int bal_h;                        // k-blocks of every tile that helper CTA pairs compute (0: none)
  // what the producer prefetches into L2 once its own loads are issued: the first pf_kb
  // k-blocks of its unit in the phase named here (tiles == 0: nothing)
  const CUtensorMap *pf_w0, *pf_w1, *pf_w2;
  int pf_tiles, pf_nsplit, pf_KB, pf_kb, pf_t1, pf_t2;  // pf_t1 / pf_t2: first tile of w1 / w2
  int pf_bal_h;
};

// CTA-level unit u -> (weight tile, K split).  CTAs 2p and 2p+1 form a pair and must hold adjacent
// tiles of the same split: pair unit u / 2 = tile_pair * nsplit + split.
__device__ __forceinline__ void chain_unit(int u, int nsplit, int& tile, int& split) {
  const int pp = u >> 1;
  tile = (pp / nsplit) * 2 + (u & 1);
  split = pp % nsplit;
}

// The work item of this CTA in a GEMM phase (there is at most one: the launch conditions keep
// tiles * nsplit within the grid): weight tile, K split, k-block range, kind.  Without balancing
// an item is a unit as above.  With balancing (bal_h > 0; one split, fewer tile pairs than CTA
// pairs, at most two tile pairs per helper pair) CTA pair t < tiles / 2 owns tile pair t and computes
// its k-blocks [0, KB - bal_h) (ITEM_MAIN); helper pair hp = pair - tiles / 2 computes the k-blocks
// [KB - bal_h, KB) of tile pair hp and, if there is one, of tile pair hp + n_help (tile2) in the
// same pass - one activation tile, two weight tiles, one accumulator each, the shape of gate / up -
// and hands the sums over (ITEM_HELP).
enum { ITEM_FULL = 0, ITEM_MAIN = 1, ITEM_HELP = 2 };
struct ChainItem { int tile, tile2, split, kb0, kb1, kind; };
__device__ __forceinline__ bool chain_item(int tiles, int nsplit, int KB, int bal_h, ChainItem& w) {
  w.tile2 = -1;
  if (bal_h == 0) {
    if ((int)blockIdx.x >= tiles * nsplit) return false;
    chain_unit(blockIdx.x, nsplit, w.tile, w.split);
    w.kb0 = (int)(((long long)w.split * KB) / nsplit);
    w.kb1 = (int)(((long long)(w.split + 1) * KB) / nsplit);
    w.kind = ITEM_FULL;
    return true;
  }
  const int pair = blockIdx.x >> 1, r = blockIdx.x & 1, tp = tiles >> 1;
  w.split = 0;
  if (pair < tp) {
    w.tile = 2 * pair + r; w.kb0 = 0; w.kb1 = KB - bal_h; w.kind = ITEM_MAIN;
    return true;
  }
  const int n_help = (gridDim.x >> 1) - tp, hp = pair - tp;
  if (hp >= tp) return false;
  w.tile = 2 * hp + r; w.kb0 = KB - bal_h; w.kb1 = KB; w.kind = ITEM_HELP;
  if (hp + n_help < tp) w.tile2 = 2 * (hp + n_help) + r;
  return true;
}

enum { CEPI_PARTIAL = 0, CEPI_SWIGLU = 1, CEPI_QKV = 2 };

// RoPE factors of one thread's feature pair index i: (cos, sin) of the first row of a chunk and
// of the angle step between consecutive rows.  The rows of a chunk are consecutive positions, so
// the factors of the following rows come from the rotation recurrence (16 steps in fp32: the
// error stays far below a bf16 ulp).  This replaces 32 table reads per chunk, which sat on the
// critical path behind the exchange barrier, by 2 reads issued one chunk ahead.
struct RopeBase { float c, s, cd, sd; };

// Epilogue of 16 accumulator columns (activation rows c0 .. c0+15) of feature f of a tile.
template <int EPI>
__device__ __forceinline__ void chain_emit(ChainCtx& c, const ChainParams& p, const int N,
                                           const int tile, const int split, const int f,
                                           const int c0, float (&v0)[16], float (&v1)[16],
                                           const RopeBase rb, const int half) {
  if (EPI == CEPI_PARTIAL) {
    float* dst = p.part + (size_t)split * p.part_stride + (size_t)(tile * kChainTile + f) +
                 (size_t)c0 * N;
#pragma unroll
    for (int j = 0; j < 16; ++j) dst[(size_t)j * N] = v0[j] + v1[j];
  } else if (EPI == CEPI_SWIGLU) {
    __nv_bfloat16* dst = p.act + (size_t)(tile * kChainTile + f) + (size_t)c0 * N;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      // silu(g) = g * sigmoid(g) = g * (0.5 + 0.5 * tanh(g / 2)): one special-function
      // instruction instead of two (exp and reciprocal; that unit gives 16 results per clock and
      // SM).  tanh.approx is good to about 2^-11 absolute, the result is rounded to bf16
      const float gt = v0[j];
      float th;
      asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(0.5f * gt));
      v0[j] = gt * fmaf(0.5f, th, 0.5f) * v1[j];
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) dst[(size_t)j * N] = __float2bfloat16_rn(v0[j]);
  } else {  // CEPI_QKV
    float bias_f = 0.f;   // projection bias of this thread's output feature, before the rotation
    if (p.bq != nullptr) {
      const __nv_bfloat16* bb = tile >= p.nq + p.nkv ? p.bv + (tile - p.nq - p.nkv) * 128
                                : tile >= p.nq ? p.bk + (tile - p.nq) * 128 : p.bq + tile * 128;
      bias_f = __bfloat162float(__ldg(bb + f));
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) v0[j] += v1[j] + bias_f;
    const bool is_v = tile >= p.nq + p.nkv;
    if (is_v) {
      // V is stored transposed (keys contiguous): 16 consecutive keys of feature row f
      __nv_bfloat16* dst = p.v + (size_t)((tile - p.nq - p.nkv) * 128 + f) * p.ldv + c0;
#pragma unroll
      for (int j = 0; j < 16; j += 8) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          __nv_bfloat162 pr = __floats2bfloat162_rn(v0[j + 2 * e], v0[j + 2 * e + 1]);
          w[e] = *reinterpret_cast<uint32_t*>(&pr);
        }
        *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    } else {
      // rotate-half RoPE: feature i < 64 pairs with i + 64, held by the warp two quarters
      // away; the chunk is exchanged through shared memory
      // each thread's 16 values are one padded row of 20 floats: four 16-byte stores, and the
      // partner's row comes back with four 16-byte loads (no bank conflicts at this stride)
      float4* xrow = reinterpret_cast<float4*>(c.xch + half * (128 * kXchRow));   // `half`: the column part of this warp
#pragma unroll
      for (int k = 0; k < 4; ++k)
        xrow[f * (kXchRow / 4) + k] = make_float4(v0[4 * k], v0[4 * k + 1], v0[4 * k + 2], v0[4 * k + 3]);
      // the 128 threads of this column part meet on their own named barrier (1 .. 4)
      asm volatile("bar.sync %0, 128;" ::"r"(half + 1) : "memory");
      const bool lo = f < 64;
      const bool is_k = tile >= p.nq;
      const int ld = is_k ? p.nkv * 128 : p.nq * 128;
      __nv_bfloat16* dst = (is_k ? p.k + (size_t)((tile - p.nq) * 128 + f)
                                 : p.q + (size_t)(tile * 128 + f)) + (size_t)c0 * ld;
      float other[16];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 o4 = xrow[(f ^ 64) * (kXchRow / 4) + k];
        other[4 * k] = o4.x; other[4 * k + 1] = o4.y; other[4 * k + 2] = o4.z; other[4 * k + 3] = o4.w;
      }
      float cv = rb.c, sv = rb.s;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        v0[j] = lo ? (v0[j] * cv - other[j] * sv) : (v0[j] * cv + other[j] * sv);
        const float cn = cv * rb.cd - sv * rb.sd;
        sv = sv * rb.cd + cv * rb.sd;
        cv = cn;
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) dst[(size_t)j * ld] = __float2bfloat16_rn(v0[j]);
      asm volatile("bar.sync %0, 128;" ::"r"(half + 1) : "memory");
    }
  }
}


template <int EPI>
__device__ __forceinline__ void chain_gemm(ChainCtx& c, const ChainParams& p, const GemmPhase& g) {
  const int BN = p.BN;
  const int half_rows = BN >> 1;  // activation rows this CTA stages (the pair MMA reads both halves)
  ChainItem w;
  const bool has = chain_item(g.tiles, g.nsplit, g.KB, g.bal_h, w);
  // weight tiles per k-block: gate and up, or the two tiles of a helper pair in a balanced QKV
  const int nw = (EPI == CEPI_SWIGLU) ? 2 : (EPI == CEPI_QKV && has && w.tile2 >= 0) ? 2 : 1;
  const int slot_bytes = nw * kChainTile * kChainTileK * 2 + half_rows * kChainTileK * 2;
  int stages = kChainRing / slot_bytes;
  if (stages > 8) stages = 8;
  // map and first row of a QKV tile (q tiles, then k, then v)
  auto qkv_src = [&](int tile, const CUtensorMap*& m, int& row) {
    m = g.w0; row = tile * kChainTile;
    if (tile >= p.nq + p.nkv) { m = g.w2; row = (tile - p.nq - p.nkv) * kChainTile; }
    else if (tile >= p.nq) { m = g.w1; row = (tile - p.nq) * kChainTile; }
  };

  if (c.warp == 0) {
    bool ok = true;
    if (c.lane == 0) {
      // ---------------- TMA producer ----------------
      const uint32_t ring0 = ptx::smem_u32(c.ring);
      const uint32_t full0 = ptx::smem_u32(&c.full[0]), empty0 = ptx::smem_u32(&c.empty[0]);
      const uint32_t full_remote0 = c.rank == 0 ? full0 : ptx::mapa_shared(full0, 0);
      const int arow = (int)c.rank * half_rows;
      uint32_t ps = 0, pslot = ring0;
      const uint64_t pol_w = ptx::l2_policy_evict_first(), pol_a = ptx::l2_policy_evict_last();
      if (has) {
        const CUtensorMap *mw = g.w0, *mw2 = g.w1;
        int wrow = w.tile * kChainTile, wrow2 = wrow;
        if (EPI == CEPI_QKV) {
          qkv_src(w.tile, mw, wrow);
          if (nw == 2) qkv_src(w.tile2, mw2, wrow2);
        }
        // lean loop: slot index, addresses and coordinates advance by additions only
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          const uint32_t par = (c.fill_bits >> ps) & 1u;
          c.fill_bits ^= 1u << ps;
          ok = ptx::mbar_wait_a(empty0 + 8u * ps, par ^ 1u, c.abort_flag);
          if (!ok) break;
          // the bytes of both CTAs are credited to the even CTA's barrier, which its MMA issuer
          // waits on
          if (c.rank == 0) ptx::mbar_expect_tx_a(full0 + 8u * ps, 2u * (uint32_t)slot_bytes);
          const uint32_t bar = full_remote0 + 8u * ps;
          const int kc = kb * kChainTileK;
          // weights pass through L2 once (evict first); the activation tile is re-read by every CTA
          // and the small buffers between phases should stay resident (evict last): -5% step time
          ptx::tma_load_2d_pair_hint(pslot, mw, bar, kc, wrow, pol_w);
          if (nw == 2) ptx::tma_load_2d_pair_hint(pslot + kChainTile * kChainTileK * 2, mw2, bar, kc, wrow2, pol_w);
          ptx::tma_load_2d_pair_hint(pslot + nw * kChainTile * kChainTileK * 2, g.amap, bar, kc, arow, pol_a);
          if (++ps == (uint32_t)stages) { ps = 0; pslot = ring0; } else pslot += (uint32_t)slot_bytes;
        }
      }
    }
    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    {
      // ---------------- L2 prefetch of this CTA's item in the next GEMM phase ----------------
      // Issued by all lanes of the warp, a k-block each: a prefetch instruction occupies its thread
      // for a while, and the producer lane is needed again right after the grid barrier.
      ChainItem n;
      if (ok && g.pf_tiles > 0 && chain_item(g.pf_tiles, g.pf_nsplit, g.pf_KB, g.pf_bal_h, n)) {
        const int kb1 = n.kb1 > n.kb0 + g.pf_kb ? n.kb0 + g.pf_kb : n.kb1;
        const bool both = g.pf_w1 != nullptr && g.pf_t1 == 0;  // gate and up: same rows of two maps
        auto src = [&](int tile, const CUtensorMap*& m, int& row) {
          m = g.pf_w0; row = tile * kChainTile;
          if (!both && g.pf_w2 != nullptr && tile >= g.pf_t2) { m = g.pf_w2; row = (tile - g.pf_t2) * kChainTile; }
          else if (!both && g.pf_w1 != nullptr && tile >= g.pf_t1) { m = g.pf_w1; row = (tile - g.pf_t1) * kChainTile; }
        };
        const CUtensorMap *m0, *m1 = nullptr;
        int r0, r1 = 0;
        src(n.tile, m0, r0);
        if (both) { m1 = g.pf_w1; r1 = r0; }
        else if (n.tile2 >= 0) src(n.tile2, m1, r1);
        for (int kb = n.kb0 + c.lane; kb < kb1; kb += 32) {
          ptx::tma_prefetch_l2_2d(m0, kb * kChainTileK, r0);
          if (m1 != nullptr) ptx::tma_prefetch_l2_2d(m1, kb * kChainTileK, r1);
        }
      }
    }
  } else if (c.warp == 1) {
    if (c.lane == 0 && c.rank == 0 && has) {
      // ---------------- MMA issuer (even CTA of the pair, for both) ----------------
      // (A ring unrolled over its slots with split 32-bit descriptors issues an MMA every 97 clk at
      // N = 192 in isolation, against 140 for this loop, but these GEMMs wait for their data, not
      // for the issue, and the larger code made the launch 4% slower: measured and taken out.)
      const uint32_t idesc = ptx::idesc_bf16(2 * kChainTile, BN);
      bool ok = true;
      const uint32_t mring0 = ptx::smem_u32(c.ring);
      const uint32_t mfull0 = ptx::smem_u32(&c.full[0]), mempty0 = ptx::smem_u32(&c.empty[0]);
      const uint64_t desc_hi = ptx::smem_desc_sw128_hi();
      uint32_t ms = 0, mslot = mring0;
      if (c.mma_units > 0) {  // the epilogue has drained both accumulators of the last unit
        ok = ptx::mbar_wait(c.acc_empty, (c.mma_units - 1) & 1u, c.abort_flag);
      }
      ptx::tc_fence_after();
      uint32_t acc_first = 0;   // 0 until the first k-block of the unit has been issued
      for (int kb = w.kb0; kb < w.kb1 && ok; ++kb) {
        const uint32_t par = (c.use_bits >> ms) & 1u;
        c.use_bits ^= 1u << ms;
        ok = ptx::mbar_wait_a(mfull0 + 8u * ms, par, c.abort_flag);
        if (!ok) break;
        const uint64_t dw0 = desc_hi | (uint64_t)(mslot >> 4);
        const uint64_t dw1 = dw0 + (kChainTile * kChainTileK * 2 >> 4);
        const uint64_t da = dw0 + ((uint64_t)nw * (kChainTile * kChainTileK * 2 >> 4));
        if (nw == 2) {
          ptx::umma_bf16_pair(c.tmem_base, dw0, da, idesc, acc_first);
          ptx::umma_bf16_pair(c.tmem_base + 256, dw1, da, idesc, acc_first);
#pragma unroll
          for (int kk = 1; kk < kChainTileK / 16; ++kk) {
            ptx::umma_bf16_pair_acc(c.tmem_base, dw0 + 2 * kk, da + 2 * kk, idesc);
            ptx::umma_bf16_pair_acc(c.tmem_base + 256, dw1 + 2 * kk, da + 2 * kk, idesc);
          }
        } else {
          ptx::umma_bf16_pair(c.tmem_base, dw0, da, idesc, acc_first);
          ptx::umma_bf16_pair(c.tmem_base + 256, dw0 + 2, da + 2, idesc, acc_first);
          ptx::umma_bf16_pair_acc(c.tmem_base, dw0 + 4, da + 4, idesc);
          ptx::umma_bf16_pair_acc(c.tmem_base + 256, dw0 + 6, da + 6, idesc);
        }
        acc_first = 1;
        ptx::umma_commit_pair_a(mempty0 + 8u * ms);   // frees the slot in both CTAs
        if (++ms == (uint32_t)stages) { ms = 0; mslot = mring0; } else mslot += (uint32_t)slot_bytes;
      }
      if (ok) ptx::umma_commit_pair(c.acc_full);  // both epilogues start
      ++c.mma_units;
    }
  }
  __syncwarp();
  if (has) {
    // ---------------- epilogue: all warps; TMEM lane quarter = warp % 4, column part = warp / 4 ----
    const int quarter = c.warp & 3;
    const int half = c.warp >> 2;                    // column part 0 .. kChainParts-1
    const int part_cols = ((BN / 16 + kChainParts - 1) / kChainParts) * 16;
    const int col0 = min(half * part_cols, BN), col1 = min(col0 + part_cols, BN);
    const int f = quarter * 32 + c.lane;  // feature inside the tile = TMEM lane
    const uint32_t t_lane = c.tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int tile = w.tile, split = w.split, kind = w.kind;
    const bool rope = EPI == CEPI_QKV && kind != ITEM_HELP && tile < p.nq + p.nkv;
    RopeBase rb{1.f, 0.f, 1.f, 0.f};
    auto rope_base = [&](int c0, RopeBase& r) {
      int m0 = c0;  // a chunk of 16 rows never straddles the variants (rows_per_variant % 16 == 0)
      if (m0 >= p.rows_per_variant) m0 -= p.rows_per_variant;  // prev variant: same table
      const float* cs = p.cos_sin + (size_t)m0 * 128 + (f & 63);
      r.c = __ldg(cs); r.s = __ldg(cs + 64);
    };
    if (rope) {
      const float* dl = p.cos_sin + (size_t)p.rows_per_variant * 128 + (f & 63);  // step row
      rb.cd = __ldg(dl); rb.sd = __ldg(dl + 64);
    }
    bool ok = ptx::mbar_wait(c.acc_full, c.units_done & 1u, c.abort_flag);
    ++c.units_done;
    if (ok && EPI == CEPI_QKV && kind == ITEM_MAIN) {
      // the helper pair's part of this tile has been written (its warps have counted up)
      bool got = true;
      if (c.lane == 0) got = ptx::flag_wait(p.tile_flags + tile, p.flag_target, c.abort_flag);
      ok = __shfl_sync(0xffffffffu, (int)got, 0) != 0;   // also orders the lanes' loads behind the acquire
    }
    if (ok) {
      ptx::tc_fence_after();
      // 16 columns (activation rows) per step in a rolled loop (the code runs once per unit, so
      // it must stay small for the instruction cache).  No register double-buffering: the four
      // warps of a scheduler cover each other's TMEM and memory latencies.  BN equals M here (M
      // is a multiple of 16), so every column is a real row.
      float a0[16], a1[16];
      if (EPI == CEPI_QKV && kind != ITEM_FULL) {
        // sums handed from a helper pair to the tile's owner, in the order that makes every
        // access a 16-byte one and every warp access 512 contiguous bytes:
        // [tile][chunk of 16 rows][4][128 features][4 rows].  The owner adds them to the first
        // accumulator's registers; a helper stores the sum of its two accumulators, or, with two
        // tiles, one accumulator per tile.
        float4* hand = reinterpret_cast<float4*>(p.part + (size_t)tile * BN * kChainTile) + f;
        float4* hand2 = reinterpret_cast<float4*>(p.part + (size_t)(w.tile2 >= 0 ? w.tile2 : tile) * BN * kChainTile) + f;
        const bool dual = w.tile2 >= 0;
        // the owner's loads (helper sums, RoPE factors) are issued one chunk ahead: the warps of
        // a column part move in step through the exchange barriers, so nothing else would cover
        // their latency
        float4 ha[4], hn[4];
        RopeBase rn = rb;
        if (kind == ITEM_MAIN && col0 < col1) {
#pragma unroll
          for (int k = 0; k < 4; ++k) ha[k] = __ldcg(hand + (size_t)(col0 >> 4) * 4 * kChainTile + k * kChainTile);
          if (rope) rope_base(col0, rb);
        }
#pragma unroll 1
        for (int c0 = col0; c0 < col1; c0 += 16) {
          ptx::tmem_ld_32x16(t_lane + c0, a0);
          ptx::tmem_ld_32x16(t_lane + 256 + c0, a1);
          const size_t cq = (size_t)(c0 >> 4) * 4 * kChainTile;   // float4 index of this chunk
          if (kind == ITEM_HELP) {
            ptx::tmem_ld_wait();
            if (dual) {
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                __stcg(hand + cq + k * kChainTile, make_float4(a0[4 * k], a0[4 * k + 1], a0[4 * k + 2], a0[4 * k + 3]));
                __stcg(hand2 + cq + k * kChainTile, make_float4(a1[4 * k], a1[4 * k + 1], a1[4 * k + 2], a1[4 * k + 3]));
              }
            } else {
#pragma unroll
              for (int k = 0; k < 4; ++k)
                __stcg(hand + cq + k * kChainTile,
                       make_float4(a0[4 * k] + a1[4 * k], a0[4 * k + 1] + a1[4 * k + 1],
                                   a0[4 * k + 2] + a1[4 * k + 2], a0[4 * k + 3] + a1[4 * k + 3]));
            }
          } else {
            if (c0 + 16 < col1) {
#pragma unroll
              for (int k = 0; k < 4; ++k) hn[k] = __ldcg(hand + cq + (4 + k) * kChainTile);
              if (rope) rope_base(c0 + 16, rn);
            }
            ptx::tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              a0[4 * k] += ha[k].x; a0[4 * k + 1] += ha[k].y; a0[4 * k + 2] += ha[k].z; a0[4 * k + 3] += ha[k].w;
            }
            chain_emit<EPI>(c, p, g.N, tile, split, f, c0, a0, a1, rb, half);
#pragma unroll
            for (int k = 0; k < 4; ++k) ha[k] = hn[k];
            rb.c = rn.c; rb.s = rn.s;
          }
        }
        if (kind == ITEM_HELP) {
          __threadfence();
          __syncwarp();
          if (c.lane == 0) {
            ptx::flag_add(p.tile_flags + tile);
            if (dual) ptx::flag_add(p.tile_flags + w.tile2);
          }
        }
      } else {
        RopeBase rn = rb;
        if (rope && col0 < col1) rope_base(col0, rb);
#pragma unroll 1
        for (int c0 = col0; c0 < col1; c0 += 16) {
          ptx::tmem_ld_32x16(t_lane + c0, a0);
          ptx::tmem_ld_32x16(t_lane + 256 + c0, a1);
          if (rope && c0 + 16 < col1) rope_base(c0 + 16, rn);   // one chunk ahead
          ptx::tmem_ld_wait();
          chain_emit<EPI>(c, p, g.N, tile, split, f, c0, a0, a1, rb, half);
          rb.c = rn.c; rb.s = rn.s;
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(c.acc_empty);
    }
  }
  // the outputs are read through TMA (async proxy) by other CTAs after the grid barrier
  ptx::fence_proxy_async_global();
}

// x[row] += sum of the partial sums (in split order); out[row] = bf16(rmsnorm(x[row]) * g).
// Two rows per CTA at a time: warps 0..3 take one, warps 4..7 the other.  The rows of x and of
// the partial sums are brought into the (idle) ring by bulk copies, so that a CTA has all of its
// 160 KB in flight at once instead of a few loads per thread.
__device__ __forceinline__ void chain_norm(ChainCtx& c, const ChainParams& p, int nsplit,
                                           const __nv_bfloat16* __restrict__ g, float* red) {
  constexpr int kGrp = kChainThreads / 2;          // threads per row
  const int grp = threadIdx.x / kGrp;              // 0 or 1
  const int t = threadIdx.x - grp * kGrp;          // index inside the group
  const int d = p.d;
  const int narr = 1 + nsplit;
  float* stage = reinterpret_cast<float*>(c.ring);  // [grp][narr][d], then the gain vector
  __nv_bfloat16* sg = reinterpret_cast<__nv_bfloat16*>(stage + (size_t)2 * narr * d);
  for (int r0 = 2 * blockIdx.x; r0 < p.M; r0 += 2 * gridDim.x) {
    if (threadIdx.x == 0) {
      const int rows = (r0 + 1 < p.M) ? 2 : 1;
      ptx::fence_proxy_async_smem();  // earlier generic accesses to the staging space come first
      ptx::mbar_expect_tx(c.norm_bar, (uint32_t)(rows * narr * d * 4 + d * 2));
      ptx::bulk_load(sg, g, d * 2, c.norm_bar);
      for (int gi = 0; gi < rows; ++gi) {
        float* dst = stage + (size_t)gi * narr * d;
        ptx::bulk_load(dst, p.x + (size_t)(r0 + gi) * d, d * 4, c.norm_bar);
        for (int s = 0; s < nsplit; ++s)
          ptx::bulk_load(dst + (size_t)(s + 1) * d,
                         p.part + (size_t)s * p.part_stride + (size_t)(r0 + gi) * d, d * 4, c.norm_bar);
      }
    }
    const bool got = ptx::mbar_wait(c.norm_bar, c.norm_uses & 1u, c.abort_flag);
    ++c.norm_uses;
    const int row = r0 + grp;
    const bool live = got && row < p.M;
    float* sx = stage + (size_t)grp * narr * d;
    float ss = 0.f;
    if (live) {
      float* xr = p.x + (size_t)row * d;
      for (int i = t * 4; i < d; i += kGrp * 4) {
        float4 v = *reinterpret_cast<const float4*>(sx + i);
        if (nsplit > 0) {
          for (int s = 0; s < nsplit; ++s) {
            const float4 pv = *reinterpret_cast<const float4*>(sx + (size_t)(s + 1) * d + i);
            v.x += pv.x; v.y += pv.y; v.z += pv.z; v.w += pv.w;
          }
          *reinterpret_cast<float4*>(xr + i) = v;
          *reinterpret_cast<float4*>(sx + i) = v;
        }
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (c.lane == 0) red[c.warp] = ss;
    // group-wide exchange: named barriers 5 and 6 (1..4 belong to the QKV epilogue)
    asm volatile("bar.sync %0, %1;" ::"r"(grp + 5), "n"(kGrp) : "memory");
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < kGrp / 32; ++i) tot += red[grp * (kGrp / 32) + i];
    if (live) {
      const float inv = rsqrtf(tot / (float)d + p.eps);
      __nv_bfloat16* outr = p.a + (size_t)row * d;
      for (int i = t * 4; i < d; i += kGrp * 4) {
        const float4 v = *reinterpret_cast<const float4*>(sx + i);
        const uint2 gw = *reinterpret_cast<const uint2*>(sg + i);
        const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162*>(&gw.x);
        const __nv_bfloat162 g23 = *reinterpret_cast<const __nv_bfloat162*>(&gw.y);
        __nv_bfloat162 o01 = __floats2bfloat162_rn(v.x * inv * __low2float(g01), v.y * inv * __high2float(g01));
        __nv_bfloat162 o23 = __floats2bfloat162_rn(v.z * inv * __low2float(g23), v.w * inv * __high2float(g23));
        *reinterpret_cast<uint2*>(outr + i) =
            make_uint2(*reinterpret_cast<uint32_t*>(&o01), *reinterpret_cast<uint32_t*>(&o23));
      }
    }
    // everyone is done with the staged rows before the next pair is loaded over them
    __syncthreads();
  }
  ptx::fence_proxy_async_global();  // `a` is the next phase's TMA operand
}

__global__ void __launch_bounds__(kChainThreads, 1)
k_dense_chain(const __grid_constant__ ChainMaps maps, const ChainParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bar_full[8], bar_empty[8], bar_acc_full, bar_acc_empty, bar_norm;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float red[kChainThreads / 32];

  ChainCtx c;
  c.ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                      ~static_cast<uintptr_t>(1023));
  c.xch = reinterpret_cast<float*>(c.ring + kChainRing);
  c.full = bar_full; c.empty = bar_empty; c.acc_full = &bar_acc_full; c.acc_empty = &bar_acc_empty; c.norm_bar = &bar_norm;
  c.abort_flag = &abort_flag;
  c.fill_bits = 0; c.use_bits = 0; c.units_done = 0; c.mma_units = 0; c.norm_uses = 0;
  c.warp = threadIdx.x >> 5; c.lane = threadIdx.x & 31;
  c.rank = ptx::cluster_ctarank();

  if (threadIdx.x == 0) {
    // an earlier kernel of this step gave up: run through without touching anything (every CTA
    // still reaches the cluster barriers below)
    abort_flag = (*reinterpret_cast<volatile int32_t*>(p.status) != 0) ? 1 : 0;
    for (int i = 0; i < 8; ++i) { ptx::mbar_init(&bar_full[i], 1); ptx::mbar_init(&bar_empty[i], 1); }
    ptx::mbar_init(&bar_acc_full, 1);
    ptx::mbar_init(&bar_acc_empty, kChainThreads);
    ptx::mbar_init(&bar_norm, 1);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&maps.wo); ptx::prefetch_tmap(&maps.wg); ptx::prefetch_tmap(&maps.wu);
    ptx::prefetch_tmap(&maps.wd); ptx::prefetch_tmap(&maps.wq); ptx::prefetch_tmap(&maps.wk);
    ptx::prefetch_tmap(&maps.wv); ptx::prefetch_tmap(&maps.a); ptx::prefetch_tmap(&maps.o);
    ptx::prefetch_tmap(&maps.act);
    ptx::prefetch_tmap(&maps.wo_n);
  }
  if (c.warp == 1) {
    ptx::tmem_alloc(&tmem_base_s, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  c.tmem_base = tmem_base_s;
  // both CTAs of a pair hold all 512 columns, so the pair MMA's accumulator address (the even
  // CTA's) names the same columns in the odd CTA; anything else would be a silent mix-up
  if (threadIdx.x == 0 && c.tmem_base != 0) abort_flag = 1;
  // the partner's barriers are initialised before any of its loads can report to them
  ptx::cluster_sync();

  const int KBd = p.d / kChainTileK, KBq = p.nq * 128 / kChainTileK, KBf = p.F / kChainTileK;
  const int tiles_d = p.d / kChainTile, tiles_f = p.F / kChainTile, tiles_qkv = p.nq + 2 * p.nkv;
  const bool has_qkv = p.phase_end > CH_QKV;

  unsigned int n_barriers = 0;
  for (int ph = p.phase_begin; ph < p.phase_end; ++ph) {
    GemmPhase g{};
    const bool dead = abort_flag != 0;   // uniform: written before the last CTA-wide barrier
    if (!dead) switch (ph) {
      case CH_OPROJ:
        g.w0 = &maps.wo; g.amap = &maps.o; g.tiles = tiles_d; g.nsplit = p.split_o; g.KB = KBq; g.N = p.d;
        g.pf_w0 = &maps.wg; g.pf_w1 = &maps.wu; g.pf_t1 = 0; g.pf_tiles = tiles_f; g.pf_nsplit = 1;
        g.pf_KB = KBd; g.pf_kb = kPfGateUp;
        chain_gemm<CEPI_PARTIAL>(c, p, g);
        break;
      case CH_NORM2:
        chain_norm(c, p, p.split_o, p.g2, red);
        break;
      case CH_GATEUP:
        g.w0 = &maps.wg; g.w1 = &maps.wu; g.amap = &maps.a; g.tiles = tiles_f; g.nsplit = 1; g.KB = KBd; g.N = p.F;
        g.pf_w0 = &maps.wd; g.pf_tiles = tiles_d; g.pf_nsplit = p.split_down; g.pf_KB = KBf; g.pf_kb = kPfDown;
        chain_gemm<CEPI_SWIGLU>(c, p, g);
        break;
      case CH_DOWN:
        g.w0 = &maps.wd; g.amap = &maps.act; g.tiles = tiles_d; g.nsplit = p.split_down; g.KB = KBf; g.N = p.d;
        if (has_qkv) {
          g.pf_w0 = &maps.wq; g.pf_w1 = &maps.wk; g.pf_w2 = &maps.wv; g.pf_t1 = p.nq; g.pf_t2 = p.nq + p.nkv;
          g.pf_tiles = tiles_qkv; g.pf_nsplit = 1; g.pf_KB = KBd; g.pf_kb = kPfQkv; g.pf_bal_h = p.bal_h;
        }
        chain_gemm<CEPI_PARTIAL>(c, p, g);
        break;
      case CH_NORM1:
        chain_norm(c, p, p.fold_norm1, p.g1, red);
        break;
      default:  // CH_QKV
        g.w0 = &maps.wq; g.w1 = &maps.wk; g.w2 = &maps.wv; g.amap = &maps.a; g.tiles = tiles_qkv;
        g.nsplit = 1; g.KB = KBd; g.N = 0; g.bal_h = p.bal_h;
        // attention runs next; meanwhile the O projection of that layer streams into L2 (gate / up
        // of that layer on top of it was measured slower: +2..4% per step for 8..32 k-blocks)
        g.pf_w0 = &maps.wo_n; g.pf_tiles = tiles_d; g.pf_nsplit = p.split_o; g.pf_KB = KBq; g.pf_kb = 64;
        chain_gemm<CEPI_QKV>(c, p, g);
        break;
    }
    if (ph + 1 < p.phase_end) {
      __syncthreads();
      if (threadIdx.x == 0) {
        ++n_barriers;
        if (abort_flag == 0 && !ptx::grid_barrier(p.bar, p.bar_base + n_barriers * gridDim.x, p.status))
          abort_flag = 1;
        if (abort_flag) atomicExch(p.status, DC_ERR_TIMEOUT);
        ptx::fence_proxy_async_all();
      }
      __syncthreads();
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  // neither CTA of a pair leaves while the other may still read its shared memory or signal its
  // barriers
  ptx::cluster_sync();
  if (c.warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(c.tmem_base, 512);
  }
  if (threadIdx.x == 0 && abort_flag) atomicExch(p.status, DC_ERR_TIMEOUT);
}

}  // namespace dc
