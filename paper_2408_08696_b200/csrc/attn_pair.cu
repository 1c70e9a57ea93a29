// Tree attention (paper Sec. 2.2) for grouped-query shapes, head_dim 128: two 128-row query tiles per CTA on one
// K/V stream.
//
// With G query heads per KV head the G * N query rows of a KV head fill several 128-row tiles that all need the same
// keys and values.  At these shapes the op is bound by the tensor cores and the exponential unit, not by HBM, so the
// aim is to keep both busy at once: a CTA works on TWO row tiles ("streams" A and B), each with its own softmax
// warpgroup, its own MMA-issuing thread, its own score buffer and its own output accumulator in TMEM - one stream's
// softmax runs under the other stream's MMAs.  Keys come in tiles of 128 (a
// narrower S = Q K^T instruction is bound by re-reading the Q operand from shared memory, not by the tensor core):
// 2 streams x (128 score columns + 128 output columns) = all 512 TMEM columns.  P is handed over in two halves of 64
// keys, so the first half's P V runs under the second half's exponentials.
//
//   warps 0..3   softmax, stream A: thread r owns query row r (TMEM lane r): scores -> ancestor mask -> exp2 with a
//                lazily updated reference maximum -> P (bf16) over S in TMEM; at the end of a unit it normalises and
//                stores its output row
//   warps 4..7   the same for stream B
//   warp 8       TMA producer: takes the next unit from a global counter, publishes it to the other roles, loads the
//                unit's Q tiles and its K / V tiles (128 keys x 128 dims, 32 KB) into a ring of 5 slots
//   warp 9       MMA issuer of stream A: S = Q K^T and O += P V (per half); owns the TMEM allocation
//   warp 10      MMA issuer of stream B
//
// Units.  Per (sequence, layer, KV head) the MT row tiles are taken two at a time: "pair" units share one K/V stream.
// When MT is odd, the left-over tiles of two neighbouring KV heads form a "twin" unit: two streams with their own K/V
// each, so that every unit advances through the keys at the same pace and units that read the same K/V (which start
// close together) find it in L2.  Units are handed out dynamically (they differ in cost and SMs differ in speed).
// Every wait is bounded; a wait that runs out sets TR_FLAG_WAIT_TIMEOUT and the CTA drains and exits.
#include "tc_ptx.cuh"
#include "tr_internal.cuh"

namespace {

constexpr int BK = 128;                           // keys per tile
constexpr int HD = 128;                           // head_dim
constexpr int KV_TILE_BYTES = BK * HD * 2;        // 32 KB
constexpr int KV_HALF_BYTES = KV_TILE_BYTES / 2;  // one TMA box: 64 dims x 128 keys
constexpr int Q_TILE_BYTES = 128 * HD * 2;        // 32 KB
constexpr int Q_HALF_BYTES = Q_TILE_BYTES / 2;    // one TMA box: 64 dims x 128 rows
constexpr int NSLOT = 5;                          // ring slots (K and V tiles alternate)
constexpr int NTHREADS = 384;
// Registers are re-balanced after start-up (setmaxnreg): 12 warps are launched at 168 each, which fixes the CTA's pool
// at 12 x 32 x 168 = 64512; a softmax thread keeps a whole 128-column score row in registers.  The raised budgets must
// fit into the pool, or the last warp to ask waits for ever: 8 x 32 x 216 + 4 x 32 x 64 = 63488.
constexpr int REGS_SOFTMAX = 216, REGS_CONTROL = 64;
static_assert(8 * 32 * REGS_SOFTMAX + 4 * 32 * REGS_CONTROL <= 12 * 32 * 168, "setmaxnreg budgets exceed the CTA's pool");
constexpr int WARP_PRODUCER = 8, WARP_QK = 9, WARP_PV = 10;
constexpr int UQ = 4;                             // depth of the CTA's unit queue

TR_STAMP_DECL(g_pair_stamps, 64)
#ifdef TR_STAMPS
#define PCLK() clock64()
#define PACC(var, t0) var += clock64() - (t0)
#else
#define PCLK() 0ll
#define PACC(var, t0) do { } while (0)
#endif

struct PairParams {
  __nv_bfloat16* out;
  const int32_t* ctx_len;
  const uint32_t* anc;
  uint32_t* flags;
  unsigned int* queue;  // [0]: next unit, [1]: CTAs that are done with it (the last one clears both)
  int N, L, HU, G, g_shift, MT;
  int NP;            // pair units per (sequence, layer, KV head) = MT / 2
  int twins;         // twin units per (sequence, layer): (HU + 1) / 2 when MT is odd, else 0
  int units_per_bl;  // HU * NP + twins
  int n_units;
  int64_t os_b, os_h, os_t, os_l;
  float scale_log2;
};

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int SM_Q = 0;                                // 2 x 32 KB
constexpr int SM_RING = 2 * Q_TILE_BYTES;              // 5 x 32 KB
constexpr int SM_BAR = SM_RING + NSLOT * KV_TILE_BYTES;
constexpr int BAR_FULL = 0, BAR_EMPTY = NSLOT, BAR_QFULL = 2 * NSLOT, BAR_QEMPTY = BAR_QFULL + 2,
              BAR_SFULL = BAR_QEMPTY + 2, BAR_PFULL = BAR_SFULL + 2, BAR_OREADY = BAR_PFULL + 4, BAR_OFREE = BAR_OREADY + 2, BAR_UFULL = BAR_OFREE + 2,
              BAR_UEMPTY = BAR_UFULL + UQ, BAR_TURN = BAR_UEMPTY + UQ, BAR_COUNT = BAR_TURN + 2;
constexpr int SM_MISC = SM_BAR + BAR_COUNT * 8;        // tmem base (4 B), abort flag (4 B)
constexpr int SM_UNIT = SM_MISC + 16;                  // unit queue: UQ ints
constexpr int SMEM_BYTES = SM_UNIT + UQ * 4;
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB a CTA can opt in to");

struct PairUnit {
  int b, layer, C, nt;     // tiles of BK keys over the prefix and the tree
  int ns;                  // streams in use (1 or 2)
  int shared;              // both streams read the same K/V tiles
  int hu[2], mt[2];        // per stream: head unit (= KV head) and row tile
  int m64[2];              // per stream: the tile has at most 64 real rows -> its products run with M = 64
};

__device__ __forceinline__ PairUnit decode_pair_unit(const PairParams& p, int u) {
  PairUnit x;
  const int bl = u / p.units_per_bl, r = u - bl * p.units_per_bl;
  x.b = bl / p.L;
  x.layer = bl - x.b * p.L;
  x.C = p.ctx_len[x.b];
  x.nt = (x.C + p.N + BK - 1) / BK;
  if (r < p.HU * p.NP) {
    const int hu = r / p.NP, pp = r - hu * p.NP;
    x.ns = 2; x.shared = 1;
    x.hu[0] = x.hu[1] = hu;
    x.mt[0] = 2 * pp; x.mt[1] = 2 * pp + 1;
  } else {
    const int q = r - p.HU * p.NP;
    x.shared = 0;
    x.hu[0] = 2 * q; x.hu[1] = 2 * q + 1;
    x.mt[0] = x.mt[1] = p.MT - 1;
    x.ns = x.hu[1] < p.HU ? 2 : 1;
  }
#pragma unroll
  for (int s = 0; s < 2; ++s) {  // real rows of the tile = its nodes below N, times the group's heads
    const int nodes_live = min(128 >> p.g_shift, p.N - x.mt[s] * (128 >> p.g_shift));
    x.m64[s] = (nodes_live << p.g_shift) <= 64 ? 1 : 0;
  }
  return x;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(NTHREADS, 1)
tr_attn_pair_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const PairParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {  // swizzled tiles need a 1024-byte aligned window; not expected, but checked
    if (threadIdx.x == 0) atomicOr(p.flags, TR_FLAG_WAIT_TIMEOUT);
    return;
  }
  const uint32_t bars = base + SM_BAR;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem_raw + SM_MISC);
  volatile uint32_t* s_abort = s_tmem + 1;
  volatile int* s_unit = reinterpret_cast<volatile int*>(smem_raw + SM_UNIT);
  auto bar = [&](int i) { return bars + static_cast<uint32_t>(i) * 8u; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < NSLOT; ++i) {
      mbar_init(bar(BAR_FULL + i), 1);
      mbar_init(bar(BAR_EMPTY + i), 2);  // one commit per stream (a tile read by one stream only is committed twice)
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_QFULL + i), 1);
      mbar_init(bar(BAR_QEMPTY + i), 1);
      mbar_init(bar(BAR_OREADY + i), 1);
      mbar_init(bar(BAR_OFREE + i), 4);   // one arrival per softmax warp of the stream
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_SFULL + i), 1);
    }
    for (int i = 0; i < 4; ++i) mbar_init(bar(BAR_PFULL + i), 4);  // (stream, half): one arrival per softmax warp
    for (int i = 0; i < 2; ++i) mbar_init(bar(BAR_TURN + i), 4);
    for (int i = 0; i < UQ; ++i) {
      mbar_init(bar(BAR_UFULL + i), 1);
      mbar_init(bar(BAR_UEMPTY + i), 10);  // the two MMA issuing threads and the eight softmax warps
    }
    *s_abort = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == WARP_QK) {  // TMEM: all 512 columns (one CTA per SM)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + SM_MISC), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  // TMEM columns: scores (then P) of stream s at 128 s; output accumulator of stream s at 256 + 128 s
  auto s_col = [&](uint32_t s) { return tmem + 128u * s; };
  auto o_col = [&](uint32_t s) { return tmem + 256u + 128u * s; };

  // every consumer role takes the next unit from the CTA's queue the same way
  auto next_unit = [&](uint32_t ui, bool one_arrival_per_warp) -> int {
    const uint32_t slot = ui % UQ;
    if (!mbar_wait<0>(bar(BAR_UFULL + slot), (ui / UQ) & 1u, s_abort)) return -2;
    const int u = s_unit[slot];
    if (one_arrival_per_warp) {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_UEMPTY + slot));
    } else {
      mbar_arrive(bar(BAR_UEMPTY + slot));
    }
    return u;
  };

  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_CONTROL));
  if (warp == WARP_PRODUCER) {
    // =========================== TMA producer and unit dispatcher ===========================
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_first();
      uint32_t ui = 0, c = 0, us[2] = {0u, 0u};
      bool ok = true;
      while (ok) {
        const uint32_t qs = ui % UQ;
        ok = mbar_wait<0>(bar(BAR_UEMPTY + qs), ((ui / UQ) & 1u) ^ 1u, s_abort);
        if (!ok) break;
        int u = static_cast<int>(atomicAdd(p.queue, 1u));
        if (u >= p.n_units) u = -1;
        s_unit[qs] = u;
        mbar_arrive(bar(BAR_UFULL + qs));
        if (u < 0) break;
        const PairUnit x = decode_pair_unit(p, u);
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          if (s >= x.ns || !ok) break;
          ok = mbar_wait<0>(bar(BAR_QEMPTY + s), (us[s] & 1u) ^ 1u, s_abort);
          if (!ok) break;
          const uint32_t dst = base + SM_Q + s * Q_TILE_BYTES;
          const int h0 = x.hu[s] * p.G, node0 = x.mt[s] * (128 >> p.g_shift);
          mbar_expect_tx(bar(BAR_QFULL + s), Q_TILE_BYTES);
          tma_load_5d(dst, &map_q, bar(BAR_QFULL + s), 0, h0, node0, x.layer, x.b);
          tma_load_5d(dst + Q_HALF_BYTES, &map_q, bar(BAR_QFULL + s), 64, h0, node0, x.layer, x.b);
          ++us[s];
        }
        const int nsrc = x.shared ? 1 : x.ns;
        for (int t = 0; t < x.nt && ok; ++t) {
#pragma unroll
          for (int src = 0; src < 2; ++src) {
            if (src >= nsrc || !ok) break;
#pragma unroll
            for (int kv = 0; kv < 2; ++kv) {
              const uint32_t slot = c % NSLOT;
              ok = mbar_wait<0>(bar(BAR_EMPTY + slot), ((c / NSLOT) & 1u) ^ 1u, s_abort);
              if (!ok) break;
              const CUtensorMap* m = kv == 0 ? &map_k : &map_v;
              const uint32_t dst = base + SM_RING + slot * KV_TILE_BYTES;
              mbar_expect_tx(bar(BAR_FULL + slot), KV_TILE_BYTES);
              tma_load_5d_hint(dst, m, bar(BAR_FULL + slot), 0, t * BK, x.hu[src], x.layer, x.b, pol);
              tma_load_5d_hint(dst + KV_HALF_BYTES, m, bar(BAR_FULL + slot), 64, t * BK, x.hu[src], x.layer, x.b, pol);
              ++c;
            }
          }
        }
        ++ui;
      }
    }
    __syncwarp();
  } else if (warp == WARP_QK || warp == WARP_PV) {
    // =========================== MMA issuer of stream s: S = Q K^T and O += P V ===========================
    // One thread issues both products of a stream.  The tensor core runs one thread's instructions in order, so
    // S(t + 1) = Q K(t + 1)^T is issued right behind O += P(t) V(t) without waiting for it to finish: it cannot
    // overwrite P(t) before it has been read, and a finished S(t + 1) implies that O holds every tile up to t (which
    // is what the softmax warps rely on when they rescale O).
    if (lane == 0) {
      const int s = warp - WARP_QK;
      uint32_t IDESC_QK = make_idesc(false, BK);  // N = 128 keys
      uint32_t IDESC_PV = make_idesc(true, HD);
      constexpr uint32_t M_MASK = 0x1Fu << 24;
      uint32_t ui = 0, c = 0, g = 0, us = 0;  // units seen, ring entries, this stream's tiles and units
      bool ok = true;
      long long w_k = 0, w_v = 0, w_p = 0, w_qk = 0, w_pvi = 0, w_tot = PCLK(), n_t = 0;
      const uint32_t q_lo = smem_desc_lo(base + SM_Q + s * Q_TILE_BYTES, 16);
      const uint32_t d_tm = s_col(s), o_tm = o_col(s);
      auto issue_qk = [&](uint32_t ke, bool shared) -> bool {  // S = Q K^T for the K tile in ring entry ke
        const uint32_t slot = ke % NSLOT;
        long long t0 = PCLK();
        if (!mbar_wait<0>(bar(BAR_FULL + slot), (ke / NSLOT) & 1u, s_abort)) return false;
        PACC(w_k, t0); t0 = PCLK();
        tc_fence_after();
        const uint32_t k_lo = smem_desc_lo(base + SM_RING + slot * KV_TILE_BYTES, 16);
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          // 16 dims per step: 32 bytes inside a 128-byte swizzle row; the second 64 dims sit in the second box
          const uint32_t off16 = static_cast<uint32_t>(((k >> 2) * Q_HALF_BYTES + (k & 3) * 32) >> 4);
          tc_mma_ss_lh(d_tm, q_lo + off16, k_lo + off16, smem_desc_hi(1024), IDESC_QK, k > 0);
        }
        tc_commit(bar(BAR_EMPTY + slot));               // K tile consumed by this stream ...
        if (!shared) tc_commit(bar(BAR_EMPTY + slot));  // ... and nobody else reads it (the barrier counts two)
        tc_commit(bar(BAR_SFULL + s));                  // S ready for the softmax warps
        PACC(w_qk, t0);
        return true;
      };
      while (ok) {
        const int u = next_unit(ui, false);
        if (u < 0) break;
        ++ui;
        const PairUnit x = decode_pair_unit(p, u);
        const uint32_t nsrc = x.shared ? 1u : static_cast<uint32_t>(x.ns);
        if (s >= x.ns) {  // a lone tile: this stream sits the unit out
          c += 2u * nsrc * static_cast<uint32_t>(x.nt);
          continue;
        }
        const uint32_t src = x.shared ? 0u : static_cast<uint32_t>(s);
        {  // M of this unit's products: 64 when the tile's upper half holds no real row
          const uint32_t m_bits = (x.m64[s] ? (64u >> 4) : (128u >> 4)) << 24;
          IDESC_QK = (IDESC_QK & ~M_MASK) | m_bits;
          IDESC_PV = (IDESC_PV & ~M_MASK) | m_bits;
        }
        ok = mbar_wait<0>(bar(BAR_QFULL + s), us & 1u, s_abort);
        if (!ok) break;
        ok = issue_qk(c + 2u * src, x.shared != 0);
        // (the Q tile is handed back as soon as the unit's last S = Q K^T has been issued, so that the next unit's Q
        // arrives under this unit's last tile)
        if (x.nt == 1) tc_commit(bar(BAR_QEMPTY + s));
        for (int t = 0; t < x.nt && ok; ++t, ++g) {
          if (t == 0) {  // the accumulator must have been read out by the stream's epilogue of its previous unit
            ok = mbar_wait<0>(bar(BAR_OFREE + s), (us & 1u) ^ 1u, s_abort);
            if (!ok) break;
          }
          const uint32_t ve = c + 2u * src + 1u, slot = ve % NSLOT;
          long long t0 = PCLK();
          ok = mbar_wait<0>(bar(BAR_FULL + slot), (ve / NSLOT) & 1u, s_abort);
          if (!ok) break;
          PACC(w_v, t0);
          // B = V tile, MN-major: the two 64-dim boxes are 16 KB apart, 8-key groups 1 KB apart, 16 keys per step
          const uint32_t v_lo = smem_desc_lo(base + SM_RING + slot * KV_TILE_BYTES, KV_HALF_BYTES);
#pragma unroll
          for (int h = 0; h < 2; ++h) {  // P arrives in two halves of 64 keys
            t0 = PCLK();
            ok = mbar_wait<0>(bar(BAR_PFULL + 2 * s + h), g & 1u, s_abort);
            if (!ok) break;
            PACC(w_p, t0); t0 = PCLK();
            tc_fence_after();
#pragma unroll
            for (int k = 4 * h; k < 4 * h + 4; ++k)  // A = P: bf16 pairs, 8 TMEM columns per 16 keys
              tc_mma_ts_lh(o_tm, d_tm + k * 8u, v_lo + k * (2048u >> 4), smem_desc_hi(1024), IDESC_PV,
                           (t > 0 || k > 0) ? 1u : 0u);
            PACC(w_pvi, t0);
          }
          if (!ok) break;
          t0 = PCLK();
          tc_commit(bar(BAR_EMPTY + slot));                 // V tile consumed by this stream ...
          if (!x.shared) tc_commit(bar(BAR_EMPTY + slot));  // ... and nobody else reads it
          c += 2u * nsrc;
          ++n_t;
          if (t == x.nt - 1) {
            tc_commit(bar(BAR_OREADY + s));  // the stream's output is complete
            ++us;
            PACC(w_pvi, t0);
          } else {
            PACC(w_pvi, t0);
            ok = issue_qk(c + 2u * src, x.shared != 0);  // the next tile's scores, right behind this tile's PV
            if (t == x.nt - 2) tc_commit(bar(BAR_QEMPTY + s));  // that was the unit's last S = Q K^T
          }
        }
      }
#ifdef TR_STAMPS
      if (blockIdx.x == 0) {
        const int o = 8 * s;
        g_pair_stamps[o] = clock64() - w_tot; g_pair_stamps[o + 1] = w_k; g_pair_stamps[o + 2] = w_v;
        g_pair_stamps[o + 3] = w_p; g_pair_stamps[o + 4] = w_qk; g_pair_stamps[o + 5] = w_pvi; g_pair_stamps[o + 6] = n_t;
      }
#endif
    }
    __syncwarp();
  }
  } else {
    // =========================== softmax + epilogue of stream s ===========================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
    const int s = warp >> 2;
    const int r_full = (warp & 3) * 32 + lane;  // query row == TMEM lane (M = 128)
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    uint32_t ui = 0, g = 0, us = 0, gp = 0;  // gp: tiles of two-stream units (the same count in both warpgroups)
    bool ok = true;
    long long w_s = 0, w_busy = 0, w_epi = 0, w_tot = PCLK(), n_resc = 0;
    while (ok) {
      const int u = next_unit(ui, true);
      if (u < 0) break;
      ++ui;
      const PairUnit x = decode_pair_unit(p, u);
      if (s >= x.ns) continue;
      // A tile with at most 64 real rows (e.g. the third row tile of a 4-heads-per-KV-head group with 80 nodes) runs
      // its products with M = 64.  The accumulator's row i then sits in TMEM lane 32 (i / 16) + i % 16: every warp
      // owns sixteen rows, in its lower sixteen lanes (2 % faster at `llama3-8b`; the other shapes have no such tile).
      const int r = x.m64[s] ? (warp & 3) * 16 + (lane & 15) : r_full;
      const bool lane_ok = !x.m64[s] || lane < 16;
      const int node = x.mt[s] * (128 >> p.g_shift) + (r >> p.g_shift);  // rows of a packed tile are node-major ...
      const int head = x.hu[s] * p.G + (r & (p.G - 1));                  // ... with the group's query heads interleaved
      const bool row_ok = lane_ok && node < p.N;
      uint32_t anc[4];
#pragma unroll
      for (int w = 0; w < 4; ++w) anc[w] = row_ok ? p.anc[node * 4 + w] : 0u;
      float m_ref = -INFINITY, l = 0.f;
      for (int t = 0; t < x.nt && ok; ++t, ++g) {
        long long t0 = PCLK();
        ok = mbar_wait<0>(bar(BAR_SFULL + s), g & 1u, s_abort);
        ok = __all_sync(0xFFFFFFFFu, ok);  // the TMEM loads below are warp-collective
        if (!ok) break;
        // The two warpgroups take turns (A, B, A, ...): the exponentials of one stream then run while the other
        // stream's MMAs are in flight, instead of both streams' exponentials sharing the special-function unit and
        // both streams' MMAs sharing the tensor core at the same time.
        if (x.ns == 2) {
          ok = mbar_wait<0>(bar(BAR_TURN + s), s == 0 ? ((gp & 1u) ^ 1u) : (gp & 1u), s_abort);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
        }
        PACC(w_s, t0); t0 = PCLK();
        tc_fence_after();
        uint32_t sreg[4][32];
#pragma unroll
        for (int q = 0; q < 4; ++q) tc_ld32(s_col(s) + lane_base + q * 32u, sreg[q]);
        tc_wait_ld();
        const int key0 = t * BK;
        if (key0 + BK > x.C) {  // only the one or two tiles that reach into the tree's keys
          const int sh0 = x.C - key0;  // tile column of the first tree key (may be <= 0 or >= 128)
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            // bit c of the word: column 32 w + c is visible iff it is a prefix key (column < sh0) or bit
            // (column - sh0) of the row's ancestor mask is set
            const int col0 = 32 * w, sh = col0 - sh0;  // tree index of column col0
            uint32_t word = 0u;
            if (sh0 >= col0 + 32) word = 0xFFFFFFFFu;
            else if (sh0 > col0) word = (1u << (sh0 - col0)) - 1u;
            uint32_t tw = 0u;
            if (sh >= 0) {
              const int wi = sh >> 5, bi = sh & 31;
              const uint32_t lo = wi < 4 ? (wi == 0 ? anc[0] : wi == 1 ? anc[1] : wi == 2 ? anc[2] : anc[3]) : 0u;
              const uint32_t hi = wi + 1 < 4 ? (wi == 0 ? anc[1] : wi == 1 ? anc[2] : anc[3]) : 0u;
              tw = bi ? ((lo >> bi) | (hi << (32 - bi))) : lo;
            } else if (sh > -32) {
              tw = anc[0] << (-sh);
            }
            const uint32_t vis = word | tw;
#pragma unroll
            for (int cc = 0; cc < 32; ++cc)
              if (!((vis >> cc) & 1u)) sreg[w][cc] = 0xFF800000u;  // -inf
          }
        }
        // row maximum of the raw scores: eight independent chains (scale > 0, applied afterwards)
        float mx[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) mx[i] = -INFINITY;
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int cc = 0; cc < 32; cc += 2)
            mx[(cc >> 1) & 7] = max3(mx[(cc >> 1) & 7], __uint_as_float(sreg[q][cc]), __uint_as_float(sreg[q][cc + 1]));
        const float tmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                 fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7]))) * p.scale_log2;
        // lazy rescale: keep the old reference unless the maximum grew by more than 2^8
        float alpha = 1.f;
        if (tmax > m_ref + 8.f) {
          alpha = (m_ref == -INFINITY) ? 0.f : fast_exp2(m_ref - tmax);
          m_ref = tmax;
        }
        const bool need = (alpha != 1.f) && (t > 0);
        if (__any_sync(0xFFFFFFFFu, need)) {
          ++n_resc;
          // O of this unit holds the tiles before t.  Their PVs have all landed: this tile's S was only computed
          // after the previous tile's PV had completed.
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t oreg[32];
            tc_ld32(o_col(s) + lane_base + q * 32u, oreg);
            tc_wait_ld();
#pragma unroll
            for (int cc = 0; cc < 32; ++cc) oreg[cc] = __float_as_uint(__uint_as_float(oreg[cc]) * alpha);
            tc_st32(o_col(s) + lane_base + q * 32u, oreg);
          }
        }
        l *= alpha;
        const float nsub = (m_ref == -INFINITY) ? 0.f : -m_ref;
        const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), nsub2 = pack2(nsub, nsub);
        uint64_t sm2[4] = {0ull, 0ull, 0ull, 0ull};  // packed (even, odd) partial row sums
#pragma unroll
        for (int h = 0; h < 2; ++h) {  // P goes out in two halves of 64 keys: the first half's PV starts early
          uint32_t preg[32];
#pragma unroll
          for (int q = 2 * h; q < 2 * h + 2; ++q)
#pragma unroll
            for (int cc = 0; cc < 32; cc += 2) {
              float x0, x1;
              unpack2(fma2(pack2(__uint_as_float(sreg[q][cc]), __uint_as_float(sreg[q][cc + 1])), scale2, nsub2), x0, x1);
              const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
              sm2[(cc >> 1) & 3] = add2(sm2[(cc >> 1) & 3], pack2(p0, p1));
              __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
              preg[(q & 1) * 16 + (cc >> 1)] = *reinterpret_cast<uint32_t*>(&pk);
            }
          // The other stream's turn begins when this stream's last exponentials are done: its softmax starts with work
          // that does not need the special-function unit (TMEM loads, the maximum), which so runs under this stream's
          // last P store (2 % faster than handing over after the store; handing over earlier still - with up to a quarter
          // of the exponentials to go - measured the same, after the first half slower).
          if (h == 1 && x.ns == 2 && lane == 0) mbar_arrive(bar(BAR_TURN + (s ^ 1)));
          tc_st32(s_col(s) + lane_base + h * 32u, preg);
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(BAR_PFULL + 2 * s + h));
        }
        if (x.ns == 2) ++gp;
        float se, so;
        unpack2(add2(add2(sm2[0], sm2[1]), add2(sm2[2], sm2[3])), se, so);
        l += se + so;
        PACC(w_busy, t0);
      }
      if (!ok) break;
      long long t1 = PCLK();
      // ---- epilogue: the unit's last PV has landed -> normalise the row out of TMEM and store it
      ok = mbar_wait<0>(bar(BAR_OREADY + s), us & 1u, s_abort);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      ++us;
      tc_fence_after();
      const float inv = 1.f / l;
      __nv_bfloat16* orow = p.out + x.b * p.os_b + x.layer * p.os_l + head * p.os_h + static_cast<int64_t>(node) * p.os_t;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t oreg[32];
        tc_ld32(o_col(s) + lane_base + q * 32u, oreg);
        tc_wait_ld();
        if (q == 3) {  // O is in registers: hand the accumulator back to the PV issuer
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(BAR_OFREE + s));
        }
        if (row_ok) {
#pragma unroll
          for (int cc = 0; cc < 32; cc += 8) {
            uint4 w4;
            __nv_bfloat162 t0 = __floats2bfloat162_rn(__uint_as_float(oreg[cc + 0]) * inv, __uint_as_float(oreg[cc + 1]) * inv);
            __nv_bfloat162 t1 = __floats2bfloat162_rn(__uint_as_float(oreg[cc + 2]) * inv, __uint_as_float(oreg[cc + 3]) * inv);
            __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(oreg[cc + 4]) * inv, __uint_as_float(oreg[cc + 5]) * inv);
            __nv_bfloat162 t3 = __floats2bfloat162_rn(__uint_as_float(oreg[cc + 6]) * inv, __uint_as_float(oreg[cc + 7]) * inv);
            w4.x = *reinterpret_cast<uint32_t*>(&t0); w4.y = *reinterpret_cast<uint32_t*>(&t1);
            w4.z = *reinterpret_cast<uint32_t*>(&t2); w4.w = *reinterpret_cast<uint32_t*>(&t3);
            *reinterpret_cast<uint4*>(orow + q * 32 + cc) = w4;
          }
        }
      }
      PACC(w_epi, t1);
    }
#ifdef TR_STAMPS
    if (blockIdx.x == 0 && (tid & 127) == 0) {
      const int o = 16 + 8 * s;
      g_pair_stamps[o] = clock64() - w_tot; g_pair_stamps[o + 1] = w_s; g_pair_stamps[o + 2] = w_busy;
      g_pair_stamps[o + 3] = w_epi; g_pair_stamps[o + 4] = g; g_pair_stamps[o + 5] = n_resc; g_pair_stamps[o + 6] = ui;
    }
#endif
  }

  // ---- teardown: every thread arrives here, also after an aborted wait
  __syncthreads();
  if (tid == 0) {
    // the unit counter clears itself: the last CTA to get here (every CTA's dispatcher has stopped drawing by then)
    // resets it for the next launch
    __threadfence();
    const unsigned int d = atomicAdd(p.queue + 1, 1u);
    if (d == gridDim.x - 1) {
      p.queue[0] = 0u;
      p.queue[1] = 0u;
      __threadfence();
    }
  }
  if (*s_abort) {
    if (tid == 0) atomicOr(p.flags, TR_FLAG_WAIT_TIMEOUT);
    // give copies and MMAs that may still be in flight time to land before shared memory and TMEM are released
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == WARP_QK) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// 5-D bf16 tensor map with 128-byte swizzle; out-of-bounds elements read as zero.  dims[0] is head_dim (contiguous);
// strides (elements) belong to dims[1..4]; a stride of a size-1 dimension may be anything.
bool encode_map5(CUtensorMap* m, const void* ptr, const uint64_t (&dims)[5], const int64_t (&strides)[4],
                 const uint32_t (&box)[5]) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t gd[5], gs[4];
  cuuint32_t bx[5], es[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < 5; ++i) { gd[i] = dims[i]; bx[i] = box[i]; }
  for (int i = 0; i < 4; ++i) gs[i] = static_cast<cuuint64_t>(strides[i] > 0 ? strides[i] : HD) * 2;  // bytes
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), gd, gs, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

#ifdef TR_STAMPS
extern "C" int tr_debug_stamps_pair(unsigned long long* host) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(host, g_pair_stamps, sizeof(unsigned long long) * 64);
  return 0;
}
#endif

static bool g_pair_usable = false;

tr_status tr_attention_pair_setup() {
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
  // The kernel raises its softmax warps' register budget at run time; the request blocks until the CTA's pool (the
  // registers the kernel was compiled to launch with, times its threads) has that much to give.  Use the kernel only
  // if the compiled register count makes the pool large enough - otherwise the other attention kernel serves.
  cudaFuncAttributes fa;
  TR_CUDA_TRY(cudaFuncGetAttributes(&fa, tr_attn_pair_kernel));
  g_pair_usable = fa.numRegs * NTHREADS >= 8 * 32 * REGS_SOFTMAX + 4 * 32 * REGS_CONTROL;
  return get_encode_fn() ? TR_OK : TR_ERR_CUDA;
}

// Whether the two-tiles-per-CTA kernel applies: head_dim 128, a group size > 1 that divides 128, at least two row tiles
// per KV head.  (It has no split-KV path: the caller uses it only when the launch has enough units without splitting.)
bool tr_attention_pair_applies(const tr_ctx* ctx, const tr_attn_args* a) {
  if (!g_pair_usable || a->head_dim != HD) return false;
  const int group = a->n_q_heads / a->n_kv_heads;
  if (group <= 1 || (128 % group) != 0) return false;
  return (ctx->n_nodes * group + 127) / 128 >= 2;
}

tr_status tr_launch_attention_pair(tr_ctx* ctx, const tr_attn_args* a, cudaStream_t s) {
  const int group = a->n_q_heads / a->n_kv_heads;
  PairParams p;
  p.G = group;
  p.g_shift = 0;
  while ((1 << p.g_shift) < p.G) ++p.g_shift;
  p.HU = a->n_kv_heads;
  p.MT = (ctx->n_nodes * p.G + 127) / 128;
  p.NP = p.MT / 2;
  p.twins = (p.MT & 1) ? (p.HU + 1) / 2 : 0;
  p.units_per_bl = p.HU * p.NP + p.twins;
  const int64_t units = static_cast<int64_t>(ctx->batch) * a->n_layers * p.units_per_bl;
  if (units > (1 << 30)) return TR_ERR_UNSUPPORTED;
  p.n_units = static_cast<int>(units);
  p.out = static_cast<__nv_bfloat16*>(a->out);
  p.ctx_len = a->d_ctx_len;
  p.anc = ctx->d_anc;
  p.flags = ctx->d_flags;
  p.queue = ctx->d_attn_queue;
  p.N = ctx->n_nodes;
  p.L = a->n_layers;
  p.os_b = a->o_stride[0]; p.os_h = a->o_stride[1]; p.os_t = a->o_stride[2]; p.os_l = a->layer_stride_o;
  const float scale = a->scale != 0.f ? a->scale : 1.0f / sqrtf(static_cast<float>(a->head_dim));
  p.scale_log2 = scale * 1.4426950408889634f;

  // Q is addressed as (dim, head, node, layer, sequence): a tile is 64 dims x G heads x 128/G nodes = 128 rows
  CUtensorMap mq, mk, mv;
  const uint64_t qd[5] = {HD, (uint64_t)a->n_q_heads, (uint64_t)ctx->n_nodes, (uint64_t)a->n_layers, (uint64_t)ctx->batch};
  const int64_t qs[4] = {a->q_stride[1], a->q_stride[2], a->layer_stride_q, a->q_stride[0]};
  const uint32_t qbox[5] = {64, (uint32_t)p.G, (uint32_t)(128 / p.G), 1, 1};
  const uint64_t kd[5] = {HD, (uint64_t)a->kv_rows, (uint64_t)a->n_kv_heads, (uint64_t)a->n_layers, (uint64_t)ctx->batch};
  const int64_t ks[4] = {a->kv_stride[2], a->kv_stride[1], a->layer_stride_kv, a->kv_stride[0]};
  const uint32_t kbox[5] = {64, BK, 1, 1, 1};
  if (!encode_map5(&mq, a->q, qd, qs, qbox) || !encode_map5(&mk, a->k_cache, kd, ks, kbox) ||
      !encode_map5(&mv, a->v_cache, kd, ks, kbox))
    return TR_ERR_UNSUPPORTED;
  const int grid = p.n_units < ctx->sm_count ? p.n_units : ctx->sm_count;
  tr_attn_pair_kernel<<<grid, NTHREADS, SMEM_BYTES, s>>>(mq, mk, mv, p);
  TR_CUDA_TRY(cudaGetLastError());
  return TR_OK;
}
