// Tree attention (paper Sec. 2.2) for head_dim 128 and 64 on the 5th-generation tensor cores: a persistent,
// warp-specialised flash-decoding kernel.
//
//   warps 0..3  epilogue: thread r normalises output row r out of TMEM and stores it, off the softmax warps' path
//   warp 8      TMA producer: Q tile (double-buffered, or single with one more ring slot: kQSingle) and a ring of
//               K / V tiles (128 keys x head_dim, bf16, 128-byte swizzle: 32 KB at head_dim 128, one 64-dim TMA box
//               per 16 KB), one mbarrier per ring slot
//   warp 9      MMA issuer 1: S = Q K^T (tcgen05.mma, both operands in shared memory, accumulator in TMEM); owns
//               the TMEM allocation
//   warp 10     MMA issuer 2: O += P V (P read from TMEM, V as an MN-major shared-memory operand)
//   warps 4..7  softmax: thread r owns query row r (= TMEM lane r): loads its S row, applies the ancestor mask
//               (a 128-bit mask kept in registers, shifted to the tile), exp2 with a lazily updated reference
//               maximum, writes P (bf16) over S in TMEM, rescales O in TMEM only when the maximum moved by
//               more than 2^8, and finally normalises and stores the output row
//
// A CTA walks units u = blockIdx.x, blockIdx.x + gridDim.x, ...; a unit is one (sequence, layer, KV head,
// query head, KV split).  TMEM: S/P double buffer (2 x 128 columns) + O double buffer (2 x 128 columns), so the
// QK^T of tile j+1 overlaps the softmax of tile j and the epilogue of a unit overlaps the next unit.
// Every wait is bounded; a wait that runs out sets TR_FLAG_WAIT_TIMEOUT and the CTA drains and exits.
#include "tc_ptx.cuh"
#include "tr_internal.cuh"

namespace {

constexpr int BK = 128;          // keys per tile
constexpr int HD_MAX = 128;      // head_dim is 128 or 64 (template argument kHD)
constexpr int NST_MAX = 6;       // ring slots (K and V tiles alternate): 5 beside a double-buffered Q tile, 6 beside a
                                 // single one (kQSingle: long units, where the Q reload between units is negligible)
constexpr int TILE_BYTES = BK * HD_MAX * 2;   // 32 KB: a tile at head_dim 128 (the shared-memory map is laid out for it)
constexpr int BOX_BYTES = BK * 64 * 2;        // one TMA box: 64 dims x 128 rows = 16 KB
constexpr int NTHREADS = 384;       // warps 0-3 epilogue, 4-7 softmax, 8 TMA producer, 9 QK issuer, 10 PV issuer, 11 idle
constexpr int WARP_PRODUCER = 8, WARP_MMA = 9, WARP_PV = 10;
// Registers are re-balanced per warpgroup after start-up (setmaxnreg): 12 warps are launched at 168 each.
constexpr int REGS_EPILOGUE = 112, REGS_SOFTMAX = 240, REGS_CONTROL = 96;

TR_STAMP_DECL(g_attn_stamps, 8)
TR_STAMP_DECL(g_attn_cta, 512)

struct TcParams {
  __nv_bfloat16* out;
  const int32_t* ctx_len;
  const uint32_t* anc;
  float* part_o;
  float* part_ml;
  uint32_t* flags;
  int N, L, S, n_units, HD;
  // Query rows are grouped per "head unit" hu: with grouped-query attention the G query heads that share a KV head
  // are packed into common 128-row tiles (row = node * G + head-in-group), MT tiles per head unit; when the group
  // size does not divide 128, every query head is its own head unit (G = 1) and kv_div maps it to its KV head.
  int HU, G, g_shift, MT, kv_div;
  int early_prefix;  // the producer may fetch prefix K/V tiles before it waits for the kernel in front (see tr.h)
  int live_warps;  // softmax warps that own at least one real row in every unit (4 unless tiles are unpacked and N <= 96)
  uint32_t div_MT[2], div_S[2], div_HU[2], div_L[2], div_kv[2];  // (multiplier, shift) for exact u32 division
  int64_t os_b, os_h, os_t, os_l;
  float scale_log2;
};

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int SM_Q = 0;                               // 2 x 32 KB
constexpr int SM_BAR = 7 * TILE_BYTES;                // Q tile(s) + ring = 7 x 32 KB, then the mbarriers
constexpr int BAR_FULL = 0, BAR_EMPTY = NST_MAX, BAR_QFULL = 2 * NST_MAX, BAR_QEMPTY = BAR_QFULL + 2,
              BAR_SFULL = BAR_QEMPTY + 2, BAR_PFULL = BAR_SFULL + 2, BAR_PVDONE = BAR_PFULL + 2,
              BAR_OFREE = BAR_PVDONE + 2, BAR_OREADY = BAR_OFREE + 2, BAR_LFULL = BAR_OREADY + 2,
              BAR_COUNT = BAR_LFULL + 2;
constexpr int SM_MISC = SM_BAR + BAR_COUNT * 8;       // tmem base (4 B), abort flag (4 B)
constexpr int SM_LM = SM_MISC + 16;                   // per O buffer: row sums l[128] and reference maxima m[128]
constexpr int SM_CTX = SM_LM + 2 * 2 * 128 * 4;        // cached context lengths
constexpr int SM_TOTAL = SM_CTX + 64 * 4;
constexpr int SMEM_BYTES = SM_TOTAL;                  // the tiles sit at the 1024-byte aligned start of the window
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB a CTA can opt in to");

struct Unit {
  int b, layer, kvh, h0, node0, split, slot;  // h0: first query head of the tile's rows; node0: its first tree node
  int t0, t1, C;
};

// u / d for 0 <= u < 2^31 with a host-computed (multiplier, shift): no hardware divide in the single-thread roles.
__device__ __forceinline__ uint32_t fast_div(uint32_t u, const uint32_t (&ms)[2]) {
  return static_cast<uint32_t>((static_cast<uint64_t>(u) * ms[0]) >> ms[1]);
}

constexpr int CTX_CACHE = 64;  // context lengths of the first 64 sequences are staged in shared memory

__device__ __forceinline__ Unit decode_unit(const TcParams& p, int u, const int* s_ctx) {
  Unit x;
  x.slot = u;
  uint32_t v = static_cast<uint32_t>(u), q;
  q = fast_div(v, p.div_MT); const uint32_t mt = v - q * p.MT; v = q;
  q = fast_div(v, p.div_S); x.split = static_cast<int>(v - q * p.S); v = q;
  q = fast_div(v, p.div_HU); const uint32_t hu = v - q * p.HU; v = q;
  q = fast_div(v, p.div_L); x.layer = static_cast<int>(v - q * p.L); v = q;
  x.b = static_cast<int>(v);
  x.h0 = static_cast<int>(hu) * p.G;
  x.node0 = static_cast<int>(mt) * (128 >> p.g_shift);
  x.kvh = static_cast<int>(fast_div(hu, p.div_kv));
  x.C = x.b < CTX_CACHE ? s_ctx[x.b] : p.ctx_len[x.b];
  const int T = (x.C + p.N + BK - 1) / BK;
  x.t0 = static_cast<int>(static_cast<int64_t>(T) * x.split / p.S);
  x.t1 = static_cast<int>(static_cast<int64_t>(T) * (x.split + 1) / p.S);
  return x;
}

// Walks this CTA's tiles in order: units blockIdx.x, blockIdx.x + gridDim.x, ... (empty units skipped), tiles
// t0..t1-1 inside each.  `ui` numbers the non-empty units, `g` the tiles, both from 0.
struct TileCursor {
  Unit x;
  int u, j, nt;
  uint32_t ui, g;
  bool valid;
  __device__ __forceinline__ void seek(const TcParams& p, const int* s_ctx) {
    while (u < p.n_units) {
      x = decode_unit(p, u, s_ctx);
      nt = x.t1 - x.t0;
      if (nt > 0) { j = 0; valid = true; return; }
      u += gridDim.x;
    }
    valid = false;
  }
  __device__ __forceinline__ void init(const TcParams& p, const int* s_ctx) {
    u = blockIdx.x; ui = 0; g = 0; j = 0; nt = 0;
    seek(p, s_ctx);
  }
  __device__ __forceinline__ void next(const TcParams& p, const int* s_ctx) {
    ++g;
    if (++j < nt) return;
    u += gridDim.x;
    ++ui;
    seek(p, s_ctx);
  }
};

// sm_100 packed / three-input float instructions: half the instruction count of the softmax's element-wise passes
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

template <int kHD, bool kQSingle, bool kPdl>
__global__ void __launch_bounds__(NTHREADS, 1)
tr_attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* base_ptr = smem_raw;
  if (base & 1023u) {  // swizzled tiles need a 1024-byte aligned window; not expected, but checked
    if (threadIdx.x == 0) atomicOr(p.flags, TR_FLAG_WAIT_TIMEOUT);
    return;
  }
  constexpr int NST = kQSingle ? 6 : 5;
  constexpr int TILE = BK * kHD * 2;   // bytes of one Q / K / V tile
  constexpr int NBOX = kHD / 64;       // 64-dim TMA boxes per tile
  constexpr int SM_RING = (kQSingle ? 1 : 2) * TILE_BYTES;
  const uint32_t bars = base + SM_BAR;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(base_ptr + SM_MISC);
  volatile uint32_t* s_abort = s_tmem + 1;
  auto bar = [&](int i) { return bars + static_cast<uint32_t>(i) * 8u; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef TR_STAMPS
  if (threadIdx.x == 0 && blockIdx.x == 0) g_attn_stamps[5] = g_attn_stamps[0];  // the previous launch's start
#endif
  TR_STAMP_MIN(g_attn_stamps, 0);
  TR_STAMP_MAX(g_attn_stamps, 1);
  int* s_ctx = reinterpret_cast<int*>(base_ptr + SM_CTX);
  auto stage_ctx_len = [&]() {
    const int nb = p.n_units / (p.L * p.HU * p.S * p.MT);  // sequences
    if (tid >= 64 && tid - 64 < CTX_CACHE && tid - 64 < nb) s_ctx[tid - 64] = p.ctx_len[tid - 64];
  };
  if (!kPdl) stage_ctx_len();

  // (the TMA producer's thread sets the barriers up, so that it can start copying before the CTA's first barrier)
  uint32_t c_early = 0;  // producer only: ring entries of the first unit issued before the dependency wait
  if (tid == WARP_PRODUCER * 32) {
    for (int i = 0; i < NST_MAX; ++i) { mbar_init(bar(BAR_FULL + i), 1); mbar_init(bar(BAR_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_QFULL + i), 1);
      mbar_init(bar(BAR_QEMPTY + i), 1);
      mbar_init(bar(BAR_SFULL + i), 1);
      mbar_init(bar(BAR_PFULL + i), 32u * static_cast<uint32_t>(p.live_warps));
      mbar_init(bar(BAR_PVDONE + i), 1);
      mbar_init(bar(BAR_OFREE + i), 128);
      mbar_init(bar(BAR_OREADY + i), 1);
      mbar_init(bar(BAR_LFULL + i), 32u * static_cast<uint32_t>(p.live_warps));
    }
    *s_abort = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (kPdl && p.early_prefix) {
      // The caller vouches that the prefix lengths and the prefix rows of the caches are not being written by
      // whatever still runs in front of this launch: the K/V tiles of this CTA's first unit that lie wholly inside
      // the prefix are requested now, under the tail of the kernel in front; Q and the tiles that reach into the
      // tree's rows follow after the wait.
      const int nb = p.n_units / (p.L * p.HU * p.S * p.MT);
      for (int i = 0; i < nb && i < CTX_CACHE; ++i) s_ctx[i] = __ldcg(p.ctx_len + i);
      const uint64_t pol = l2_policy_evict_first();
      int u = blockIdx.x;
      Unit x = decode_unit(p, u, s_ctx);
      while (x.t0 >= x.t1 && u + static_cast<int>(gridDim.x) < p.n_units) { u += gridDim.x; x = decode_unit(p, u, s_ctx); }
      if (x.t0 < x.t1) {
        const int t_end = min(x.t1, x.C / BK);  // tiles below hold prefix keys only
        for (int t = x.t0; t < t_end && c_early + 2u <= static_cast<uint32_t>(NST); ++t) {
#pragma unroll
          for (int kv = 0; kv < 2; ++kv) {
            const uint32_t slot = c_early % NST;
            const CUtensorMap* m = kv == 0 ? &map_k : &map_v;
            const uint32_t dst = base + SM_RING + slot * TILE_BYTES;
            mbar_expect_tx(bar(BAR_FULL + slot), TILE);
            tma_load_5d_hint(dst, m, bar(BAR_FULL + slot), 0, t * BK, x.kvh, x.layer, x.b, pol);
            if (NBOX == 2)
              tma_load_5d_hint(dst + BOX_BYTES, m, bar(BAR_FULL + slot), 64, t * BK, x.kvh, x.layer, x.b, pol);
            ++c_early;
          }
        }
      }
    }
  }
  if (warp == WARP_MMA) {  // TMEM: all 512 columns (one CTA per SM)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + SM_MISC), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (kPdl) {
    // launched with programmatic dependent launch (short launches only): everything above touches only this CTA's
    // shared memory and TMEM; the context lengths, Q/K/V and the partial buffers belong to whatever ran before
    tr_grid_dependency_wait();
    stage_ctx_len();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  TR_STAMP_MAX(g_attn_stamps, 2);
  float* s_lm = reinterpret_cast<float*>(base_ptr + SM_LM);  // [2 O buffers][l: 128 | m: 128]

  // Each warpgroup first re-sizes its register budget: the light roles hand registers to the softmax warps.
  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_CONTROL));
  if (warp == WARP_PRODUCER) {
    // =========================== TMA producer ===========================
    if (lane == 0) {
      uint32_t ui = 0, c = 0;  // non-empty units done by this CTA; ring entries issued
      bool ok = true;
      const uint64_t pol = l2_policy_evict_first();
      for (int u = blockIdx.x; u < p.n_units && ok; u += gridDim.x) {
        const Unit x = decode_unit(p, u, s_ctx);
        if (x.t0 >= x.t1) continue;
        const uint32_t qb = kQSingle ? 0u : (ui & 1u);
        ok = mbar_wait(bar(BAR_QEMPTY + qb), ((kQSingle ? ui : (ui >> 1)) & 1u) ^ 1u, s_abort);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_QFULL + qb), TILE);
        tma_load_5d(base + SM_Q + qb * TILE_BYTES, &map_q, bar(BAR_QFULL + qb), 0, x.h0, x.node0, x.layer, x.b);
        if (NBOX == 2)
          tma_load_5d(base + SM_Q + qb * TILE_BYTES + BOX_BYTES, &map_q, bar(BAR_QFULL + qb), 64, x.h0, x.node0, x.layer,
                      x.b);
        for (int t = x.t0; t < x.t1 && ok; ++t) {
#pragma unroll
          for (int kv = 0; kv < 2; ++kv) {
            if (c < c_early) { ++c; continue; }  // requested before the dependency wait
            const uint32_t slot = c % NST, par = ((c / NST) & 1u) ^ 1u;
            ok = mbar_wait(bar(BAR_EMPTY + slot), par, s_abort);
            if (!ok) break;
            const CUtensorMap* m = kv == 0 ? &map_k : &map_v;
            const uint32_t dst = base + SM_RING + slot * TILE_BYTES;
            mbar_expect_tx(bar(BAR_FULL + slot), TILE);
            tma_load_5d_hint(dst, m, bar(BAR_FULL + slot), 0, t * BK, x.kvh, x.layer, x.b, pol);
            if (NBOX == 2)
              tma_load_5d_hint(dst + BOX_BYTES, m, bar(BAR_FULL + slot), 64, t * BK, x.kvh, x.layer, x.b, pol);
            ++c;
          }
        }
        ++ui;
      }
    }
    __syncwarp();
  } else if (warp == WARP_MMA) {
    // =========================== MMA issuer 1: S = Q K^T ===========================
    // The two products are issued by two threads in different warps (this one and WARP_PV): an issue loop is one
    // thread's dependent instruction stream (waits, descriptor arithmetic, commits), and a single thread issuing
    // both left the tensor pipe waiting for it.  One flat stream of tiles over all of this CTA's units; tile g uses
    // S/P buffer g&1 and ring entries 2g (K) and 2g+1 (V).  This thread runs ahead of the PV issuer as far as the
    // S/P buffers and the ring allow - also across a unit boundary, so the first scores of the next unit are ready
    // when the softmax warps finish the current one.
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = make_idesc(false);
      bool ok = true;
      TileCursor kc;
      kc.init(p, s_ctx);
      while (ok && kc.valid) {
        const uint32_t sb = kc.g & 1u, c = 2u * kc.g, slot = c % NST, qb = kQSingle ? 0u : (kc.ui & 1u);
        if (kc.j == 0) {
          ok = mbar_wait(bar(BAR_QFULL + qb), (kQSingle ? kc.ui : (kc.ui >> 1)) & 1u, s_abort);
          if (!ok) break;
        }
        // the S/P buffer is free once the PV of tile g-2 has completed
        ok = mbar_wait(bar(BAR_PVDONE + sb), ((kc.g >> 1) & 1u) ^ 1u, s_abort);
        if (!ok) break;
        ok = mbar_wait(bar(BAR_FULL + slot), (c / NST) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
        // descriptors are stepped by adding to their low words, to keep the instruction stream short
        const uint32_t q_lo = smem_desc_lo(base + SM_Q + qb * TILE_BYTES, 16);
        const uint32_t k_lo = smem_desc_lo(base + SM_RING + slot * TILE_BYTES, 16);
        const uint32_t s_tm = tmem + sb * 128u;
#pragma unroll
        for (int k = 0; k < kHD / 16; ++k) {
          const uint32_t off16 = static_cast<uint32_t>(((k >> 2) * BOX_BYTES + (k & 3) * 32) >> 4);
          tc_mma_ss_lh(s_tm, q_lo + off16, k_lo + off16, smem_desc_hi(1024), IDESC_QK, k > 0);
        }
        tc_commit(bar(BAR_EMPTY + slot));                          // K tile consumed
        tc_commit(bar(BAR_SFULL + sb));                            // S ready for the softmax warps
        if (kc.j == kc.nt - 1) tc_commit(bar(BAR_QEMPTY + qb));    // unit's last QK: Q buffer free when it finishes
        kc.next(p, s_ctx);
      }
    }
    __syncwarp();
  } else if (warp == WARP_PV) {
    // =========================== MMA issuer 2: O += P V ===========================
    if (lane == 0) {
      constexpr uint32_t IDESC_PV = make_idesc(true, kHD);  // N = head_dim
      bool ok = true;
      TileCursor vc;
      vc.init(p, s_ctx);
      while (ok && vc.valid) {
        const uint32_t sb = vc.g & 1u, ob = vc.ui & 1u, c = 2u * vc.g + 1u, vslot = c % NST;
        if (vc.j == 0) {  // the O buffer must have been drained by the epilogue of unit ui-2
          ok = mbar_wait(bar(BAR_OFREE + ob), ((vc.ui >> 1) & 1u) ^ 1u, s_abort);
          if (!ok) break;
        }
        ok = mbar_wait(bar(BAR_FULL + vslot), (c / NST) & 1u, s_abort);
        if (!ok) break;
        ok = mbar_wait(bar(BAR_PFULL + sb), (vc.g >> 1) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
        const uint32_t v_lo = smem_desc_lo(base + SM_RING + vslot * TILE_BYTES, BOX_BYTES);
        const uint32_t o_tm = tmem + 256u + ob * 128u, p_tm = tmem + sb * 128u;
        const uint32_t acc0 = vc.j > 0 ? 1u : 0u;
#pragma unroll
        for (int k = 0; k < BK / 16; ++k) {
          // A = P (bf16 pairs, 8 TMEM columns per 16 keys); B = V tile, MN-major: 64-dim boxes 16 KB apart,
          // 8-key groups 1 KB apart, 16 keys per step = 2 KB
          tc_mma_ts_lh(o_tm, p_tm + k * 8u, v_lo + k * (2048u >> 4), smem_desc_hi(1024), IDESC_PV, k > 0 ? 1u : acc0);
        }
        tc_commit(bar(BAR_EMPTY + vslot));                             // V tile consumed
        tc_commit(bar(BAR_PVDONE + sb));                               // P consumed, O updated
        if (vc.j == vc.nt - 1) tc_commit(bar(BAR_OREADY + ob));        // the unit's output is complete
        vc.next(p, s_ctx);
      }
    }
    __syncwarp();
  }
  } else if (warp >= 4) {
    // =========================== softmax / correction ===========================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
    const int r = (warp & 3) * 32 + lane;                 // query row == TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    uint32_t anc[4];
    uint32_t ui = 0, g = 0;
    // A warp whose 32 rows lie past the tree's last node in every unit (80 nodes leave rows 96..127 of an unpacked tile
    // empty) is not counted by the barriers of this role and goes straight to the teardown: its scores, exponentials
    // and P rows would never be used.
    bool ok = (warp & 3) < p.live_warps;
    for (int u = blockIdx.x; u < p.n_units && ok; u += gridDim.x) {
      const Unit x = decode_unit(p, u, s_ctx);
      const int nt = x.t1 - x.t0;
      {  // this row's tree node (rows of a packed tile are node-major) and its ancestor mask
        const int node = x.node0 + (r >> p.g_shift);
#pragma unroll
        for (int w = 0; w < 4; ++w) anc[w] = (nt > 0 && node < p.N) ? p.anc[node * 4 + w] : 0u;
      }
      float m_ref = -INFINITY, l = 0.f;
      const uint32_t ob = ui & 1u;
      for (int j = 0; j < nt && ok; ++j, ++g) {
        const uint32_t sb = g & 1u;
        ok = mbar_wait<0>(bar(BAR_SFULL + sb), (g >> 1) & 1u, s_abort);
        ok = __all_sync(0xFFFFFFFFu, ok);  // the TMEM loads below are warp-collective
        if (!ok) break;
        tc_fence_after();
        uint32_t sreg[4][32];
#pragma unroll
        for (int q = 0; q < 4; ++q) tc_ld32(tmem + lane_base + sb * 128u + q * 32u, sreg[q]);
        tc_wait_ld();
        // visibility of the tile's 128 keys for this row
        const int key0 = (x.t0 + j) * BK;
        uint32_t vis[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
        const bool masked = key0 + BK > x.C;
        if (masked) {
          const int s = x.C - key0;  // tile column of the first tree key (may be <= 0 or >= 128)
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            // bit c of word w: column 32w + c; visible iff column < s, or bit (column - s) of anc
            uint32_t word = 0;
            const int col0 = 32 * w;
            const int sh = col0 - s;  // tree index of column col0
            // prefix part
            if (s >= col0 + 32) word = 0xFFFFFFFFu;
            else if (s > col0) word = (1u << (s - col0)) - 1u;
            // tree part: bits of the 128-bit anc starting at tree index sh
            uint32_t tw = 0;
            if (sh >= 0) {
              const int wi = sh >> 5, bi = sh & 31;
              const uint32_t lo = wi < 4 ? (wi == 0 ? anc[0] : wi == 1 ? anc[1] : wi == 2 ? anc[2] : anc[3]) : 0u;
              const uint32_t hi = wi + 1 < 4 ? (wi == 0 ? anc[1] : wi == 1 ? anc[2] : anc[3]) : 0u;
              tw = bi ? ((lo >> bi) | (hi << (32 - bi))) : lo;
            } else if (sh > -32) {
              tw = anc[0] << (-sh);
            }
            vis[w] = word | tw;
          }
        }
        if (masked) {  // only the one or two tiles that reach into the tree's keys
#pragma unroll
          for (int q = 0; q < 4; ++q)
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (!((vis[q] >> c) & 1u)) sreg[q][c] = 0xFF800000u;  // -inf
        }
        // row maximum of the raw scores: eight independent chains (scale > 0, applied afterwards)
        float mx[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) mx[i] = -INFINITY;
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int c = 0; c < 32; c += 2)  // three-input max: two scores per instruction
            mx[(c >> 1) & 7] = max3(mx[(c >> 1) & 7], __uint_as_float(sreg[q][c]), __uint_as_float(sreg[q][c + 1]));
        const float tmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                 fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7]))) * p.scale_log2;
        // lazy rescale: keep the old reference unless the maximum grew by more than 2^8
        float alpha = 1.f;
        if (tmax > m_ref + 8.f) {
          alpha = (m_ref == -INFINITY) ? 0.f : fast_exp2(m_ref - tmax);
          m_ref = tmax;
        }
        const bool need = (alpha != 1.f) && (j > 0);
        if (__any_sync(0xFFFFFFFFu, need)) {
          // O of this unit holds tiles < j; PV(j-1) must have landed before it is rescaled
          const uint32_t pb = (g - 1u) & 1u;
          ok = mbar_wait<0>(bar(BAR_PVDONE + pb), ((g - 1u) >> 1) & 1u, s_abort);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int q = 0; q < kHD / 32; ++q) {
            uint32_t oreg[32];
            tc_ld32(tmem + lane_base + 256u + ob * 128u + q * 32u, oreg);
            tc_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) oreg[c] = __float_as_uint(__uint_as_float(oreg[c]) * alpha);
            tc_st32(tmem + lane_base + 256u + ob * 128u + q * 32u, oreg);
          }
        }
        l *= alpha;
        const float nsub = (m_ref == -INFINITY) ? 0.f : -m_ref;
        const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), nsub2 = pack2(nsub, nsub);
        uint64_t sm2[4] = {0ull, 0ull, 0ull, 0ull};  // packed (even, odd) partial row sums
        uint32_t preg[2][32];
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            float x0, x1;
            unpack2(fma2(pack2(__uint_as_float(sreg[q][c]), __uint_as_float(sreg[q][c + 1])), scale2, nsub2), x0, x1);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
            sm2[(c >> 1) & 3] = add2(sm2[(c >> 1) & 3], pack2(p0, p1));
            __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
            preg[q >> 1][(q & 1) * 16 + (c >> 1)] = *reinterpret_cast<uint32_t*>(&pk);
          }
        float se, so;
        unpack2(add2(add2(sm2[0], sm2[1]), add2(sm2[2], sm2[3])), se, so);
        const float sum = se + so;
        l += sum;
        tc_st32(tmem + lane_base + sb * 128u, preg[0]);
        tc_st32(tmem + lane_base + sb * 128u + 32u, preg[1]);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar(BAR_PFULL + sb));
      }
      if (!ok) break;
      if (nt <= 0) continue;  // empty split: the epilogue warps write its (empty) partial
      // ---- hand the unit to the epilogue warps: row sum and reference maximum go through shared memory.  The
      //      slot was last read by the epilogue of unit ui-2, which signalled OFREE when it was done with it.
      ok = mbar_wait<0>(bar(BAR_OFREE + ob), ((ui >> 1) & 1u) ^ 1u, s_abort);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      s_lm[ob * 256 + r] = l;
      s_lm[ob * 256 + 128 + r] = m_ref;
      mbar_arrive(bar(BAR_LFULL + ob));
      ++ui;
    }
  } else {
    // =========================== epilogue ===========================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_EPILOGUE));
    // Thread r owns output row r: waits until the unit's last PV has landed (OREADY) and the softmax warps have
    // published the row sums (LFULL), then normalises O out of TMEM and stores it (bf16 rows, or the fp32
    // partial of a KV split), so the softmax warps never stop at a unit boundary.
    const int r = warp * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    uint32_t ui = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < p.n_units && ok; u += gridDim.x) {
      const Unit x = decode_unit(p, u, s_ctx);
      const int nt = x.t1 - x.t0;
      const int node = x.node0 + (r >> p.g_shift);      // rows of a packed tile are node-major ...
      const int head = x.h0 + (r & (p.G - 1));          // ... with the group's query heads interleaved
      const bool row_ok = node < p.N;
      float* po = p.part_o + (static_cast<size_t>(x.slot) * ATTN_PART_ROWS + r) * 128;
      float* pml = p.part_ml + (static_cast<size_t>(x.slot) * ATTN_PART_ROWS + r) * 2;
      if (nt <= 0) {  // empty split: contributes nothing
        if (p.S > 1 && row_ok) {
          pml[0] = -INFINITY;
          pml[1] = 0.f;
        }
        continue;
      }
      const uint32_t ob = ui & 1u, par = (ui >> 1) & 1u;
      ok = mbar_wait<0>(bar(BAR_LFULL + ob), par, s_abort) && mbar_wait<0>(bar(BAR_OREADY + ob), par, s_abort);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const float l = s_lm[ob * 256 + r], m_ref = s_lm[ob * 256 + 128 + r];
      const float inv = 1.f / l;
      __nv_bfloat16* orow = p.out + x.b * p.os_b + x.layer * p.os_l + head * p.os_h + static_cast<int64_t>(node) * p.os_t;
#pragma unroll
      for (int q = 0; q < kHD / 32; ++q) {
        uint32_t oreg[32];
        tc_ld32(tmem + lane_base + 256u + ob * 128u + q * 32u, oreg);
        tc_wait_ld();
        if (q == kHD / 32 - 1) {  // O (and l, m) are in registers: hand the buffer back to the MMA and softmax warps
          tc_fence_before();
          mbar_arrive(bar(BAR_OFREE + ob));
        }
        if (row_ok) {
          if (p.S == 1) {
#pragma unroll
            for (int c = 0; c < 32; c += 8) {
              uint4 w;
              __nv_bfloat162 t0 = __floats2bfloat162_rn(__uint_as_float(oreg[c + 0]) * inv, __uint_as_float(oreg[c + 1]) * inv);
              __nv_bfloat162 t1 = __floats2bfloat162_rn(__uint_as_float(oreg[c + 2]) * inv, __uint_as_float(oreg[c + 3]) * inv);
              __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(oreg[c + 4]) * inv, __uint_as_float(oreg[c + 5]) * inv);
              __nv_bfloat162 t3 = __floats2bfloat162_rn(__uint_as_float(oreg[c + 6]) * inv, __uint_as_float(oreg[c + 7]) * inv);
              w.x = *reinterpret_cast<uint32_t*>(&t0); w.y = *reinterpret_cast<uint32_t*>(&t1);
              w.z = *reinterpret_cast<uint32_t*>(&t2); w.w = *reinterpret_cast<uint32_t*>(&t3);
              *reinterpret_cast<uint4*>(orow + q * 32 + c) = w;
            }
          } else {
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              *reinterpret_cast<float4*>(po + q * 32 + c) =
                  make_float4(__uint_as_float(oreg[c]), __uint_as_float(oreg[c + 1]), __uint_as_float(oreg[c + 2]),
                              __uint_as_float(oreg[c + 3]));
          }
        }
      }
      if (p.S > 1 && row_ok) {
        pml[0] = m_ref;
        pml[1] = l;
      }
      ++ui;
    }
  }

  // ---- teardown: every thread arrives here, also after an aborted wait
  __syncthreads();
  TR_STAMP_MIN(g_attn_stamps, 3);
  TR_STAMP_MAX(g_attn_stamps, 4);
#ifdef TR_STAMPS
  if (threadIdx.x == 0 && blockIdx.x < 256) {
    unsigned smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    g_attn_cta[blockIdx.x] = tr_globaltimer();
    g_attn_cta[256 + blockIdx.x] = smid;
  }
#endif
  if (*s_abort) {
    if (tid == 0) atomicOr(p.flags, TR_FLAG_WAIT_TIMEOUT);
    // give copies and MMAs that may still be in flight time to land before shared memory and TMEM are released
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == WARP_MMA) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------
// 5-D bf16 tensor map with 128-byte swizzle; out-of-bounds elements read as zero.  dims[0] is head_dim (contiguous);
// strides (elements) belong to dims[1..4]; a stride of a size-1 dimension may be anything.
bool encode_map(CUtensorMap* m, const void* ptr, const uint64_t (&dims)[5], const int64_t (&strides)[4],
                const uint32_t (&box)[5]) {
  const int64_t HD = static_cast<int64_t>(dims[0]);
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

// Merge of the per-split partials written by tr_attn_tc_kernel: out = sum_s 2^(m_s - m*) O_s / sum_s 2^(m_s - m*) l_s.
// One CTA per (8 tile rows, tile); 32 lanes x float4 cover the 128 dims of a row.  Slots are numbered like the
// units: (((b, layer, head unit), split), tile).
__global__ void __launch_bounds__(256) tr_attn_tc_combine_kernel(const TcParams p) {
  tr_grid_dependency_wait();  // launched with programmatic dependent launch: the partials come from the kernel before
  // the kernel behind this one may be scheduled now (it waits for this grid before it reads what is written here);
  // a following attention launch uses the time to set itself up and, if allowed, to request prefix K/V
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5);  // row of the tile
  const int d = (threadIdx.x & 31) * 4;
  if (d >= p.HD) return;                              // head_dim 64: half the lanes have no column
  const uint32_t t = blockIdx.y;                        // (b, layer, head unit, tile)
  const uint32_t blh = t / p.MT, mt = t - blh * p.MT;
  const uint32_t bl = blh / p.HU, hu = blh - bl * p.HU;
  const uint32_t b = bl / p.L, layer = bl - b * p.L;
  const int node = static_cast<int>(mt) * (128 >> p.g_shift) + (r >> p.g_shift);
  const int head = static_cast<int>(hu) * p.G + (r & (p.G - 1));
  if (node >= p.N) return;
  float mstar = -INFINITY;
  for (int s = 0; s < p.S; ++s) {
    const size_t slot = (static_cast<size_t>(blh) * p.S + s) * p.MT + mt;
    mstar = fmaxf(mstar, p.part_ml[(slot * ATTN_PART_ROWS + r) * 2]);
  }
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float den = 0.f;
  for (int s = 0; s < p.S; ++s) {
    const size_t slot = (static_cast<size_t>(blh) * p.S + s) * p.MT + mt;
    const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + (slot * ATTN_PART_ROWS + r) * 2);
    const float w = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - mstar);
    const float4 o = *reinterpret_cast<const float4*>(p.part_o + (slot * ATTN_PART_ROWS + r) * 128 + d);
    acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
    den += w * ml.y;
  }
  const float inv = 1.f / den;
  __nv_bfloat16* op = p.out + b * p.os_b + layer * p.os_l + head * p.os_h + static_cast<int64_t>(node) * p.os_t + d;
  __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
  uint2 w2;
  w2.x = *reinterpret_cast<uint32_t*>(&lo);
  w2.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(op) = w2;
}

}  // namespace

#ifdef TR_STAMPS
extern "C" int tr_debug_stamps_attn_cta(unsigned long long* host) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(host, g_attn_cta, sizeof(unsigned long long) * 512);
  return 0;
}
extern "C" int tr_debug_stamps_attn(unsigned long long* host, int reset) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(host, g_attn_stamps, sizeof(unsigned long long) * 8);
  if (reset) {
    unsigned long long init[8] = {~0ull, 0, 0, ~0ull, 0, 0, 0, 0};
    cudaMemcpyToSymbol(g_attn_stamps, init, sizeof(init));
  }
  return 0;
}
#endif

tr_status tr_attention_tc_setup() {
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_tc_kernel<128, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_tc_kernel<128, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_tc_kernel<128, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_tc_kernel<64, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_tc_kernel<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_tc_kernel<64, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
  return get_encode_fn() ? TR_OK : TR_ERR_CUDA;
}

// Number of KV splits of a launch with `base_units` units before splitting: one unit per SM at most when there are
// fewer units than SMs (a->splits > 0 forces a count; never more than there are key tiles or partial slots).
int tr_attention_pick_splits(const tr_ctx* ctx, const tr_attn_args* a, int base_units, int tile_keys) {
  const int tiles = (a->max_ctx + ctx->n_nodes + tile_keys - 1) / tile_keys;
  int S = a->splits;
  if (S <= 0) {
    S = base_units >= ctx->sm_count ? 1 : ctx->sm_count / base_units;
    if (S > 16) S = 16;
  }
  if (S > tiles) S = tiles;
  while (S > 1 && static_cast<int64_t>(base_units) * S > ATTN_MAX_PART_SLOTS) --S;
  return S < 1 ? 1 : S;
}

// (M, k) with floor(u / d) == (u * M) >> k for all 0 <= u < 2^31: k = 31 + ceil(log2 d), M = ceil(2^k / d) < 2^32.
static void magic_u32(uint32_t d, uint32_t (&ms)[2]) {
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;
  const uint32_t k = 31 + l;
  ms[0] = static_cast<uint32_t>(((1ull << k) + d - 1) / d);
  ms[1] = k;
}

tr_status tr_launch_attention_tc(tr_ctx* ctx, const tr_attn_args* a, cudaStream_t s) {
  if (a->head_dim != 128 && a->head_dim != 64) return TR_ERR_UNSUPPORTED;
  const uint64_t HD = static_cast<uint64_t>(a->head_dim);
  // grouped-query attention: pack the group's heads into common row tiles when the group size divides 128
  const int group = a->n_q_heads / a->n_kv_heads;
  const bool packed = group > 1 && (128 % group) == 0;
  TcParams p;
  p.G = packed ? group : 1;
  p.g_shift = 0;
  while ((1 << p.g_shift) < p.G) ++p.g_shift;
  p.HU = packed ? a->n_kv_heads : a->n_q_heads;
  p.kv_div = packed ? 1 : group;
  p.MT = (ctx->n_nodes * p.G + 127) / 128;
  p.early_prefix = a->prefix_stable ? 1 : 0;
  p.live_warps = (p.MT == 1 && p.G == 1) ? (ctx->n_nodes + 31) / 32 : 4;
  const int64_t base = static_cast<int64_t>(ctx->batch) * a->n_layers * p.HU * p.MT;
  if (base > (1 << 30)) return TR_ERR_UNSUPPORTED;
  p.out = static_cast<__nv_bfloat16*>(a->out);
  p.ctx_len = a->d_ctx_len;
  p.anc = ctx->d_anc;
  p.part_o = ctx->d_attn_part_o;
  p.part_ml = ctx->d_attn_part_ml;
  p.flags = ctx->d_flags;
  p.N = ctx->n_nodes; p.L = a->n_layers; p.HD = a->head_dim;
  p.os_b = a->o_stride[0]; p.os_h = a->o_stride[1]; p.os_t = a->o_stride[2]; p.os_l = a->layer_stride_o;
  const float scale = a->scale != 0.f ? a->scale : 1.0f / sqrtf(static_cast<float>(a->head_dim));
  p.scale_log2 = scale * 1.4426950408889634f;
  p.S = tr_attention_pick_splits(ctx, a, static_cast<int>(base), BK);
  if (p.S > 1 && base * p.S > ATTN_MAX_PART_SLOTS) return TR_ERR_UNSUPPORTED;
  // grouped-query shapes with at least two row tiles per KV head and enough work without splitting the keys: two
  // tiles per CTA on one K/V stream
  if (p.S == 1 && tr_attention_pair_applies(ctx, a)) return tr_launch_attention_pair(ctx, a, s);
  p.n_units = static_cast<int>(base * p.S);
  magic_u32(static_cast<uint32_t>(p.MT), p.div_MT);
  magic_u32(static_cast<uint32_t>(p.S), p.div_S);
  magic_u32(static_cast<uint32_t>(p.HU), p.div_HU);
  magic_u32(static_cast<uint32_t>(p.L), p.div_L);
  magic_u32(static_cast<uint32_t>(p.kv_div), p.div_kv);

  // Q is addressed as (dim, head, node, layer, sequence): in the usual [.., node, head, dim] layout the head
  // stride is the smaller one, and the tile (64 dims x 1 head x 128 nodes) lands in shared memory as 128 rows.
  CUtensorMap mq, mk, mv;
  const uint64_t qd[5] = {HD, (uint64_t)a->n_q_heads, (uint64_t)ctx->n_nodes, (uint64_t)a->n_layers, (uint64_t)ctx->batch};
  const int64_t qs[4] = {a->q_stride[1], a->q_stride[2], a->layer_stride_q, a->q_stride[0]};
  const uint32_t qbox[5] = {64, (uint32_t)p.G, (uint32_t)(128 / p.G), 1, 1};  // G heads x 128/G nodes = 128 rows
  const uint64_t kd[5] = {HD, (uint64_t)a->kv_rows, (uint64_t)a->n_kv_heads, (uint64_t)a->n_layers, (uint64_t)ctx->batch};
  const int64_t ks[4] = {a->kv_stride[2], a->kv_stride[1], a->layer_stride_kv, a->kv_stride[0]};
  const uint32_t kbox[5] = {64, BK, 1, 1, 1};
  if (!encode_map(&mq, a->q, qd, qs, qbox) || !encode_map(&mk, a->k_cache, kd, ks, kbox) ||
      !encode_map(&mv, a->v_cache, kd, ks, kbox))
    return TR_ERR_UNSUPPORTED;
  const int grid = p.n_units < ctx->sm_count ? p.n_units : ctx->sm_count;
  // Grouped-query shapes (several row tiles per KV head, long units, K/V re-read from L2): one Q buffer and a sixth
  // ring slot; otherwise Q is double-buffered so that short units overlap their Q load.
  // A short launch (fewer units than SMs, split along the keys) between other short kernels, typically one layer's
  // attention, uses programmatic dependent launch: it hides the launch latency (503 -> 475 us for 32 per-layer launches
  // at the 7B shape).  Long launches gain nothing from it and measured about 1.5 % slower.
  if (a->head_dim == 128) {
    if (p.MT > 1)
      tr_attn_tc_kernel<128, true, false><<<grid, NTHREADS, SMEM_BYTES, s>>>(mq, mk, mv, p);
    else if (p.S > 1)
      TR_CUDA_TRY(tr_launch_pdl(tr_attn_tc_kernel<128, false, true>, dim3(grid), dim3(NTHREADS), SMEM_BYTES, s, mq, mk, mv, p));
    else
      tr_attn_tc_kernel<128, false, false><<<grid, NTHREADS, SMEM_BYTES, s>>>(mq, mk, mv, p);
  } else {
    if (p.MT > 1)
      tr_attn_tc_kernel<64, true, false><<<grid, NTHREADS, SMEM_BYTES, s>>>(mq, mk, mv, p);
    else if (p.S > 1)
      TR_CUDA_TRY(tr_launch_pdl(tr_attn_tc_kernel<64, false, true>, dim3(grid), dim3(NTHREADS), SMEM_BYTES, s, mq, mk, mv, p));
    else
      tr_attn_tc_kernel<64, false, false><<<grid, NTHREADS, SMEM_BYTES, s>>>(mq, mk, mv, p);
  }
  TR_CUDA_TRY(cudaGetLastError());
  if (p.S > 1)
    TR_CUDA_TRY(tr_launch_pdl(tr_attn_tc_combine_kernel, dim3(16, static_cast<unsigned>(base)), dim3(256), 0, s, p));
  return TR_OK;
}
