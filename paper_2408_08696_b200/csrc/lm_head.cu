// Output layer fused with argtopk (paper Sec. 2.1: p = M(x), x^0..x^{k-1} = argtopk(p)): the last linear layer of the
// model, logits[r, v] = sum_h hidden[r, h] * weight[v, h], evaluated on the 5th-generation tensor cores with the
// per-row top-k taken directly from the accumulators, so the [rows, V] logits are never written to memory.
//
// The op is bound by the one pass over the weight matrix.  Each CTA owns a contiguous slice of the vocabulary and
// streams it exactly once: TMA brings 64-wide hidden slabs of the weight slice (up to 256 vocabulary rows, the MMA's N)
// and of the hidden states (128 rows, the MMA's M; rows past the real ones read as zero, re-read from L2) into a ring
// of stages, tcgen05.mma accumulates the [128, <=256] fp32 logits tile in TMEM, and the epilogue warps - two threads
// per row, on alternate 32-column blocks - scan the accumulator columns in ascending vocabulary order, each keeping a
// sorted top list in registers.  A slice wider than 256 is cut into chunks with two accumulators in TMEM, so the
// epilogue of one chunk runs under the main loop of the next.  Each (CTA, column half) writes its k best (value, index)
// keys per row; a small second kernel merges the lists.
//
//   warp 0      TMA producer
//   warp 1      MMA issuer, owns the TMEM allocation
//   warps 2..9  epilogue (TMEM lane quarter = warp & 3; warps 2..5 take the even 32-column blocks, 6..9 the odd ones)
//
// Order: value descending, equal values by lower index - the 64-bit key of the top-k kernel, so the merge is exact.
// Every wait is bounded; a wait that runs out sets TR_FLAG_WAIT_TIMEOUT and the CTA drains and exits.
#include "tc_ptx.cuh"
#include "tr_internal.cuh"

typedef unsigned long long u64;

namespace {

constexpr int LM_BK = 64;                       // hidden elements per stage: one 128-byte swizzle row
constexpr int LM_MAX_STAGES = 8;
constexpr int LM_A_BYTES = 128 * LM_BK * 2;     // 16 KB: 128 query rows
constexpr int LM_RING_BYTES = 224 * 1024;       // stages of LM_A_BYTES + NC * 128 bytes each
constexpr int LM_THREADS = 320;
constexpr int LM_MAX_NC = 256;                  // widest chunk = the MMA's largest N (narrower chunks hide more
                                                // epilogues but re-read the hidden states more often: measured slower)
constexpr int LM_SM_BAR = LM_RING_BYTES;
constexpr int LM_BAR_FULL = 0, LM_BAR_EMPTY = LM_MAX_STAGES, LM_BAR_ACC_FULL = 2 * LM_MAX_STAGES,
              LM_BAR_ACC_EMPTY = LM_BAR_ACC_FULL + 2, LM_BAR_COUNT = LM_BAR_ACC_EMPTY + 2;
constexpr int LM_SM_MISC = LM_SM_BAR + LM_BAR_COUNT * 8;  // tmem base, abort flag
constexpr int LM_SMEM_BYTES = LM_SM_MISC + 16;
static_assert(LM_SMEM_BYTES <= 232448, "exceeds the 227 KB a CTA can opt in to");
constexpr int LM_MERGE_THREADS = 256;
constexpr int LM_MERGE_CAND = 256;

struct LmParams {
  u64* part;        // [rows][parts][k], parts = 2 * vocabulary slices
  uint32_t* flags;
  int R;            // rows in all (groups of 128: CTA = (vocabulary slice, row group), the groups of a slice adjacent)
  int groups;       // row groups
  int V, H;         // vocabulary size, hidden size
  int cols_per_cta; // vocabulary slice of one CTA
  int NC;           // width of a chunk = the MMA's N (a multiple of 16, <= 256)
  int n_main;       // chunks per full slice
  int nstage;       // ring stages in use
  int k, parts;
};

__device__ __forceinline__ u64 lm_key(float v, uint32_t idx) {
  uint32_t b = __float_as_uint(v);
  if (b == 0x80000000u) b = 0u;  // -0 and +0 compare equal: the index decides
  const uint32_t s = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return (static_cast<u64>(s) << 32) | static_cast<u64>(0xFFFFFFFFu - idx);
}
__device__ __forceinline__ float lm_key_value(u64 key) {
  const uint32_t s = static_cast<uint32_t>(key >> 32);
  return __uint_as_float((s & 0x80000000u) ? (s & 0x7FFFFFFFu) : ~s);
}

template <int KMAX>
__global__ void __launch_bounds__(LM_THREADS, 1)
tr_lm_head_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const LmParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {  // swizzled tiles need a 1024-byte aligned window; not expected, but checked
    if (threadIdx.x == 0) atomicOr(p.flags, TR_FLAG_WAIT_TIMEOUT);
    return;
  }
  const uint32_t bars = base + LM_SM_BAR;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem_raw + LM_SM_MISC);
  volatile uint32_t* s_abort = s_tmem + 1;
  auto bar = [&](int i) { return bars + static_cast<uint32_t>(i) * 8u; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // this CTA's slice, row group and chunks: chunk c starts at v_begin + c * NC.  The CTAs of one slice (one per row
  // group) have neighbouring indices, run at the same time and stream the same weight rows: the first to ask brings
  // them in from HBM, the others find them in L2.
  const int slice = blockIdx.x / p.groups, row0 = (blockIdx.x - slice * p.groups) * 128;
  const int v_begin = slice * p.cols_per_cta;
  const int v_end = min(p.V, v_begin + p.cols_per_cta);
  int n_chunks = 0;
  for (int c = 0; c < p.n_main; ++c) n_chunks += (v_begin + c * p.NC < v_end) ? 1 : 0;
  const int ksteps = (p.H + LM_BK - 1) / LM_BK;
  const uint32_t stage_bytes = LM_A_BYTES + static_cast<uint32_t>(p.NC) * LM_BK * 2;  // a multiple of 1024
  const uint32_t nstage = static_cast<uint32_t>(p.nstage);

  if (tid == 0) {
    for (int i = 0; i < LM_MAX_STAGES; ++i) { mbar_init(bar(LM_BAR_FULL + i), 1); mbar_init(bar(LM_BAR_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar(LM_BAR_ACC_FULL + i), 1); mbar_init(bar(LM_BAR_ACC_EMPTY + i), 256); }
    *s_abort = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {  // TMEM: all 512 columns (one CTA per SM): two accumulators of up to 256 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + LM_SM_MISC), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  // (programmatic dependent launch) the hidden states belong to whatever ran before on this stream
  tr_grid_dependency_wait();

  if (warp == 0) {
    // =========================== TMA producer ===========================
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_first();  // the weight is read once; the hidden states stay in L2
      const int k_shift = static_cast<int>((static_cast<uint32_t>(slice) * 11u) % static_cast<uint32_t>(ksteps));
      uint32_t it = 0;
      bool ok = true;
      for (int c = 0; c < n_chunks && ok; ++c) {
        const int v0 = v_begin + c * p.NC;
        for (int ks = 0; ks < ksteps; ++ks, ++it) {
          const uint32_t s = it % nstage;
          ok = mbar_wait(bar(LM_BAR_EMPTY + s), ((it / nstage) & 1u) ^ 1u, s_abort);
          if (!ok) break;
          const uint32_t dst = base + s * stage_bytes;
          mbar_expect_tx(bar(LM_BAR_FULL + s), stage_bytes);
          // every CTA starts its walk over the hidden dimension at a different slab (the sum does not care), so
          // that the CTAs, whose slices are a fixed large stride apart, do not march through DRAM in lockstep
          int kq = ks + k_shift;
          kq = kq >= ksteps ? kq - ksteps : kq;
          if (p.groups == 1) tma_load_2d_hint(dst + LM_A_BYTES, &map_b, bar(LM_BAR_FULL + s), kq * LM_BK, v0, pol);
          else tma_load_2d(dst + LM_A_BYTES, &map_b, bar(LM_BAR_FULL + s), kq * LM_BK, v0);  // shared through L2
          tma_load_2d(dst, &map_a, bar(LM_BAR_FULL + s), kq * LM_BK, row0);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      const uint32_t idesc = make_idesc(false, static_cast<uint32_t>(p.NC));
      uint32_t it = 0;
      bool ok = true;
      for (int c = 0; c < n_chunks && ok; ++c) {
        const uint32_t buf = c & 1u;
        // the accumulator must have been drained by the epilogue of chunk c-2
        ok = mbar_wait(bar(LM_BAR_ACC_EMPTY + buf), ((c >> 1) & 1u) ^ 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
        for (int ks = 0; ks < ksteps; ++ks, ++it) {
          const uint32_t s = it % nstage;
          ok = mbar_wait(bar(LM_BAR_FULL + s), (it / nstage) & 1u, s_abort);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a = base + s * stage_bytes, b = a + LM_A_BYTES;
#pragma unroll
          for (int kk = 0; kk < LM_BK / 16; ++kk)  // both operands K-major, 128-byte swizzle: 32 bytes per K step
            tc_mma_ss(tmem + buf * 256u, smem_desc(a + kk * 32, 16, 1024), smem_desc(b + kk * 32, 16, 1024), idesc,
                      (ks > 0 || kk > 0) ? 1u : 0u);
          tc_commit(bar(LM_BAR_EMPTY + s));  // stage consumed
        }
        if (ok) tc_commit(bar(LM_BAR_ACC_FULL + buf));  // the chunk's logits are complete
      }
    }
    __syncwarp();
  } else {
    // =========================== epilogue: running top list per (row, column half) ===========================
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    const int r = q * 32 + lane;  // query row == TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
    float val[KMAX];
    int idx[KMAX];
#pragma unroll
    for (int i = 0; i < KMAX; ++i) { val[i] = -INFINITY; idx[i] = -1; }
    bool ok = true;
    for (int c = 0; c < n_chunks && ok; ++c) {
      const uint32_t buf = c & 1u;
      ok = mbar_wait<40>(bar(LM_BAR_ACC_FULL + buf), (c >> 1) & 1u, s_abort);
      ok = __all_sync(0xFFFFFFFFu, ok);  // the TMEM loads below are warp-collective
      if (!ok) break;
      tc_fence_after();
      const int width = p.NC;
      const int cbase = v_begin + c * p.NC;
      const int vlim = min(v_end, cbase + width);  // columns at or past it belong to nobody or to the next chunk / CTA
      bool released = false;
      for (int c0 = 32 * half; c0 < width; c0 += 64) {
        uint32_t x[32];
        tc_ld32(tmem + lane_base + buf * 256u + c0, x);
        tc_wait_ld();
        if (c0 + 64 >= width) {  // this warp's last load of the chunk: hand the accumulator back
          tc_fence_before();
          mbar_arrive(bar(LM_BAR_ACC_EMPTY + buf));
          released = true;
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int v = cbase + c0 + i;
          const float cv = __uint_as_float(x[i]);
          // ascending vocabulary order + strict comparisons: among equal values the lower index stays in front
          if (v < vlim && cv > val[KMAX - 1]) {
            // Insert into the sorted list without a serial chain: entry t keeps its value if the new one does not
            // beat it, takes its upper neighbour's if the new one beats that too, and the new one otherwise.  Every
            // entry depends on two comparisons only (a compare-and-swap cascade costs ~8 dependent steps, and the
            // 32 rows of a warp insert at different columns, so nearly every column pays one insertion per warp).
            bool gt[KMAX];
#pragma unroll
            for (int t = 0; t < KMAX; ++t) gt[t] = cv > val[t];
#pragma unroll
            for (int t = KMAX - 1; t > 0; --t) {
              val[t] = gt[t] ? (gt[t - 1] ? val[t - 1] : cv) : val[t];
              idx[t] = gt[t] ? (gt[t - 1] ? idx[t - 1] : v) : idx[t];
            }
            val[0] = gt[0] ? cv : val[0];
            idx[0] = gt[0] ? v : idx[0];
          }
        }
      }
      if (!released) {  // no block of this chunk fell to this half
        tc_fence_before();
        mbar_arrive(bar(LM_BAR_ACC_EMPTY + buf));
      }
    }
    if (ok && row0 + r < p.R) {
      u64* dst = p.part + (static_cast<size_t>(row0 + r) * p.parts + 2 * slice + half) * p.k;
#pragma unroll
      for (int i = 0; i < KMAX; ++i)
        if (i < p.k) dst[i] = idx[i] >= 0 ? lm_key(val[i], static_cast<uint32_t>(idx[i])) : 0ull;
    }
  }

  // ---- teardown: every thread arrives here, also after an aborted wait
  __syncthreads();
  if (*s_abort) {
    if (tid == 0) atomicOr(p.flags, TR_FLAG_WAIT_TIMEOUT);
    // give copies and MMAs that may still be in flight time to land before shared memory and TMEM are released
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// Merge of the per-(CTA, half) lists: one CTA per row.  Every list is sorted, so its first key is its maximum; the
// k-th largest of those maxima (tau) is a lower bound of the row's k-th largest key, and the few keys >= tau are ranked
// by counting.  Keys are distinct (the index is part of the key); empty list entries are 0.
__global__ void __launch_bounds__(LM_MERGE_THREADS)
tr_lm_head_merge_kernel(const u64* __restrict__ part, int parts, int k, int32_t* __restrict__ topk_idx,
                        float* __restrict__ topk_val) {
  extern __shared__ u64 s_keys[];
  __shared__ u64 s_cand[LM_MERGE_CAND];
  __shared__ u64 s_wmax[LM_MERGE_THREADS / 32];
  __shared__ u64 s_tau;
  __shared__ int s_cnt;
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = parts * k;
  auto warp_max = [](u64 x) {
    const uint32_t hi = static_cast<uint32_t>(x >> 32), lo = static_cast<uint32_t>(x);
    const uint32_t mh = __reduce_max_sync(0xFFFFFFFFu, hi);
    const uint32_t ml = __reduce_max_sync(0xFFFFFFFFu, hi == mh ? lo : 0u);
    return (static_cast<u64>(mh) << 32) | ml;
  };
  auto emit = [&](int rank, u64 key) {
    topk_idx[static_cast<size_t>(row) * k + rank] = key ? static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(key)) : 0;
    if (topk_val) topk_val[static_cast<size_t>(row) * k + rank] = key ? lm_key_value(key) : -INFINITY;
  };
  tr_grid_dependency_wait();
  const u64* rp = part + static_cast<size_t>(row) * n;
  for (int i = tid; i < n; i += LM_MERGE_THREADS) s_keys[i] = __ldcg(rp + i);
  if (tid == 0) s_cnt = 0;
  __syncthreads();
  if (warp == 0) {  // tau: k rounds of "largest list maximum below the previous one" (0 if fewer than k lists are filled)
    u64 last = ~0ull;
    for (int rnd = 0; rnd < k; ++rnd) {
      u64 best = 0ull;
      for (int i = lane; i < parts; i += 32) {
        const u64 x = s_keys[i * k];
        if (x < last && x > best) best = x;
      }
      last = warp_max(best);
    }
    if (lane == 0) s_tau = last;
  }
  __syncthreads();
  const u64 tau = s_tau;
  for (int i = tid; i < n; i += LM_MERGE_THREADS) {
    const u64 x = s_keys[i];
    if (x != 0ull && x >= tau) {
      const int pos = atomicAdd(&s_cnt, 1);
      if (pos < LM_MERGE_CAND) s_cand[pos] = x;
    }
  }
  __syncthreads();
  const int cnt = s_cnt;
  if (cnt <= LM_MERGE_CAND) {
    if (tid < cnt) {
      const u64 mine = s_cand[tid];
      int larger = 0;
      for (int i = 0; i < cnt; ++i) larger += (s_cand[i] > mine) ? 1 : 0;
      if (larger < k) emit(larger, mine);
    }
    if (tid >= cnt && tid < k) emit(tid, 0ull);  // fewer than k candidates in total (cannot happen for V >= k)
    return;
  }
  // more keys at or above tau than the candidate buffer holds (long runs of equal values): k rounds over all keys
  u64 last = ~0ull;
  for (int rnd = 0; rnd < k; ++rnd) {
    u64 best = 0ull;
    for (int i = tid; i < n; i += LM_MERGE_THREADS) {
      const u64 x = s_keys[i];
      if (x < last && x > best) best = x;
    }
    best = warp_max(best);
    if (lane == 0) s_wmax[warp] = best;
    __syncthreads();
    u64 m = 0ull;
#pragma unroll
    for (int w = 0; w < LM_MERGE_THREADS / 32; ++w) m = s_wmax[w] > m ? s_wmax[w] : m;
    last = m;
    if (tid == 0) emit(rnd, m);
    __syncthreads();
  }
}

// 2-D bf16 tensor map [rows, cols] (cols contiguous), 128-byte swizzle, box = (64 columns, box_rows); out-of-bounds
// elements read as zero.
bool lm_encode_map(CUtensorMap* m, const void* ptr, uint64_t cols, uint64_t rows, int64_t row_stride, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t gd[2] = {cols, rows};
  cuuint64_t gs[1] = {static_cast<cuuint64_t>(row_stride) * 2};
  cuuint32_t bx[2] = {LM_BK, box_rows}, es[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
         CUDA_SUCCESS;
}

}  // namespace

tr_status tr_lm_head_setup() {
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_lm_head_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, LM_SMEM_BYTES));
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_lm_head_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, LM_SMEM_BYTES));
  return get_encode_fn() ? TR_OK : TR_ERR_CUDA;
}

// Vocabulary slice per CTA (V spread over at most sm_count / groups slices, a multiple of 16), cut into equal chunks of
// at most 256 columns, and as many ring stages as fit.
static void lm_partition(const tr_ctx* ctx, int groups, LmParams* p, int* n_slices) {
  const int max_slices = ctx->sm_count / groups > 0 ? ctx->sm_count / groups : 1;
  int w = (ctx->vocab + max_slices - 1) / max_slices;
  w = (w + 15) / 16 * 16;
  p->cols_per_cta = w;
  *n_slices = (ctx->vocab + w - 1) / w;
  p->n_main = (w + LM_MAX_NC - 1) / LM_MAX_NC;
  p->NC = ((w + p->n_main - 1) / p->n_main + 15) / 16 * 16;
  const int stage = LM_A_BYTES + p->NC * LM_BK * 2;
  p->nstage = LM_RING_BYTES / stage < LM_MAX_STAGES ? LM_RING_BYTES / stage : LM_MAX_STAGES;
}

tr_status tr_launch_lm_head(tr_ctx* ctx, const void* d_hidden, int64_t hidden_stride, const void* d_weight,
                            int64_t weight_stride, int hidden_dim, int32_t* d_topk_idx, float* d_topk_val,
                            cudaStream_t s) {
  const int rows = ctx->batch * ctx->n_nodes;
  LmParams p;
  // rows beyond 128 form further row groups; a vocabulary slice is then worked on by one CTA per group at the same
  // time, so that the weight still comes from HBM once
  p.groups = (rows + 127) / 128;
  if (p.groups > ctx->sm_count) return TR_ERR_UNSUPPORTED;
  int n_slices = 0;
  lm_partition(ctx, p.groups, &p, &n_slices);
  p.flags = ctx->d_flags;
  p.V = ctx->vocab;
  p.H = hidden_dim;
  p.k = ctx->k;
  p.R = rows;
  p.parts = 2 * n_slices;
  p.part = ctx->d_lm_part;
  if (p.parts > ctx->lm_parts_cap) return TR_ERR_UNSUPPORTED;
  if (static_cast<size_t>(p.parts) * p.k * sizeof(u64) > 40 * 1024) return TR_ERR_UNSUPPORTED;  // merge kernel's staging
  CUtensorMap ma, mb;
  if (!lm_encode_map(&mb, d_weight, static_cast<uint64_t>(hidden_dim), static_cast<uint64_t>(ctx->vocab), weight_stride,
                     static_cast<uint32_t>(p.NC)) ||
      !lm_encode_map(&ma, d_hidden, static_cast<uint64_t>(hidden_dim), static_cast<uint64_t>(rows), hidden_stride, 128))
    return TR_ERR_UNSUPPORTED;
  const dim3 grid(static_cast<unsigned>(n_slices * p.groups));
  if (ctx->k <= 8)
    TR_CUDA_TRY(tr_launch_pdl(tr_lm_head_kernel<8>, grid, dim3(LM_THREADS), LM_SMEM_BYTES, s, ma, mb, p));
  else
    TR_CUDA_TRY(tr_launch_pdl(tr_lm_head_kernel<16>, grid, dim3(LM_THREADS), LM_SMEM_BYTES, s, ma, mb, p));
  TR_CUDA_TRY(tr_launch_pdl(tr_lm_head_merge_kernel, dim3(rows), dim3(LM_MERGE_THREADS),
                            sizeof(u64) * p.parts * p.k, s, static_cast<const u64*>(ctx->d_lm_part), p.parts, p.k,
                            d_topk_idx, d_topk_val));
  return TR_OK;
}
