// Fused per-node argmax + top-k over fp32 vocabulary logits (paper Sec. 2.1: argtopk, x^0 = argmax).
//
// Order: value descending, equal values by lower index.  Every (value, index) pair is packed into one 64-bit key
// whose unsigned order IS that order, so all keys are distinct and "top-k" means "the k largest keys" - any split /
// merge order gives the same answer, bit for bit.
//
// One thread-block cluster per logits row, P = 1, 2, 4 or 8 CTAs; CTA p scans a contiguous part of the row in chunks
// of 4096 values (16 per thread in registers, 128-bit streaming loads).  The hot loop works on the float values only:
//   threshold : tau = k-th largest of the chunk's 16 half-warp maxima (at least k values of the part are >= tau, so
//               the part's k best keys are among the values >= tau); tau only grows from chunk to chunk
//   candidates: the few values >= tau are turned into keys and pushed to shared memory (threads whose own maximum is
//               below tau skip the scan)
//   part list : candidates ranked by counting -> the part's k best keys, stored straight into the shared memory of
//               the cluster's first CTA (distributed shared memory)
//   merge     : after one cluster barrier the first CTA ranks the P * k keys by counting and writes the row's top-k.
// No global scratch, no atomics on global memory, no second kernel.  Massive ties (more candidates than the buffer
// holds) take an exact, slower path that selects round by round from global memory.
#include "tr_internal.cuh"

namespace {

typedef unsigned long long u64;
constexpr int CHUNK = TOPK_SEG_ELEMS;        // values per CTA and iteration
constexpr int E = TOPK_ELEMS_PER_THREAD;     // values per thread and iteration
constexpr int CAND_CAP = 512;
constexpr int MAX_PARTS = 8;

// float -> uint32 whose unsigned order is the float order (-0 and +0 coincide), and back
__device__ __forceinline__ uint32_t ord_u32(float v) {
  uint32_t b = __float_as_uint(v);
  if (b == 0x80000000u) b = 0u;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord_to_float(uint32_t s) {
  return __uint_as_float((s & 0x80000000u) ? (s ^ 0x80000000u) : ~s);
}
__device__ __forceinline__ u64 topk_key(float v, uint32_t idx) {
  return (static_cast<u64>(ord_u32(v)) << 32) | static_cast<u64>(0xFFFFFFFFu - idx);
}
__device__ __forceinline__ u64 warp_max_u64(u64 x) {
  const uint32_t hi = static_cast<uint32_t>(x >> 32), lo = static_cast<uint32_t>(x);
  const uint32_t mh = __reduce_max_sync(0xFFFFFFFFu, hi);
  const uint32_t ml = __reduce_max_sync(0xFFFFFFFFu, hi == mh ? lo : 0u);
  return (static_cast<u64>(mh) << 32) | ml;
}
__device__ __forceinline__ float max3f(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// store into the shared memory of the cluster's CTA 0 (same offset as the local address `p`)
__device__ __forceinline__ void st_leader_u64(const void* p, u64 v) {
  const uint32_t local = static_cast<uint32_t>(__cvta_generic_to_shared(p));
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(0u));
  asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(remote), "l"(v) : "memory");
}

// kSample: rank z = fl32(fl32(logit * inv_t) + gumbel) instead of the logits (Sec. 5.3 temperature sampling: with k = 1
// the result is the token drawn at temperature 1 / inv_t by the Gumbel-max rule).  Two roundings, no fused multiply-add:
// the decision is reproducible with plain float32 arithmetic.
template <bool kVec, bool kSample>
__global__ void __launch_bounds__(TOPK_THREADS)
tr_topk_kernel(const float* __restrict__ logits, int V, int k, int chunks_per_part, int32_t* __restrict__ topk_idx,
               const float* __restrict__ gumbel, float inv_t) {
  __shared__ u64 s_cand[CAND_CAP];
  __shared__ u64 s_all[MAX_PARTS * TR_MAX_K];  // CTA 0 of the cluster: every part's list
  __shared__ u64 s_red[TOPK_THREADS / 32];
  __shared__ uint32_t s_gmax[2][16];
  __shared__ int s_cnt;

  const int part = blockIdx.x, P = gridDim.x, row = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31;
  const float* rowp = logits + static_cast<size_t>(row) * V;
  const float* rowg = kSample ? gumbel + static_cast<size_t>(row) * V : nullptr;
  const int part_base = part * chunks_per_part * CHUNK;
  const int part_end = min(V, part_base + chunks_per_part * CHUNK);

  if (tid == 0) s_cnt = 0;
  // first half of a cluster barrier: before a CTA stores into the first CTA's shared memory (below), every CTA of the
  // cluster must have started
  if (P > 1) asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  // (programmatic dependent launch) the logits belong to whatever ran before on this stream
  tr_grid_dependency_wait();
  // The kernel behind this one (accept / update / retrieve) may be scheduled from here on and run its preamble; it
  // waits for this grid to finish before it reads the result.  (Only after the wait above: whatever that kernel
  // fetches early must come from kernels that are complete by now.)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  auto index_of = [&](int base, int j) -> int {
    return kVec ? base + (j >> 2) * (TOPK_THREADS * 4) + tid * 4 + (j & 3) : base + j * TOPK_THREADS + tid;
  };
  auto load_chunk = [&](int base, float (&v)[E]) {
    if (kVec) {
#pragma unroll
      for (int j = 0; j < E / 4; ++j) {
        const int i0 = base + j * (TOPK_THREADS * 4) + tid * 4;
        float4 t = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (i0 < part_end) {
          t = __ldcs(reinterpret_cast<const float4*>(rowp + i0));
          if (kSample) {
            const float4 g = __ldcs(reinterpret_cast<const float4*>(rowg + i0));
            t.x = __fadd_rn(__fmul_rn(t.x, inv_t), g.x); t.y = __fadd_rn(__fmul_rn(t.y, inv_t), g.y);
            t.z = __fadd_rn(__fmul_rn(t.z, inv_t), g.z); t.w = __fadd_rn(__fmul_rn(t.w, inv_t), g.w);
          }
        }
        v[4 * j] = t.x; v[4 * j + 1] = t.y; v[4 * j + 2] = t.z; v[4 * j + 3] = t.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const int i = base + j * TOPK_THREADS + tid;
        float x = -INFINITY;
        if (i < part_end) {
          x = __ldcs(rowp + i);
          if (kSample) x = __fadd_rn(__fmul_rn(x, inv_t), __ldcs(rowg + i));
        }
        v[j] = x;
      }
    }
  };

  // ---- scan the part chunk by chunk; the next chunk's loads are in flight while the current one is examined
  uint32_t tau_ord = 0u;  // below every value, -inf included
  float v[E], vn[E];
  if (part_base < part_end) load_chunk(part_base, v);
  for (int c = 0; c < chunks_per_part; ++c) {
    const int base = part_base + c * CHUNK;
    if (base >= part_end) break;  // uniform over the CTA
    const bool more = (c + 1 < chunks_per_part) && (base + CHUNK < part_end);
    if (more) load_chunk(base + CHUNK, vn);
    // thread maximum (values only: -0 == +0, no NaN by precondition), then the maxima of the 16 half-warp groups
    float m = max3f(v[0], v[1], v[2]);
#pragma unroll
    for (int j = 3; j + 1 < E; j += 2) m = max3f(m, v[j], v[j + 1]);
    m = fmaxf(m, v[E - 1]);
    {
      const unsigned mask = (lane < 16) ? 0x0000FFFFu : 0xFFFF0000u;
      const uint32_t gm = __reduce_max_sync(mask, ord_u32(m));
      if ((lane & 15) == 0) s_gmax[c & 1][tid >> 4] = gm;
    }
    __syncthreads();
    // every warp works the threshold out for itself: the group maximum with fewer than k larger and at least k
    // larger-or-equal ones is the k-th largest.  Groups past the row's end hold -inf; with fewer than k real groups
    // the threshold is -inf and every value of the chunk is a candidate.
    {
      const uint32_t mine = s_gmax[c & 1][lane & 15];
      int larger = 0, ge = 0;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const uint32_t g = s_gmax[c & 1][i];
        larger += (g > mine) ? 1 : 0;
        ge += (g >= mine) ? 1 : 0;
      }
      const unsigned hit = __ballot_sync(0xFFFFFFFFu, larger < k && ge >= k);
      const uint32_t tau_c = hit ? __shfl_sync(0xFFFFFFFFu, mine, __ffs(hit) - 1) : 0u;  // k <= 16 groups: always a hit
      tau_ord = max(tau_ord, tau_c);
    }
    const float tau = ord_to_float(tau_ord);
    if (m >= tau) {
#pragma unroll
      for (int j = 0; j < E; ++j) {
        if (v[j] >= tau) {
          const int i = index_of(base, j);
          if (i < part_end) {
            const int p = atomicAdd(&s_cnt, 1);
            if (p < CAND_CAP) s_cand[p] = topk_key(v[j], i);
          }
        }
      }
    }
    if (more) {
#pragma unroll
      for (int j = 0; j < E; ++j) v[j] = vn[j];
    }
  }
  __syncthreads();

  // ---- the part's k best keys -> list `part` in the first CTA's shared memory (unused entries are 0)
  u64* my_list = s_all + part * TR_MAX_K;
  const int cnt = s_cnt;
  if (P > 1) asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
  if (cnt <= CAND_CAP) {
    for (int t = tid; t < cnt; t += TOPK_THREADS) {
      const u64 mine = s_cand[t];
      int larger = 0;
      for (int i = 0; i < cnt; ++i) larger += (s_cand[i] > mine) ? 1 : 0;
      if (larger < k) st_leader_u64(my_list + larger, mine);
    }
    if (tid >= cnt && tid < k) st_leader_u64(my_list + tid, 0ull);
  } else {
    // More candidates than the buffer holds (massive ties or adversarial layouts): select straight from global
    // memory, round by round, the whole CTA taking part.
    u64 last = ~0ull;
    for (int r = 0; r < k; ++r) {
      u64 best = 0;
      for (int i = part_base + tid; i < part_end; i += TOPK_THREADS) {
        float x = __ldcg(rowp + i);
        if (kSample) x = __fadd_rn(__fmul_rn(x, inv_t), __ldcg(rowg + i));
        const u64 key = topk_key(x, i);
        if (key < last && key > best) best = key;
      }
      best = warp_max_u64(best);
      __syncthreads();  // the previous round's readers are done with s_red
      if (lane == 0) s_red[tid >> 5] = best;
      __syncthreads();
      u64 mx = 0;
#pragma unroll
      for (int w = 0; w < TOPK_THREADS / 32; ++w) mx = s_red[w] > mx ? s_red[w] : mx;
      last = mx;
      if (tid == 0) st_leader_u64(my_list + r, mx);
    }
  }

  // ---- merge in the cluster's first CTA
  if (P > 1) {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    if (part != 0) return;  // the lists are delivered; only the first CTA goes on
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  } else {
    __syncthreads();
  }
  const int n = P * TR_MAX_K;
  if (tid < n && (tid & (TR_MAX_K - 1)) < k) {
    const u64 mine = s_all[tid];
    if (mine != 0ull) {
      int larger = 0;
      for (int q = 0; q < P; ++q)
        for (int i = 0; i < k; ++i) larger += (s_all[q * TR_MAX_K + i] > mine) ? 1 : 0;
      if (larger < k)
        topk_idx[static_cast<size_t>(row) * k + larger] = static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(mine));
    }
  }
}

}  // namespace

tr_status tr_launch_topk(tr_ctx* ctx, const float* d_logits, int32_t* d_topk_idx, cudaStream_t s,
                         const float* d_gumbel, float inv_temperature, int k_override) {
  const int rows = ctx->batch * ctx->n_nodes;
  const int k = k_override > 0 ? k_override : ctx->k;
  const int chunks = (ctx->vocab + CHUNK - 1) / CHUNK;
  int P = 1;
  while (P < MAX_PARTS && P < chunks) P *= 2;
  const int cpp = (chunks + P - 1) / P;
  bool vec = (ctx->vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(d_logits) & 15) == 0);
  if (d_gumbel) vec = vec && ((reinterpret_cast<uintptr_t>(d_gumbel) & 15) == 0);

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(P, rows);
  cfg.blockDim = dim3(TOPK_THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = P;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const int V = ctx->vocab;
  cudaError_t e;
  if (d_gumbel)
    e = vec ? cudaLaunchKernelEx(&cfg, tr_topk_kernel<true, true>, d_logits, V, k, cpp, d_topk_idx, d_gumbel, inv_temperature)
            : cudaLaunchKernelEx(&cfg, tr_topk_kernel<false, true>, d_logits, V, k, cpp, d_topk_idx, d_gumbel, inv_temperature);
  else
    e = vec ? cudaLaunchKernelEx(&cfg, tr_topk_kernel<true, false>, d_logits, V, k, cpp, d_topk_idx, d_gumbel, 1.f)
            : cudaLaunchKernelEx(&cfg, tr_topk_kernel<false, false>, d_logits, V, k, cpp, d_topk_idx, d_gumbel, 1.f);
  TR_CUDA_TRY(e);
  return TR_OK;
}
