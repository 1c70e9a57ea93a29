// Fused per-node argmax + top-k over fp32 vocabulary logits (paper Sec. 2.1: argtopk, x^0 = argmax).
//
// Order: value descending, equal values by lower index.  Every (value, index) pair is packed into one 64-bit key
// whose unsigned order IS that order, so all keys are distinct and "top-k" means "the k largest keys" - any split /
// merge order gives the same answer, bit for bit.
//
// One thread-block cluster per logits row, P = 1, 2, 4 or 8 CTAs of 128 threads; CTA p scans a contiguous part of the
// row in chunks of 4096 values (32 per thread in registers, 128-bit streaming loads).  The kernel is short and all its
// CTAs are resident at once, so its duration is the memory latency plus the instructions every warp issues: the hot
// loop works on the float values only and keeps the per-warp instruction count low.
//   threshold : tau = k-th largest of the chunk's 16 quarter-warp maxima (at least k values of the part are >= tau,
//               so the part's k best keys are among the values >= tau); tau only grows from chunk to chunk
//   candidates: the few values >= tau are turned into keys and pushed to shared memory (threads whose own maximum is
//               below tau skip the scan; the others test four values at a time)
//   part list : candidates ranked by counting (four threads per candidate) -> the part's k best keys, stored straight
//               into the shared memory of EVERY CTA of the cluster (distributed shared memory)
//   merge     : after one cluster barrier every CTA holds all P lists and ranks its own k keys among them by counting
//               (four threads per key; the other warps have left by then); a key with fewer than k keys above it is
//               written to its place of the row's top-k.  Keys are distinct, so the P CTAs write disjoint places.
// No global scratch, no atomics on global memory, no second kernel.  Massive ties (more candidates than the buffer
// holds) take an exact, slower path that selects round by round from global memory.
#include "tr_internal.cuh"

namespace {

typedef unsigned long long u64;
constexpr int KT = 128;                      // threads per CTA
constexpr int E = 32;                        // values per thread and iteration
constexpr int CHUNK = KT * E;                // values per CTA and iteration (4096)
constexpr int CAND_CAP = 512;                // candidate keys a CTA can hold
constexpr int MAX_PARTS = 8;
TR_STAMP_DECL(g_stamps, 16)

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
// store into the shared memory of every CTA of the cluster (same offset as the local address `p`)
__device__ __forceinline__ void st_all_u64(const void* p, u64 v, int n_ctas) {
  const uint32_t local = static_cast<uint32_t>(__cvta_generic_to_shared(p));
  for (int r = 0; r < n_ctas; ++r) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(r));
    asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(remote), "l"(v) : "memory");
  }
}
__device__ __forceinline__ int count_gt(const ulonglong2& a, u64 x) { return (a.x > x) + (a.y > x); }

// kSample: the clusters blockIdx.y >= rows_plain rank z = fl32(fl32(logit * inv_t) + gumbel) instead of the logits
// (Sec. 5.3 temperature sampling: with k = 1 the result is the token drawn at temperature 1 / inv_t by the Gumbel-max
// rule) and write their k_sample best to out_sample.  Two roundings, no fused multiply-add: the decision is
// reproducible with plain float32 arithmetic.  rows_plain = 0: every cluster samples; rows_plain = rows with 2 * rows
// clusters: the model's top-k and the draw of every row in one launch, side by side.
template <bool kVec, bool kSample>
__global__ void __launch_bounds__(KT)
tr_topk_kernel(const float* __restrict__ logits, int V, int k_plain, int chunks_per_part,
               int32_t* __restrict__ out_plain, const float* __restrict__ gumbel, float inv_t, int rows_plain,
               int k_sample, int32_t* __restrict__ out_sample) {
  __shared__ __align__(16) u64 s_cand[CAND_CAP + 32];        // candidates, then up to 32 zeros of padding
  __shared__ __align__(16) u64 s_all[MAX_PARTS * TR_MAX_K];  // every part's list (each CTA gets a copy)
  __shared__ u64 s_red[KT / 32];
  __shared__ uint32_t s_gmax[16];
  __shared__ uint32_t s_tau;
  __shared__ int s_cnt;

  const int part = blockIdx.x, P = gridDim.x;
  const bool sample = kSample && static_cast<int>(blockIdx.y) >= rows_plain;  // the same for a whole cluster
  const int row = sample ? blockIdx.y - rows_plain : blockIdx.y;
  const int k = sample ? k_sample : k_plain;
  int32_t* __restrict__ topk_idx = sample ? out_sample : out_plain;
  const int tid = threadIdx.x, lane = tid & 31;
  const float* rowp = logits + static_cast<size_t>(row) * V;
  const float* rowg = kSample ? gumbel + static_cast<size_t>(row) * V : nullptr;
  const int part_base = part * chunks_per_part * CHUNK;
  const int part_end = min(V, part_base + chunks_per_part * CHUNK);

  TR_STAMP_MIN(g_stamps, 0);
  if (tid == 0) { s_tau = 0u; s_cnt = 0; }  // tau = 0 is below every value, -inf included
  // first half of a cluster barrier: before a CTA stores into another CTA's shared memory (below), every CTA of the
  // cluster must have started
  if (P > 1) asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  // (programmatic dependent launch) the logits belong to whatever ran before on this stream
  tr_grid_dependency_wait();
  TR_STAMP_MIN(g_stamps, 1);
  TR_STAMP_MAX(g_stamps, 2);
  // The kernel behind this one (accept / update / retrieve) may be scheduled from here on and run its preamble; it
  // waits for this grid to finish before it reads the result.  (Only after the wait above: whatever that kernel
  // fetches early must come from kernels that are complete by now.)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // value j of this thread: vector layout - float4 number j/4 of the chunk's tid-th slot; scalar layout - strided
  auto index_of = [&](int base, int j) -> int {
    return kVec ? base + (j >> 2) * (KT * 4) + tid * 4 + (j & 3) : base + j * KT + tid;
  };
  auto load_chunk = [&](int base, float (&v)[E]) {
    if (kVec) {
#pragma unroll
      for (int j = 0; j < E / 4; ++j) {
        const int i0 = base + j * (KT * 4) + tid * 4;
        float4 t = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (i0 < part_end) {
          t = __ldcs(reinterpret_cast<const float4*>(rowp + i0));
          if (kSample && sample) {
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
        const int i = base + j * KT + tid;
        float x = -INFINITY;
        if (i < part_end) {
          x = __ldcs(rowp + i);
          if (kSample && sample) x = __fadd_rn(__fmul_rn(x, inv_t), __ldcs(rowg + i));
        }
        v[j] = x;
      }
    }
  };

  // ---- scan the part chunk by chunk; the next chunk's loads are in flight while the current one is examined
  float v[E], vn[E];
  if (part_base < part_end) load_chunk(part_base, v);
  TR_STAMP_MIN(g_stamps, 6);
  for (int c = 0; c < chunks_per_part; ++c) {
    const int base = part_base + c * CHUNK;
    if (base >= part_end) break;  // uniform over the CTA
    const bool more = (c + 1 < chunks_per_part) && (base + CHUNK < part_end);
    if (more) load_chunk(base + CHUNK, vn);
    // maxima of groups of four values and of the thread (values only: -0 == +0, no NaN by precondition), then the
    // maxima of the 16 quarter-warp groups
    float g4[E / 4];
#pragma unroll
    for (int j = 0; j < E / 4; ++j) g4[j] = fmaxf(max3f(v[4 * j], v[4 * j + 1], v[4 * j + 2]), v[4 * j + 3]);
    float m = max3f(g4[0], g4[1], g4[2]);
#pragma unroll
    for (int j = 3; j + 1 < E / 4; j += 2) m = max3f(m, g4[j], g4[j + 1]);
    m = fmaxf(m, g4[E / 4 - 1]);
    {
      const uint32_t gm = __reduce_max_sync(0xFFu << (lane & 24), ord_u32(m));
      if ((lane & 7) == 0) s_gmax[tid >> 3] = gm;
    }
    __syncthreads();
    // the first warp works the threshold out: the group maximum with fewer than k larger and at least k
    // larger-or-equal ones is the k-th largest (lane = (group, half): each lane counts over 8 of the 16 maxima).
    // Groups past the row's end hold -inf; with fewer than k real groups the threshold is -inf and every value of the
    // chunk is a candidate.
    if (tid < 32) {
      const uint32_t mine = s_gmax[lane & 15];
      int larger = 0, ge = 0;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t g = s_gmax[(lane >> 4) * 8 + u];
        larger += (g > mine) ? 1 : 0;
        ge += (g >= mine) ? 1 : 0;
      }
      larger += __shfl_xor_sync(0xFFFFFFFFu, larger, 16);
      ge += __shfl_xor_sync(0xFFFFFFFFu, ge, 16);
      const unsigned hit = __ballot_sync(0xFFFFFFFFu, larger < k && ge >= k);
      const uint32_t tau_c = hit ? __shfl_sync(0xFFFFFFFFu, mine, __ffs(hit) - 1) : 0u;  // k <= 16 groups: always a hit
      if (lane == 0) s_tau = max(s_tau, tau_c);
    }
    __syncthreads();
    const float tau = ord_to_float(s_tau);
    TR_STAMP_MIN(g_stamps, 7);
    if (m >= tau) {  // a few threads per warp
#pragma unroll
      for (int j = 0; j < E / 4; ++j) {
        if (g4[j] >= tau) {
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            if (v[4 * j + u] >= tau) {
              const int i = index_of(base, 4 * j + u);
              if (i < part_end) {
                const int pos = atomicAdd(&s_cnt, 1);
                if (pos < CAND_CAP) s_cand[pos] = topk_key(v[4 * j + u], i);
              }
            }
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
  const int cnt = s_cnt;
  if (cnt <= CAND_CAP && tid < 32) s_cand[cnt + tid] = 0ull;  // zeros (below every key) pad the last round of 32
  __syncthreads();
  TR_STAMP_MAX(g_stamps, 3);
  TR_STAMP_MIN(g_stamps, 8);

  // ---- the part's k best keys -> list `part` in every CTA's shared memory (unused entries are 0)
  u64* my_list = s_all + part * TR_MAX_K;
  if (P > 1) asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
  if (cnt <= CAND_CAP) {
    // rank by counting, four threads per candidate: thread (c, s) counts the keys above candidate c among the
    // entries s, s + 4, s + 8, ... - eight independent loads per round of 32 entries
    const int s4 = tid & 3;
    for (int c0 = 0; c0 < cnt; c0 += KT / 4) {
      const int c = c0 + (tid >> 2);
      const u64 mine = c < cnt ? s_cand[c] : ~0ull;
      int larger = 0;
      for (int i0 = 0; i0 < cnt; i0 += 32) {
        u64 e[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) e[u] = s_cand[i0 + s4 + 4 * u];
#pragma unroll
        for (int u = 0; u < 8; ++u) larger += (e[u] > mine) ? 1 : 0;
      }
      larger += __shfl_xor_sync(0xFFFFFFFFu, larger, 1);
      larger += __shfl_xor_sync(0xFFFFFFFFu, larger, 2);
      if (s4 == 0 && c < cnt && larger < k) st_all_u64(my_list + larger, mine, P);
    }
    // entries the part cannot fill, and the unused tail of the list, are 0
    if (tid < TR_MAX_K && (tid >= k || tid >= cnt)) st_all_u64(my_list + tid, 0ull, P);
  } else {
    // More candidates than the buffer holds (massive ties or adversarial layouts): select straight from global
    // memory, round by round, the whole CTA taking part.
    u64 last = ~0ull;
    for (int r = 0; r < k; ++r) {
      u64 best = 0;
      for (int i = part_base + tid; i < part_end; i += KT) {
        float x = __ldcg(rowp + i);
        if (kSample && sample) x = __fadd_rn(__fmul_rn(x, inv_t), __ldcg(rowg + i));
        const u64 key = topk_key(x, i);
        if (key < last && key > best) best = key;
      }
      best = warp_max_u64(best);
      __syncthreads();  // the previous round's readers are done with s_red
      if (lane == 0) s_red[tid >> 5] = best;
      __syncthreads();
      u64 mx = 0;
#pragma unroll
      for (int w = 0; w < KT / 32; ++w) mx = s_red[w] > mx ? s_red[w] : mx;
      last = mx;
      if (tid == 0) st_all_u64(my_list + r, mx, P);
    }
    if (tid >= k && tid < TR_MAX_K) st_all_u64(my_list + tid, 0ull, P);
  }

  // ---- every CTA now ranks its own list's keys among all lists
  TR_STAMP_MIN(g_stamps, 9);
  if (P > 1) {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    TR_STAMP_MIN(g_stamps, 10);
    // The final ranking takes 4 threads per key.  Threads without a key leave here: a warp that waits at the cluster
    // barrier is not idle for the SM's schedulers, and with four or five CTAs per SM the waiting warps slowed the
    // working ones down (1.6 us of the kernel at 80 rows x 32000).
    if (tid >= 4 * (k <= 8 ? 8 : TR_MAX_K)) return;
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  } else {
    __syncthreads();
  }
  TR_STAMP_MIN(g_stamps, 11);
  TR_STAMP_MAX(g_stamps, 4);
  if (tid < 4 * (k <= 8 ? 8 : TR_MAX_K)) {
    // four threads per key: thread (i, q) counts the keys of lists q and q + 4 above key i of this part's list (every
    // list has TR_MAX_K entries, zeros behind its k keys; with k <= 8 the first half of a list is enough)
    const int i = tid >> 2, q = tid & 3;
    const u64 mine = my_list[i];
    int larger = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int ql = q + 4 * h;
      if (ql < P) {
        const ulonglong2* lp = reinterpret_cast<const ulonglong2*>(s_all + ql * TR_MAX_K);
        const ulonglong2 a0 = lp[0], a1 = lp[1], a2 = lp[2], a3 = lp[3];
        larger += count_gt(a0, mine) + count_gt(a1, mine) + count_gt(a2, mine) + count_gt(a3, mine);
        if (k > 8) {
          const ulonglong2 a4 = lp[4], a5 = lp[5], a6 = lp[6], a7 = lp[7];
          larger += count_gt(a4, mine) + count_gt(a5, mine) + count_gt(a6, mine) + count_gt(a7, mine);
        }
      }
    }
    larger += __shfl_xor_sync(0xFFFFFFFFu, larger, 1);
    larger += __shfl_xor_sync(0xFFFFFFFFu, larger, 2);
    if (q == 0 && mine != 0ull && larger < k)
      topk_idx[static_cast<size_t>(row) * k + larger] = static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(mine));
  }
  TR_STAMP_MAX(g_stamps, 5);
  TR_STAMP_MIN(g_stamps, 12);
}

}  // namespace

#ifdef TR_STAMPS
extern "C" int tr_debug_stamps_topk(unsigned long long* host, int reset) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(host, g_stamps, sizeof(unsigned long long) * 16);
  if (reset) {
    unsigned long long init[16] = {~0ull, ~0ull, 0, 0, 0, 0, 0, 0};
    cudaMemcpyToSymbol(g_stamps, init, sizeof(init));
  }
  return 0;
}
#endif

tr_status tr_launch_topk(tr_ctx* ctx, const float* d_logits, int32_t* d_topk_idx, cudaStream_t s,
                         const float* d_gumbel, float inv_temperature, int32_t* d_drawn) {
  // without noise: the rows' top-k.  With noise: the same launch also holds one more cluster per row that ranks
  // logit * inv_temperature + noise and writes its first entry (the draw) to d_drawn.
  const int rows = ctx->batch * ctx->n_nodes;
  const int k = ctx->k;
  const int chunks = (ctx->vocab + CHUNK - 1) / CHUNK;
  int P = 1;
  while (P < MAX_PARTS && P < chunks) P *= 2;
  const int cpp = (chunks + P - 1) / P;
  bool vec = (ctx->vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(d_logits) & 15) == 0);
  if (d_gumbel) vec = vec && ((reinterpret_cast<uintptr_t>(d_gumbel) & 15) == 0);
  if (d_gumbel && (!d_drawn || 2 * rows > 65535)) return TR_ERR_UNSUPPORTED;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(P, d_gumbel ? 2 * rows : rows);
  cfg.blockDim = dim3(KT);
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
    e = vec ? cudaLaunchKernelEx(&cfg, tr_topk_kernel<true, true>, d_logits, V, k, cpp, d_topk_idx, d_gumbel,
                                 inv_temperature, rows, 1, d_drawn)
            : cudaLaunchKernelEx(&cfg, tr_topk_kernel<false, true>, d_logits, V, k, cpp, d_topk_idx, d_gumbel,
                                 inv_temperature, rows, 1, d_drawn);
  else
    e = vec ? cudaLaunchKernelEx(&cfg, tr_topk_kernel<true, false>, d_logits, V, k, cpp, d_topk_idx, d_gumbel, 1.f, rows, 1,
                                 d_drawn)
            : cudaLaunchKernelEx(&cfg, tr_topk_kernel<false, false>, d_logits, V, k, cpp, d_topk_idx, d_gumbel, 1.f, rows, 1,
                                 d_drawn);
  TR_CUDA_TRY(e);
  return TR_OK;
}
