// Fused per-node argmax + top-k over fp32 vocabulary logits (paper Sec. 2.1: argtopk, x^0 = argmax).
//
// Order: value descending, equal values by lower index.  Every (value, index) pair is packed into one
// 64-bit key whose unsigned order IS that order, so all keys are distinct and "top-k" means "the k largest
// keys" - any split / merge order gives the same answer, bit for bit.
//
// A logits row is cut into segments of TOPK_SEG_ELEMS; one CTA per (segment, row) keeps its 16 values per
// thread in registers (128-bit loads), finds a threshold that is guaranteed not to exceed the segment's
// k-th largest key (the k-th largest of the per-thread maxima), collects the few keys at or above it and
// selects the segment's top-k exactly.  The last CTA of a row to finish (atomic ticket, no waiting) merges the
// per-segment lists into the row's final top-k.
#include "tr_internal.cuh"

typedef unsigned long long u64;
constexpr int TOPK_MERGE_CAP = 1024;

__device__ __forceinline__ u64 topk_key(float v, uint32_t idx) {
  uint32_t b = __float_as_uint(v);
  if (b == 0x80000000u) b = 0u;  // -0 and +0 compare equal: the index decides
  const uint32_t s = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return (static_cast<u64>(s) << 32) | static_cast<u64>(0xFFFFFFFFu - idx);
}

__device__ __forceinline__ u64 warp_max_u64(u64 x) {
  const uint32_t hi = static_cast<uint32_t>(x >> 32), lo = static_cast<uint32_t>(x);
  const uint32_t mh = __reduce_max_sync(0xFFFFFFFFu, hi);
  const uint32_t ml = __reduce_max_sync(0xFFFFFFFFu, hi == mh ? lo : 0u);
  return (static_cast<u64>(mh) << 32) | ml;
}

// The k largest keys of arr[0..n) in descending order, one warp; out[r] = 0 when fewer than r+1 keys exist.
// Each round takes the largest key strictly below the previous winner (keys are distinct).
__device__ __forceinline__ void warp_select_topk(const u64* arr, int n, int k, u64* out, int lane) {
  u64 last = ~0ull;
  for (int r = 0; r < k; ++r) {
    u64 best = 0;
    for (int i = lane; i < n; i += 32) {
      const u64 x = arr[i];
      if (x < last && x > best) best = x;
    }
    last = warp_max_u64(best);
    if (lane == 0) out[r] = last;  // once 0 (nothing left) it stays 0
  }
}

template <bool kVec>
__global__ void __launch_bounds__(TOPK_THREADS)
tr_topk_kernel(const float* __restrict__ logits, int V, int k, int segs, u64* __restrict__ part,
               unsigned int* __restrict__ ticket, int32_t* __restrict__ topk_idx) {
  constexpr int E = TOPK_ELEMS_PER_THREAD;
  constexpr int NW = TOPK_THREADS / 32;
  __shared__ u64 s_wtop[NW * TR_MAX_K];
  __shared__ u64 s_cand[TR_MAX_K * E];
  __shared__ u64 s_out[TR_MAX_K];
  __shared__ u64 s_merge[TOPK_MERGE_CAP];
  __shared__ int s_cnt;
  __shared__ int s_last;

  const int seg = blockIdx.x;
  const int row = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* rowp = logits + static_cast<size_t>(row) * V;
  const int seg_base = seg * TOPK_SEG_ELEMS;

  u64 key[E];
  if (kVec) {
    float4 v[E / 4];
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      const int i0 = seg_base + j * (TOPK_THREADS * 4) + tid * 4;
      v[j] = (i0 < V) ? __ldcs(reinterpret_cast<const float4*>(rowp + i0)) : make_float4(0, 0, 0, 0);
    }
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      const int i0 = seg_base + j * (TOPK_THREADS * 4) + tid * 4;
      const bool ok = i0 < V;  // V % 4 == 0 on this path
      key[4 * j + 0] = ok ? topk_key(v[j].x, i0 + 0) : 0ull;
      key[4 * j + 1] = ok ? topk_key(v[j].y, i0 + 1) : 0ull;
      key[4 * j + 2] = ok ? topk_key(v[j].z, i0 + 2) : 0ull;
      key[4 * j + 3] = ok ? topk_key(v[j].w, i0 + 3) : 0ull;
    }
  } else {
    float v[E];
#pragma unroll
    for (int j = 0; j < E; ++j) {
      const int i = seg_base + j * TOPK_THREADS + tid;
      v[j] = (i < V) ? __ldcs(rowp + i) : 0.f;
    }
#pragma unroll
    for (int j = 0; j < E; ++j) {
      const int i = seg_base + j * TOPK_THREADS + tid;
      key[j] = (i < V) ? topk_key(v[j], i) : 0ull;
    }
  }
  if (tid == 0) s_cnt = 0;

  // (1) per-thread maximum, (2) each warp's k largest thread maxima
  u64 tmax = 0;
#pragma unroll
  for (int j = 0; j < E; ++j) tmax = key[j] > tmax ? key[j] : tmax;
  {
    u64 cur = tmax;
    for (int r = 0; r < k; ++r) {
      const u64 w = warp_max_u64(cur);
      if (lane == r) s_wtop[warp * k + r] = w;
      if (cur == w) cur = 0;  // the (unique) winner retires; if w == 0 nothing changes
    }
  }
  __syncthreads();
  // (3) threshold = k-th largest thread maximum of the CTA: at least k keys of the segment are >= it, and
  //     only the <= k threads holding those maxima can hold keys >= it, so at most k*E candidates follow.
  u64 tau = ~0ull;
  for (int r = 0; r < k; ++r) {
    u64 best = 0;
    for (int i = lane; i < NW * k; i += 32) {
      const u64 x = s_wtop[i];
      if (x < tau && x > best) best = x;
    }
    tau = warp_max_u64(best);
    if (tau == 0) break;  // fewer than k non-empty threads: every valid key is a candidate
  }
#pragma unroll
  for (int j = 0; j < E; ++j) {
    if (key[j] != 0 && key[j] >= tau) {
      const int p = atomicAdd(&s_cnt, 1);
      s_cand[p] = key[j];
    }
  }
  __syncthreads();
  // (4) exact top-k of the candidates -> this segment's partial list
  u64* my_part = part + (static_cast<size_t>(row) * segs + seg) * k;
  if (warp == 0) warp_select_topk(s_cand, s_cnt, k, my_part, lane);
  // (5) ticket: the last CTA of the row merges all partial lists
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(&ticket[row], 1u);
    s_last = (t == static_cast<unsigned int>(segs - 1));
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const u64* row_part = part + static_cast<size_t>(row) * segs * k;
  const int n = segs * k;
  const bool staged = n <= TOPK_MERGE_CAP;  // one parallel fetch of every partial list, then rounds in shared memory
  if (staged) {
    for (int i = tid; i < n; i += TOPK_THREADS) s_merge[i] = __ldcg(row_part + i);
    __syncthreads();
  }
  if (warp == 0) {
    u64 last = ~0ull;
    for (int r = 0; r < k; ++r) {
      u64 best = 0;
      for (int i = lane; i < n; i += 32) {
        const u64 x = staged ? s_merge[i] : __ldcg(row_part + i);
        if (x < last && x > best) best = x;
      }
      last = warp_max_u64(best);
      if (lane == 0) s_out[r] = last;
    }
    __syncwarp();
    if (lane < k) topk_idx[static_cast<size_t>(row) * k + lane] =
        static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(s_out[lane]));
    if (lane == 0) ticket[row] = 0u;  // ready for the next launch
  }
}

tr_status tr_launch_topk(tr_ctx* ctx, const float* d_logits, int32_t* d_topk_idx, cudaStream_t s) {
  const int rows = ctx->batch * ctx->n_nodes;
  dim3 grid(ctx->topk_segs, rows);
  const bool vec = (ctx->vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(d_logits) & 15) == 0);
  if (vec)
    tr_topk_kernel<true><<<grid, TOPK_THREADS, 0, s>>>(d_logits, ctx->vocab, ctx->k, ctx->topk_segs,
                                                       ctx->d_topk_part, ctx->d_topk_ticket, d_topk_idx);
  else
    tr_topk_kernel<false><<<grid, TOPK_THREADS, 0, s>>>(d_logits, ctx->vocab, ctx->k, ctx->topk_segs,
                                                        ctx->d_topk_part, ctx->d_topk_ticket, d_topk_idx);
  TR_CUDA_TRY(cudaGetLastError());
  return TR_OK;
}
