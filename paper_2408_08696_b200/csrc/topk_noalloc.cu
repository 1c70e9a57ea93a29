// Top-k for callers that cannot allocate device memory: tr_topk_noalloc and the segment / ticket top-k kernel it runs.
//
// The kernel cuts a logits row into segments of TOPK_SEG_ELEMS; one CTA per (segment, row) keeps its 16 values per
// thread in registers (128-bit loads), finds a threshold that cannot exceed the segment's k-th largest key (the k-th
// largest of the 16 half-warp maxima), collects the few keys at or above it and selects the segment's top-k exactly.
// The per-segment lists go to scratch memory; the last CTA of a row to finish (atomic ticket, nobody waits) merges
// them into the row's final top-k.  Order: value descending, equal values by lower index - every (value, index) pair is
// one 64-bit key whose unsigned order is that order, so any split / merge order gives the same answer bit for bit.
// (The context path, tr_verify_update, uses the scratch-free cluster kernel of topk.cu instead.)
#include <mutex>

#include "tr_internal.cuh"

namespace {

typedef unsigned long long u64;
constexpr int TOPK_MERGE_CAP = 1024;
constexpr int TOPK_CAND_CAP = 512;

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

template <bool kVec>
__global__ void __launch_bounds__(TOPK_THREADS, 5)
tr_topk_seg_kernel(const float* __restrict__ logits, int V, int k, int segs, u64* __restrict__ part,
                   unsigned int* __restrict__ ticket, int32_t* __restrict__ topk_idx) {
  constexpr int E = TOPK_ELEMS_PER_THREAD;
  constexpr int G = TOPK_THREADS / 16;  // half-warp groups: 16 >= TR_MAX_K
  __shared__ u64 s_gmax[G];
  __shared__ u64 s_cand[TOPK_CAND_CAP];
  __shared__ u64 s_out[TR_MAX_K];
  __shared__ u64 s_merge[TOPK_MERGE_CAP];
  __shared__ u64 s_tau;
  __shared__ int s_cnt;
  __shared__ int s_last;

  const int seg = blockIdx.x;
  const int row = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* rowp = logits + static_cast<size_t>(row) * V;
  const int seg_base = seg * TOPK_SEG_ELEMS;

  // ---- (1) 16 values per thread in registers; running maximum with its index (first = lowest index wins ties)
  float v[E];
  int idx0[E / 4];  // index of each 4-group's first element (vector path) -- scalar path uses j * THREADS + tid
  if (kVec) {
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      const int i0 = seg_base + j * (TOPK_THREADS * 4) + tid * 4;
      idx0[j] = i0;
      float4 t = (i0 < V) ? __ldcs(reinterpret_cast<const float4*>(rowp + i0))
                          : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      v[4 * j] = t.x; v[4 * j + 1] = t.y; v[4 * j + 2] = t.z; v[4 * j + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int j = 0; j < E; ++j) {
      const int i = seg_base + j * TOPK_THREADS + tid;
      v[j] = (i < V) ? __ldcs(rowp + i) : -INFINITY;
    }
  }
  auto index_of = [&](int j) -> int {
    return kVec ? idx0[j >> 2] + (j & 3) : seg_base + j * TOPK_THREADS + tid;
  };
  if (tid == 0) s_cnt = 0;
  float bv = v[0];
  int bj = 0;
#pragma unroll
  for (int j = 1; j < E; ++j)
    if (v[j] > bv) { bv = v[j]; bj = j; }  // -0 == +0 here as well; indices ascend with j
  int bi = 0;
#pragma unroll
  for (int j = 0; j < E; ++j) bi = (bj == j) ? index_of(j) : bi;
  const u64 tmax = (bi < V) ? topk_key(bv, bi) : 0ull;  // padding threads past the row's end hold no key

  // ---- (2) maxima of the 16 half-warp groups; threshold = k-th largest of them.  At least k keys of the segment
  //          are >= it, so the segment's top-k lies among the keys >= it.
  {
    const unsigned mask = (lane < 16) ? 0x0000FFFFu : 0xFFFF0000u;
    const uint32_t hi = static_cast<uint32_t>(tmax >> 32), lo = static_cast<uint32_t>(tmax);
    const uint32_t mh = __reduce_max_sync(mask, hi);
    const uint32_t ml = __reduce_max_sync(mask, hi == mh ? lo : 0u);
    if ((lane & 15) == 0) s_gmax[tid >> 4] = (static_cast<u64>(mh) << 32) | ml;
  }
  __syncthreads();
  // rank by counting, by half a warp for the whole CTA: the group maximum that has exactly k-1 larger ones is the
  // threshold; with fewer than k non-empty groups the threshold is 0 and every key is a candidate
  if (warp == 0) {
    const u64 mine = lane < G ? s_gmax[lane] : 0ull;
    int larger = 0;
#pragma unroll
    for (int i = 0; i < G; ++i) larger += (s_gmax[i] > mine) ? 1 : 0;
    const unsigned hit = __ballot_sync(0xFFFFFFFFu, lane < G && mine != 0ull && larger == k - 1);
    if (hit == 0u) {
      if (lane == 0) s_tau = 0ull;
    } else if (lane == __ffs(hit) - 1) {
      s_tau = mine;
    }
  }
  __syncthreads();
  const u64 tau = s_tau;
  // ---- (3) candidates: only threads whose own maximum reaches the threshold look at their values
  if (tmax != 0 && tmax >= tau) {
    const uint32_t tau_hi = static_cast<uint32_t>(tau >> 32);
#pragma unroll
    for (int j = 0; j < E; ++j) {
      const int i = index_of(j);
      // cheap filter on the value alone, then the exact (value, index) comparison
      if (i < V && static_cast<uint32_t>(topk_key(v[j], 0u) >> 32) >= tau_hi) {
        const u64 key = topk_key(v[j], i);
        if (key >= tau) {
          const int p = atomicAdd(&s_cnt, 1);
          if (p < TOPK_CAND_CAP) s_cand[p] = key;
        }
      }
    }
  }
  __syncthreads();
  // ---- (4) exact top-k of the candidates -> this segment's partial list
  u64* my_part = part + (static_cast<size_t>(row) * segs + seg) * k;
  const int cnt = s_cnt;
  if (cnt <= TOPK_CAND_CAP) {
    // rank by counting: candidate with r larger ones is the segment's r-th entry; unused entries are 0
    for (int t = tid; t < cnt; t += TOPK_THREADS) {
      const u64 mine = s_cand[t];
      int larger = 0;
      for (int i = 0; i < cnt; ++i) larger += (s_cand[i] > mine) ? 1 : 0;
      if (larger < k) my_part[larger] = mine;
    }
    if (tid >= cnt && tid < k) my_part[tid] = 0ull;
    // (these writes are published by the barrier below together with thread 0's fence, which is cumulative)
  } else {
    // More candidates than the buffer holds (only with massive ties or adversarial layouts): select straight
    // from the registers, round by round, the whole CTA taking part.
    u64 last = ~0ull;
    for (int r = 0; r < k; ++r) {
      u64 best = 0;
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const int i = index_of(j);
        const u64 key = (i < V) ? topk_key(v[j], i) : 0ull;
        if (key < last && key > best) best = key;
      }
      best = warp_max_u64(best);
      __syncthreads();  // previous round's readers are done with s_gmax
      if (lane == 0) s_gmax[warp] = best;
      __syncthreads();
      u64 m = 0;
#pragma unroll
      for (int w = 0; w < TOPK_THREADS / 32; ++w) m = s_gmax[w] > m ? s_gmax[w] : m;
      last = m;
      if (tid == 0) my_part[r] = m;
    }
  }
  // ---- (5) ticket: the last CTA of the row merges all partial lists
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
  if (staged) {
    // every partial key counts the keys above it; the k keys with fewer than k above them are the answer
    for (int t = tid; t < n; t += TOPK_THREADS) {
      const u64 mine = s_merge[t];
      if (mine == 0ull) continue;
      int larger = 0;
      for (int i = 0; i < n; ++i) larger += (s_merge[i] > mine) ? 1 : 0;
      if (larger < k)
        topk_idx[static_cast<size_t>(row) * k + larger] = static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(mine));
    }
    if (tid == 0) ticket[row] = 0u;  // ready for the next launch
  } else if (warp == 0) {
    u64 last = ~0ull;
    for (int r = 0; r < k; ++r) {
      u64 best = 0;
      for (int i = lane; i < n; i += 32) {
        const u64 x = __ldcg(row_part + i);
        if (x < last && x > best) best = x;
      }
      last = warp_max_u64(best);
      if (lane == 0) s_out[r] = last;
    }
    __syncwarp();
    if (lane < k) topk_idx[static_cast<size_t>(row) * k + lane] =
        static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(s_out[lane]));
    if (lane == 0) ticket[row] = 0u;
  }
}

}  // namespace

// ---------------------------------------------------------------------------------------------------
// tr_topk_noalloc: the kernel above with its scratch in a fixed device array instead of allocated memory.
//
// Some callers of this library cannot allocate device memory at all: a plug-in running inside a serving
// process that has handed every byte of HBM to its own pool (cudaMalloc simply fails there), or code on a
// latency-critical path where the implicit device-wide synchronisation of cudaMalloc / cudaFree is not
// acceptable.  tr_init allocates, so such callers cannot even create a context.  For them the per-segment
// candidate lists and the per-row tickets of the top-k kernel live in the file-scope array below, which every
// device that loads this library carries until the process exits.
constexpr int NOALLOC_MAX_ROWS = 4096;            // logits rows per call
constexpr int NOALLOC_MAX_PART = 65536;           // rows * segments * k partial keys per call
constexpr size_t NOALLOC_TICKET_BYTES = sizeof(unsigned int) * NOALLOC_MAX_ROWS;
constexpr size_t NOALLOC_BYTES = NOALLOC_TICKET_BYTES + sizeof(u64) * NOALLOC_MAX_PART;  // 528 KB

static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

namespace {
constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;
unsigned char* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};  // device address of the array, per device
}  // namespace

extern "C" tr_status tr_topk_noalloc_limits(int32_t* max_rows, int32_t* max_partial_keys) {
  if (!max_rows || !max_partial_keys) return TR_ERR_INVALID_ARG;
  *max_rows = NOALLOC_MAX_ROWS;
  *max_partial_keys = NOALLOC_MAX_PART;
  return TR_OK;
}

extern "C" tr_status tr_topk_noalloc(const float* d_logits, int32_t rows, int32_t vocab, int32_t k,
                                     int32_t* d_topk_idx, void* stream) {
  if (!d_logits || !d_topk_idx || rows < 1 || k < 1 || k > TR_MAX_K || vocab < k) return TR_ERR_INVALID_ARG;
  const int segs = (vocab + TOPK_SEG_ELEMS - 1) / TOPK_SEG_ELEMS;
  if (rows > NOALLOC_MAX_ROWS || static_cast<int64_t>(rows) * segs * k > NOALLOC_MAX_PART || rows > 65535)
    return TR_ERR_UNSUPPORTED;  // beyond the fixed scratch: see tr_topk_noalloc_limits
  int dev = -1;
  TR_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return TR_ERR_UNSUPPORTED;
  unsigned char* base = nullptr;
  {
    // First call on this device: look up where this device keeps its copy of the array.  In host code the
    // array's name is only a handle; the kernel must be given the address the runtime reports for it.
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
      void* p = nullptr;
      TR_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
      g_noalloc_ptr[dev] = static_cast<unsigned char*>(p);
    }
    base = g_noalloc_ptr[dev];
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned int* ticket = reinterpret_cast<unsigned int*>(base);
  u64* part = reinterpret_cast<u64*>(base + NOALLOC_TICKET_BYTES);
  // The array keeps whatever the previous call left behind.  The tickets must start at zero; the partial lists
  // are fully rewritten by every call before they are read.
  TR_CUDA_TRY(cudaMemsetAsync(ticket, 0, sizeof(unsigned int) * rows, s));
  const dim3 grid(segs, rows);
  const bool vec = (vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(d_logits) & 15) == 0);
  if (vec)
    tr_topk_seg_kernel<true><<<grid, TOPK_THREADS, 0, s>>>(d_logits, vocab, k, segs, part, ticket, d_topk_idx);
  else
    tr_topk_seg_kernel<false><<<grid, TOPK_THREADS, 0, s>>>(d_logits, vocab, k, segs, part, ticket, d_topk_idx);
  TR_CUDA_TRY(cudaGetLastError());
  return TR_OK;
}

