// Internal declarations shared by the translation units of libtr.so.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <vector>

#include "tr.h"

#define TR_CUDA_TRY(expr)                                  \
  do {                                                     \
    cudaError_t e__ = (expr);                              \
    if (e__ != cudaSuccess) {                              \
      tr_set_last_cuda_error(e__, #expr, __FILE__, __LINE__); \
      return (e__ == cudaErrorMemoryAllocation) ? TR_ERR_NOMEM : TR_ERR_CUDA; \
    }                                                      \
  } while (0)

void tr_set_last_cuda_error(cudaError_t e, const char* what, const char* file, int line);

// The top-k kernels scan a logits row in pieces of TOPK_SEG_ELEMS values: 16 per thread of a 256-thread CTA.
constexpr int TOPK_THREADS = 256;
constexpr int TOPK_ELEMS_PER_THREAD = 16;
constexpr int TOPK_SEG_ELEMS = TOPK_THREADS * TOPK_ELEMS_PER_THREAD;  // 4096

// Split-KV attention partials: [slot][ATTN_PART_ROWS][D] fp32 + [slot][ATTN_PART_ROWS][2] (m, l).
constexpr int ATTN_PART_ROWS = 128;
constexpr int ATTN_MAX_PART_SLOTS = 1024;

// Layer groups of tr_step_host's copy / compute pipeline.  Measured at the 7B shape (73 MB in, 21 MB out per step):
// 2 groups 1.55 ms, 4 groups 1.60, 8 groups 1.70, 16 groups 1.79 - every extra copy operation costs more than the
// shorter un-overlapped tail saves; one group (no overlap of the copy out) 2.1 ms.
constexpr int TR_IO_GROUPS = 2;

struct tr_ctx {
  int device = 0;
  int vocab = 0, k = 0, n_nodes = 0, batch = 0, depth_max = 0;
  int sm_count = 148;
  std::vector<int32_t> h_parent, h_rank, h_depth;
  // device tables
  int32_t* d_parent = nullptr;   // [N]
  int32_t* d_rank = nullptr;     // [N]
  int32_t* d_depth = nullptr;    // [N]
  int32_t* d_level_off = nullptr;  // [depth_max + 2]: nodes of level d are [off[d], off[d+1])
  uint32_t* d_anc = nullptr;     // [N][4] bit j of row i: j is i or an ancestor of i
  int32_t* d_M = nullptr;        // [batch][V][k]
  // scratch
  unsigned int* d_seq_ticket = nullptr;       // [batch]: CTAs of a sequence that passed tr_commit's read phase
  int32_t* d_sampled = nullptr;               // [batch*N] tokens drawn by tr_verify_update_sampled
  unsigned long long* d_lm_part = nullptr;    // [batch*N][lm_parts_cap][k] per-CTA lists of tr_lm_head_topk
  int lm_parts_cap = 0;
  float* d_attn_part_o = nullptr;   // [slots][128][128]
  float* d_attn_part_ml = nullptr;  // [slots][128][2]
  unsigned int* d_attn_queue = nullptr;  // [2] unit counter of the two-tiles-per-CTA attention kernel (clears itself)
  uint32_t* d_flags = nullptr;
  // tr_step_host: host->device and device->host copy streams and the events that chain them to the caller's stream
  cudaStream_t io_in = nullptr, io_out = nullptr;
  cudaEvent_t ev_start = nullptr, ev_logits = nullptr, ev_out = nullptr;
  cudaEvent_t ev_in[TR_IO_GROUPS] = {}, ev_attn[TR_IO_GROUPS] = {};
  int update_rule = 0, update_scope = 0;  // TR_UPDATE_*
};

// Launch with programmatic dependent launch: the kernel may be scheduled while the previous kernel of the stream is
// still draining; it must execute tr_grid_dependency_wait() before it touches anything that kernel wrote.
template <typename... KArgs, typename... Args>
inline cudaError_t tr_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                 Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void tr_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Timeline instrumentation for development builds (-DTR_STAMPS): each translation unit keeps a few %globaltimer
// stamps (earliest / latest over its CTAs) that a debug entry point copies out.  Compiled out of the product build.
#ifdef TR_STAMPS
#define TR_STAMP_DECL(name, n) static __device__ unsigned long long name[n];
#ifdef __CUDACC__
__device__ __forceinline__ unsigned long long tr_globaltimer() {
#ifdef TR_STAMPS_CLK  // SM cycle counter instead of the global timer: only differences inside one CTA mean anything
  return static_cast<unsigned long long>(clock64());
#else
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
#endif
}
// "MIN": the first CTA's time of the latest launch (plain store); "MAX": the latest time over all CTAs so far
#define TR_STAMP_MIN(arr, i) do { if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0) arr[i] = tr_globaltimer(); } while (0)
#ifdef TR_STAMPS_NOMAX  // only the first CTA's plain stores: no atomics that could disturb what is being timed
#define TR_STAMP_MAX(arr, i) do { } while (0)
#else
#define TR_STAMP_MAX(arr, i) do { if (threadIdx.x == 0) atomicMax(&arr[i], tr_globaltimer()); } while (0)
#endif
#endif
#else
#define TR_STAMP_DECL(name, n)
#define TR_STAMP_MIN(arr, i) do { } while (0)
#define TR_STAMP_MAX(arr, i) do { } while (0)
#endif

// launchers (host functions defined next to their kernels)
// With d_gumbel: the same launch also draws one token per row - the first entry of the ranking of
// z = fl32(fl32(logit * inv_temperature) + gumbel) - into d_drawn [batch * N] (temperature sampling).
tr_status tr_launch_topk(tr_ctx* ctx, const float* d_logits, int32_t* d_topk_idx, cudaStream_t s,
                         const float* d_gumbel = nullptr, float inv_temperature = 1.f, int32_t* d_drawn = nullptr);
// d_target [batch, N] (optional): the token every node's children are matched against, instead of topk[:, 0]
// tree_early: d_tree was written at least two kernels back on the stream (the kernel directly in front did not write it)
tr_status tr_launch_tail(tr_ctx* ctx, const int32_t* d_tree, const tr_step_out* out, cudaStream_t s,
                         const int32_t* d_target = nullptr, bool tree_early = false);
tr_status tr_launch_commit(tr_ctx* ctx, const tr_commit_args* a, const int32_t* d_acc_nodes,
                           const int32_t* d_out_tokens, const int32_t* d_n_new, cudaStream_t s);
tr_status tr_launch_build_tree(tr_ctx* ctx, const int32_t* d_root, int32_t* d_tree, cudaStream_t s);
tr_status tr_launch_attention_tc(tr_ctx* ctx, const tr_attn_args* a, cudaStream_t s);
tr_status tr_attention_tc_setup();
bool tr_attention_pair_applies(const tr_ctx* ctx, const tr_attn_args* a);
tr_status tr_launch_attention_pair(tr_ctx* ctx, const tr_attn_args* a, cudaStream_t s);
tr_status tr_attention_pair_setup();
tr_status tr_lm_head_setup();
tr_status tr_launch_lm_head(tr_ctx* ctx, const void* d_hidden, int64_t hidden_stride, const void* d_weight,
                            int64_t weight_stride, int hidden_dim, int32_t* d_topk_idx, float* d_topk_val, cudaStream_t s);
int tr_attention_pick_splits(const tr_ctx* ctx, const tr_attn_args* a, int base_units, int tile_keys);
