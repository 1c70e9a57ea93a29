// Host side of the C ABI: context, template validation and derived tables, matrix state, status.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "tr_internal.cuh"

static thread_local char g_last_error[512] = "";

void tr_set_last_cuda_error(cudaError_t e, const char* what, const char* file, int line) {
  snprintf(g_last_error, sizeof(g_last_error), "%s:%d: %s -> %s", file, line, what, cudaGetErrorString(e));
}

extern "C" const char* tr_status_string(tr_status s) {
  switch (s) {
    case TR_OK: return "ok";
    case TR_ERR_INVALID_ARG: return "invalid argument";
    case TR_ERR_TEMPLATE: return "malformed tree template";
    case TR_ERR_UNSUPPORTED: return "unsupported configuration";
    case TR_ERR_CUDA: return g_last_error[0] ? g_last_error : "CUDA error";
    case TR_ERR_NOMEM: return "out of device memory";
    case TR_ERR_DEVICE_FLAG: return "device flag set";
    default: return "unknown status";
  }
}

extern "C" tr_status tr_template_from_branching(const int32_t* b, int32_t nb, int32_t max_nodes,
                                                int32_t* parent_out, int32_t* rank_out, int32_t* n_out) {
  if (!b || !parent_out || !rank_out || !n_out || nb < 1 || max_nodes < 1 || max_nodes > TR_MAX_NODES)
    return TR_ERR_INVALID_ARG;
  for (int i = 0; i < nb; ++i)
    if (b[i] < 0) return TR_ERR_INVALID_ARG;
  int depth[TR_MAX_NODES];
  int n = 1;
  parent_out[0] = -1;
  rank_out[0] = 0;
  depth[0] = 0;
  for (int head = 0; head < n && n < max_nodes; ++head) {
    const int d = depth[head];
    const int bd = b[d < nb ? d : nb - 1];
    const int kids = bd - rank_out[head];
    for (int r = 0; r < kids && n < max_nodes; ++r) {
      parent_out[n] = head;
      rank_out[n] = r;
      depth[n] = d + 1;
      ++n;
    }
  }
  *n_out = n;
  return TR_OK;
}

static tr_status free_all(tr_ctx* c) {
  cudaFree(c->d_parent);
  cudaFree(c->d_rank);
  cudaFree(c->d_depth);
  cudaFree(c->d_level_off);
  cudaFree(c->d_anc);
  cudaFree(c->d_M);
  cudaFree(c->d_seq_ticket);
  cudaFree(c->d_lm_part);
  cudaFree(c->d_sampled);
  if (c->io_in) cudaStreamDestroy(c->io_in);
  if (c->io_out) cudaStreamDestroy(c->io_out);
  for (cudaEvent_t e : {c->ev_start, c->ev_logits, c->ev_out}) if (e) cudaEventDestroy(e);
  for (int g = 0; g < TR_IO_GROUPS; ++g) {
    if (c->ev_in[g]) cudaEventDestroy(c->ev_in[g]);
    if (c->ev_attn[g]) cudaEventDestroy(c->ev_attn[g]);
  }
  cudaFree(c->d_attn_part_o);
  cudaFree(c->d_attn_part_ml);
  cudaFree(c->d_attn_queue);
  cudaFree(c->d_flags);
  delete c;
  return TR_OK;
}

extern "C" tr_status tr_init(tr_ctx** out, int32_t vocab, int32_t k, const int32_t* parent, const int32_t* rank,
                             int32_t n_nodes, int32_t batch, int32_t device) {
  if (!out || !parent || !rank) return TR_ERR_INVALID_ARG;
  *out = nullptr;
  if (k < 1 || k > TR_MAX_K || vocab < k || batch < 1 || device < 0) return TR_ERR_INVALID_ARG;
  if (n_nodes < 1 || n_nodes > TR_MAX_NODES) return TR_ERR_TEMPLATE;
  if (static_cast<int64_t>(batch) * n_nodes > 65535) return TR_ERR_UNSUPPORTED;  // logits rows are a grid's y extent
  // Template checks: layer order, parents before children, siblings contiguous enough for Algorithm 1.
  if (parent[0] != -1) return TR_ERR_TEMPLATE;
  std::vector<int32_t> depth(n_nodes, 0);
  for (int i = 1; i < n_nodes; ++i) {
    if (parent[i] < 0 || parent[i] >= i) return TR_ERR_TEMPLATE;
    if (rank[i] < 0 || rank[i] >= k) return TR_ERR_TEMPLATE;
    depth[i] = depth[parent[i]] + 1;
    if (depth[i] < depth[i - 1]) return TR_ERR_TEMPLATE;
  }
  int ndev = 0;
  TR_CUDA_TRY(cudaGetDeviceCount(&ndev));
  if (device >= ndev) return TR_ERR_INVALID_ARG;
  TR_CUDA_TRY(cudaSetDevice(device));

  tr_ctx* c = new (std::nothrow) tr_ctx();
  if (!c) return TR_ERR_NOMEM;
  c->device = device;
  c->vocab = vocab;
  c->k = k;
  c->n_nodes = n_nodes;
  c->batch = batch;
  c->h_parent.assign(parent, parent + n_nodes);
  c->h_rank.assign(rank, rank + n_nodes);
  c->h_depth = depth;
  c->depth_max = depth[n_nodes - 1];
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) == cudaSuccess) c->sm_count = prop.multiProcessorCount;

  std::vector<int32_t> level_off(c->depth_max + 2, 0);
  for (int i = 0; i < n_nodes; ++i) level_off[depth[i] + 1] = i + 1;
  std::vector<uint32_t> anc(static_cast<size_t>(n_nodes) * 4, 0u);
  for (int i = 0; i < n_nodes; ++i)
    for (int j = i; j >= 0; j = parent[j]) anc[i * 4 + (j >> 5)] |= 1u << (j & 31);

#define TR_INIT_TRY(expr)                    \
  do {                                       \
    cudaError_t e__ = (expr);                \
    if (e__ != cudaSuccess) {                \
      tr_set_last_cuda_error(e__, #expr, __FILE__, __LINE__); \
      free_all(c);                           \
      return (e__ == cudaErrorMemoryAllocation) ? TR_ERR_NOMEM : TR_ERR_CUDA; \
    }                                        \
  } while (0)

  const size_t nb = sizeof(int32_t) * n_nodes;
  TR_INIT_TRY(cudaMalloc(&c->d_parent, nb));
  TR_INIT_TRY(cudaMalloc(&c->d_rank, nb));
  TR_INIT_TRY(cudaMalloc(&c->d_depth, nb));
  TR_INIT_TRY(cudaMalloc(&c->d_level_off, sizeof(int32_t) * level_off.size()));
  TR_INIT_TRY(cudaMalloc(&c->d_anc, sizeof(uint32_t) * anc.size()));
  TR_INIT_TRY(cudaMemcpy(c->d_parent, parent, nb, cudaMemcpyHostToDevice));
  TR_INIT_TRY(cudaMemcpy(c->d_rank, rank, nb, cudaMemcpyHostToDevice));
  TR_INIT_TRY(cudaMemcpy(c->d_depth, depth.data(), nb, cudaMemcpyHostToDevice));
  TR_INIT_TRY(cudaMemcpy(c->d_level_off, level_off.data(), sizeof(int32_t) * level_off.size(), cudaMemcpyHostToDevice));
  TR_INIT_TRY(cudaMemcpy(c->d_anc, anc.data(), sizeof(uint32_t) * anc.size(), cudaMemcpyHostToDevice));

  const size_t m_bytes = sizeof(int32_t) * static_cast<size_t>(batch) * vocab * k;
  TR_INIT_TRY(cudaMalloc(&c->d_M, m_bytes));
  TR_INIT_TRY(cudaMemset(c->d_M, 0, m_bytes));

  const size_t rows = static_cast<size_t>(batch) * n_nodes;
  TR_INIT_TRY(cudaMalloc(&c->d_seq_ticket, sizeof(unsigned int) * batch));
  TR_INIT_TRY(cudaMemset(c->d_seq_ticket, 0, sizeof(unsigned int) * batch));
  TR_INIT_TRY(cudaMalloc(&c->d_sampled, sizeof(int32_t) * rows));
  c->lm_parts_cap = 2 * c->sm_count;  // two lists per CTA
  TR_INIT_TRY(cudaMalloc(&c->d_lm_part, sizeof(unsigned long long) * rows * c->lm_parts_cap * k));

  TR_INIT_TRY(cudaMalloc(&c->d_attn_part_o, sizeof(float) * ATTN_MAX_PART_SLOTS * ATTN_PART_ROWS * 128));
  TR_INIT_TRY(cudaMalloc(&c->d_attn_part_ml, sizeof(float) * ATTN_MAX_PART_SLOTS * ATTN_PART_ROWS * 2));
  TR_INIT_TRY(cudaMalloc(&c->d_attn_queue, sizeof(unsigned int) * 2));
  TR_INIT_TRY(cudaMemset(c->d_attn_queue, 0, sizeof(unsigned int) * 2));
  // streams and events of tr_step_host's copy pipeline
  TR_INIT_TRY(cudaStreamCreateWithFlags(&c->io_in, cudaStreamNonBlocking));
  TR_INIT_TRY(cudaStreamCreateWithFlags(&c->io_out, cudaStreamNonBlocking));
  TR_INIT_TRY(cudaEventCreateWithFlags(&c->ev_start, cudaEventDisableTiming));
  TR_INIT_TRY(cudaEventCreateWithFlags(&c->ev_logits, cudaEventDisableTiming));
  TR_INIT_TRY(cudaEventCreateWithFlags(&c->ev_out, cudaEventDisableTiming));
  for (int g = 0; g < TR_IO_GROUPS; ++g) {
    TR_INIT_TRY(cudaEventCreateWithFlags(&c->ev_in[g], cudaEventDisableTiming));
    TR_INIT_TRY(cudaEventCreateWithFlags(&c->ev_attn[g], cudaEventDisableTiming));
  }
  TR_INIT_TRY(cudaMalloc(&c->d_flags, sizeof(uint32_t)));
  TR_INIT_TRY(cudaMemset(c->d_flags, 0, sizeof(uint32_t)));
  TR_INIT_TRY(cudaDeviceSynchronize());
#undef TR_INIT_TRY
  {
    tr_status st = tr_attention_tc_setup();
    if (st == TR_OK) st = tr_attention_pair_setup();
    if (st == TR_OK) st = tr_lm_head_setup();
    if (st != TR_OK) {
      free_all(c);
      return st;
    }
  }
  *out = c;
  return TR_OK;
}

extern "C" tr_status tr_destroy(tr_ctx* ctx) {
  if (!ctx) return TR_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  return free_all(ctx);
}

extern "C" tr_status tr_set_update_rule(tr_ctx* ctx, int32_t rule, int32_t scope) {
  if (!ctx || (rule != TR_UPDATE_LAST && rule != TR_UPDATE_FIRST && rule != TR_UPDATE_CUR) ||
      (scope != TR_UPDATE_ALL_DRAFT && scope != TR_UPDATE_ONLY_ACCEPTED))
    return TR_ERR_INVALID_ARG;
  ctx->update_rule = rule;
  ctx->update_scope = scope;
  return TR_OK;
}

extern "C" int32_t tr_max_new_tokens(const tr_ctx* ctx) { return ctx ? ctx->depth_max + 1 : 0; }

extern "C" tr_status tr_matrix_zero(tr_ctx* ctx, void* stream) {
  if (!ctx) return TR_ERR_INVALID_ARG;
  const size_t bytes = sizeof(int32_t) * static_cast<size_t>(ctx->batch) * ctx->vocab * ctx->k;
  TR_CUDA_TRY(cudaMemsetAsync(ctx->d_M, 0, bytes, static_cast<cudaStream_t>(stream)));
  return TR_OK;
}

// Seeded fill (Sec. 5.2 initialisation study, "Random"): every entry is a counter-based hash of its position.
__global__ void tr_matrix_fill_kernel(int32_t* __restrict__ M, size_t n, int V, uint64_t seed) {
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    uint64_t z = seed + 0x9E3779B97F4A7C15ull * (static_cast<uint64_t>(i) + 1ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    M[i] = static_cast<int32_t>(((z >> 32) * static_cast<uint64_t>(V)) >> 32);
  }
}

extern "C" tr_status tr_matrix_fill(tr_ctx* ctx, int32_t mode, uint64_t seed, void* stream) {
  if (!ctx || (mode != TR_FILL_ZERO && mode != TR_FILL_SEEDED)) return TR_ERR_INVALID_ARG;
  if (mode == TR_FILL_ZERO) return tr_matrix_zero(ctx, stream);
  const size_t n = static_cast<size_t>(ctx->batch) * ctx->vocab * ctx->k;
  const int blocks = static_cast<int>(n / 256 + 1 < 1184 ? n / 256 + 1 : 1184);
  tr_matrix_fill_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(ctx->d_M, n, ctx->vocab, seed);
  TR_CUDA_TRY(cudaGetLastError());
  return TR_OK;
}

extern "C" int32_t* tr_matrix_device_ptr(tr_ctx* ctx, int32_t seq) {
  if (!ctx || seq < 0 || seq >= ctx->batch) return nullptr;
  return ctx->d_M + static_cast<size_t>(seq) * ctx->vocab * ctx->k;
}

extern "C" tr_status tr_matrix_import(tr_ctx* ctx, int32_t seq, const int32_t* host_M) {
  int32_t* dst = tr_matrix_device_ptr(ctx, seq);
  if (!dst || !host_M) return TR_ERR_INVALID_ARG;
  const size_t n = static_cast<size_t>(ctx->vocab) * ctx->k;
  for (size_t i = 0; i < n; ++i)
    if (host_M[i] < 0 || host_M[i] >= ctx->vocab) return TR_ERR_INVALID_ARG;  // keep M within [0, V)
  TR_CUDA_TRY(cudaMemcpy(dst, host_M, n * sizeof(int32_t), cudaMemcpyHostToDevice));
  return TR_OK;
}

extern "C" tr_status tr_matrix_export(tr_ctx* ctx, int32_t seq, int32_t* host_M) {
  int32_t* src = tr_matrix_device_ptr(ctx, seq);
  if (!src || !host_M) return TR_ERR_INVALID_ARG;
  TR_CUDA_TRY(cudaMemcpy(host_M, src, sizeof(int32_t) * static_cast<size_t>(ctx->vocab) * ctx->k,
                         cudaMemcpyDeviceToHost));
  return TR_OK;
}

extern "C" tr_status tr_device_flags(tr_ctx* ctx, uint32_t* host_flags) {
  if (!ctx || !host_flags) return TR_ERR_INVALID_ARG;
  TR_CUDA_TRY(cudaSetDevice(ctx->device));
  TR_CUDA_TRY(cudaDeviceSynchronize());
  TR_CUDA_TRY(cudaMemcpy(host_flags, ctx->d_flags, sizeof(uint32_t), cudaMemcpyDeviceToHost));
  return TR_OK;
}

extern "C" tr_status tr_build_tree(tr_ctx* ctx, const int32_t* d_root, int32_t* d_tree, void* stream) {
  if (!ctx || !d_root || !d_tree) return TR_ERR_INVALID_ARG;
  return tr_launch_build_tree(ctx, d_root, d_tree, static_cast<cudaStream_t>(stream));
}

extern "C" tr_status tr_verify_update(tr_ctx* ctx, const float* d_logits, const int32_t* d_tree,
                                      const tr_step_out* out, void* stream) {
  if (!ctx || !d_logits || !d_tree || !out) return TR_ERR_INVALID_ARG;
  if (!out->d_topk_idx || !out->d_n_new || !out->d_acc_nodes || !out->d_out_tokens || !out->d_next_root ||
      !out->d_next_tree)
    return TR_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  tr_status st = tr_launch_topk(ctx, d_logits, out->d_topk_idx, s);
  if (st != TR_OK) return st;
  return tr_launch_tail(ctx, d_tree, out, s, nullptr, true);
}

extern "C" tr_status tr_verify_update_sampled(tr_ctx* ctx, const float* d_logits, const float* d_gumbel,
                                              float inv_temperature, const int32_t* d_tree, const tr_step_out* out,
                                              int32_t* d_sampled, void* stream) {
  if (!ctx || !d_logits || !d_gumbel || !d_tree || !out) return TR_ERR_INVALID_ARG;
  if (!(inv_temperature > 0.f) || !(inv_temperature < INFINITY)) return TR_ERR_INVALID_ARG;
  if (!out->d_topk_idx || !out->d_n_new || !out->d_acc_nodes || !out->d_out_tokens || !out->d_next_root ||
      !out->d_next_tree)
    return TR_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* drawn = d_sampled ? d_sampled : ctx->d_sampled;
  // one launch, two clusters per row: the model's top-k (the candidates stored in the matrix, whatever is drawn) and
  // the draw - the first entry of the same ranking applied to logit / T + noise
  tr_status st = tr_launch_topk(ctx, d_logits, out->d_topk_idx, s, d_gumbel, inv_temperature, drawn);
  if (st != TR_OK) return st;
  return tr_launch_tail(ctx, d_tree, out, s, drawn, true);
}

extern "C" tr_status tr_verify_update_topk(tr_ctx* ctx, const int32_t* d_tree, const tr_step_out* out, void* stream) {
  if (!ctx || !d_tree || !out) return TR_ERR_INVALID_ARG;
  if (!out->d_topk_idx || !out->d_n_new || !out->d_acc_nodes || !out->d_out_tokens || !out->d_next_root ||
      !out->d_next_tree)
    return TR_ERR_INVALID_ARG;
  return tr_launch_tail(ctx, d_tree, out, static_cast<cudaStream_t>(stream));
}

extern "C" tr_status tr_lm_head_topk(tr_ctx* ctx, const void* d_hidden, int64_t hidden_stride, const void* d_weight,
                                     int64_t weight_stride, int32_t hidden_dim, int32_t* d_topk_idx, float* d_topk_val,
                                     void* stream) {
  if (!ctx || !d_hidden || !d_weight || !d_topk_idx) return TR_ERR_INVALID_ARG;
  if (hidden_dim < 8 || (hidden_dim % 8) != 0) return TR_ERR_INVALID_ARG;
  if (hidden_stride < hidden_dim || weight_stride < hidden_dim || (hidden_stride % 8) != 0 || (weight_stride % 8) != 0)
    return TR_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_hidden) & 15) != 0 || (reinterpret_cast<uintptr_t>(d_weight) & 15) != 0)
    return TR_ERR_INVALID_ARG;
  return tr_launch_lm_head(ctx, d_hidden, hidden_stride, d_weight, weight_stride, hidden_dim, d_topk_idx, d_topk_val,
                           static_cast<cudaStream_t>(stream));
}

static tr_status check_attn_args(const tr_ctx* ctx, const tr_attn_args* a) {
  if (!ctx || !a || !a->q || !a->k_cache || !a->v_cache || !a->out || !a->d_ctx_len) return TR_ERR_INVALID_ARG;
  if (a->n_q_heads < 1 || a->n_kv_heads < 1 || a->n_q_heads % a->n_kv_heads != 0) return TR_ERR_INVALID_ARG;
  if (a->head_dim != 64 && a->head_dim != 128) return TR_ERR_UNSUPPORTED;
  if (!(a->scale >= 0.f) || a->scale > 1e30f) return TR_ERR_INVALID_ARG;  // 0 selects 1/sqrt(head_dim)
  if (a->n_layers < 1 || a->max_ctx < 0 || a->kv_rows < a->max_ctx + ctx->n_nodes || a->splits < 0)
    return TR_ERR_INVALID_ARG;
  const uintptr_t ptrs[4] = {(uintptr_t)a->q, (uintptr_t)a->k_cache, (uintptr_t)a->v_cache, (uintptr_t)a->out};
  for (uintptr_t p : ptrs)
    if (p & 15) return TR_ERR_INVALID_ARG;
  const int64_t strides[12] = {a->q_stride[0],  a->q_stride[1],  a->q_stride[2],  a->kv_stride[0],
                               a->kv_stride[1], a->kv_stride[2], a->o_stride[0],  a->o_stride[1],
                               a->o_stride[2],  a->layer_stride_q, a->layer_stride_kv, a->layer_stride_o};
  for (int64_t s : strides)
    if (s < 0 || (s & 7)) return TR_ERR_INVALID_ARG;
  if (a->q_stride[2] < a->head_dim || a->kv_stride[2] < a->head_dim || a->o_stride[2] < a->head_dim)
    return TR_ERR_INVALID_ARG;
  return TR_OK;
}

extern "C" tr_status tr_tree_attention(tr_ctx* ctx, const tr_attn_args* a, void* stream) {
  tr_status st = check_attn_args(ctx, a);
  if (st != TR_OK) return st;
  return tr_launch_attention_tc(ctx, a, static_cast<cudaStream_t>(stream));
}

extern "C" tr_status tr_commit(tr_ctx* ctx, const tr_commit_args* a, const int32_t* d_acc_nodes,
                               const int32_t* d_out_tokens, const int32_t* d_n_new, void* stream) {
  if (!ctx || !a || !a->k_cache || !a->v_cache || !a->d_ctx_len || !a->d_tokens || !a->d_n_tokens || !d_acc_nodes ||
      !d_out_tokens || !d_n_new)
    return TR_ERR_INVALID_ARG;
  if (a->n_kv_heads < 1 || a->n_layers < 1 || a->kv_rows < ctx->n_nodes || a->token_capacity < 1)
    return TR_ERR_INVALID_ARG;
  if (a->head_dim < 8 || a->head_dim % 8 != 0 || a->head_dim > 256) return TR_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(a->k_cache) & 15) || (reinterpret_cast<uintptr_t>(a->v_cache) & 15))
    return TR_ERR_INVALID_ARG;
  const int64_t strides[4] = {a->kv_stride[0], a->kv_stride[1], a->kv_stride[2], a->layer_stride_kv};
  for (int64_t s : strides)
    if (s < 0 || (s & 7)) return TR_ERR_INVALID_ARG;
  if (a->kv_stride[2] < a->head_dim) return TR_ERR_INVALID_ARG;
  return tr_launch_commit(ctx, a, d_acc_nodes, d_out_tokens, d_n_new, static_cast<cudaStream_t>(stream));
}

extern "C" tr_status tr_step_host(tr_ctx* ctx, const tr_attn_args* a, const tr_step_out* d_out,
                                  const tr_host_io* io, void* stream) {
  tr_status st = check_attn_args(ctx, a);
  if (st != TR_OK) return st;
  if (!d_out || !io || !io->h_q || !io->h_tree_k || !io->h_tree_v || !io->h_logits || !io->h_ctx_len ||
      !io->d_logits_staging || !io->d_tree || !io->h_out || !io->h_n_new || !io->h_out_tokens || !io->h_next_tree)
    return TR_ERR_INVALID_ARG;
  TR_CUDA_TRY(cudaSetDevice(ctx->device));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int B = ctx->batch, N = ctx->n_nodes, L = a->n_layers, D = a->head_dim;
  const size_t esz = sizeof(__nv_bfloat16);
  // queries: the staging tensor must be dense [B, L, N, Hq, D]
  if (a->q_stride[2] != (int64_t)a->n_q_heads * D || a->q_stride[1] != D ||
      a->layer_stride_q != (int64_t)N * a->n_q_heads * D || a->q_stride[0] != (int64_t)L * N * a->n_q_heads * D ||
      a->o_stride[2] != a->q_stride[2] || a->o_stride[1] != D || a->layer_stride_o != a->layer_stride_q ||
      a->o_stride[0] != a->q_stride[0])
    return TR_ERR_INVALID_ARG;
  if (a->kv_stride[2] != D) return TR_ERR_UNSUPPORTED;
  for (int bq = 0; bq < B; ++bq)
    if (io->h_ctx_len[bq] < 0 || io->h_ctx_len[bq] > a->max_ctx) return TR_ERR_INVALID_ARG;
  // The layers are independent, so the step is pipelined over groups of layers on three streams: while group g's
  // attention runs, group g+1's inputs are on their way in and group g-1's output is on its way out (PCIe carries
  // both directions at once).  Host -> device on io_in, kernels on the caller's stream, device -> host on io_out.
  const int G = L < TR_IO_GROUPS ? L : TR_IO_GROUPS;
  TR_CUDA_TRY(cudaEventRecord(ctx->ev_start, s));  // whatever the caller queued before comes first on all three
  TR_CUDA_TRY(cudaStreamWaitEvent(ctx->io_in, ctx->ev_start, 0));
  TR_CUDA_TRY(cudaStreamWaitEvent(ctx->io_out, ctx->ev_start, 0));
  // the prefix lengths the kernels read on the device are this call's host values (the tree rows are placed by them)
  TR_CUDA_TRY(cudaMemcpyAsync(const_cast<int32_t*>(a->d_ctx_len), io->h_ctx_len, sizeof(int32_t) * B,
                              cudaMemcpyHostToDevice, ctx->io_in));
  const size_t q_layer = static_cast<size_t>(N) * a->n_q_heads * D;  // elements of one (sequence, layer) of Q / out
  for (int g = 0; g < G; ++g) {
    const int l0 = static_cast<int>(static_cast<int64_t>(L) * g / G), l1 = static_cast<int>(static_cast<int64_t>(L) * (g + 1) / G);
    const int nl = l1 - l0;
    for (int b = 0; b < B; ++b) {
      const int C = io->h_ctx_len[b];
      const size_t q_off = (static_cast<size_t>(b) * L + l0) * q_layer;
      TR_CUDA_TRY(cudaMemcpyAsync((__nv_bfloat16*)a->q + q_off, (const __nv_bfloat16*)io->h_q + q_off, nl * q_layer * esz,
                                  cudaMemcpyHostToDevice, ctx->io_in));
      // this step's tree K/V rows go behind the sequence's prefix: the N rows of one head are contiguous (N*D
      // elements) and heads are kv_stride[1] apart; when the layers are Hkv heads apart as well (a dense cache), the
      // group's (layer, head) pairs form one run of equally spaced rows and a single strided copy moves them all
      const bool dense = a->layer_stride_kv == static_cast<int64_t>(a->n_kv_heads) * a->kv_stride[1];
      const int ncopies = dense ? 1 : nl;
      for (int i = 0; i < ncopies; ++i) {
        const int l = l0 + i;
        const size_t src_off = (static_cast<size_t>(b) * L + l) * a->n_kv_heads * N * D;
        const size_t dst_off = b * a->kv_stride[0] + l * a->layer_stride_kv + static_cast<size_t>(C) * a->kv_stride[2];
        const size_t height = static_cast<size_t>(dense ? nl : 1) * a->n_kv_heads;
        TR_CUDA_TRY(cudaMemcpy2DAsync((__nv_bfloat16*)a->k_cache + dst_off, a->kv_stride[1] * esz,
                                      (const __nv_bfloat16*)io->h_tree_k + src_off, (size_t)N * D * esz,
                                      (size_t)N * D * esz, height, cudaMemcpyHostToDevice, ctx->io_in));
        TR_CUDA_TRY(cudaMemcpy2DAsync((__nv_bfloat16*)a->v_cache + dst_off, a->kv_stride[1] * esz,
                                      (const __nv_bfloat16*)io->h_tree_v + src_off, (size_t)N * D * esz,
                                      (size_t)N * D * esz, height, cudaMemcpyHostToDevice, ctx->io_in));
      }
    }
    TR_CUDA_TRY(cudaEventRecord(ctx->ev_in[g], ctx->io_in));
    TR_CUDA_TRY(cudaStreamWaitEvent(s, ctx->ev_in[g], 0));
    tr_attn_args ag = *a;
    ag.q = (const __nv_bfloat16*)a->q + l0 * a->layer_stride_q;
    ag.k_cache = (const __nv_bfloat16*)a->k_cache + l0 * a->layer_stride_kv;
    ag.v_cache = (const __nv_bfloat16*)a->v_cache + l0 * a->layer_stride_kv;
    ag.out = (__nv_bfloat16*)a->out + l0 * a->layer_stride_o;
    ag.n_layers = nl;
    st = tr_tree_attention(ctx, &ag, stream);
    if (st != TR_OK) return st;
    TR_CUDA_TRY(cudaEventRecord(ctx->ev_attn[g], s));
    TR_CUDA_TRY(cudaStreamWaitEvent(ctx->io_out, ctx->ev_attn[g], 0));
    for (int b = 0; b < B; ++b) {
      const size_t q_off = (static_cast<size_t>(b) * L + l0) * q_layer;
      TR_CUDA_TRY(cudaMemcpyAsync((__nv_bfloat16*)io->h_out + q_off, (const __nv_bfloat16*)a->out + q_off, nl * q_layer * esz,
                                  cudaMemcpyDeviceToHost, ctx->io_out));
    }
  }
  const size_t lg_bytes = sizeof(float) * static_cast<size_t>(B) * N * ctx->vocab;
  TR_CUDA_TRY(cudaMemcpyAsync(io->d_logits_staging, io->h_logits, lg_bytes, cudaMemcpyHostToDevice, ctx->io_in));
  TR_CUDA_TRY(cudaEventRecord(ctx->ev_logits, ctx->io_in));
  TR_CUDA_TRY(cudaStreamWaitEvent(s, ctx->ev_logits, 0));
  tr_step_out o = *d_out;
  o.d_next_tree = io->d_tree;
  st = tr_verify_update(ctx, io->d_logits_staging, io->d_tree, &o, stream);
  if (st != TR_OK) return st;
  const int W = ctx->depth_max + 1;
  TR_CUDA_TRY(cudaMemcpyAsync(io->h_n_new, o.d_n_new, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, s));
  TR_CUDA_TRY(cudaMemcpyAsync(io->h_out_tokens, o.d_out_tokens, sizeof(int32_t) * B * W, cudaMemcpyDeviceToHost, s));
  TR_CUDA_TRY(cudaMemcpyAsync(io->h_next_tree, io->d_tree, sizeof(int32_t) * B * N, cudaMemcpyDeviceToHost, s));
  TR_CUDA_TRY(cudaEventRecord(ctx->ev_out, ctx->io_out));
  TR_CUDA_TRY(cudaStreamWaitEvent(s, ctx->ev_out, 0));  // the caller's stream ends after the last copy out
  TR_CUDA_TRY(cudaStreamSynchronize(s));
  return TR_OK;
}
