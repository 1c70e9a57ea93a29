// Acceptance, matrix update and next-tree retrieval in one kernel (paper Sec. 2.2 verification, Sec. 3.3
// update, Sec. 3.2 / Algorithm 1 retrieval), plus the stand-alone retrieval kernel behind tr_build_tree.
//
// One CTA per sequence, one thread per tree node (N <= 128).
//   accept : node c is correct iff every edge on its root path matches, S[x] == argmax[parent(x)]; each thread
//            walks its own path (<= depth_max steps); the deepest correct node, lowest index among equals, is
//            found with one packed-key maximum (warp reduce + shared memory).
//   update : M[S[i]] <- topk[i] for all i; when a token repeats, only the highest i writes, which is what the
//            sequential loop "for i: M[S[i]] = O[i]" leaves behind - deterministic, no write races.  (TR_UPDATE_CUR,
//            the paper's uncontrolled update, lets every occurrence store its row element by element instead.)
//   BFS    : S'[0] = argmax[last accepted]; level by level S'[i] = M[S'[parent i]][rank i], reading the rows
//            written a moment ago by this same CTA (ordered by __syncthreads()).
#include "tr_internal.cuh"

constexpr int TAIL_THREADS = 128;

// Template tables staged in shared memory once per kernel (one parallel fetch instead of dependent global loads).
struct TailTables {
  int32_t parent[TR_MAX_NODES];
  int32_t rank[TR_MAX_NODES];
  int32_t depth[TR_MAX_NODES];
  int32_t level_off[TR_MAX_NODES + 2];
};

__device__ __forceinline__ void load_tables(TailTables& t, int n, int depth_max, const int32_t* __restrict__ parent,
                                            const int32_t* __restrict__ rank, const int32_t* __restrict__ depth,
                                            const int32_t* __restrict__ level_off, int tid) {
  if (tid < n) {
    t.parent[tid] = parent[tid];
    t.rank[tid] = rank[tid];
    t.depth[tid] = depth[tid];
  }
  for (int i = tid; i < depth_max + 2; i += TAIL_THREADS) t.level_off[i] = level_off[i];
}

__device__ __forceinline__ void bfs_expand(const int32_t* __restrict__ M, int V, int k, int n,
                                           const int32_t* parent, const int32_t* rank,
                                           const int32_t* level_off, int depth_max,
                                           int32_t* s_tree /* shared [n], s_tree[0] set */, int tid) {
  // one dependent round of gathers per level; every node of a level is looked up in parallel
  for (int d = 1; d <= depth_max; ++d) {
    __syncthreads();
    const int lo = level_off[d], hi = level_off[d + 1];
    const int i = lo + tid;
    if (i < hi) s_tree[i] = __ldcg(M + static_cast<size_t>(s_tree[parent[i]]) * k + rank[i]);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(TAIL_THREADS)
tr_build_tree_kernel(const int32_t* __restrict__ M_all, int V, int k, int n, const int32_t* __restrict__ parent,
                     const int32_t* __restrict__ rank, const int32_t* __restrict__ level_off, int depth_max,
                     const int32_t* __restrict__ root, int32_t* __restrict__ tree, uint32_t* __restrict__ flags) {
  __shared__ int32_t s_tree[TR_MAX_NODES];
  __shared__ TailTables tb;
  const int b = blockIdx.x, tid = threadIdx.x;
  const int32_t* M = M_all + static_cast<size_t>(b) * V * k;
  load_tables(tb, n, depth_max, parent, rank, rank, level_off, tid);
  if (tid == 0) {
    int32_t r = root[b];
    if (r < 0 || r >= V) {
      atomicOr(flags, TR_FLAG_BAD_TOKEN);
      r = 0;
    }
    s_tree[0] = r;
  }
  bfs_expand(M, V, k, n, tb.parent, tb.rank, tb.level_off, depth_max, s_tree, tid);
  if (tid < n) tree[static_cast<size_t>(b) * n + tid] = s_tree[tid];
}

__global__ void __launch_bounds__(TAIL_THREADS)
tr_tail_kernel(int32_t* __restrict__ M_all, int V, int k, int n, const int32_t* __restrict__ parent,
               const int32_t* __restrict__ rank, const int32_t* __restrict__ depth,
               const int32_t* __restrict__ level_off, int depth_max, const int32_t* tree_in,
               const int32_t* __restrict__ topk_idx, int32_t* __restrict__ n_new, int32_t* __restrict__ acc_nodes,
               int32_t* __restrict__ out_tokens, int32_t* __restrict__ next_root, int32_t* tree_out,
               uint32_t* __restrict__ flags, const uint32_t* __restrict__ anc, int update_rule, int update_scope,
               const int32_t* __restrict__ target, int tree_early) {
  __shared__ int32_t s_S[TR_MAX_NODES];
  __shared__ int32_t s_argmax[TR_MAX_NODES];  // the token each node's children must match: argmax, or the given draw
  __shared__ int32_t s_tree[TR_MAX_NODES];
  __shared__ uint32_t s_best[TAIL_THREADS / 32];
  __shared__ TailTables tb;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  load_tables(tb, n, depth_max, parent, rank, depth, level_off, tid);
  int32_t* M = M_all + static_cast<size_t>(b) * V * k;
  const int32_t* topk = topk_idx + static_cast<size_t>(b) * n * k;
  const int W = depth_max + 1;

  // the kernel behind this one may be scheduled now; it must wait for this grid before it reads anything written here
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  int32_t tok = 0;
  int32_t row[TR_MAX_K];
  bool tok_ok = false;
  // tree_early: the tree was written at least two kernels back on this stream (tr_verify_update: the top-k kernel sits
  // in between and has itself waited for its predecessor), so it may be fetched while the top-k kernel is still running
  if (tree_early && tid < n) tok = tree_in[static_cast<size_t>(b) * n + tid];
  // Everything above was fetched while the kernel in front may still have been running (programmatic dependent
  // launch); its output is read only from here on.
  tr_grid_dependency_wait();
  if (tid < n) {
    if (!tree_early) tok = tree_in[static_cast<size_t>(b) * n + tid];
    tok_ok = (tok >= 0 && tok < V);
    bool ids_ok = tok_ok;
    s_S[tid] = tok;
    // the candidates are stored into M and later used as row indices: anything outside [0, V) is replaced by token 0
#pragma unroll
    for (int c = 0; c < TR_MAX_K; ++c) {
      int32_t x = c < k ? topk[tid * k + c] : 0;  // fetched once, with the tokens
      if (x < 0 || x >= V) { x = 0; ids_ok = false; }
      row[c] = x;
    }
    int32_t want = row[0];
    if (target) {
      want = target[static_cast<size_t>(b) * n + tid];
      if (want < 0 || want >= V) { want = 0; ids_ok = false; }
    }
    s_argmax[tid] = want;
    if (!ids_ok) atomicOr(flags, TR_FLAG_BAD_TOKEN);
  }
  __syncthreads();

  // ---- accept: walk this node's root path
  uint32_t keyv = 0;
  if (tid < n) {
    bool ok = true;
    for (int x = tid; x > 0;) {
      const int p = tb.parent[x];
      ok = ok && (s_S[x] == s_argmax[p]);
      x = p;
    }
    // deeper first, then lower index; +1 keeps every valid key above the 0 of idle threads
    if (ok) keyv = (static_cast<uint32_t>(tb.depth[tid]) << 8 | static_cast<uint32_t>(255 - tid)) + 1u;
  }
  const uint32_t wbest = __reduce_max_sync(0xFFFFFFFFu, keyv);
  if (lane == 0) s_best[warp] = wbest;
  __syncthreads();
  uint32_t best = 0;
#pragma unroll
  for (int w = 0; w < TAIL_THREADS / 32; ++w) best = max(best, s_best[w]);
  const int leaf = 255 - static_cast<int>((best - 1u) & 0xFFu);
  const int acc_len = static_cast<int>((best - 1u) >> 8);  // accepted drafts = depth of the leaf
  const int32_t bonus = s_argmax[leaf];

  if (tid == 0) {
    n_new[b] = acc_len + 1;
    next_root[b] = bonus;
    int x = leaf;
    for (int d = acc_len; d >= 0; --d) {  // fill the path backwards
      acc_nodes[b * W + d] = x;
      if (d > 0) out_tokens[b * W + d - 1] = s_S[x];
      x = tb.parent[x];
    }
    out_tokens[b * W + acc_len] = bonus;
    for (int d = acc_len + 1; d < W; ++d) {
      acc_nodes[b * W + d] = -1;
      out_tokens[b * W + d] = -1;
    }
    s_tree[0] = bonus;
  }

  // ---- update: one occurrence of each token writes its whole row - the last one by default, the first one
  //      under TR_UPDATE_FIRST; under TR_UPDATE_ONLY_ACCEPTED only nodes on the accepted path take part
  //      (node i is on it iff i is the accepted leaf or one of its ancestors: bit i of the leaf's mask)
  uint32_t in_scope = 1u;
  if (update_scope == TR_UPDATE_ONLY_ACCEPTED && tid < n) in_scope = (anc[leaf * 4 + (tid >> 5)] >> (tid & 31)) & 1u;
  if (update_scope == TR_UPDATE_ONLY_ACCEPTED) {  // the competitors below must be in scope too
    __syncthreads();                               // (everyone is past reading s_S for the acceptance walk)
    if (tid < n && !in_scope) s_S[tid] = -1 - tid;  // a value no token equals
    __syncthreads();
  }
  if (tid < n && tok_ok && in_scope) {
    bool last = true;
    if (update_rule == TR_UPDATE_FIRST) {
      for (int j = 0; j < tid; ++j) last = last && (s_S[j] != tok);
    } else if (update_rule == TR_UPDATE_LAST) {
      for (int j = tid + 1; j < n; ++j) last = last && (s_S[j] != tok);
    }  // TR_UPDATE_CUR: every occurrence stores; the 32-bit stores of different occurrences land in any order
    if (last) {
      int32_t* dst = M + static_cast<size_t>(tok) * k;
#pragma unroll
      for (int c = 0; c < TR_MAX_K; ++c)
        if (c < k) dst[c] = row[c];
    }
  }
  // ---- retrieve the next tree from the updated matrix (bfs_expand starts with a __syncthreads())
  bfs_expand(M, V, k, n, tb.parent, tb.rank, tb.level_off, depth_max, s_tree, tid);
  if (tid < n) tree_out[static_cast<size_t>(b) * n + tid] = s_tree[tid];
}

tr_status tr_launch_build_tree(tr_ctx* ctx, const int32_t* d_root, int32_t* d_tree, cudaStream_t s) {
  tr_build_tree_kernel<<<ctx->batch, TAIL_THREADS, 0, s>>>(ctx->d_M, ctx->vocab, ctx->k, ctx->n_nodes, ctx->d_parent,
                                                           ctx->d_rank, ctx->d_level_off, ctx->depth_max, d_root,
                                                           d_tree, ctx->d_flags);
  TR_CUDA_TRY(cudaGetLastError());
  return TR_OK;
}

tr_status tr_launch_tail(tr_ctx* ctx, const int32_t* d_tree, const tr_step_out* out, cudaStream_t s,
                         const int32_t* d_target, bool tree_early) {
  TR_CUDA_TRY(tr_launch_pdl(tr_tail_kernel, dim3(ctx->batch), dim3(TAIL_THREADS), 0, s, ctx->d_M, ctx->vocab, ctx->k,
                            ctx->n_nodes, ctx->d_parent, ctx->d_rank, ctx->d_depth, ctx->d_level_off, ctx->depth_max,
                            d_tree, out->d_topk_idx, out->d_n_new, out->d_acc_nodes, out->d_out_tokens,
                            out->d_next_root, out->d_next_tree, ctx->d_flags, ctx->d_anc, ctx->update_rule,
                            ctx->update_scope, d_target, tree_early ? 1 : 0));
  return TR_OK;
}
