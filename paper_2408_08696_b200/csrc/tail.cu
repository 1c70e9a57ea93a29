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
TR_STAMP_DECL(g_tail_stamps, 8)

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

// One dependent round of gathers per level; every node of a level is looked up in parallel.  Thread i is node i and
// holds its parent, rank and depth in registers (depth -1: no node), so that a level's chain is just barrier -> parent's
// token from shared memory -> the gather -> store.
__device__ __forceinline__ void bfs_expand(const int32_t* __restrict__ M, int k, int my_parent, int my_rank,
                                           int my_depth, int depth_max,
                                           int32_t* s_tree /* shared [n], s_tree[0] set */, int tid) {
  for (int d = 1; d <= depth_max; ++d) {
    __syncthreads();
    if (d == my_depth) s_tree[tid] = __ldcg(M + static_cast<size_t>(s_tree[my_parent]) * k + my_rank);
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
  __syncthreads();
  int my_depth = -1;  // (this kernel gets no depth table: the level whose range holds the node)
  if (tid < n)
    for (int d = 0; d <= depth_max; ++d)
      if (tid >= tb.level_off[d] && tid < tb.level_off[d + 1]) my_depth = d;
  bfs_expand(M, k, tid < n ? tb.parent[tid] : 0, tid < n ? tb.rank[tid] : 0, my_depth, depth_max, s_tree, tid);
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
  __shared__ __align__(16) int32_t s_S[TR_MAX_NODES];
  __shared__ int32_t s_argmax[TR_MAX_NODES];  // the token each node's children must match: argmax, or the given draw
  __shared__ int32_t s_tree[TR_MAX_NODES];
  __shared__ uint32_t s_best[TAIL_THREADS / 32];
  __shared__ uint32_t s_match[TAIL_THREADS / 32];
  __shared__ uint32_t s_anc[TR_MAX_NODES][4];
  __shared__ TailTables tb;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  TR_STAMP_MIN(g_tail_stamps, 0);
  // the kernel behind this one may be scheduled now; it must wait for this grid before it reads anything written here
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- static tables (written by tr_init): fetched while the kernel in front may still be running
  load_tables(tb, n, depth_max, parent, rank, depth, level_off, tid);
  // (this thread's own entries, for the retrieval at the end)
  const int my_parent = tid < n ? tb.parent[tid] : 0, my_rank = tid < n ? tb.rank[tid] : 0;
  const int my_depth = tid < n ? tb.depth[tid] : -1;
  uint32_t my_anc[4] = {0u, 0u, 0u, 0u};  // bit j: node j is this node or one of its ancestors
  if (tid < n) {
    const uint4 a = *reinterpret_cast<const uint4*>(anc + tid * 4);
    my_anc[0] = a.x; my_anc[1] = a.y; my_anc[2] = a.z; my_anc[3] = a.w;
    *reinterpret_cast<uint4*>(s_anc[tid]) = a;
  }
  int32_t* M = M_all + static_cast<size_t>(b) * V * k;
  const int32_t* topk = topk_idx + static_cast<size_t>(b) * n * k;
  const int W = depth_max + 1;
  int32_t tok = 0;
  int32_t row[TR_MAX_K];
  bool tok_ok = false;
  // tree_early: the tree was written at least two kernels back on this stream (tr_verify_update: the top-k kernel sits
  // in between and has itself waited for its predecessor), so it may be fetched while the top-k kernel is still running
  if (tree_early && tid < n) tok = tree_in[static_cast<size_t>(b) * n + tid];
  // Everything above was fetched while the kernel in front may still have been running (programmatic dependent
  // launch); its output is read only from here on.
  tr_grid_dependency_wait();
  TR_STAMP_MAX(g_tail_stamps, 1);
  if (tid < n) {
    if (!tree_early) tok = tree_in[static_cast<size_t>(b) * n + tid];
    // the candidates are stored into M and later used as row indices: anything outside [0, V) is replaced by token 0
    if ((k & 3) == 0 && (reinterpret_cast<uintptr_t>(topk) & 15) == 0) {
#pragma unroll
      for (int c = 0; c < TR_MAX_K; c += 4) {
        int4 x = make_int4(0, 0, 0, 0);
        if (c < k) x = __ldcg(reinterpret_cast<const int4*>(topk + tid * k + c));
        row[c] = x.x; row[c + 1] = x.y; row[c + 2] = x.z; row[c + 3] = x.w;
      }
    } else {
#pragma unroll
      for (int c = 0; c < TR_MAX_K; ++c) row[c] = c < k ? __ldcg(topk + tid * k + c) : 0;
    }
    int32_t want = target ? __ldcg(target + static_cast<size_t>(b) * n + tid) : 0;
    tok_ok = (tok >= 0 && tok < V);
    bool ids_ok = tok_ok;
#pragma unroll
    for (int c = 0; c < TR_MAX_K; ++c)
      if (row[c] < 0 || row[c] >= V) { row[c] = 0; ids_ok = false; }
    if (!target) want = row[0];
    else if (want < 0 || want >= V) { want = 0; ids_ok = false; }
    s_S[tid] = tok;
    s_argmax[tid] = want;
    if (!ids_ok) atomicOr(flags, TR_FLAG_BAD_TOKEN);
  } else {
    s_S[tid] = -1 - tid;  // padding up to TR_MAX_NODES: a value no token equals
  }
  __syncthreads();
  TR_STAMP_MAX(g_tail_stamps, 2);

  // ---- accept: edge (parent(i), i) matches iff S[i] equals the token wanted after the parent; node i is correct iff
  //      every edge on its root path matches, i.e. iff no node of its ancestor mask fails (the root always passes)
  const bool edge_ok = tid < n && (tid == 0 || s_S[tid] == s_argmax[tb.parent[tid]]);
  const uint32_t mword = __ballot_sync(0xFFFFFFFFu, edge_ok);
  if (lane == 0) s_match[warp] = mword;
  __syncthreads();
  uint32_t keyv = 0;
  if (tid < n) {
    const uint32_t bad = (my_anc[0] & ~s_match[0]) | (my_anc[1] & ~s_match[1]) | (my_anc[2] & ~s_match[2]) |
                         (my_anc[3] & ~s_match[3]);
    // deeper first, then lower index; +1 keeps every valid key above the 0 of idle threads
    if (bad == 0u) keyv = (static_cast<uint32_t>(tb.depth[tid]) << 8 | static_cast<uint32_t>(255 - tid)) + 1u;
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
  // the accepted path = the leaf's ancestor mask; its node at depth d goes to slot d
  const uint32_t on_path = (tid < n) ? (s_anc[leaf][tid >> 5] >> (tid & 31)) & 1u : 0u;
  if (on_path) {
    const int d = tb.depth[tid];
    acc_nodes[b * W + d] = tid;
    if (d > 0) out_tokens[b * W + d - 1] = tok;
  }
  if (tid > acc_len && tid < W) {
    acc_nodes[b * W + tid] = -1;
    out_tokens[b * W + tid] = -1;
  }
  if (tid == 0) {
    n_new[b] = acc_len + 1;
    next_root[b] = bonus;
    out_tokens[b * W + acc_len] = bonus;
    s_tree[0] = bonus;
  }

  TR_STAMP_MAX(g_tail_stamps, 3);
  // ---- update: one occurrence of each token writes its whole row - the last one by default, the first one
  //      under TR_UPDATE_FIRST; under TR_UPDATE_ONLY_ACCEPTED only nodes on the accepted path take part
  const uint32_t in_scope = (update_scope == TR_UPDATE_ONLY_ACCEPTED) ? on_path : 1u;
  if (update_scope == TR_UPDATE_ONLY_ACCEPTED) {  // the competitors below must be in scope too
    __syncthreads();                               // (everyone is past reading s_S for the acceptance)
    if (tid < n && !in_scope) s_S[tid] = -1 - tid;
    __syncthreads();
  }
  if (tid < n && tok_ok && in_scope) {
    // does the same token occur at a later (Last) / earlier (First) node?  s_S is padded with values no token equals
    bool other = false;
    if (update_rule != TR_UPDATE_CUR) {
      const bool want_later = update_rule == TR_UPDATE_LAST;
      const int n4 = (n + 3) & ~3;
#pragma unroll 4
      for (int j = 0; j < n4; j += 4) {
        const int4 x = *reinterpret_cast<const int4*>(s_S + j);
        other |= (x.x == tok) & ((j > tid) == want_later) & (j != tid);
        other |= (x.y == tok) & ((j + 1 > tid) == want_later) & (j + 1 != tid);
        other |= (x.z == tok) & ((j + 2 > tid) == want_later) & (j + 2 != tid);
        other |= (x.w == tok) & ((j + 3 > tid) == want_later) & (j + 3 != tid);
      }
    }  // TR_UPDATE_CUR: every occurrence stores; the 32-bit stores of different occurrences land in any order
    if (!other) {
      int32_t* dst = M + static_cast<size_t>(tok) * k;
      if ((k & 3) == 0 && update_rule != TR_UPDATE_CUR) {
#pragma unroll
        for (int c = 0; c < TR_MAX_K; c += 4)
          if (c < k) *reinterpret_cast<int4*>(dst + c) = make_int4(row[c], row[c + 1], row[c + 2], row[c + 3]);
      } else {
#pragma unroll
        for (int c = 0; c < TR_MAX_K; ++c)
          if (c < k) dst[c] = row[c];
      }
    }
  }
  TR_STAMP_MAX(g_tail_stamps, 4);
  // ---- retrieve the next tree from the updated matrix (bfs_expand starts with a __syncthreads())
  bfs_expand(M, k, my_parent, my_rank, my_depth, depth_max, s_tree, tid);
  if (tid < n) tree_out[static_cast<size_t>(b) * n + tid] = s_tree[tid];
  TR_STAMP_MAX(g_tail_stamps, 5);
}

#ifdef TR_STAMPS
extern "C" int tr_debug_stamps_tail(unsigned long long* host, int reset) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(host, g_tail_stamps, sizeof(unsigned long long) * 8);
  if (reset) {
    unsigned long long init[8] = {~0ull, 0, 0, 0, 0, 0, 0, 0};
    cudaMemcpyToSymbol(g_tail_stamps, init, sizeof(init));
  }
  return 0;
}
#endif

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
