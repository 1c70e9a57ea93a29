/*
 * tr.h - C ABI of the Token Recycling (TR) verify-and-recycle step for one NVIDIA B200 (sm_100a).
 *
 * One TR decoding step (paper Sec. 3 and Sec. 5.4) is
 *     retrieve a draft tree from the adjacency matrix   -> tr_build_tree
 *     model forward with tree attention                  -> tr_tree_attention (attention only)
 *     verify (argmax per node, longest correct path),
 *     update the matrix with every node's top-k,
 *     retrieve the next tree                             -> tr_verify_update
 *
 * Conventions
 *   - Every pointer is marked HOST or DEVICE.  DEVICE pointers are caller-owned (for example PyTorch
 *     tensors) unless stated; the library never frees them.
 *   - `stream` is a cudaStream_t passed as void*; NULL is the legacy default stream.
 *   - All entry points return a tr_status; none throws, aborts or synchronises the device unless its
 *     comment says so.  Argument errors are detected on the host before any launch.
 *   - tr_build_tree, tr_tree_attention and tr_verify_update allocate nothing, read nothing back and do
 *     not synchronise, so they can be recorded in a CUDA graph.
 *   - Anomalies only the device can see (a token id outside [0, vocab)) set a sticky bit in a flag word
 *     (tr_device_flags); the offending access is skipped or clamped.  Kernels never trap.
 *   - Notation follows the paper: V = vocabulary size, k = candidates per token, M = adjacency matrix
 *     [V, k], S = merged sequence (tree tokens in layer order, root first), N = tree nodes incl. root.
 */
#ifndef TR_H_
#define TR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tr_ctx tr_ctx; /* opaque; owns M, the template tables and the kernels' scratch */

typedef int32_t tr_status;
#define TR_OK 0
#define TR_ERR_INVALID_ARG (-1)
#define TR_ERR_TEMPLATE (-2)
#define TR_ERR_UNSUPPORTED (-3)
#define TR_ERR_CUDA (-4)
#define TR_ERR_NOMEM (-5)
#define TR_ERR_DEVICE_FLAG (-6)

#define TR_MAX_NODES 128 /* ancestor masks are 128-bit */
#define TR_MAX_K 16

/* Device flag bits (tr_device_flags). */
#define TR_FLAG_BAD_TOKEN 1u    /* a token id (tree, root, given top-k or draw) was outside [0, V): row skipped / id replaced by 0 */
#define TR_FLAG_WAIT_TIMEOUT 2u /* a bounded wait inside a kernel ran out (should never happen) */
#define TR_FLAG_CACHE_FULL 4u   /* tr_commit: no room for another tree behind the grown prefix; sequence left as is */

const char* tr_status_string(tr_status s);

/*
 * Static tree template by rule (Sec. 3.2: static, imbalanced - earlier siblings get more children).
 * A node at depth d whose rank among its siblings is r gets max(0, b[min(d, nb-1)] - r) children; children
 * are appended parent by parent, rank ascending (layer order), and the list is cut at max_nodes.
 * HOST in: b[nb].  HOST out: parent_out[max_nodes], rank_out[max_nodes] (parent[0] = -1), *n_out = node count.
 * Errors: TR_ERR_INVALID_ARG on NULL / non-positive sizes / max_nodes > TR_MAX_NODES.
 */
tr_status tr_template_from_branching(const int32_t* b, int32_t nb, int32_t max_nodes,
                                     int32_t* parent_out, int32_t* rank_out, int32_t* n_out);

/*
 * Create a context on `device` (Sec. 3.1): allocates `batch` adjacency matrices M[V, k] (int32, zeroed: the
 * paper's cold start), uploads the template and the tables derived from it (depth, ancestor bitmasks),
 * and allocates the scratch the kernels need.  Synchronises once.
 * HOST in: parent[n_nodes], rank[n_nodes] - the static tree in layer order: parent[0] = -1, 0 <= parent[i] < i,
 *   depth non-decreasing, 0 <= rank[i] < k (rank = the column of M a node is drawn from, Appendix tree figure).
 * Errors: TR_ERR_INVALID_ARG (vocab < k, k < 1 or > TR_MAX_K, batch < 1, NULL), TR_ERR_TEMPLATE
 *   (malformed tree, n_nodes > TR_MAX_NODES), TR_ERR_UNSUPPORTED (batch * n_nodes > 65535), TR_ERR_CUDA / TR_ERR_NOMEM.
 */
tr_status tr_init(tr_ctx** out, int32_t vocab, int32_t k, const int32_t* parent, const int32_t* rank,
                  int32_t n_nodes, int32_t batch, int32_t device);
tr_status tr_destroy(tr_ctx* ctx); /* frees everything tr_init allocated; synchronises */

/* Matrix state (Sec. 3.1: zero initialisation, or "hot start" = keep / restore an earlier matrix). */
tr_status tr_matrix_zero(tr_ctx* ctx, void* stream);                                /* all sequences */
/*
 * Fill all sequences' matrices on the device (Sec. 5.2, study of initialisations: zeros, or random token ids).
 *   TR_FILL_ZERO   : every entry 0 (= tr_matrix_zero)
 *   TR_FILL_SEEDED : entry number i of the context's [batch, V, k] array (i = (b * V + token) * k + column) is
 *                    (hi32(mix(seed + 0x9E3779B97F4A7C15 * (i + 1))) * V) >> 32, where mix is the splitmix64 finaliser
 *                    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9; z ^= z >> 27; z *= 0x94D049BB133111EB; z ^= z >> 31
 *                    (64-bit wrap-around arithmetic) - uniform token ids in [0, V), reproducible on any host.
 * Errors: TR_ERR_INVALID_ARG (NULL, unknown mode).  Does not synchronise.
 */
#define TR_FILL_ZERO 0
#define TR_FILL_SEEDED 1
tr_status tr_matrix_fill(tr_ctx* ctx, int32_t mode, uint64_t seed, void* stream);
tr_status tr_matrix_import(tr_ctx* ctx, int32_t seq, const int32_t* host_M);        /* HOST [V*k]; synchronises */
tr_status tr_matrix_export(tr_ctx* ctx, int32_t seq, int32_t* host_M);              /* HOST [V*k]; synchronises */
int32_t* tr_matrix_device_ptr(tr_ctx* ctx, int32_t seq);                            /* DEVICE, borrowed; NULL on error */

/*
 * Draft tree retrieval (Sec. 3.2, Algorithm 1): for every sequence b, tree[b][0] = root[b] and
 * tree[b][i] = M_b[tree[b][parent[i]]][rank[i]], layer by layer.
 * DEVICE in: d_root[batch].  DEVICE out: d_tree[batch * N] (the merged sequence S per sequence).
 * A root outside [0, V) sets TR_FLAG_BAD_TOKEN and is treated as token 0.
 */
tr_status tr_build_tree(tr_ctx* ctx, const int32_t* d_root, int32_t* d_tree, void* stream);

/*
 * Tree attention (Sec. 2.2): for every sequence b, layer l, query head h and tree node i,
 *   out[b,l,i,h,:] = softmax_j( scale * q[b,l,i,h,:] . k[b,l,g,j,:] ) @ v[b,l,g,j,:],  g = h / (Hq / Hkv),
 * over the keys j in [0, C_b) (the prefix, all visible) and j = C_b + t for tree nodes t that are node i
 * itself or one of its ancestors.  C_b = d_ctx_len[b]; the tree's K/V rows sit right after the prefix.
 * bf16 inputs and output, fp32 accumulation.  Rows j >= C_b + N of the cache are never used, but rows below
 * kv_rows may be fetched and must hold finite numbers.
 *
 * Addressing (strides in ELEMENTS; head_dim is contiguous):
 *   q  : q   + b*q_stride[0]  + l*layer_stride_q  + h*q_stride[1]  + i*q_stride[2]
 *   k,v: k   + b*kv_stride[0] + l*layer_stride_kv + g*kv_stride[1] + j*kv_stride[2]
 *   out: out + b*o_stride[0]  + l*layer_stride_o  + h*o_stride[1]  + i*o_stride[2]
 * All base pointers 16-byte aligned and all strides multiples of 8 elements.
 * n_layers > 1 runs that many independent layers in one launch (layers of a real model are sequential;
 * this is for callers that hold all layers' q already, e.g. benchmarks).
 * The call uses scratch of the context (split-KV partials, a unit counter): calls on one context must not overlap
 * on the device (one stream, or streams ordered by events).
 * Early start (prefix_stable != 0).  A short launch (fewer units than SMs, e.g. one layer of one sequence) is split
 * along the keys and launched so that it may begin while the kernel in front of it on the stream is still draining.
 * By default it touches no global memory until that kernel has finished.  With prefix_stable the caller vouches that
 * d_ctx_len and the cache rows below C_b (the prefix) are NOT written by the kernel directly in front of this call
 * (nor by a kernel that this one let start early before its own inputs were complete): the launch then requests its
 * prefix K/V tiles at once and only q, the tree's K/V rows and the output wait.  True for the usual caller - the
 * kernel in front writes this layer's q and tree rows - and false directly behind tr_commit, which moves rows into
 * the prefix and changes d_ctx_len.  Ignored by launches that are not split.
 * Errors: TR_ERR_INVALID_ARG (NULL, bad head counts, alignment), TR_ERR_UNSUPPORTED (head_dim not 64/128).
 */
typedef struct {
  const void* q;       /* DEVICE bf16 */
  const void* k_cache; /* DEVICE bf16 */
  const void* v_cache; /* DEVICE bf16 */
  void* out;           /* DEVICE bf16 */
  int32_t n_q_heads, n_kv_heads, head_dim;
  const int32_t* d_ctx_len; /* DEVICE [batch] prefix lengths C_b, each <= max_ctx */
  int32_t max_ctx;          /* upper bound of C_b, used for launch sizing */
  int32_t kv_rows;          /* token rows addressable per (b, l, g) slice, >= max_ctx + N */
  int64_t q_stride[3], kv_stride[3], o_stride[3]; /* (sequence, head, token) */
  int32_t n_layers;
  int64_t layer_stride_q, layer_stride_kv, layer_stride_o;
  float scale;    /* 0 -> 1/sqrt(head_dim) */
  int32_t splits; /* 0 -> chosen by the library; >0 forces that many KV splits (testing) */
  int32_t prefix_stable; /* non-zero: see above ("Early start") */
} tr_attn_args;
tr_status tr_tree_attention(tr_ctx* ctx, const tr_attn_args* args, void* stream);

/*
 * Verify, recycle and retrieve (Sec. 2.1 argtopk, Sec. 2.2 verification, Sec. 3.3 update, Algorithm 1):
 *   topk[b,i,:]  = indices of the k largest logits of node i, largest first, equal values by lower index
 *   acceptance   : node c is correct iff parent(c) is correct and tree[c] == topk[parent(c)][0]; the deepest
 *                  correct node wins (lowest layer-order index among equals)
 *   out_tokens   = tokens of the accepted path below the root, then topk[last accepted][0]; n_new = their count
 *   M_b[tree[i]] = topk[i,:] for every node i in increasing i (a repeated token keeps its last row)
 *   next_tree    = tr_build_tree on the updated M_b rooted at the last emitted token (= next_root)
 * DEVICE in : d_logits [batch, N, V] fp32 row-major (no NaN), d_tree [batch, N].
 * DEVICE out: d_topk_idx [batch,N,k], d_n_new [batch], d_acc_nodes [batch, depth_max+1] (unused tail = -1),
 *             d_out_tokens [batch, depth_max+1] (unused tail = -1), d_next_root [batch], d_next_tree [batch,N].
 *             d_next_tree may alias d_tree.  depth_max+1 = tr_max_new_tokens(ctx).
 */
typedef struct {
  int32_t* d_topk_idx;
  int32_t* d_n_new;
  int32_t* d_acc_nodes;
  int32_t* d_out_tokens;
  int32_t* d_next_root;
  int32_t* d_next_tree;
} tr_step_out;
tr_status tr_verify_update(tr_ctx* ctx, const float* d_logits, const int32_t* d_tree, const tr_step_out* out,
                           void* stream);
int32_t tr_max_new_tokens(const tr_ctx* ctx); /* depth of the template + 1 (Appendix: maximum acceptance length) */

/*
 * The same step from a top-k that is already on the device (for example from tr_lm_head_topk): everything
 * tr_verify_update does after its argtopk.  out->d_topk_idx [batch, N, k] is an INPUT here (indices in [0, V),
 * column 0 the argmax); the other members of `out` are written as by tr_verify_update.  An index outside [0, V)
 * sets TR_FLAG_BAD_TOKEN and is treated as token 0 (the matrix never holds an id outside the vocabulary).
 * d_tree and d_topk_idx may have been written by the kernel directly in front on the same stream.
 */
tr_status tr_verify_update_topk(tr_ctx* ctx, const int32_t* d_tree, const tr_step_out* out, void* stream);

/*
 * Verification under temperature sampling (Sec. 5.3 "Temperature Sampling": TR keeps its speed-up at T = 0.3 .. 1.0 and
 * loses a little when drawn tokens fall outside the stored top-k; the paper does not spell the acceptance rule out).
 * Rule implemented ("sample, then match"): every node i draws one token
 *     x_i = argmax_v ( fl32( fl32(logits[i,v] * inv_temperature) + gumbel[i,v] ) ),   lowest v among equal values,
 * which for standard Gumbel noise g = -log(-log(u)) is a draw from softmax(logits[i] / T), T = 1 / inv_temperature
 * (Gumbel-max); a draft child c is correct iff tree[c] == x_parent(c); out_tokens are the accepted drafts followed by
 * the draw of the last accepted node.  Everything else is tr_verify_update: M_b[tree[i]] = argtopk(logits[i]) for
 * every node (the stored candidates are the model's top-k, not the draws), next tree from the updated matrix.
 * The emitted tokens are exactly those of token-by-token sampling with the same noise.  With gumbel == 0 the call
 * equals tr_verify_update.
 * DEVICE in : d_logits, d_gumbel [batch, N, V] fp32 (the noise is the caller's: any generator, one row per node);
 *             inv_temperature > 0 and finite (else TR_ERR_INVALID_ARG); d_tree [batch, N].
 * DEVICE out: as tr_verify_update; d_sampled [batch, N] int32 receives the draws (NULL: kept in the context).
 * Two passes over the logits and one over the noise, side by side in one launch (two clusters per row: top-k and
 * draw); 2 * batch * n_nodes must not exceed 65535 (TR_ERR_UNSUPPORTED).  Allocates nothing, does not synchronise.
 */
tr_status tr_verify_update_sampled(tr_ctx* ctx, const float* d_logits, const float* d_gumbel, float inv_temperature,
                                   const int32_t* d_tree, const tr_step_out* out, int32_t* d_sampled, void* stream);

/*
 * Output layer fused with argtopk (Sec. 2.1: p = M(x), x^0..x^{k-1} = argtopk(p); Sec. 5.4: the forward pass is most of
 * a step).  For the rows = batch * N tree nodes,
 *     logits[r, v] = sum_h hidden[r, h] * weight[v, h]      bf16 inputs, fp32 accumulation on the tensor cores
 *     topk[r, :]   = indices of the k largest logits of row r, largest first, equal values by lower index
 * and the [rows, V] logits are never written to memory: every CTA streams one slice of the weight once and keeps the
 * per-row candidates of its slice; a second small kernel merges the slices.  The comparison is made on the fp32
 * accumulators; their summation order is the hardware's, so two logits closer than fp32 rounding of a length-hidden
 * dot product may come out in either order (inputs whose products and sums are exact give exact results).
 * DEVICE in : d_hidden [rows, hidden_dim] bf16, row stride hidden_stride elements; d_weight [V, hidden_dim] bf16 (the
 *             layout of a linear layer's weight), row stride weight_stride elements.  Both 16-byte aligned, strides
 *             multiples of 8 and >= hidden_dim, hidden_dim a multiple of 8 (else TR_ERR_INVALID_ARG).  No NaN.
 * DEVICE out: d_topk_idx [rows, k] int32; d_topk_val [rows, k] fp32 (the accumulated logits at those indices) or NULL.
 * Rows are processed in groups of 128; the CTAs that work on the same vocabulary slice for different groups run side
 * by side, so the weight is fetched from HBM once and shared through L2.  Allocates nothing, reads nothing back, does
 * not synchronise; uses scratch of the context (not re-entrant per context).
 */
tr_status tr_lm_head_topk(tr_ctx* ctx, const void* d_hidden, int64_t hidden_stride, const void* d_weight,
                          int64_t weight_stride, int32_t hidden_dim, int32_t* d_topk_idx, float* d_topk_val,
                          void* stream);

/*
 * Update-rule variants the paper compares (Sec. 5.2 "Update Strategies" and "Effect of Rejected Tokens"; Appendix
 * "Explanation of Three Update Strategies").  Takes effect for the following tr_verify_update calls.
 *   rule : TR_UPDATE_LAST  (default) - a repeated token keeps the row of its last occurrence
 *          TR_UPDATE_FIRST           - ... of its first occurrence
 *          TR_UPDATE_CUR             - the paper's own uncontrolled update: every occurrence stores its row, one 32-bit
 *                                      element at a time, with nothing ordering the occurrences - each element of a
 *                                      repeated token's row ends up as that element of ONE of its occurrences, and
 *                                      different elements may come from different occurrences; not reproducible
 *                                      from run to run (rows of tokens that occur once are as under the other rules)
 *   scope: TR_UPDATE_ALL_DRAFT (default) - every node of the tree updates its token's row
 *          TR_UPDATE_ONLY_ACCEPTED       - only the nodes of the accepted path do
 */
#define TR_UPDATE_LAST 0
#define TR_UPDATE_FIRST 1
#define TR_UPDATE_CUR 2
#define TR_UPDATE_ALL_DRAFT 0
#define TR_UPDATE_ONLY_ACCEPTED 1
tr_status tr_set_update_rule(tr_ctx* ctx, int32_t rule, int32_t scope);

/*
 * Commit the accepted path (Sec. 5.4: besides the matrix, a step also advances the token list and the KV cache).
 * Call after tr_verify_update with its outputs.  For every sequence b with n = n_new[b] and accepted nodes
 * a_0 = 0 (root), a_1, ..., a_{n-1} (acc_nodes[b]):
 *   K/V : for every layer and KV head, cache row C_b + a_i moves to row C_b + i (i = 1..n-1; the root's row is in
 *         place), so rows [0, C_b + n) are the new prefix in order;
 *   text: out_tokens[b][0..n) (the accepted drafts and the extra greedy token) are appended at
 *         d_tokens[b * token_capacity + n_tokens[b]];
 *   then C_b += n and n_tokens[b] += n.  ctx_len lives on the device, so a captured graph keeps replaying while
 *   the prefix grows (tr_tree_attention reads it there).
 * A sequence for which C_b + n + N > kv_rows or n_tokens[b] + n > token_capacity is left untouched and
 * TR_FLAG_CACHE_FULL is set.
 * DEVICE in/out: k_cache, v_cache (bf16, same addressing as tr_tree_attention), d_ctx_len [batch], d_tokens
 *   [batch, token_capacity] int32, d_n_tokens [batch].  DEVICE in: d_acc_nodes, d_out_tokens [batch, depth_max+1],
 *   d_n_new [batch] as written by tr_verify_update.
 * Errors: TR_ERR_INVALID_ARG (NULL, bad sizes / alignment), TR_ERR_UNSUPPORTED (head_dim not a multiple of 8).
 */
typedef struct {
  void* k_cache; /* DEVICE bf16 */
  void* v_cache; /* DEVICE bf16 */
  int32_t n_kv_heads, head_dim, n_layers, kv_rows;
  int64_t kv_stride[3]; /* (sequence, head, token) in elements */
  int64_t layer_stride_kv;
  int32_t* d_ctx_len;
  int32_t* d_tokens;
  int32_t token_capacity;
  int32_t* d_n_tokens;
} tr_commit_args;
tr_status tr_commit(tr_ctx* ctx, const tr_commit_args* args, const int32_t* d_acc_nodes, const int32_t* d_out_tokens,
                    const int32_t* d_n_new, void* stream);

/* Copies the sticky flag word to HOST and synchronises the device. */
tr_status tr_device_flags(tr_ctx* ctx, uint32_t* host_flags);

/*
 * One whole step from HOST buffers (pinned memory recommended): copies this step's inputs to the device,
 * runs tr_tree_attention over n_layers layers, then tr_verify_update, copies the results back and waits.
 * The prefix K/V (rows [0, C_b)) and the current tree stay resident in device buffers the caller owns.
 * HOST in : h_q [batch, L, N, Hq, D] bf16; h_tree_k / h_tree_v [batch, L, Hkv, N, D] bf16 (this step's tree
 *           rows, written to cache rows C_b..C_b+N-1; h_ctx_len[batch] gives C_b and is copied to a->d_ctx_len, the
 *           device array the attention kernel reads, at the start of the call); h_logits [batch, N, V] fp32.
 * DEVICE  : a->q / a->out must be buffers of that shape (used as staging), a->k_cache / a->v_cache the caches
 *           with kv_stride/layer_stride_kv as described above; d_logits_staging [batch,N,V]; d_tree [batch,N]
 *           current tree (updated in place to the next tree); d_out as in tr_verify_update.
 * HOST out: h_out [batch, L, N, Hq, D] bf16; h_n_new [batch]; h_out_tokens [batch, depth_max+1];
 *           h_next_tree [batch, N].
 * The layers are independent, so the copies are pipelined against the attention launches over groups of layers on
 * two internal copy streams of the context (inputs of group g+1 and outputs of group g-1 move while group g
 * computes); everything is ordered after the work already queued on `stream`, which is synchronised before returning.
 */
typedef struct {
  const void* h_q;
  const void* h_tree_k;
  const void* h_tree_v;
  const float* h_logits;
  const int32_t* h_ctx_len;
  float* d_logits_staging;
  int32_t* d_tree;
  void* h_out;
  int32_t* h_n_new;
  int32_t* h_out_tokens;
  int32_t* h_next_tree;
} tr_host_io;
tr_status tr_step_host(tr_ctx* ctx, const tr_attn_args* a, const tr_step_out* d_out, const tr_host_io* io,
                       void* stream);

/*
 * Top-k without any allocation (the paper has no counterpart; this entry point exists for deployment reasons).
 *
 * Who needs it: code that must not, or cannot, allocate device memory - for example a plug-in inside a serving
 * process whose memory pool already owns all of HBM, so that cudaMalloc fails, or a latency-critical loop that
 * cannot afford the device-wide synchronisation cudaMalloc and cudaFree imply.  tr_init allocates, so these
 * callers cannot hold a context; this function needs none.
 *
 * What it computes: exactly the top-k part of tr_verify_update - for each of `rows` logits rows the indices of the
 * k largest values, largest first, equal values by lower index - with a kernel that cuts every row into segments of
 * 4096 values, keeps per-segment candidate lists in scratch memory and lets the last CTA of a row (a per-row ticket)
 * merge them.  That scratch lives in a fixed 528 KB device array inside the library, held by every GPU that loads the
 * library until the process exits.
 * DEVICE in : d_logits [rows, vocab] fp32 row-major.   DEVICE out: d_topk_idx [rows, k] int32.
 * Limits    : rows <= 4096 and rows * ceil(vocab / 4096) * k <= 65536 (tr_topk_noalloc_limits reports both);
 *             anything larger returns TR_ERR_UNSUPPORTED and launches nothing.  1 <= k <= TR_MAX_K <= vocab.
 * The call allocates nothing and frees nothing; it enqueues one small memset and one kernel on `stream`.
 * First call on a device: it asks the runtime for the device address of the array (once per device, with that
 * device current).  Make this first call outside any stream capture.
 * Sharing  : all calls on a device use the same array.  Calls issued to one stream are safe back to back (the
 * tickets are cleared at the start of each call); calls that may overlap on the GPU (different streams, or
 * different host threads feeding different streams) race on it and must be serialised by the caller.
 */
tr_status tr_topk_noalloc(const float* d_logits, int32_t rows, int32_t vocab, int32_t k, int32_t* d_topk_idx,
                          void* stream);
tr_status tr_topk_noalloc_limits(int32_t* max_rows, int32_t* max_partial_keys); /* HOST out */

#ifdef __cplusplus
}
#endif
#endif /* TR_H_ */
