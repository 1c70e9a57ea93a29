// Commit of the accepted path (paper Sec. 5.4: besides the matrix, a step advances the token list and the KV cache): the
// accepted nodes' K/V rows are compacted to the end of the prefix, the confirmed tokens are appended, the prefix
// length grows - all on the device, so the step graph replays without the host.
//
// One CTA per (sequence, layer, KV head).  Moves go in increasing path position with a barrier in between: the
// source of position i is tree row a_i >= i, so it is never one of the rows written for positions < i, while a
// later position may overwrite the source of an earlier one only after that one has been read.
// The CTA that arrives last at a per-sequence ticket - by then every CTA of the sequence has read C_b - appends
// the tokens and advances C_b and the token count.
#include "tr_internal.cuh"

namespace {

struct CommitParams {
  __nv_bfloat16* k;
  __nv_bfloat16* v;
  int Hkv, D, L, kv_rows, N, W;
  int64_t s_b, s_h, s_t, s_l;
  int32_t* ctx_len;
  int32_t* tokens;
  int token_capacity;
  int32_t* n_tokens;
  const int32_t* acc_nodes;
  const int32_t* out_tokens;
  const int32_t* n_new;
  unsigned int* ticket;  // [batch]
  uint32_t* flags;
};

__global__ void __launch_bounds__(64) tr_commit_kernel(const CommitParams p) {
  __shared__ int s_last;
  int u = blockIdx.x;
  const int g = u % p.Hkv; u /= p.Hkv;
  const int layer = u % p.L; u /= p.L;
  const int b = u;
  const int tid = threadIdx.x;
  const int C = p.ctx_len[b];
  const int n = p.n_new[b];
  const int ntok = p.n_tokens[b];
  const bool fits = n >= 1 && n <= p.W && C + n + p.N <= p.kv_rows && ntok + n <= p.token_capacity;
  if (fits) {
    const int chunks = p.D / 8;                // 16-byte chunks per row
    const int which = tid / chunks;            // 0: K, 1: V (threads beyond 2 * chunks idle)
    const int ch = tid % chunks;
    __nv_bfloat16* base = (which == 0 ? p.k : p.v) + b * p.s_b + layer * p.s_l + g * p.s_h;
    for (int i = 1; i < n; ++i) {
      const int a = p.acc_nodes[b * p.W + i];
      if (which < 2 && a != i && a > 0 && a < p.N) {
        const uint4 row = *reinterpret_cast<const uint4*>(base + static_cast<int64_t>(C + a) * p.s_t + ch * 8);
        *reinterpret_cast<uint4*>(base + static_cast<int64_t>(C + i) * p.s_t + ch * 8) = row;
      }
      __syncthreads();
    }
  }
  // ---- ticket: every CTA of the sequence has read C_b and n_tokens[b] before anyone changes them
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(&p.ticket[b], 1u);
    s_last = (t == static_cast<unsigned int>(p.L * p.Hkv - 1));
  }
  __syncthreads();
  if (!s_last) return;
  if (tid == 0) p.ticket[b] = 0u;
  if (!fits) {
    if (tid == 0) atomicOr(p.flags, TR_FLAG_CACHE_FULL);
    return;
  }
  for (int i = tid; i < n; i += blockDim.x)
    p.tokens[static_cast<int64_t>(b) * p.token_capacity + ntok + i] = p.out_tokens[b * p.W + i];
  if (tid == 0) {
    p.ctx_len[b] = C + n;
    p.n_tokens[b] = ntok + n;
  }
}

}  // namespace

tr_status tr_launch_commit(tr_ctx* ctx, const tr_commit_args* a, const int32_t* d_acc_nodes,
                           const int32_t* d_out_tokens, const int32_t* d_n_new, cudaStream_t s) {
  CommitParams p;
  p.k = static_cast<__nv_bfloat16*>(a->k_cache);
  p.v = static_cast<__nv_bfloat16*>(a->v_cache);
  p.Hkv = a->n_kv_heads; p.D = a->head_dim; p.L = a->n_layers; p.kv_rows = a->kv_rows;
  p.N = ctx->n_nodes; p.W = ctx->depth_max + 1;
  p.s_b = a->kv_stride[0]; p.s_h = a->kv_stride[1]; p.s_t = a->kv_stride[2]; p.s_l = a->layer_stride_kv;
  p.ctx_len = a->d_ctx_len; p.tokens = a->d_tokens; p.token_capacity = a->token_capacity; p.n_tokens = a->d_n_tokens;
  p.acc_nodes = d_acc_nodes; p.out_tokens = d_out_tokens; p.n_new = d_n_new;
  p.ticket = ctx->d_seq_ticket;
  p.flags = ctx->d_flags;
  const int64_t blocks = static_cast<int64_t>(ctx->batch) * a->n_layers * a->n_kv_heads;
  if (blocks > (1ll << 30)) return TR_ERR_UNSUPPORTED;
  tr_commit_kernel<<<static_cast<unsigned>(blocks), 64, 0, s>>>(p);
  TR_CUDA_TRY(cudaGetLastError());
  return TR_OK;
}
