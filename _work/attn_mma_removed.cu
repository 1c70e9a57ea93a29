// Tree attention (paper Sec. 2.2), warp-level tensor-core version: split-KV flash-decoding over the prefix
// K/V with the tree's ancestor mask applied to the trailing N keys.
//
// One CTA per (sequence, layer, query head, KV split); warp w owns query rows 16w..16w+15 (N <= 128 -> <= 8
// warps).  K/V tiles of 64 keys are double-buffered in shared memory with cp.async (rows past C+N are
// zero-filled, never fetched), 16-byte chunks XOR-swizzled so ldmatrix is conflict-free.  QK^T and PV use
// mma.sync.m16n8k16 bf16 with fp32 accumulation and an online softmax in the exp2 domain.  The ancestor
// bitmask of each thread's two rows stays in registers.  With more than one split the unnormalised partial
// output and its (max, sum) go to scratch and a small combine kernel finishes the softmax.
#include "tr_internal.cuh"

namespace {

constexpr int BN = 64;  // keys per tile

struct AttnParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  __nv_bfloat16* out;
  const int32_t* ctx_len;
  const uint32_t* anc;
  float* part_o;
  float* part_ml;
  int N, Hq, Hkv, L, S;
  int64_t qs_b, qs_h, qs_t, qs_l;
  int64_t ks_b, ks_h, ks_t, ks_l;
  int64_t os_b, os_h, os_t, os_l;
  float scale_log2;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

template <int D>
__device__ __forceinline__ void load_tile(const __nv_bfloat16* __restrict__ g, int64_t row_stride, int row0,
                                          int rows_valid_end, __nv_bfloat16* s, int tid, int nthreads) {
  constexpr int CH = D / 8;  // 16-byte chunks per row
  for (int c = tid; c < BN * CH; c += nthreads) {
    const int r = c / CH, ch = c % CH;
    const int grow = row0 + r;
    const bool ok = grow < rows_valid_end;
    const __nv_bfloat16* src = g + static_cast<int64_t>(ok ? grow : 0) * row_stride + ch * 8;
    cp_async16(smem_u32(s + r * D + ((ch ^ (r & 7)) * 8)), src, ok ? 16 : 0);
  }
}

template <int D>
__global__ void __launch_bounds__(256) tr_attn_mma_kernel(const AttnParams p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __nv_bfloat16* sK = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [2][BN][D]
  __nv_bfloat16* sV = sK + 2 * BN * D;                             // [2][BN][D]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x;
  const int g = lane >> 2, t = lane & 3;
  const int group = p.Hq / p.Hkv;
  int u = blockIdx.x;
  const int gq = u % group;  u /= group;
  const int split = u % p.S; u /= p.S;
  const int kvh = u % p.Hkv; u /= p.Hkv;
  const int layer = u % p.L; u /= p.L;
  const int b = u;
  const int h = kvh * group + gq;

  const int C = p.ctx_len[b];
  const int n_keys = C + p.N;
  const int T = (n_keys + BN - 1) / BN;
  const int t0 = static_cast<int>(static_cast<int64_t>(T) * split / p.S);
  const int t1 = static_cast<int>(static_cast<int64_t>(T) * (split + 1) / p.S);

  const __nv_bfloat16* qp = p.q + b * p.qs_b + layer * p.qs_l + h * p.qs_h;
  const __nv_bfloat16* kp = p.k + b * p.ks_b + layer * p.ks_l + kvh * p.ks_h;
  const __nv_bfloat16* vp = p.v + b * p.ks_b + layer * p.ks_l + kvh * p.ks_h;

  const int r_lo = warp * 16 + g, r_hi = r_lo + 8;
  // Q fragments (A operand) straight from global memory; rows past N read as zero
  uint32_t qf[D / 16][4];
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const int c = ks * 16 + 2 * t;
    qf[ks][0] = r_lo < p.N ? *reinterpret_cast<const uint32_t*>(qp + r_lo * p.qs_t + c) : 0u;
    qf[ks][1] = r_hi < p.N ? *reinterpret_cast<const uint32_t*>(qp + r_hi * p.qs_t + c) : 0u;
    qf[ks][2] = r_lo < p.N ? *reinterpret_cast<const uint32_t*>(qp + r_lo * p.qs_t + c + 8) : 0u;
    qf[ks][3] = r_hi < p.N ? *reinterpret_cast<const uint32_t*>(qp + r_hi * p.qs_t + c + 8) : 0u;
  }
  uint32_t anc_lo[4], anc_hi[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    anc_lo[w] = r_lo < p.N ? p.anc[r_lo * 4 + w] : 0u;
    anc_hi[w] = r_hi < p.N ? p.anc[r_hi * 4 + w] : 0u;
  }

  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  if (t0 < t1) {
    load_tile<D>(kp, p.ks_t, t0 * BN, n_keys, sK, tid, nthreads);
    load_tile<D>(vp, p.ks_t, t0 * BN, n_keys, sV, tid, nthreads);
  }
  cp_async_commit();

  for (int tile = t0; tile < t1; ++tile) {
    const int buf = (tile - t0) & 1;
    if (tile + 1 < t1) {
      load_tile<D>(kp, p.ks_t, (tile + 1) * BN, n_keys, sK + (buf ^ 1) * BN * D, tid, nthreads);
      load_tile<D>(vp, p.ks_t, (tile + 1) * BN, n_keys, sV + (buf ^ 1) * BN * D, tid, nthreads);
    }
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    const uint32_t kb = smem_u32(sK + buf * BN * D), vb = smem_u32(sV + buf * BN * D);

    // ---- S = Q K^T
    float s[BN / 8][4];
#pragma unroll
    for (int i = 0; i < BN / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
    {
      const int m = lane >> 3;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
        for (int np = 0; np < BN / 16; ++np) {
          const int row = np * 16 + (m >> 1) * 8 + (lane & 7);
          const int ch = ks * 2 + (m & 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(kb + (row * D + ((ch ^ (row & 7)) * 8)) * 2, b0, b1, b2, b3);
          mma_bf16(s[2 * np], qf[ks], b0, b1);
          mma_bf16(s[2 * np + 1], qf[ks], b2, b3);
        }
      }
    }
    // ---- scale, mask, online softmax
    const int key0 = tile * BN;
    const bool need_mask = key0 + BN > C;
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float x = s[nt][e] * p.scale_log2;
        if (need_mask) {
          const int key = key0 + nt * 8 + 2 * t + (e & 1);
          const int j = key - C;
          if (j >= 0) {
            const int jw = j >> 5;  // explicit selects keep the mask words in registers
            const uint32_t wl = jw == 0 ? anc_lo[0] : jw == 1 ? anc_lo[1] : jw == 2 ? anc_lo[2] : anc_lo[3];
            const uint32_t wh = jw == 0 ? anc_hi[0] : jw == 1 ? anc_hi[1] : jw == 2 ? anc_hi[2] : anc_hi[3];
            const bool vis = (j < p.N) && ((((e < 2) ? wl : wh) >> (j & 31)) & 1u);
            if (!vis) x = -INFINITY;
          }
        }
        s[nt][e] = x;
        if (e < 2) mx_lo = fmaxf(mx_lo, x); else mx_hi = fmaxf(mx_hi, x);
      }
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xFFFFFFFFu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xFFFFFFFFu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xFFFFFFFFu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xFFFFFFFFu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float sub_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, sub_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
    const float al_lo = exp2f(m_lo - sub_lo), al_hi = exp2f(m_hi - sub_hi);  // exp2(-inf) = 0 on first tile
    m_lo = mn_lo; m_hi = mn_hi;
    float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
    for (int nt = 0; nt < BN / 8; ++nt) {
      s[nt][0] = exp2f(s[nt][0] - sub_lo); s[nt][1] = exp2f(s[nt][1] - sub_lo);
      s[nt][2] = exp2f(s[nt][2] - sub_hi); s[nt][3] = exp2f(s[nt][3] - sub_hi);
      sum_lo += s[nt][0] + s[nt][1];
      sum_hi += s[nt][2] + s[nt][3];
    }
    l_lo = l_lo * al_lo + sum_lo;
    l_hi = l_hi * al_hi + sum_hi;
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
      o[i][0] *= al_lo; o[i][1] *= al_lo; o[i][2] *= al_hi; o[i][3] *= al_hi;
    }
    // ---- O += P V
    {
      const int m = lane >> 3;
#pragma unroll
      for (int kk = 0; kk < BN / 16; ++kk) {
        uint32_t pa[4];
        pa[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
        pa[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
        pa[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
        pa[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
        for (int dp = 0; dp < D / 16; ++dp) {
          const int row = kk * 16 + (m & 1) * 8 + (lane & 7);
          const int ch = dp * 2 + (m >> 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_trans(vb + (row * D + ((ch ^ (row & 7)) * 8)) * 2, b0, b1, b2, b3);
          mma_bf16(o[2 * dp], pa, b0, b1);
          mma_bf16(o[2 * dp + 1], pa, b2, b3);
        }
      }
    }
    __syncthreads();  // everyone is done with `buf` before the next iteration refills it
  }
  cp_async_wait<0>();

  l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 2);

  if (p.S == 1) {
    __nv_bfloat16* op = p.out + b * p.os_b + layer * p.os_l + h * p.os_h;
    const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;  // every real row sees at least its own key
#pragma unroll
    for (int nt = 0; nt < D / 8; ++nt) {
      const int c = nt * 8 + 2 * t;
      if (r_lo < p.N)
        *reinterpret_cast<__nv_bfloat162*>(op + r_lo * p.os_t + c) = __floats2bfloat162_rn(o[nt][0] * inv_lo, o[nt][1] * inv_lo);
      if (r_hi < p.N)
        *reinterpret_cast<__nv_bfloat162*>(op + r_hi * p.os_t + c) = __floats2bfloat162_rn(o[nt][2] * inv_hi, o[nt][3] * inv_hi);
    }
  } else {
    const size_t slot = blockIdx.x;
    float* po = p.part_o + slot * ATTN_PART_ROWS * 128;
    float* pml = p.part_ml + slot * ATTN_PART_ROWS * 2;
#pragma unroll
    for (int nt = 0; nt < D / 8; ++nt) {
      const int c = nt * 8 + 2 * t;
      if (r_lo < p.N) *reinterpret_cast<float2*>(po + r_lo * 128 + c) = make_float2(o[nt][0], o[nt][1]);
      if (r_hi < p.N) *reinterpret_cast<float2*>(po + r_hi * 128 + c) = make_float2(o[nt][2], o[nt][3]);
    }
    if (t == 0) {
      if (r_lo < p.N) { pml[r_lo * 2] = m_lo; pml[r_lo * 2 + 1] = l_lo; }
      if (r_hi < p.N) { pml[r_hi * 2] = m_hi; pml[r_hi * 2 + 1] = l_hi; }
    }
  }
}

// Merge the per-split partial softmaxes: out = sum_s 2^(m_s - m*) O_s / sum_s 2^(m_s - m*) l_s.
// One CTA per (8 tree nodes, query-head unit): 32 lanes x float4 cover the 128 (or 64) dims of a row.
constexpr int COMBINE_ROWS = 8;
__global__ void __launch_bounds__(COMBINE_ROWS * 32) tr_attn_combine_kernel(const AttnParams p, int D) {
  const int row = blockIdx.x * COMBINE_ROWS + (threadIdx.x >> 5);  // tree node
  const int d = (threadIdx.x & 31) * 4;
  if (row >= p.N || d >= D) return;
  int u = blockIdx.y;           // (b, layer, kv head, q-in-group)
  const int group = p.Hq / p.Hkv;
  const int gq = u % group;
  const int blg = u / group;
  const int kvh = blg % p.Hkv;
  const int layer = (blg / p.Hkv) % p.L;
  const int b = blg / (p.Hkv * p.L);
  const int h = kvh * group + gq;
  float mstar = -INFINITY;
  for (int s = 0; s < p.S; ++s) {
    const size_t slot = (static_cast<size_t>(blg) * p.S + s) * group + gq;
    mstar = fmaxf(mstar, p.part_ml[(slot * ATTN_PART_ROWS + row) * 2]);
  }
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float den = 0.f;
  for (int s = 0; s < p.S; ++s) {
    const size_t slot = (static_cast<size_t>(blg) * p.S + s) * group + gq;
    const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + (slot * ATTN_PART_ROWS + row) * 2);
    const float w = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - mstar);
    const float4 o = *reinterpret_cast<const float4*>(p.part_o + (slot * ATTN_PART_ROWS + row) * 128 + d);
    acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
    den += w * ml.y;
  }
  const float inv = 1.f / den;
  __nv_bfloat16* op = p.out + b * p.os_b + layer * p.os_l + h * p.os_h + row * p.os_t + d;
  __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
  uint2 w2;
  w2.x = *reinterpret_cast<uint32_t*>(&lo);
  w2.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(op) = w2;
}

}  // namespace

// `fill_once`: the caller is a persistent one-CTA-per-SM kernel, so the split count is chosen to give every SM at
// most one unit (no second, partly filled round); otherwise about two CTAs' worth of units per SM.
int tr_attention_pick_splits(const tr_ctx* ctx, const tr_attn_args* a, int base_units, int tile_keys, bool fill_once) {
  const int tiles = (a->max_ctx + ctx->n_nodes + tile_keys - 1) / tile_keys;
  int S = a->splits;
  if (S <= 0) {
    if (fill_once) {
      S = base_units >= ctx->sm_count ? 1 : ctx->sm_count / base_units;
    } else {
      const int want = 2 * ctx->sm_count;
      S = base_units >= want ? 1 : (want + base_units - 1) / base_units;
    }
    if (S > 16) S = 16;
  }
  if (S > tiles) S = tiles;
  while (S > 1 && static_cast<int64_t>(base_units) * S > ATTN_MAX_PART_SLOTS) --S;
  return S < 1 ? 1 : S;
}

// Opt in to the shared memory the kernels need; once per device, from tr_init (not a stream operation).
tr_status tr_attention_mma_setup() {
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   4 * BN * 128 * (int)sizeof(__nv_bfloat16)));
  TR_CUDA_TRY(cudaFuncSetAttribute(tr_attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   4 * BN * 64 * (int)sizeof(__nv_bfloat16)));
  return TR_OK;
}

static AttnParams make_params(tr_ctx* ctx, const tr_attn_args* a);

// Split-KV merge for either attention kernel (both write the same partial format).
void tr_launch_attention_combine(tr_ctx* ctx, const tr_attn_args* a, int S, cudaStream_t s) {
  AttnParams p = make_params(ctx, a);
  p.S = S;
  const unsigned base = static_cast<unsigned>(ctx->batch) * a->n_layers * a->n_q_heads;
  tr_attn_combine_kernel<<<dim3((ctx->n_nodes + COMBINE_ROWS - 1) / COMBINE_ROWS, base), COMBINE_ROWS * 32, 0, s>>>(
      p, a->head_dim);
}

static AttnParams make_params(tr_ctx* ctx, const tr_attn_args* a) {
  AttnParams p;
  p.q = static_cast<const __nv_bfloat16*>(a->q);
  p.k = static_cast<const __nv_bfloat16*>(a->k_cache);
  p.v = static_cast<const __nv_bfloat16*>(a->v_cache);
  p.out = static_cast<__nv_bfloat16*>(a->out);
  p.ctx_len = a->d_ctx_len;
  p.anc = ctx->d_anc;
  p.part_o = ctx->d_attn_part_o;
  p.part_ml = ctx->d_attn_part_ml;
  p.N = ctx->n_nodes; p.Hq = a->n_q_heads; p.Hkv = a->n_kv_heads; p.L = a->n_layers;
  p.qs_b = a->q_stride[0]; p.qs_h = a->q_stride[1]; p.qs_t = a->q_stride[2]; p.qs_l = a->layer_stride_q;
  p.ks_b = a->kv_stride[0]; p.ks_h = a->kv_stride[1]; p.ks_t = a->kv_stride[2]; p.ks_l = a->layer_stride_kv;
  p.os_b = a->o_stride[0]; p.os_h = a->o_stride[1]; p.os_t = a->o_stride[2]; p.os_l = a->layer_stride_o;
  const float scale = a->scale != 0.f ? a->scale : 1.0f / sqrtf(static_cast<float>(a->head_dim));
  p.scale_log2 = scale * 1.4426950408889634f;
  p.S = 1;
  return p;
}

tr_status tr_launch_attention_mma(tr_ctx* ctx, const tr_attn_args* a, cudaStream_t s) {
  AttnParams p = make_params(ctx, a);
  const int64_t base = static_cast<int64_t>(ctx->batch) * a->n_layers * a->n_q_heads;
  if (base > (1 << 30)) return TR_ERR_UNSUPPORTED;
  p.S = tr_attention_pick_splits(ctx, a, static_cast<int>(base), BN, false);
  if (p.S > 1 && base * p.S > ATTN_MAX_PART_SLOTS) return TR_ERR_UNSUPPORTED;
  const int nwarps = (ctx->n_nodes + 15) / 16;
  const int D = a->head_dim;
  const size_t smem = static_cast<size_t>(4) * BN * D * sizeof(__nv_bfloat16);
  const dim3 grid(static_cast<unsigned>(base * p.S));
  if (D == 128)
    tr_attn_mma_kernel<128><<<grid, nwarps * 32, smem, s>>>(p);
  else
    tr_attn_mma_kernel<64><<<grid, nwarps * 32, smem, s>>>(p);
  TR_CUDA_TRY(cudaGetLastError());
  if (p.S > 1) {
    tr_launch_attention_combine(ctx, a, p.S, s);
    TR_CUDA_TRY(cudaGetLastError());
  }
  return TR_OK;
}
