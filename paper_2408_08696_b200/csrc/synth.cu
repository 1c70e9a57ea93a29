// Device half of the synthetic toy model (see tr_synth.h): patches the tree-dependent logits in place.
#include <cuda_runtime.h>
#include "tr_synth.h"

__global__ void trs_patch_kernel(float* __restrict__ logits, const float* __restrict__ noise,
                                 const int32_t* __restrict__ tree, int32_t* __restrict__ prev_col,
                                 const int32_t* __restrict__ succ, float boost, int rows, int V) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const size_t base = static_cast<size_t>(r) * V;
  const int prev = prev_col[r];
  if (prev >= 0) logits[base + prev] = noise[base + prev];
  int tok = tree[r];
  if (tok < 0 || tok >= V) tok = 0;
  const int c = succ[tok];
  logits[base + c] = __fadd_rn(noise[base + c], boost);
  prev_col[r] = c;
}

extern "C" int32_t trs_patch_logits(float* d_logits, const float* d_noise, const int32_t* d_tree,
                                    int32_t* d_prev_col, const int32_t* d_succ, float boost, int32_t rows,
                                    int32_t V, void* stream) {
  trs_patch_kernel<<<(rows + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
      d_logits, d_noise, d_tree, d_prev_col, d_succ, boost, rows, V);
  return static_cast<int32_t>(cudaGetLastError());
}
