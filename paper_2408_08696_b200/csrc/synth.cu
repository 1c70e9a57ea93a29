// Device half of the synthetic toy model (see tr_synth.h): patches the tree-dependent logits in place.
#include <cuda_runtime.h>
#include "tr_synth.h"

__global__ void trs_patch_kernel(float* __restrict__ logits, const float* __restrict__ noise,
                                 const int32_t* __restrict__ tree, int32_t* __restrict__ prev_col,
                                 const int32_t* __restrict__ succ, float boost, int rows, int V) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the tree comes from the kernel in front (dependent launch)
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
  cudaLaunchConfig_t cfg = {};
  // one warp per CTA: small enough to slip onto an SM beside a resident CTA of a large kernel running concurrently
  cfg.gridDim = dim3((rows + 31) / 32);
  cfg.blockDim = dim3(32);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int r = rows, v = V;
  return static_cast<int32_t>(cudaLaunchKernelEx(&cfg, trs_patch_kernel, d_logits, d_noise, d_tree, d_prev_col, d_succ,
                                                 boost, r, v));
}
