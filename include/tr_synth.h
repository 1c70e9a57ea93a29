/*
 * tr_synth.h - device side of the synthetic "toy model" used by the tests and the benchmark (libtr_synth.so).
 * It is an input generator, not part of the Token Recycling step: it only rewrites, on the device, the few
 * logits that depend on the current tree so that a multi-step loop can run without host round trips.
 * The paper has no counterpart (its logits come from a real LLM, Sec. 4.1).
 */
#ifndef TR_SYNTH_H_
#define TR_SYNTH_H_
#include <stdint.h>
#ifdef __cplusplus
extern "C" {
#endif
/*
 * For every row r (one tree node of one sequence; rows = batch * N):
 *   if prev_col[r] >= 0: logits[r, prev_col[r]] = noise[r, prev_col[r]]          (undo the last boost)
 *   c = succ[tree[r]];   logits[r, c] = noise[r, c] + boost;   prev_col[r] = c   (one fp32 add)
 * DEVICE: logits, noise [rows, V] fp32 (logits initially a copy of noise); tree [rows] int32 token ids in [0, V);
 * prev_col [rows] int32 (initialise to -1); succ [V] int32.  Returns 0, or a cudaError_t value.
 */
int32_t trs_patch_logits(float* d_logits, const float* d_noise, const int32_t* d_tree, int32_t* d_prev_col,
                         const int32_t* d_succ, float boost, int32_t rows, int32_t V, void* stream);
#ifdef __cplusplus
}
#endif
#endif
