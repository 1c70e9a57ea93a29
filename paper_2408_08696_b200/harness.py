"""Device-side set-up of a synthetic workload: uploads the seeded inputs, creates the context and drives the
step through the C-ABI binding.  Plumbing only (allocation, copies, launches, CUDA graphs); used by the GPU
tests, the smoke check and the benchmark."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as tr
from . import synth


def bf16_tensor(bits_u16, device):
    """uint16 bit patterns (numpy) -> torch.bfloat16 tensor on `device`."""
    return torch.from_numpy(np.ascontiguousarray(bits_u16).view(np.int16)).to(device).view(torch.bfloat16)


L2_BYTES = 126 << 20


def rotation_larger_than_l2(w: synth.Workload, factor=1.5):
    """Number of rotating logits buffers whose total size exceeds `factor` x the L2 capacity, so that in a loop that
    cycles through them every step's logits come from HBM, not from a warm L2 (at least 4)."""
    per_step = w.batch * w.n_nodes * w.vocab * 4
    n = max(4, -(-int(factor * L2_BYTES) // per_step))
    return n if n <= 64 else 4      # a workload this small lives in L2 whatever is rotated


class DeviceWorkload:
    def __init__(self, w: synth.Workload, n_layers=None, device=0, n_rot=4, with_attention=True, splits=0,
                 zero_matrix=False):
        self.w = w
        self.dev = torch.device("cuda", device)
        self.L = w.n_layers if n_layers is None else n_layers
        self.n_rot = n_rot
        self.parent, self.rank = tr.tr_template_from_branching(w.branching, w.n_nodes)
        self.ctx = tr.tr_init(w.vocab, w.k, self.parent, self.rank, batch=w.batch, device=device)
        B, N, V = w.batch, w.n_nodes, w.vocab
        # --- integer loop state
        self.M0 = np.zeros((B, V, w.k), dtype=np.int32) if zero_matrix else synth.seeded_matrix(w)
        for b in range(B):
            tr.tr_matrix_import(self.ctx, b, self.M0[b])
        self.root0 = synth.root_tokens(w)
        self.succ = synth.zipf_successors(w)
        self.noise = synth.noise_logits(w, n_rot)                       # host copy for the checker's side
        self.d_noise = torch.from_numpy(self.noise).to(self.dev)
        self.d_logits = self.d_noise.clone()                           # [R, B, N, V], patched in place
        self.d_prev_col = torch.full((n_rot, B, N), -1, dtype=torch.int32, device=self.dev)
        self.d_succ = torch.from_numpy(self.succ).to(self.dev)
        self.d_root = torch.from_numpy(self.root0).to(self.dev)
        self.d_tree = torch.zeros(B, N, dtype=torch.int32, device=self.dev)
        self.out_struct, self.out = tr.make_step_out(self.ctx)
        self.out_struct.d_next_tree = self.d_tree.data_ptr()           # next tree replaces the current one
        tr.tr_build_tree(self.ctx, self.d_root, self.d_tree)
        # --- attention state
        self.attn = None
        if with_attention:
            q, k, v = synth.attention_inputs(w, self.L)
            self.q, self.k, self.v = (bf16_tensor(x, self.dev) for x in (q, k, v))
            self.o = torch.zeros_like(self.q)
            self.d_ctx_len = torch.tensor(list(w.ctx), dtype=torch.int32, device=self.dev)
            self.attn = tr.make_attn_args(self.ctx, self.q, self.k, self.v, self.o, self.d_ctx_len, w.max_ctx,
                                          splits=splits)
        torch.cuda.synchronize(self.dev)

    def patch(self, r, stream=None):
        """Toy model: rewrite the tree-dependent entries of rotating logits buffer r for the current tree."""
        tr.trs_patch_logits(self.d_logits[r], self.d_noise[r], self.d_tree, self.d_prev_col[r], self.d_succ,
                            self.w.boost, stream)

    # one whole step: toy-model logits for the current tree, attention over all layers, verify/update/retrieve
    def step(self, i, stream=None):
        r = i % self.n_rot
        self.patch(r, stream)
        if self.attn is not None:
            tr.tr_tree_attention(self.ctx, self.attn, stream)
        tr.tr_verify_update(self.ctx, self.d_logits[r], self.d_tree, self.out_struct, stream)

    def _capture_steps(self, s, side, rots):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for r in rots:
                if self.attn is not None:
                    side.wait_stream(s)
                    self.patch(r, side)
                    tr.tr_tree_attention(self.ctx, self.attn, s)
                    s.wait_stream(side)
                else:
                    self.patch(r, s)
                tr.tr_verify_update(self.ctx, self.d_logits[r], self.d_tree, self.out_struct, s)
        return g

    def capture_graphs(self):
        """One CUDA graph per rotating logits buffer: graph r is one whole step on buffer r.  A step's own kernels form
        a chain - attention, top-k, accept/update/retrieve - and, on a side branch that joins the chain in front of
        the top-k kernel, the toy model patches buffer r for the tree the previous step left (harness work: it
        stands for the rest of the model's forward pass, which produces the logits while the step's attention
        runs).  Every graph reads the current tree, so the graphs may be replayed in any order; the checker follows
        the same order of buffers."""
        s, side = torch.cuda.Stream(self.dev), torch.cuda.Stream(self.dev)
        torch.cuda.synchronize(self.dev)
        with torch.cuda.stream(s):
            graphs = [self._capture_steps(s, side, [r]) for r in range(self.n_rot)]
        torch.cuda.synchronize(self.dev)
        return graphs

    def capture_round(self):
        """One CUDA graph holding n_rot consecutive steps (buffers 0 .. n_rot-1): the steps follow one another
        inside the graph, which spares the launch gap between separate graph launches."""
        s, side = torch.cuda.Stream(self.dev), torch.cuda.Stream(self.dev)
        torch.cuda.synchronize(self.dev)
        with torch.cuda.stream(s):
            g = self._capture_steps(s, side, list(range(self.n_rot)))
        torch.cuda.synchronize(self.dev)
        return g

    def reset(self):
        """Back to the state right after construction (matrices, first tree, un-patched logits), so that a loop can
        be run again from step 0 - for instance to check replayed graphs against the CPU checker."""
        torch.cuda.synchronize(self.dev)
        for b in range(self.w.batch):
            tr.tr_matrix_import(self.ctx, b, self.M0[b])
        self.d_logits.copy_(self.d_noise)
        self.d_prev_col.fill_(-1)
        tr.tr_build_tree(self.ctx, self.d_root, self.d_tree)
        torch.cuda.synchronize(self.dev)

    def kernels_per_step(self):
        n = 3  # logits patch (harness), top-k (one cluster per row), accept/update/retrieve
        if self.attn is not None:
            n += 1
            base = self.w.batch * self.L * self.w.n_q_heads
            if self.attn.splits != 1 and base < 148:
                n += 1  # split-KV combine
        return n

    def snapshot(self):
        torch.cuda.synchronize(self.dev)
        return {k: v.cpu().numpy().copy() for k, v in self.out.items()} | {"tree": self.d_tree.cpu().numpy().copy()}

    def close(self):
        tr.tr_destroy(self.ctx)
