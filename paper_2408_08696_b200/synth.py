"""Seeded synthetic inputs shaped like the paper's LLM workloads.

This module only *draws inputs* (random tensors, the toy successor table, the
workload shapes).  It holds none of the method's arithmetic and is the one
module that both the CUDA path's callers and the CPU checker's tests may use.
All draws are numpy (host) so either side can regenerate any slice.

Workloads stand in for the paper's SpecBench / MBPP runs with Vicuna and Code
Llama models (Sec. 4.1): the shapes are those models' attention shapes and
vocabulary sizes; tokens, logits and K/V are synthetic.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    vocab: int
    k: int
    branching: tuple
    n_nodes: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ctx: tuple            # one prefix length per sequence
    boost: float
    steps: int
    seed: int
    zipf_a: float = 1.1

    @property
    def batch(self):
        return len(self.ctx)

    @property
    def max_ctx(self):
        return max(self.ctx)


def _u_ctx(seed, n, lo, hi):
    r = np.random.Generator(np.random.Philox(key=seed))
    return tuple(int(x) for x in r.integers(lo, hi + 1, size=n))


WORKLOADS = {
    "tiny": Workload("tiny", 1000, 8, (4, 2, 1), 15, 1, 4, 4, 64, (128,), 4.0, 50, 0x5EED0000),
    "llama2-7b": Workload("llama2-7b", 32000, 8, (8, 4, 3, 2, 2, 1), 80, 32, 32, 32, 128,
                          (1024,), 3.0, 256, 0x5EED0001),
    "llama2-13b": Workload("llama2-13b", 32000, 8, (8, 4, 3, 2, 2, 1), 80, 40, 40, 40, 128,
                           (4096,), 3.0, 256, 0x5EED0002),
    "llama3-8b": Workload("llama3-8b", 128256, 8, (8, 4, 3, 2, 2, 1), 80, 32, 32, 8, 128,
                          (8192,), 3.0, 256, 0x5EED0003),
    "llama2-70b-b8": Workload("llama2-70b-b8", 32000, 8, (8, 4, 3, 2, 2, 1), 80, 80, 64, 8, 128,
                              _u_ctx(0x5EED0004, 8, 1024, 4096), 3.0, 128, 0x5EED0004),
}


def _rng(seed, stream):
    return np.random.Generator(np.random.Philox(key=[int(seed) & 0xFFFFFFFFFFFFFFFF, int(stream)]))


# ---- bf16 helpers (input preparation only) --------------------------------
def f32_to_bf16_bits(x):
    """Round float32 to bfloat16 (round to nearest even); returns uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b):
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ---- tensors ---------------------------------------------------------------
POOL_LOG2 = 22


def normal_pool(seed):
    """2^22 N(0,1) draws rounded to bf16, as uint16 bits.  Large K/V/Q tensors
    are cut from this pool at seeded offsets (`pool_slice`) so that any
    (sequence, layer, head) slice can be regenerated on the host without
    materialising the whole tensor."""
    x = _rng(seed, 1).standard_normal(1 << POOL_LOG2, dtype=np.float32)
    return f32_to_bf16_bits(x)


def pool_offsets(seed, stream, count, span):
    """`count` seeded start offsets into the pool, each leaving room for `span`
    elements, aligned to 64 elements."""
    hi = ((1 << POOL_LOG2) - span) // 64
    return _rng(seed, stream).integers(0, hi, size=count, dtype=np.int64) * 64


def pool_slice(pool, off, shape):
    n = int(np.prod(shape))
    return pool[off:off + n].reshape(shape)


STREAM_Q, STREAM_K, STREAM_V, STREAM_NOISE, STREAM_SUCC, STREAM_M, STREAM_ROOT = 10, 11, 12, 13, 14, 15, 16
STREAM_HID, STREAM_W, STREAM_GUMBEL = 17, 18, 19


def attention_inputs(w: Workload, n_layers=None, pool=None):
    """bf16 bit patterns (uint16) for one workload:
       q  [B, L, N, Hq, D]
       k  [B, L, Hkv, R, D],  v likewise, R = max_ctx + N; for sequence b the
          prefix is rows 0..ctx[b]-1 and the tree rows follow at ctx[b]...
          Rows past ctx[b] + N are zero.
    """
    L = w.n_layers if n_layers is None else n_layers
    pool = normal_pool(w.seed) if pool is None else pool
    B, N, Hq, Hkv, D = w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim
    R = w.max_ctx + N
    q = np.empty((B, L, N, Hq, D), dtype=np.uint16)
    k = np.zeros((B, L, Hkv, R, D), dtype=np.uint16)
    v = np.zeros((B, L, Hkv, R, D), dtype=np.uint16)
    oq = pool_offsets(w.seed, STREAM_Q, B * L, N * Hq * D).reshape(B, L)
    ok = pool_offsets(w.seed, STREAM_K, B * L * Hkv, R * D).reshape(B, L, Hkv)
    ov = pool_offsets(w.seed, STREAM_V, B * L * Hkv, R * D).reshape(B, L, Hkv)
    for b in range(B):
        rows = w.ctx[b] + N
        for l in range(L):
            q[b, l] = pool_slice(pool, oq[b, l], (N, Hq, D))
            for g in range(Hkv):
                k[b, l, g, :rows] = pool_slice(pool, ok[b, l, g], (rows, D))
                v[b, l, g, :rows] = pool_slice(pool, ov[b, l, g], (rows, D))
    return q, k, v


def attention_slice(w: Workload, pool, b, l, g):
    """(k, v) uint16 [ctx[b] + N, D] of one (sequence, layer, kv head) and
    q uint16 [N, Hq, D] of that (sequence, layer): the same values
    `attention_inputs` produces, regenerated without the full tensors."""
    B, N, Hq, Hkv, D = w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim
    L = w.n_layers
    R = w.max_ctx + N
    rows = w.ctx[b] + N
    oq = pool_offsets(w.seed, STREAM_Q, B * L, N * Hq * D).reshape(B, L)
    ok = pool_offsets(w.seed, STREAM_K, B * L * Hkv, R * D).reshape(B, L, Hkv)
    ov = pool_offsets(w.seed, STREAM_V, B * L * Hkv, R * D).reshape(B, L, Hkv)
    return (pool_slice(pool, oq[b, l], (N, Hq, D)),
            pool_slice(pool, ok[b, l, g], (rows, D)),
            pool_slice(pool, ov[b, l, g], (rows, D)))


def lm_head_inputs(w: Workload, kind="normal", hidden_dim=None):
    """bf16 bit patterns (uint16) of the last hidden states [B * N, hidden] and of the output layer's weight
    [V, hidden], hidden = n_q_heads * head_dim unless given.
      kind "normal": independent N(0,1) draws, rounded to bf16;
      kind "small-int": integers in [-3, 3] (hidden states in [-2, 2]): every product and partial sum is a small
        integer, so the logits are exact in any accumulation order and full of ties."""
    H = w.n_q_heads * w.head_dim if hidden_dim is None else hidden_dim
    rows = w.batch * w.n_nodes
    if kind == "small-int":
        hid = _rng(w.seed, STREAM_HID).integers(-2, 3, size=(rows, H)).astype(np.float32)
        wt = _rng(w.seed, STREAM_W).integers(-3, 4, size=(w.vocab, H)).astype(np.float32)
    else:
        hid = _rng(w.seed, STREAM_HID).standard_normal((rows, H), dtype=np.float32)
        wt = _rng(w.seed, STREAM_W).standard_normal((w.vocab, H), dtype=np.float32)
    return f32_to_bf16_bits(hid), f32_to_bf16_bits(wt)


def noise_logits(w: Workload, n_rot=4):
    """float32 [n_rot, B, N, V] N(0,1) noise matrices that rotate over steps."""
    return _rng(w.seed, STREAM_NOISE).standard_normal(
        (n_rot, w.batch, w.n_nodes, w.vocab), dtype=np.float32)


def gumbel_noise(w: Workload, n_rot=4):
    """float32 [n_rot, B, N, V] standard Gumbel draws g = -log(-log(u)), u uniform in (0, 1): the random numbers of
    temperature sampling, rotating over steps like the noise logits."""
    u = _rng(w.seed, STREAM_GUMBEL).random((n_rot, w.batch, w.n_nodes, w.vocab), dtype=np.float32)
    u = np.clip(u, np.float32(1e-20), np.float32(1.0 - 2.0 ** -24))
    return (-np.log(-np.log(u.astype(np.float64)))).astype(np.float32)


def zipf_successors(w: Workload):
    """succ[t]: the toy model's preferred successor of token t.  Ranks are drawn
    from Zipf(a) truncated to [1, V] by inverse CDF in float64; id = rank - 1."""
    ranks = np.arange(1, w.vocab + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-w.zipf_a))
    cdf /= cdf[-1]
    u = _rng(w.seed, STREAM_SUCC).random(w.vocab)
    return np.minimum(np.searchsorted(cdf, u, side="left"), w.vocab - 1).astype(np.int32)


def seeded_matrix(w: Workload):
    """int32 [B, V, k] adjacency matrices filled with uniform token ids."""
    return _rng(w.seed, STREAM_M).integers(0, w.vocab, size=(w.batch, w.vocab, w.k), dtype=np.int32)


def root_tokens(w: Workload):
    return _rng(w.seed, STREAM_ROOT).integers(0, w.vocab, size=(w.batch,), dtype=np.int32)


def step_logits(noise, S, succ, boost):
    """Toy model output for one sequence: a copy of `noise` [N, V] with `boost`
    added (one float32 add) at column succ[S[i]] of row i."""
    out = np.array(noise, dtype=np.float32, copy=True)
    rows = np.arange(out.shape[0])
    cols = succ[np.asarray(S)]
    out[rows, cols] = out[rows, cols] + np.float32(boost)
    return out
