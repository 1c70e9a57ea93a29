"""ctypes binding of libtr.so / libtr_synth.so: the same names as include/tr.h, argument marshalling only.

Every function takes PyTorch CUDA tensors (device memory and streams are PyTorch's; all arithmetic runs in
the library's kernels) and raises TrError on a non-zero status.  There is no CPU fallback: if the shared
library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_TR_PATH = os.path.join(_PKG, "libtr.so")
LIB_SYNTH_PATH = os.path.join(_PKG, "libtr_synth.so")

if not os.path.exists(LIB_TR_PATH) or not os.path.exists(LIB_SYNTH_PATH):
    raise ImportError(
        "libtr.so / libtr_synth.so not built: run `python -m paper_2408_08696_b200.build` "
        "(needs nvcc; there is no fallback path)")

lib = C.CDLL(LIB_TR_PATH)
lib_synth = C.CDLL(LIB_SYNTH_PATH)

TR_OK = 0
TR_ERR_INVALID_ARG, TR_ERR_TEMPLATE, TR_ERR_UNSUPPORTED, TR_ERR_CUDA, TR_ERR_NOMEM, TR_ERR_DEVICE_FLAG = -1, -2, -3, -4, -5, -6
TR_FLAG_BAD_TOKEN, TR_FLAG_WAIT_TIMEOUT, TR_FLAG_CACHE_FULL = 1, 2, 4
TR_MAX_NODES, TR_MAX_K = 128, 16
TR_UPDATE_LAST, TR_UPDATE_FIRST, TR_UPDATE_CUR, TR_UPDATE_ALL_DRAFT, TR_UPDATE_ONLY_ACCEPTED = 0, 1, 2, 0, 1
TR_FILL_ZERO, TR_FILL_SEEDED = 0, 1


class TrError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s: status %d (%s)" % (where, status, lib.tr_status_string(status).decode()))


class tr_attn_args(C.Structure):
    _fields_ = [
        ("q", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p), ("out", C.c_void_p),
        ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("d_ctx_len", C.c_void_p), ("max_ctx", C.c_int32), ("kv_rows", C.c_int32),
        ("q_stride", C.c_int64 * 3), ("kv_stride", C.c_int64 * 3), ("o_stride", C.c_int64 * 3),
        ("n_layers", C.c_int32),
        ("layer_stride_q", C.c_int64), ("layer_stride_kv", C.c_int64), ("layer_stride_o", C.c_int64),
        ("scale", C.c_float), ("splits", C.c_int32), ("prefix_stable", C.c_int32),
    ]


class tr_step_out(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("d_topk_idx", "d_n_new", "d_acc_nodes", "d_out_tokens", "d_next_root", "d_next_tree")]


class tr_commit_args(C.Structure):
    _fields_ = [
        ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("n_layers", C.c_int32), ("kv_rows", C.c_int32),
        ("kv_stride", C.c_int64 * 3), ("layer_stride_kv", C.c_int64),
        ("d_ctx_len", C.c_void_p), ("d_tokens", C.c_void_p), ("token_capacity", C.c_int32), ("d_n_tokens", C.c_void_p),
    ]


class tr_host_io(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("h_q", "h_tree_k", "h_tree_v", "h_logits", "h_ctx_len", "d_logits_staging", "d_tree",
                 "h_out", "h_n_new", "h_out_tokens", "h_next_tree")]


_P32 = C.POINTER(C.c_int32)
lib.tr_status_string.restype = C.c_char_p
lib.tr_status_string.argtypes = [C.c_int32]
lib.tr_template_from_branching.argtypes = [_P32, C.c_int32, C.c_int32, _P32, _P32, _P32]
lib.tr_init.argtypes = [C.POINTER(C.c_void_p), C.c_int32, C.c_int32, _P32, _P32, C.c_int32, C.c_int32, C.c_int32]
lib.tr_destroy.argtypes = [C.c_void_p]
lib.tr_matrix_zero.argtypes = [C.c_void_p, C.c_void_p]
lib.tr_matrix_fill.argtypes = [C.c_void_p, C.c_int32, C.c_uint64, C.c_void_p]
lib.tr_matrix_import.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
lib.tr_matrix_export.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
lib.tr_matrix_device_ptr.restype = C.c_void_p
lib.tr_matrix_device_ptr.argtypes = [C.c_void_p, C.c_int32]
lib.tr_build_tree.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.tr_tree_attention.argtypes = [C.c_void_p, C.POINTER(tr_attn_args), C.c_void_p]
lib.tr_verify_update.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(tr_step_out), C.c_void_p]
lib.tr_max_new_tokens.argtypes = [C.c_void_p]
lib.tr_set_update_rule.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
lib.tr_device_flags.argtypes = [C.c_void_p, C.POINTER(C.c_uint32)]
lib.tr_step_host.argtypes = [C.c_void_p, C.POINTER(tr_attn_args), C.POINTER(tr_step_out), C.POINTER(tr_host_io),
                             C.c_void_p]
lib.tr_commit.argtypes = [C.c_void_p, C.POINTER(tr_commit_args), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.tr_topk_noalloc.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
lib.tr_topk_noalloc_limits.argtypes = [_P32, _P32]
lib.tr_verify_update_topk.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(tr_step_out), C.c_void_p]
lib.tr_verify_update_sampled.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p,
                                         C.POINTER(tr_step_out), C.c_void_p, C.c_void_p]
lib.tr_lm_head_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p,
                                C.c_void_p, C.c_void_p]
lib_synth.trs_patch_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                       C.c_int32, C.c_int32, C.c_void_p]


def _check(status, where):
    if status != TR_OK:
        raise TrError(status, where)


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dev(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype):
        raise TypeError("%s must be a CUDA tensor of dtype %s" % (name, dtype))
    return C.c_void_p(t.data_ptr())


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(_P32)


# ---------------------------------------------------------------------------------------------------
def tr_template_from_branching(b, max_nodes):
    """-> (parent, rank) int32 numpy arrays in layer order."""
    b_arr, b_ptr = _i32(b)
    cap = max(1, min(int(max_nodes), TR_MAX_NODES))
    parent = np.zeros(cap, dtype=np.int32)
    rank = np.zeros(cap, dtype=np.int32)
    n = C.c_int32(0)
    _check(lib.tr_template_from_branching(b_ptr, len(b_arr), int(max_nodes), parent.ctypes.data_as(_P32),
                                          rank.ctypes.data_as(_P32), C.byref(n)), "tr_template_from_branching")
    return parent[: n.value].copy(), rank[: n.value].copy()


class Context:
    """Owns a tr_ctx handle; `ctx.handle` is what the tr_* functions take."""

    def __init__(self, handle, vocab, k, n_nodes, batch, device):
        self.handle = C.c_void_p(handle)
        self.vocab, self.k, self.n_nodes, self.batch, self.device = vocab, k, n_nodes, batch, device
        self.max_new = lib.tr_max_new_tokens(self.handle)

    def close(self):
        if self.handle:
            lib.tr_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def tr_init(vocab, k, parent, rank, batch=1, device=0):
    p_arr, p_ptr = _i32(parent)
    r_arr, r_ptr = _i32(rank)
    if len(p_arr) != len(r_arr):
        raise ValueError("parent and rank differ in length")
    h = C.c_void_p()
    _check(lib.tr_init(C.byref(h), vocab, k, p_ptr, r_ptr, len(p_arr), batch, device), "tr_init")
    return Context(h.value, vocab, k, len(p_arr), batch, device)


def tr_destroy(ctx):
    ctx.close()


def tr_matrix_zero(ctx, stream=None):
    _check(lib.tr_matrix_zero(ctx.handle, _stream(stream)), "tr_matrix_zero")


def tr_matrix_fill(ctx, mode, seed=0, stream=None):
    _check(lib.tr_matrix_fill(ctx.handle, int(mode), C.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF), _stream(stream)),
           "tr_matrix_fill")


def tr_matrix_import(ctx, seq, host_M):
    a = np.ascontiguousarray(host_M, dtype=np.int32)
    if a.size != ctx.vocab * ctx.k:
        raise ValueError("host_M must hold V*k entries")
    _check(lib.tr_matrix_import(ctx.handle, seq, a.ctypes.data_as(C.c_void_p)), "tr_matrix_import")


def tr_matrix_export(ctx, seq):
    a = np.empty((ctx.vocab, ctx.k), dtype=np.int32)
    _check(lib.tr_matrix_export(ctx.handle, seq, a.ctypes.data_as(C.c_void_p)), "tr_matrix_export")
    return a


def tr_matrix_device_ptr(ctx, seq):
    return lib.tr_matrix_device_ptr(ctx.handle, seq)


def tr_build_tree(ctx, d_root, d_tree, stream=None):
    _check(lib.tr_build_tree(ctx.handle, _dev(d_root, torch.int32, "d_root"), _dev(d_tree, torch.int32, "d_tree"),
                             _stream(stream)), "tr_build_tree")


def make_attn_args(ctx, q, k_cache, v_cache, out, d_ctx_len, max_ctx, scale=0.0, splits=0, prefix_stable=False):
    """q/out: bf16 [B, L, N, Hq, D]; k_cache/v_cache: bf16 [B, L, Hkv, R, D]; d_ctx_len int32 [B].
    Any strides with a contiguous last dimension are passed through."""
    a = tr_attn_args()
    a.q, a.out = _dev(q, torch.bfloat16, "q"), _dev(out, torch.bfloat16, "out")
    a.k_cache, a.v_cache = _dev(k_cache, torch.bfloat16, "k_cache"), _dev(v_cache, torch.bfloat16, "v_cache")
    a.d_ctx_len = _dev(d_ctx_len, torch.int32, "d_ctx_len")
    B, L, N, Hq, D = q.shape
    Bk, Lk, Hkv, R, Dk = k_cache.shape
    if (Bk, Lk, Dk) != (B, L, D) or v_cache.shape != k_cache.shape or out.shape != q.shape:
        raise ValueError("attention tensor shapes disagree")
    if v_cache.stride() != k_cache.stride() or q.stride(4) != 1 or k_cache.stride(4) != 1 or out.stride(4) != 1:
        raise ValueError("unsupported strides")
    if B != ctx.batch or N != ctx.n_nodes:
        raise ValueError("batch / node count differ from the context")
    a.n_q_heads, a.n_kv_heads, a.head_dim = Hq, Hkv, D
    a.max_ctx, a.kv_rows = int(max_ctx), R
    a.q_stride = (C.c_int64 * 3)(q.stride(0), q.stride(3), q.stride(2))
    a.kv_stride = (C.c_int64 * 3)(k_cache.stride(0), k_cache.stride(2), k_cache.stride(3))
    a.o_stride = (C.c_int64 * 3)(out.stride(0), out.stride(3), out.stride(2))
    a.n_layers = L
    a.layer_stride_q, a.layer_stride_kv, a.layer_stride_o = q.stride(1), k_cache.stride(1), out.stride(1)
    a.scale, a.splits = float(scale), int(splits)
    a.prefix_stable = 1 if prefix_stable else 0
    return a


def tr_tree_attention(ctx, args, stream=None):
    _check(lib.tr_tree_attention(ctx.handle, C.byref(args), _stream(stream)), "tr_tree_attention")


def make_step_out(ctx, device=None):
    """Allocates the int32 output tensors of tr_verify_update; returns (struct, dict of tensors)."""
    dev = torch.device("cuda", ctx.device) if device is None else device
    B, N, k, W = ctx.batch, ctx.n_nodes, ctx.k, ctx.max_new
    t = dict(topk_idx=torch.zeros(B, N, k, dtype=torch.int32, device=dev),
             n_new=torch.zeros(B, dtype=torch.int32, device=dev),
             acc_nodes=torch.zeros(B, W, dtype=torch.int32, device=dev),
             out_tokens=torch.zeros(B, W, dtype=torch.int32, device=dev),
             next_root=torch.zeros(B, dtype=torch.int32, device=dev),
             next_tree=torch.zeros(B, N, dtype=torch.int32, device=dev))
    s = tr_step_out()
    for name in t:
        setattr(s, "d_" + name, C.c_void_p(t[name].data_ptr()))
    return s, t


def tr_verify_update(ctx, d_logits, d_tree, out_struct, stream=None):
    if tuple(d_logits.shape) != (ctx.batch, ctx.n_nodes, ctx.vocab) or not d_logits.is_contiguous():
        raise ValueError("d_logits must be contiguous [batch, N, V]")
    _check(lib.tr_verify_update(ctx.handle, _dev(d_logits, torch.float32, "d_logits"),
                                _dev(d_tree, torch.int32, "d_tree"), C.byref(out_struct), _stream(stream)),
           "tr_verify_update")


def tr_verify_update_sampled(ctx, d_logits, d_gumbel, inv_temperature, d_tree, out_struct, d_sampled=None,
                             stream=None):
    """Verification under temperature sampling: d_gumbel is standard Gumbel noise of the logits' shape."""
    shape = (ctx.batch, ctx.n_nodes, ctx.vocab)
    if tuple(d_logits.shape) != shape or tuple(d_gumbel.shape) != shape or not d_logits.is_contiguous() \
            or not d_gumbel.is_contiguous():
        raise ValueError("d_logits and d_gumbel must be contiguous [batch, N, V]")
    smp = None
    if d_sampled is not None:
        if d_sampled.numel() != ctx.batch * ctx.n_nodes or not d_sampled.is_contiguous():
            raise ValueError("d_sampled must be contiguous with batch*N elements")
        smp = _dev(d_sampled, torch.int32, "d_sampled")
    _check(lib.tr_verify_update_sampled(ctx.handle, _dev(d_logits, torch.float32, "d_logits"),
                                        _dev(d_gumbel, torch.float32, "d_gumbel"), float(inv_temperature),
                                        _dev(d_tree, torch.int32, "d_tree"), C.byref(out_struct), smp,
                                        _stream(stream)), "tr_verify_update_sampled")


def tr_verify_update_topk(ctx, d_tree, out_struct, stream=None):
    """The step from a top-k already in out_struct.d_topk_idx (for example written by tr_lm_head_topk)."""
    _check(lib.tr_verify_update_topk(ctx.handle, _dev(d_tree, torch.int32, "d_tree"), C.byref(out_struct),
                                     _stream(stream)), "tr_verify_update_topk")


def tr_lm_head_topk(ctx, d_hidden, d_weight, d_topk_idx, d_topk_val=None, stream=None):
    """d_hidden bf16 [batch * N, hidden], d_weight bf16 [V, hidden] (inner dimension contiguous);
    d_topk_idx int32 [batch * N, k] (any shape with that many elements), d_topk_val float32 likewise or None."""
    rows = ctx.batch * ctx.n_nodes
    if d_hidden.dim() != 2 or d_weight.dim() != 2 or d_hidden.shape[0] != rows or d_weight.shape[0] != ctx.vocab \
            or d_hidden.shape[1] != d_weight.shape[1] or d_hidden.stride(1) != 1 or d_weight.stride(1) != 1:
        raise ValueError("d_hidden must be [batch*N, hidden] and d_weight [V, hidden], inner dimension contiguous")
    if d_topk_idx.numel() != rows * ctx.k or not d_topk_idx.is_contiguous():
        raise ValueError("d_topk_idx must be contiguous with batch*N*k elements")
    val = None
    if d_topk_val is not None:
        if d_topk_val.numel() != rows * ctx.k or not d_topk_val.is_contiguous():
            raise ValueError("d_topk_val must be contiguous with batch*N*k elements")
        val = _dev(d_topk_val, torch.float32, "d_topk_val")
    _check(lib.tr_lm_head_topk(ctx.handle, _dev(d_hidden, torch.bfloat16, "d_hidden"), d_hidden.stride(0),
                               _dev(d_weight, torch.bfloat16, "d_weight"), d_weight.stride(0), d_hidden.shape[1],
                               _dev(d_topk_idx, torch.int32, "d_topk_idx"), val, _stream(stream)), "tr_lm_head_topk")


def make_commit_args(ctx, k_cache, v_cache, d_ctx_len, d_tokens, d_n_tokens):
    """k_cache/v_cache: bf16 [B, L, Hkv, R, D]; d_ctx_len, d_n_tokens int32 [B]; d_tokens int32 [B, capacity]."""
    a = tr_commit_args()
    a.k_cache, a.v_cache = _dev(k_cache, torch.bfloat16, "k_cache"), _dev(v_cache, torch.bfloat16, "v_cache")
    B, L, Hkv, R, D = k_cache.shape
    if v_cache.shape != k_cache.shape or v_cache.stride() != k_cache.stride() or k_cache.stride(4) != 1:
        raise ValueError("unsupported cache layout")
    if B != ctx.batch or tuple(d_tokens.shape[:1]) != (B,) or not d_tokens.is_contiguous():
        raise ValueError("batch differs from the context")
    a.n_kv_heads, a.head_dim, a.n_layers, a.kv_rows = Hkv, D, L, R
    a.kv_stride = (C.c_int64 * 3)(k_cache.stride(0), k_cache.stride(2), k_cache.stride(3))
    a.layer_stride_kv = k_cache.stride(1)
    a.d_ctx_len = _dev(d_ctx_len, torch.int32, "d_ctx_len")
    a.d_tokens = _dev(d_tokens, torch.int32, "d_tokens")
    a.token_capacity = d_tokens.shape[1]
    a.d_n_tokens = _dev(d_n_tokens, torch.int32, "d_n_tokens")
    return a


def tr_commit(ctx, args, d_acc_nodes, d_out_tokens, d_n_new, stream=None):
    _check(lib.tr_commit(ctx.handle, C.byref(args), _dev(d_acc_nodes, torch.int32, "d_acc_nodes"),
                         _dev(d_out_tokens, torch.int32, "d_out_tokens"), _dev(d_n_new, torch.int32, "d_n_new"),
                         _stream(stream)), "tr_commit")


def tr_set_update_rule(ctx, rule=TR_UPDATE_LAST, scope=TR_UPDATE_ALL_DRAFT):
    _check(lib.tr_set_update_rule(ctx.handle, rule, scope), "tr_set_update_rule")


def tr_device_flags(ctx):
    f = C.c_uint32(0)
    _check(lib.tr_device_flags(ctx.handle, C.byref(f)), "tr_device_flags")
    return f.value


def tr_step_host(ctx, args, out_struct, io, stream=None):
    _check(lib.tr_step_host(ctx.handle, C.byref(args), C.byref(out_struct), C.byref(io), _stream(stream)),
           "tr_step_host")


def tr_topk_noalloc_limits():
    a, b = C.c_int32(0), C.c_int32(0)
    _check(lib.tr_topk_noalloc_limits(C.byref(a), C.byref(b)), "tr_topk_noalloc_limits")
    return a.value, b.value


def tr_topk_noalloc(d_logits, k, d_topk_idx, stream=None):
    """Top-k of every row of d_logits [rows, vocab] (fp32, contiguous) into d_topk_idx [rows, k] (int32) without a
    context and without allocating: for callers that cannot call cudaMalloc.  The first call on a device should
    happen outside stream capture; calls that overlap on the GPU share one scratch array and must be serialised."""
    if d_logits.dim() != 2 or not d_logits.is_contiguous() or tuple(d_topk_idx.shape) != (d_logits.shape[0], k) \
            or not d_topk_idx.is_contiguous():
        raise ValueError("d_logits must be contiguous [rows, vocab] and d_topk_idx contiguous [rows, k]")
    rows, vocab = d_logits.shape
    st = lib.tr_topk_noalloc(_dev(d_logits, torch.float32, "d_logits"), rows, vocab, k,
                             _dev(d_topk_idx, torch.int32, "d_topk_idx"), _stream(stream))
    if st == TR_ERR_UNSUPPORTED:
        mr, mp = tr_topk_noalloc_limits()
        raise TrError(st, "tr_topk_noalloc: beyond the fixed scratch (rows <= %d, rows*segments*k <= %d)" % (mr, mp))
    _check(st, "tr_topk_noalloc")


def trs_patch_logits(d_logits, d_noise, d_tree, d_prev_col, d_succ, boost, stream=None):
    rows = d_tree.numel()
    V = d_logits.shape[-1]
    err = lib_synth.trs_patch_logits(_dev(d_logits, torch.float32, "d_logits"), _dev(d_noise, torch.float32, "d_noise"),
                                     _dev(d_tree, torch.int32, "d_tree"), _dev(d_prev_col, torch.int32, "d_prev_col"),
                                     _dev(d_succ, torch.int32, "d_succ"), float(boost), rows, V, _stream(stream))
    if err:
        raise RuntimeError("trs_patch_logits: cudaError %d" % err)
