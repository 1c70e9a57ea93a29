"""GPU parity of the output layer fused with argtopk (tr_lm_head_topk) against the CPU oracle.

Small-integer inputs make every product and partial sum exact, so the logits are the same numbers in any
accumulation order: indices and values are then compared bit for bit, ties included.  With normal inputs the fp32
accumulators differ from the float64 logits by rounding; the returned values are compared within the worst-case
bound of a length-`hidden` fp32 summation, and the indices must be exactly the oracle's wherever the oracle's ranking
is decided by more than twice a margin of eight typical rounding errors (elsewhere any order of the near-equal logits
is valid, as long as every rank holds a value that belongs there)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import tr_oracle as orc
from paper_2408_08696_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tr():
    from paper_2408_08696_b200 import build
    build.build()
    from paper_2408_08696_b200 import binding
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return binding


def _bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _run(tr, w, hid_bits, wt_bits, pad=0):
    parent, rank = tr.tr_template_from_branching(w.branching, w.n_nodes)
    ctx = tr.tr_init(w.vocab, w.k, parent, rank, batch=w.batch)
    rows, H = hid_bits.shape
    d_h, d_w = _bf16(hid_bits), _bf16(wt_bits)
    if pad:  # row strides larger than the hidden size
        big_h = torch.zeros(rows, H + pad, dtype=torch.bfloat16, device="cuda")
        big_w = torch.zeros(w.vocab, H + pad, dtype=torch.bfloat16, device="cuda")
        big_h[:, :H] = d_h
        big_w[:, :H] = d_w
        big_h[:, H:] = 7.0   # must not be read
        big_w[:, H:] = 7.0
        d_h, d_w = big_h[:, :H], big_w[:, :H]
    idx = torch.full((rows, w.k), -7, dtype=torch.int32, device="cuda")
    val = torch.zeros(rows, w.k, dtype=torch.float32, device="cuda")
    tr.tr_lm_head_topk(ctx, d_h, d_w, idx, val)
    torch.cuda.synchronize()
    assert tr.tr_device_flags(ctx) == 0
    tr.tr_destroy(ctx)
    return idx.cpu().numpy(), val.cpu().numpy()


def _wl(name="tiny", **kw):
    return dataclasses.replace(synth.WORKLOADS[name], **kw)


CASES = {
    "tiny": (_wl(), None),
    "tiny-k16-hidden200": (_wl(k=16), 200),                          # K tail (hidden % 64 != 0), 16 candidates
    "vocab-1003-ragged": (_wl(vocab=1003), None),                    # last CTA's slice is ragged, V % 16 != 0
    "two-row-groups": (_wl(ctx=(128, 128, 128, 128, 128, 128, 128, 128, 128, 128, 128)), None),  # 165 rows > 128
    "llama3-vocab-chunks": (_wl("llama3-8b", n_q_heads=2, n_kv_heads=2), None),   # 128256 tokens: 4 chunks per CTA
    "llama2-7b": (_wl("llama2-7b"), None),                           # the bench shape: 80 x 4096 x 32000
    "llama2-70b-b8": (_wl("llama2-70b-b8"), None),                   # 640 rows = 5 row groups side by side, hidden 8192
}


@pytest.mark.parametrize("case", list(CASES))
def test_lm_head_small_integers_exact(tr, case):
    w, H = CASES[case]
    hid, wt = synth.lm_head_inputs(w, kind="small-int", hidden_dim=H)
    want_idx, logits = orc.lm_head_topk(synth.bf16_bits_to_f32(hid), synth.bf16_bits_to_f32(wt), w.k)
    idx, val = _run(tr, w, hid, wt)
    assert np.array_equal(idx, want_idx)
    assert np.array_equal(val.astype(np.float64), np.take_along_axis(logits, want_idx, axis=1))


@pytest.mark.parametrize("case", ["tiny", "tiny-k16-hidden200", "llama2-7b"])
def test_lm_head_normal_inputs_within_rounding(tr, case):
    w, H = CASES[case]
    hid, wt = synth.lm_head_inputs(w, hidden_dim=H)
    fh, fw = synth.bf16_bits_to_f32(hid), synth.bf16_bits_to_f32(wt)
    want_idx, logits = orc.lm_head_topk(fh, fw, w.k + 1)
    idx, val = _run(tr, w, hid, wt, pad=8 if case == "tiny" else 0)
    # fp32 summation of `hidden` products, each step rounding (or truncating) a partial sum of at most a few times
    # the largest logit L: every value is within the worst case hidden * 2^-23 * L (checked below), and typically
    # within sqrt(hidden) * 2^-23 * L; eight times that is the margin below which two logits count as undecided.
    L = float(np.abs(logits).max())
    tol = fh.shape[1] * 2.0 ** -23 * L
    margin = 8.0 * np.sqrt(fh.shape[1]) * 2.0 ** -23 * L
    got_logits = np.take_along_axis(logits, idx.astype(np.int64), axis=1)
    assert np.abs(val - got_logits).max() <= tol
    assert np.median(np.abs(val - got_logits)) <= margin / 8
    top = np.take_along_axis(logits, want_idx, axis=1)            # oracle's k+1 best values per row
    decided = 0
    for r in range(idx.shape[0]):
        assert len(set(idx[r])) == w.k
        assert (np.diff(got_logits[r]) <= margin).all()                  # non-increasing up to the margin
        assert (got_logits[r] >= top[r, :w.k] - margin).all()            # each rank holds a value that belongs there
        gaps = np.abs(np.diff(top[r]))                                   # between ranks i and i+1, i < k
        if (gaps > 2 * margin).all():
            assert np.array_equal(idx[r], want_idx[r, :w.k])
            decided += 1
    assert decided >= 0.8 * idx.shape[0]                                 # the margin is not what makes the test pass


def test_lm_head_feeds_the_step(tr):
    """tr_lm_head_topk -> tr_verify_update_topk equals the oracle's step on the oracle's logits."""
    w = _wl()
    hid, wt = synth.lm_head_inputs(w, kind="small-int")
    _, logits = orc.lm_head_topk(synth.bf16_bits_to_f32(hid), synth.bf16_bits_to_f32(wt), w.k)
    parent, rank = tr.tr_template_from_branching(w.branching, w.n_nodes)
    M0 = synth.seeded_matrix(w)
    root = synth.root_tokens(w)
    ctx = tr.tr_init(w.vocab, w.k, parent, rank, batch=w.batch)
    tr.tr_matrix_import(ctx, 0, M0[0])
    d_tree = torch.zeros(w.batch, w.n_nodes, dtype=torch.int32, device="cuda")
    tr.tr_build_tree(ctx, torch.from_numpy(root).cuda(), d_tree)
    out_struct, out = tr.make_step_out(ctx)
    torch.cuda.synchronize()
    S = d_tree.cpu().numpy()[0].astype(np.int64)
    tr.tr_lm_head_topk(ctx, _bf16(hid), _bf16(wt), out["topk_idx"])
    tr.tr_verify_update_topk(ctx, d_tree, out_struct)
    torch.cuda.synchronize()
    assert tr.tr_device_flags(ctx) == 0
    M = M0[0].astype(np.int64).copy()
    res = orc.verify_update(M, S, logits.astype(np.float32), np.asarray(parent), np.asarray(rank))
    assert np.array_equal(tr.tr_matrix_export(ctx, 0), M)
    n_new = int(out["n_new"].cpu()[0])
    assert n_new == res["n_new"]
    assert np.array_equal(out["out_tokens"].cpu().numpy()[0, :n_new], np.asarray(res["out_tokens"]))
    assert np.array_equal(out["next_tree"].cpu().numpy()[0], np.asarray(res["next_tree"]))
    tr.tr_destroy(ctx)


def test_lm_head_argument_errors(tr):
    w = _wl()
    parent, rank = tr.tr_template_from_branching(w.branching, w.n_nodes)
    ctx = tr.tr_init(w.vocab, w.k, parent, rank, batch=w.batch)
    rows = w.batch * w.n_nodes
    idx = torch.zeros(rows, w.k, dtype=torch.int32, device="cuda")
    h = torch.zeros(rows, 132, dtype=torch.bfloat16, device="cuda")      # hidden size not a multiple of 8
    wt = torch.zeros(w.vocab, 132, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tr.TrError):
        tr.tr_lm_head_topk(ctx, h, wt, idx)
    h = torch.zeros(rows, 136, dtype=torch.bfloat16, device="cuda")[:, 4:132]   # base not 16-byte aligned
    wt = torch.zeros(w.vocab, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tr.TrError):
        tr.tr_lm_head_topk(ctx, h, wt, idx)
    tr.tr_destroy(ctx)
