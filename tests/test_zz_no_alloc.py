"""The allocation-free top-k entry point, for callers that cannot call cudaMalloc (a process whose memory pool
owns the whole device, or a loop that cannot take cudaMalloc's device-wide synchronisation).  It must give
exactly what the context-based path gives - and what the CPU oracle's argtopk gives - on calls in a row (the scratch
array is shared and keeps the previous call's contents).  Collected last on purpose: a failure here cannot hide
other tests' results."""
import numpy as np
import pytest
import torch

from oracle import tr_oracle as orc

pytestmark = pytest.mark.gpu


def _context_topk(tr, logits, k):
    rows, V = logits.shape
    parent, rank = tr.tr_template_from_branching((1,), rows)
    ctx = tr.tr_init(V, k, parent, rank)
    out_struct, out = tr.make_step_out(ctx)
    tr.tr_verify_update(ctx, torch.from_numpy(logits).cuda().reshape(1, rows, V),
                        torch.zeros(1, rows, dtype=torch.int32, device="cuda"), out_struct)
    torch.cuda.synchronize()
    got = out["topk_idx"].cpu().numpy().reshape(rows, k)
    tr.tr_destroy(ctx)
    return got


def test_no_alloc_topk_matches_context_path_twice_in_a_row():
    from paper_2408_08696_b200 import build
    build.build()
    from paper_2408_08696_b200 import binding as tr
    assert torch.cuda.is_available()
    rng = np.random.default_rng(2024)
    k = 8
    cases = [rng.standard_normal((80, 32000)).astype(np.float32),          # 8 segments per row
             rng.integers(-2, 3, size=(80, 32000)).astype(np.float32),     # same shape, tie-heavy, right after
             rng.standard_normal((33, 4099)).astype(np.float32)]           # ragged vocabulary, fewer rows
    expected = [_context_topk(tr, x, k) for x in cases]
    outs = []
    for x in cases:                                                         # back to back on one stream
        d_x = torch.from_numpy(x).cuda()
        d_out = torch.full((x.shape[0], k), -7, dtype=torch.int32, device="cuda")
        tr.tr_topk_noalloc(d_x, k, d_out)
        outs.append((d_x, d_out))
    torch.cuda.synchronize()
    for (d_x, d_out), exp in zip(outs, expected):
        assert (d_out.cpu().numpy() == exp).all()                          # integer indices: bit-exact
        assert (d_out.cpu().numpy() == orc.argtopk(d_x.cpu().numpy(), k)).all()


def test_no_alloc_rejects_sizes_beyond_the_fixed_scratch():
    from paper_2408_08696_b200 import binding as tr
    max_rows, max_part = tr.tr_topk_noalloc_limits()
    assert (max_rows, max_part) == (4096, 65536)
    d_out = torch.zeros(max_rows + 1, 8, dtype=torch.int32, device="cuda")
    with pytest.raises(tr.TrError) as e:
        tr.tr_topk_noalloc(torch.zeros(max_rows + 1, 64, device="cuda"), 8, d_out)
    assert e.value.status == tr.TR_ERR_UNSUPPORTED and "fixed scratch" in str(e.value)
    with pytest.raises(tr.TrError):                                         # 2048 rows * 5 segments * 8 > 65536
        tr.tr_topk_noalloc(torch.zeros(2048, 4096 * 4 + 1, device="cuda"), 8, d_out[:2048])
