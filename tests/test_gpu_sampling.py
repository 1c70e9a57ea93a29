"""GPU parity of verification under temperature sampling (tr_verify_update_sampled) against the CPU oracle: the draw
is an argmax of float32 multiply-then-add results, so every integer output is compared bit for bit."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import tr_oracle as orc
from paper_2408_08696_b200 import synth
from tests.oracle_loop import OracleLoop, compare_step

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tr():
    from paper_2408_08696_b200 import build
    build.build()
    from paper_2408_08696_b200 import binding
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return binding


@pytest.fixture(scope="module")
def harness(tr):
    from paper_2408_08696_b200 import harness
    return harness


def _loop(harness, tr, w, steps, temperature, zero_noise=False):
    dw = harness.DeviceWorkload(w, with_attention=False)
    ol = OracleLoop(w)
    g = synth.gumbel_noise(w, dw.n_rot)
    if zero_noise:
        g[:] = 0
    d_g = torch.from_numpy(g).to(dw.dev)
    d_x = torch.full((w.batch, w.n_nodes), -1, dtype=torch.int32, device=dw.dev)
    inv_t = np.float32(1.0 / temperature)
    mats = []
    for i in range(steps):
        r = i % dw.n_rot
        dw.patch(r)
        tr.tr_verify_update_sampled(dw.ctx, dw.d_logits[r], d_g[r], float(inv_t), dw.d_tree, dw.out_struct, d_x)
        snap = dw.snapshot()
        drawn = d_x.cpu().numpy()
        recs = []
        for b in range(w.batch):
            logits = synth.step_logits(ol.noise[r, b], ol.S[b], ol.succ, w.boost)
            rec = orc.verify_update_sampled(ol.M[b], ol.S[b], logits, g[r, b], inv_t, ol.parent, ol.rank)
            assert np.array_equal(drawn[b], rec["sampled"]), "draws differ (seq %d, step %d)" % (b, i)
            ol.S[b] = rec["next_tree"]
            recs.append(rec)
        compare_step(recs, snap, dw.ctx.max_new)
        mats.append(np.mean([rec["n_new"] for rec in recs]))
    for b in range(w.batch):
        assert (tr.tr_matrix_export(dw.ctx, b) == ol.M[b]).all(), "matrix differs after the loop"
    assert tr.tr_device_flags(dw.ctx) == 0
    dw.close()
    return float(np.mean(mats))


@pytest.mark.parametrize("temperature", [0.3, 0.7, 1.0])
def test_sampled_loop_tiny(harness, tr, temperature):
    mat = _loop(harness, tr, synth.WORKLOADS["tiny"], 30, temperature)
    assert 1.0 <= mat <= 4.0


def test_sampled_loop_llama2_7b_shape_and_batch(harness, tr):
    _loop(harness, tr, synth.WORKLOADS["llama2-7b"], 8, 0.7)
    _loop(harness, tr, dataclasses.replace(synth.WORKLOADS["tiny"], ctx=(128, 128, 128), vocab=1003), 10, 1.0)  # scalar loads


def test_sampling_without_noise_is_greedy_verification(harness, tr):
    """gumbel == 0: the draw is the argmax at any temperature, so the step equals tr_verify_update's."""
    w = synth.WORKLOADS["tiny"]
    mat_s = _loop(harness, tr, w, 20, 0.5, zero_noise=True)
    dw = harness.DeviceWorkload(w, with_attention=False)
    ol = OracleLoop(w)
    mats = []
    for i in range(20):
        dw.step(i)
        recs = ol.step(i)
        compare_step(recs, dw.snapshot(), dw.ctx.max_new)
        mats.append(np.mean([rec["n_new"] for rec in recs]))
    dw.close()
    assert mat_s == float(np.mean(mats))


def test_sampling_argument_errors(harness, tr):
    w = synth.WORKLOADS["tiny"]
    dw = harness.DeviceWorkload(w, with_attention=False)
    d_g = torch.zeros_like(dw.d_logits[0])
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(tr.TrError):
            tr.tr_verify_update_sampled(dw.ctx, dw.d_logits[0], d_g, bad, dw.d_tree, dw.out_struct)
    dw.close()


def test_sampling_rejects_more_rows_than_one_launch_can_hold(tr):
    """The top-k and the draw of a row are two clusters of one launch: 2 * batch * N must fit into the grid's second
    dimension.  A batch that tr_init accepts (batch * N <= 65535) but that is too large for the sampled call gets
    TR_ERR_UNSUPPORTED before anything is launched; the greedy call still works."""
    n, batch, V, k = 80, 410, 16, 1                      # 32 800 rows: 2 x that is more than 65 535
    parent, rank = tr.tr_template_from_branching((1,), n)
    ctx = tr.tr_init(V, k, parent, rank, batch=batch)
    out_struct, out = tr.make_step_out(ctx)
    d_logits = torch.zeros(batch, n, V, device="cuda")
    d_logits[:, :, 3] = 1.0
    d_tree = torch.zeros(batch, n, dtype=torch.int32, device="cuda")
    with pytest.raises(tr.TrError) as e:
        tr.tr_verify_update_sampled(ctx, d_logits, torch.zeros_like(d_logits), 1.0, d_tree, out_struct)
    assert e.value.status == tr.TR_ERR_UNSUPPORTED
    tr.tr_verify_update(ctx, d_logits, d_tree, out_struct)
    torch.cuda.synchronize()
    assert (out["topk_idx"].cpu().numpy() == 3).all() and tr.tr_device_flags(ctx) == 0
    tr.tr_destroy(ctx)
