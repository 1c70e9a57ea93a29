"""GPU parity: every kernel, called through the C-ABI binding, against the CPU oracle on the same seeded inputs.
Integer outputs are compared bit for bit; attention within max|diff| <= 2e-2 and relative L2 <= 1e-2."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import tr_oracle as orc
from paper_2408_08696_b200 import synth
from tests.oracle_loop import OracleLoop, attention_close, compare_step, oracle_attention

pytestmark = pytest.mark.gpu

ATOL, RTOL = 2e-2, 1e-2


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


# ------------------------------------------------------------------ argmax + top-k
def _topk_case(tr, logits, k, branching=(1,), n=None):
    rows, V = logits.shape
    n = rows if n is None else n
    parent, rank = tr.tr_template_from_branching(branching, n)
    assert len(parent) == n
    ctx = tr.tr_init(V, k, parent, rank, batch=rows // n)
    out_struct, out = tr.make_step_out(ctx)
    d_logits = torch.from_numpy(logits).cuda().reshape(rows // n, n, V)
    d_tree = torch.zeros(rows // n, n, dtype=torch.int32, device="cuda")
    tr.tr_verify_update(ctx, d_logits, d_tree, out_struct)
    torch.cuda.synchronize()
    got = out["topk_idx"].cpu().numpy().reshape(rows, k)
    assert tr.tr_device_flags(ctx) == 0
    tr.tr_destroy(ctx)
    return got


@pytest.mark.parametrize("V,k", [(1000, 8), (32000, 8), (33, 8), (4097, 8), (8191, 4), (12289, 16), (8, 8),
                                 (50001, 1), (128256, 8)])
def test_topk_matches_oracle_random(tr, V, k):
    rng = np.random.default_rng(V * 31 + k)
    x = rng.standard_normal((15, V)).astype(np.float32)
    assert (_topk_case(tr, x, k) == orc.argtopk(x, k)).all()


@pytest.mark.parametrize("V", [1000, 4099, 32000])
def test_topk_ties_and_special_values(tr, V):
    rng = np.random.default_rng(V)
    x = rng.integers(-2, 3, size=(15, V)).astype(np.float32)          # five distinct values: ties everywhere
    x[1] = 0.0
    x[2] = -np.inf
    x[3, ::2] = -0.0
    x[3, 1::2] = 0.0
    x[4] = np.float32(3.0)
    x[4, V - 1] = np.float32(3.5)                                     # winner in the ragged last segment
    x[5, : V // 2] = -np.inf
    x[6] = np.arange(V, dtype=np.float32)                             # ascending: top-k at the very end
    x[7] = -np.arange(V, dtype=np.float32)
    x[8] = np.inf
    x[9, :] = -1e30
    x[9, 4096 % V] = 1e-30
    assert (_topk_case(tr, x, 8) == orc.argtopk(x, 8)).all()


def test_topk_all_equal_rows_k16_take_the_overflow_path(tr):
    # 16 candidates per token and constant rows: more keys reach the threshold than the candidate buffer holds
    V = 9000
    x = np.zeros((15, V), dtype=np.float32)
    x[1] = -np.inf
    x[2, 100:] = 1.0
    assert (_topk_case(tr, x, 16) == orc.argtopk(x, 16)).all()


def test_topk_adversarial_all_top_in_one_thread(tr):
    # every one of a thread's 16 register slots beats the rest of the segment: the candidate buffer's bound
    V = 8192
    x = np.full((15, V), -5.0, dtype=np.float32)
    for t in range(16):
        x[:, 4 * 7 + (t // 4) * 1024 + t % 4] = 10.0 - t               # the 16 elements of thread 7, segment 0
    x[:, 5000] = 9.5
    assert (_topk_case(tr, x, 8) == orc.argtopk(x, 8)).all()


# ------------------------------------------------------------------ retrieval
def test_build_tree_matches_oracle(tr):
    w = synth.WORKLOADS["llama2-70b-b8"]
    parent, rank = tr.tr_template_from_branching(w.branching, w.n_nodes)
    ctx = tr.tr_init(w.vocab, w.k, parent, rank, batch=w.batch)
    M = synth.seeded_matrix(w)
    for b in range(w.batch):
        tr.tr_matrix_import(ctx, b, M[b])
        assert (tr.tr_matrix_export(ctx, b) == M[b]).all()
    roots = synth.root_tokens(w)
    d_root = torch.from_numpy(roots).cuda()
    d_tree = torch.zeros(w.batch, w.n_nodes, dtype=torch.int32, device="cuda")
    tr.tr_build_tree(ctx, d_root, d_tree)
    got = d_tree.cpu().numpy()
    for b in range(w.batch):
        assert (got[b] == orc.bfs_tree(M[b], parent, rank, int(roots[b]))).all()
    # zero matrix (cold start, Sec. 3.1): all drafts are token 0
    tr.tr_matrix_zero(ctx)
    tr.tr_build_tree(ctx, d_root, d_tree)
    got = d_tree.cpu().numpy()
    assert (got[:, 0] == roots).all() and (got[:, 1:] == 0).all()
    assert tr.tr_device_flags(ctx) == 0
    # a root outside the vocabulary sets the flag and is treated as token 0; nothing traps
    d_root[0] = w.vocab + 5
    tr.tr_build_tree(ctx, d_root, d_tree)
    assert tr.tr_device_flags(ctx) & tr.TR_FLAG_BAD_TOKEN
    tr.tr_destroy(ctx)


# ------------------------------------------------------------------ verify / update / retrieve loop
def _run_loop(harness, w, steps, zero_matrix=False, graphs=False, check_every=1):
    dw = harness.DeviceWorkload(w, with_attention=False, zero_matrix=zero_matrix)
    ol = OracleLoop(w, zero_matrix=zero_matrix)
    assert (dw.d_tree.cpu().numpy() == np.stack(ol.S)).all()
    g = dw.capture_graphs() if graphs else None
    mats = []
    for i in range(steps):
        if graphs:
            g[i % dw.n_rot].replay()
        else:
            dw.step(i)
        recs = ol.step(i)
        if i % check_every == 0 or i == steps - 1:
            compare_step(recs, dw.snapshot(), dw.ctx.max_new)
        mats.append(np.mean([r["n_new"] for r in recs]))
    from paper_2408_08696_b200 import binding as tr
    for b in range(w.batch):
        assert (tr.tr_matrix_export(dw.ctx, b) == ol.M[b]).all(), "matrix differs after the loop"
    assert tr.tr_device_flags(dw.ctx) == 0
    dw.close()
    return float(np.mean(mats))


def test_loop_tiny_50_steps(harness):
    mat = _run_loop(harness, synth.WORKLOADS["tiny"], 50)
    assert 1.0 <= mat <= 7.0


def test_loop_tiny_cold_start_zero_matrix(harness):
    _run_loop(harness, synth.WORKLOADS["tiny"], 30, zero_matrix=True)     # all-equal drafts: duplicate handling


def test_loop_llama2_7b_shape(harness):
    _run_loop(harness, synth.WORKLOADS["llama2-7b"], 24)


def test_loop_llama2_7b_all_256_steps_of_the_workload_as_graph_replays(harness):
    """The benchmark's workload from its first step to its last (256 steps, the replayed single-step graphs): every
    integer output of every step and the matrix at the end, bit for bit.  About a minute of oracle time."""
    _run_loop(harness, synth.WORKLOADS["llama2-7b"], 256, graphs=True)


def test_loop_batched_8_sequences_via_graph(harness):
    _run_loop(harness, synth.WORKLOADS["llama2-70b-b8"], 12, graphs=True)


def test_loop_large_vocab(harness):
    _run_loop(harness, synth.WORKLOADS["llama3-8b"], 6)


def test_loop_large_vocab_32_steps_as_graph_replays(harness):
    _run_loop(harness, synth.WORKLOADS["llama3-8b"], 32, graphs=True)


@pytest.mark.parametrize("rule,only_accepted", [("first", False), ("last", True), ("first", True)])
@pytest.mark.parametrize("zero_matrix", [False, True])
def test_loop_update_rule_variants(harness, tr, rule, only_accepted, zero_matrix):
    """The update strategies the paper compares (First / Last, all drafts / only accepted); the zero matrix makes
    every draft the same token, so the duplicate handling decides every row."""
    w = synth.WORKLOADS["tiny"]
    dw = harness.DeviceWorkload(w, with_attention=False, zero_matrix=zero_matrix)
    tr.tr_set_update_rule(dw.ctx, tr.TR_UPDATE_FIRST if rule == "first" else tr.TR_UPDATE_LAST,
                          tr.TR_UPDATE_ONLY_ACCEPTED if only_accepted else tr.TR_UPDATE_ALL_DRAFT)
    ol = OracleLoop(w, zero_matrix=zero_matrix, rule=rule, only_accepted=only_accepted)
    for i in range(25):
        dw.step(i)
        compare_step(ol.step(i), dw.snapshot(), dw.ctx.max_new)
    assert (tr.tr_matrix_export(dw.ctx, 0) == ol.M[0]).all()
    with pytest.raises(tr.TrError):
        tr.tr_set_update_rule(dw.ctx, 7, 0)
    dw.close()


def test_duplicate_tokens_last_writer_wins(tr):
    # Appendix "Explanation of Three Update Strategies": S = [a, b, c, a, d] keeps O[3] for a.
    parent = np.array([-1, 0, 0, 0, 0], dtype=np.int32)
    rank = np.array([0, 0, 1, 2, 3], dtype=np.int32)
    V, k = 64, 4
    ctx = tr.tr_init(V, k, parent, rank)
    out_struct, out = tr.make_step_out(ctx)
    S = np.array([[10, 11, 12, 10, 13]], dtype=np.int32)
    rng = np.random.default_rng(0)
    logits = rng.standard_normal((1, 5, V)).astype(np.float32)
    d_tree = torch.from_numpy(S).cuda()
    tr.tr_verify_update(ctx, torch.from_numpy(logits).cuda(), d_tree, out_struct)
    torch.cuda.synchronize()
    M = tr.tr_matrix_export(ctx, 0)
    O = orc.argtopk(logits[0], k)
    assert (M[10] == O[3]).all() and not (M[10] == O[0]).all()
    assert (M[11] == O[1]).all() and (M[12] == O[2]).all() and (M[13] == O[4]).all()
    touched = np.zeros(V, bool); touched[[10, 11, 12, 13]] = True
    assert (M[~touched] == 0).all()
    tr.tr_destroy(ctx)


def _random_template(rng, n, k):
    """An irregular static tree in level order: every node draws its own number of children (ranks 0..c-1)."""
    parent, rank, level = [-1], [0], [0]
    while len(parent) < n:
        nxt = []
        for p_ in level:
            for r in range(int(rng.integers(0, min(k, 4) + 1))):
                if len(parent) < n:
                    parent.append(p_)
                    rank.append(r)
                    nxt.append(len(parent) - 1)
        if not nxt:                                    # nobody drew a child: the level's first node gets one
            parent.append(level[0])
            rank.append(0)
            nxt.append(len(parent) - 1)
        level = nxt
    return np.array(parent, dtype=np.int32), np.array(rank, dtype=np.int32)


@pytest.mark.parametrize("seed", range(12))
def test_verify_update_seeded_random_configurations(tr, seed):
    """Irregular templates (children counts differ inside a level), small vocabularies (duplicate tokens in the tree),
    tie-heavy integer logits with planted continuations, every update rule and scope, 1-4 sequences: three chained
    steps each, every integer output and the matrix against the oracle."""
    rng = np.random.default_rng(7000 + seed)
    k = int(rng.choice([1, 2, 4, 5, 8, 12, 16]))
    n = int(rng.choice([1, 2, 7, 31, 80, 97, 128]))
    V = int(rng.choice([max(k, 16), 97, 1000, 4099]))
    B = int(rng.integers(1, 5))
    rule = ["last", "first"][int(rng.integers(2))]
    only_accepted = bool(rng.integers(2))
    parent, rank = _random_template(rng, n, k)
    ctx = tr.tr_init(V, k, parent, rank, batch=B)
    tr.tr_set_update_rule(ctx, tr.TR_UPDATE_FIRST if rule == "first" else tr.TR_UPDATE_LAST,
                          tr.TR_UPDATE_ONLY_ACCEPTED if only_accepted else tr.TR_UPDATE_ALL_DRAFT)
    M = [rng.integers(0, V, size=(V, k)).astype(np.int32) for _ in range(B)]
    for b in range(B):
        tr.tr_matrix_import(ctx, b, M[b])
    roots = rng.integers(0, V, size=B).astype(np.int32)
    d_tree = torch.zeros(B, n, dtype=torch.int32, device="cuda")
    tr.tr_build_tree(ctx, torch.from_numpy(roots).cuda(), d_tree)
    S = d_tree.cpu().numpy().copy()
    for b in range(B):
        assert (S[b] == orc.bfs_tree(M[b], parent, rank, int(roots[b]))).all()
    out_struct, out = tr.make_step_out(ctx)
    children = [[j for j in range(n) if parent[j] == i] for i in range(n)]
    for step in range(3):
        logits = rng.integers(-3, 4, size=(B, n, V)).astype(np.float32)
        for b in range(B):
            for i in range(n):
                if children[i] and rng.random() < 0.6:        # the model "agrees" with one of the node's drafts
                    logits[b, i, S[b, children[i][int(rng.integers(len(children[i])))]]] += 10.0
        tr.tr_verify_update(ctx, torch.from_numpy(logits).cuda(), d_tree, out_struct)
        torch.cuda.synchronize()
        got = {name: t.cpu().numpy() for name, t in out.items()}
        for b in range(B):
            rec = orc.verify_update(M[b], S[b], logits[b], parent, rank, rule=rule, only_accepted=only_accepted)
            m = rec["n_new"]
            assert (got["topk_idx"][b] == rec["topk"]).all()
            assert got["n_new"][b] == m
            assert got["acc_nodes"][b, :m].tolist() == rec["acc_nodes"]
            assert got["out_tokens"][b, :m].tolist() == rec["out_tokens"]
            assert got["next_root"][b] == rec["next_root"]
            assert (got["next_tree"][b] == rec["next_tree"]).all()
            assert (tr.tr_matrix_export(ctx, b) == M[b]).all()
            S[b] = rec["next_tree"]
        d_tree.copy_(out["next_tree"])
    assert tr.tr_device_flags(ctx) == 0
    tr.tr_destroy(ctx)


# ------------------------------------------------------------------ tree attention
def _attention_case(harness, w, n_layers, splits=0):
    dw = harness.DeviceWorkload(w, n_layers=n_layers, splits=splits)
    from paper_2408_08696_b200 import binding as tr
    tr.tr_tree_attention(dw.ctx, dw.attn)
    torch.cuda.synchronize()
    got = dw.o.float().cpu().numpy()                                   # [B, L, N, Hq, D]
    q, k, v = synth.attention_inputs(w, n_layers)
    worst = (0.0, 0.0)
    for b in range(w.batch):
        for l in range(n_layers):
            ref = oracle_attention(w, q, k, v, b, l, dw.parent)
            assert np.isfinite(got[b, l]).all()
            for h in range(w.n_q_heads):
                mx, rel = attention_close(got[b, l, :, h], ref[:, h])
                assert mx <= ATOL and rel <= RTOL, (b, l, h, mx, rel)
                worst = (max(worst[0], mx), max(worst[1], rel))
    assert tr.tr_device_flags(dw.ctx) == 0
    dw.close()
    return worst


@pytest.mark.parametrize("splits", [0, 1, 2, 3, 5])
def test_attention_tiny(harness, splits):
    _attention_case(harness, synth.WORKLOADS["tiny"], 1, splits)


@pytest.mark.parametrize("ctx", [0, 1, 63, 64, 65, 77, 200])
def test_attention_ragged_context(harness, ctx):
    w = dataclasses.replace(synth.WORKLOADS["tiny"], ctx=(ctx,))
    _attention_case(harness, w, 2)
    _attention_case(harness, w, 1, splits=4)


@pytest.mark.parametrize("splits", [0, 1, 4])
def test_attention_head_dim_128_full_tree(harness, splits):
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], n_q_heads=4, n_kv_heads=4, ctx=(333,))
    _attention_case(harness, w, 2, splits)


def test_attention_gqa_and_batch_with_mixed_contexts(harness):
    w = dataclasses.replace(synth.WORKLOADS["llama2-70b-b8"], n_q_heads=8, n_kv_heads=2, ctx=(100, 257, 31))
    _attention_case(harness, w, 2)
    _attention_case(harness, w, 1, splits=3)


@pytest.mark.parametrize("hq,hkv", [(6, 2), (8, 1), (4, 2), (16, 2)])
def test_attention_group_sizes(harness, hq, hkv):
    """Grouped-query attention: group sizes that divide 128 share packed row tiles (2, 8; 8 heads of one KV head
    fill five tiles with the 80-node tree), others (3) fall back to one tile per query head."""
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], n_q_heads=hq, n_kv_heads=hkv, ctx=(150,))
    _attention_case(harness, w, 1)
    _attention_case(harness, w, 2, splits=2)


def test_attention_two_tiles_per_cta_kernel_largest_tree_and_wide_groups(harness):
    """128 nodes with 4 heads per KV head (four full row tiles = two pair units per KV head), and 16 / 32 heads per KV
    head (8 / 4 nodes per tile; ten and twenty row tiles) on the default tree."""
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], branching=(10, 10), n_nodes=128, n_q_heads=8, n_kv_heads=2,
                            ctx=(200, 77), vocab=3000, k=16)
    _attention_case(harness, w, 2, splits=1)
    for hq, hkv in ((16, 1), (32, 1)):
        w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], n_q_heads=hq, n_kv_heads=hkv, ctx=(150,))
        _attention_case(harness, w, 1, splits=1)


@pytest.mark.parametrize("hq,hkv,ctxs,L", [
    (8, 1, (150,), 1),          # 8 heads per KV head: five row tiles = two pairs and a lone left-over tile
    (8, 2, (100, 257), 2),      # 4 per KV head: three tiles = one pair per KV head + one twin of the two left-overs
    (12, 3, (333,), 2),         # odd number of KV heads: pairs, one twin and one lone tile
    (4, 2, (64,), 3),           # 2 per KV head: two tiles, pairs only; the prefix ends on a tile boundary
    (8, 2, (0, 1, 63), 1),      # empty and tiny prefixes: the tree block alone spans two key tiles
    (32, 8, (1200, 40), 2),     # the llama3-8b head layout, two sequences of very different length
])
def test_attention_two_tiles_per_cta_kernel(harness, hq, hkv, ctxs, L):
    """The grouped-query kernel that runs two row tiles per CTA on one K/V stream (pair, twin and lone units, 64-key
    tiles, dynamic unit queue), forced by asking for no KV split; every output row against the oracle."""
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], n_q_heads=hq, n_kv_heads=hkv, ctx=ctxs)
    _attention_case(harness, w, L, splits=1)
    _attention_case(harness, w, L, splits=1)      # a second launch finds the unit counter cleared


@pytest.mark.parametrize("head_dim", [128, 64])
def test_attention_other_memory_layouts_and_explicit_scale(harness, tr, head_dim):
    """The same tensors in other layouts - token-major caches [B, L, R, Hkv, D], head-major queries and outputs
    [B, L, Hq, N, D], a padded last-but-one stride - addressed through the stride arguments, with a scale that is not
    1/sqrt(head_dim)."""
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], n_q_heads=4, n_kv_heads=2, head_dim=head_dim, ctx=(140, 77))
    L, scale = 2, 0.11
    parent, rank = tr.tr_template_from_branching(w.branching, w.n_nodes)
    ctx = tr.tr_init(w.vocab, w.k, parent, rank, batch=w.batch)
    q, k, v = synth.attention_inputs(w, L)                              # [B,L,N,Hq,D], [B,L,Hkv,R,D]
    dq, dk, dv = (harness.bf16_tensor(x, "cuda") for x in (q, k, v))
    B, N, Hq, Hkv, D = w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, head_dim
    R = k.shape[3]
    # token-major caches with 8 elements of padding after every (token, head) row group
    k_tm = torch.zeros(B, L, R, Hkv, D + 8, dtype=torch.bfloat16, device="cuda")
    v_tm = torch.zeros_like(k_tm)
    k_tm[..., :D] = dk.permute(0, 1, 3, 2, 4)
    v_tm[..., :D] = dv.permute(0, 1, 3, 2, 4)
    k_view, v_view = k_tm[..., :D].permute(0, 1, 3, 2, 4), v_tm[..., :D].permute(0, 1, 3, 2, 4)   # [B,L,Hkv,R,D] views
    q_hm = dq.permute(0, 1, 3, 2, 4).contiguous()                       # stored [B,L,Hq,N,D]
    o_hm = torch.zeros_like(q_hm)
    q_view, o_view = q_hm.permute(0, 1, 3, 2, 4), o_hm.permute(0, 1, 3, 2, 4)
    d_ctx = torch.tensor(list(w.ctx), dtype=torch.int32, device="cuda")
    for splits in (0, 2, 1):        # 1: no KV split - at head_dim 128 the two-tiles-per-CTA kernel (2 heads per KV head)
        o_hm.zero_()
        a = tr.make_attn_args(ctx, q_view, k_view, v_view, o_view, d_ctx, w.max_ctx, scale=scale, splits=splits)
        tr.tr_tree_attention(ctx, a)
        torch.cuda.synchronize()
        got = o_view.float().cpu().numpy()
        for b in range(B):
            for l in range(L):
                c = w.ctx[b]
                ref = orc.tree_attention(synth.bf16_bits_to_f32(q[b, l]).astype(np.float64),
                                         synth.bf16_bits_to_f32(k[b, l][:, :c + N]).astype(np.float64),
                                         synth.bf16_bits_to_f32(v[b, l][:, :c + N]).astype(np.float64), c,
                                         np.asarray(parent), scale=scale)
                for h in range(Hq):
                    mx, rel = attention_close(got[b, l, :, h], ref[:, h])
                    assert mx <= ATOL and rel <= RTOL, (splits, b, l, h, mx, rel)
    assert tr.tr_device_flags(ctx) == 0
    tr.tr_destroy(ctx)


def test_largest_tree_128_nodes_attention_and_loop(harness):
    # the maximum template size (ancestor masks are 128-bit; the attention tile has 128 query rows)
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], branching=(10, 10), n_nodes=128, n_q_heads=2, n_kv_heads=2,
                            ctx=(200,), vocab=3000, k=16)
    _attention_case(harness, w, 1)
    _attention_case(harness, w, 1, splits=3)
    w64 = dataclasses.replace(w, head_dim=64)
    _attention_case(harness, w64, 1)
    _run_loop(harness, w, 6)


@pytest.mark.parametrize("branching,n_nodes,k,boost", [
    ((1,) * 24, 25, 8, 9.0),                 # a chain: depth 24, accepted paths get long with a strong toy model
    ((2,) * 6, 127, 8, 4.0),                 # full binary tree, depth 6
    ((16,), 17, 16, 4.0),                    # a star: one level, every rank up to k - 1 = 15
    ((8, 4, 3, 2, 2, 1, 1, 1, 1, 1), 110, 8, 6.0),   # the default shape made deeper (Fig. 3b's knob)
    ((12, 6, 3, 1), 120, 12, 3.0),           # ... and broader (Fig. 3a's knob)
])
def test_loop_template_breadth_and_depth_sweep(harness, branching, n_nodes, k, boost):
    w = dataclasses.replace(synth.WORKLOADS["tiny"], branching=branching, n_nodes=n_nodes, k=k, boost=boost,
                            vocab=2000)
    mat = _run_loop(harness, w, 20)
    parent, _ = orc.template_from_branching(branching, n_nodes)
    assert 1.0 <= mat <= max(orc.node_depth(parent)) + 1          # Appendix: at most depth + 1 tokens per step


@pytest.mark.parametrize("hq,hkv,head_dim,ctx,splits", [
    (2, 2, 128, 30000, 0),      # 235 key tiles per unit, split along the keys over the SMs + merge
    (2, 2, 128, 30000, 1),      # ... and as one unit per head: 235 tiles through one CTA's ring
    (8, 2, 128, 30000, 1),      # the two-tiles-per-CTA kernel on a long stream
    (2, 1, 64, 33000, 0),       # head_dim 64, a prefix longer than 2^15 keys
])
def test_attention_long_context(harness, hq, hkv, head_dim, ctx, splits):
    """Prefixes of 30 000 and more keys (hundreds of key tiles per unit: ring wrap-arounds, barrier phases, the running
    maximum over a long row), one layer, every head against the oracle."""
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], n_q_heads=hq, n_kv_heads=hkv, head_dim=head_dim, ctx=(ctx,))
    _attention_case(harness, w, 1, splits=splits)


@pytest.mark.parametrize("hq,hkv,ctxs", [(32, 32, (1024,)), (8, 2, (300, 77)), (4, 4, (50,))])
def test_attention_per_layer_launches_with_early_prefix_requests(harness, tr, hq, hkv, ctxs):
    """One launch per layer, back to back on a stream and as a replayed graph, with the caller's promise that prefix
    lengths and prefix K/V are stable (prefix_stable): a launch may then request its prefix tiles while the launch in
    front (the previous layer's merge of split partials) is still running.  Every head of every layer against the
    oracle; the outputs must not depend on the promise."""
    L = 4
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], n_q_heads=hq, n_kv_heads=hkv, ctx=ctxs)
    dw = harness.DeviceWorkload(w, n_layers=L)
    q, k, v = synth.attention_inputs(w, L)
    ref = [[oracle_attention(w, q, k, v, b, l, dw.parent) for l in range(L)] for b in range(w.batch)]

    def check():
        torch.cuda.synchronize()
        got = dw.o.float().cpu().numpy()
        for b in range(w.batch):
            for l in range(L):
                for h in range(hq):
                    mx, rel = attention_close(got[b, l, :, h], ref[b][l][:, h])
                    assert mx <= ATOL and rel <= RTOL, (b, l, h, mx, rel)

    for stable in (False, True):
        args = [tr.make_attn_args(dw.ctx, dw.q[:, l:l + 1], dw.k[:, l:l + 1], dw.v[:, l:l + 1], dw.o[:, l:l + 1],
                                  dw.d_ctx_len, w.max_ctx, prefix_stable=stable) for l in range(L)]
        dw.o.zero_()
        for a in args:
            tr.tr_tree_attention(dw.ctx, a)
        check()
        s = torch.cuda.Stream(dw.dev)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(s):
            with torch.cuda.graph(g, stream=s):
                for a in args:
                    tr.tr_tree_attention(dw.ctx, a, s)
        for _ in range(3):
            dw.o.zero_()
            g.replay()
            check()
    assert tr.tr_device_flags(dw.ctx) == 0
    dw.close()


def test_attention_single_node_tree(harness):
    w = dataclasses.replace(synth.WORKLOADS["tiny"], n_nodes=1, branching=(1,), ctx=(50,))
    _attention_case(harness, w, 1)


def test_attention_llama2_7b_full_size_every_head(harness):
    """The benchmark's launch configuration (32 layers x 32 heads in one launch, 1024-token prefix); the oracle
    checks every one of the 1024 (layer, head) outputs."""
    w = synth.WORKLOADS["llama2-7b"]
    dw = harness.DeviceWorkload(w)
    from paper_2408_08696_b200 import binding as tr
    tr.tr_tree_attention(dw.ctx, dw.attn)
    torch.cuda.synchronize()
    pool = synth.normal_pool(w.seed)
    got_all = dw.o.float().cpu().numpy()                               # [1, L, N, Hq, D]
    worst = (0.0, 0.0)
    for l in range(w.n_layers):
        for h in range(w.n_q_heads):
            qs, ks, vs = synth.attention_slice(w, pool, 0, l, h)
            ref = orc.tree_attention(synth.bf16_bits_to_f32(qs[:, h:h + 1]), synth.bf16_bits_to_f32(ks)[None],
                                     synth.bf16_bits_to_f32(vs)[None], w.ctx[0], dw.parent)
            mx, rel = attention_close(got_all[0, l, :, h], ref[:, 0])
            assert mx <= ATOL and rel <= RTOL, (l, h, mx, rel)
            worst = (max(worst[0], mx), max(worst[1], rel))
    assert np.isfinite(got_all).all()
    assert tr.tr_device_flags(dw.ctx) == 0
    dw.close()


@pytest.mark.parametrize("name", ["llama2-13b", "llama3-8b", "llama2-70b-b8"])
def test_attention_other_workload_shapes_three_layers_sampled(harness, name):
    """The other workloads' full head counts, group sizes and context lengths (4096; 8192 with 4 query heads per KV
    head; eight sequences of 1024..4096 with 8 per KV head), three layers each in one launch; the oracle checks a
    seeded sample of 72 (sequence, layer, query head) outputs."""
    w = synth.WORKLOADS[name]
    L = 3
    dw = harness.DeviceWorkload(w, n_layers=L)
    from paper_2408_08696_b200 import binding as tr
    tr.tr_tree_attention(dw.ctx, dw.attn)
    torch.cuda.synchronize()
    assert tr.tr_device_flags(dw.ctx) == 0
    q, k, v = synth.attention_inputs(w, L)
    group = w.n_q_heads // w.n_kv_heads
    rng = np.random.default_rng(7)
    seen = set()
    for _ in range(72):
        b, l, h = int(rng.integers(0, w.batch)), int(rng.integers(0, L)), int(rng.integers(0, w.n_q_heads))
        seen.add(l)
        g, c = h // group, w.ctx[b]
        ref = orc.tree_attention(synth.bf16_bits_to_f32(q[b, l, :, h:h + 1]),
                                 synth.bf16_bits_to_f32(k[b, l, g:g + 1, : c + w.n_nodes]),
                                 synth.bf16_bits_to_f32(v[b, l, g:g + 1, : c + w.n_nodes]), c, dw.parent)
        got = dw.o[b, l, :, h].float().cpu().numpy()
        mx, rel = attention_close(got, ref[:, 0])
        assert mx <= ATOL and rel <= RTOL, (name, b, l, h, mx, rel)
    assert len(seen) == L
    assert torch.isfinite(dw.o.float()).all()
    dw.close()


# ------------------------------------------------------------------ the whole step as a CUDA graph
@pytest.mark.parametrize("hq,hkv,ctxs,L", [(32, 32, (300,), 5),          # cut-down 7B shape: 160 one-tile units, no split
                                           (16, 4, (300, 513), 7),       # grouped-query, two sequences, packed tiles
                                           (4, 4, (90,), 1)])            # fewer units than SMs: split-KV + combine
def test_step_graph_with_attention_matches_oracle(harness, tr, hq, hkv, ctxs, L):
    """The graphs the benchmark replays - toy-model patch on a side branch, tree attention, top-k, accept / update /
    retrieve - replayed in rotation order: every integer output after every replay, the matrix at the end, and the
    attention output of the last replay, against the oracle."""
    w = dataclasses.replace(synth.WORKLOADS["llama2-7b"], n_q_heads=hq, n_kv_heads=hkv, ctx=ctxs, n_layers=L)
    dw = harness.DeviceWorkload(w, n_rot=3)
    ol = OracleLoop(w, n_rot=3)
    graphs = dw.capture_graphs()
    steps = 10
    for i in range(steps):
        dw.o.zero_()
        graphs[i % dw.n_rot].replay()
        compare_step(ol.step(i), dw.snapshot(), dw.ctx.max_new)
    got = dw.o.float().cpu().numpy()
    q, k, v = synth.attention_inputs(w, L)
    for b in range(w.batch):
        assert (tr.tr_matrix_export(dw.ctx, b) == ol.M[b]).all()
        for l in range(L):
            ref = oracle_attention(w, q, k, v, b, l, dw.parent)
            for h in range(hq):
                mx, rel = attention_close(got[b, l, :, h], ref[:, h])
                assert mx <= ATOL and rel <= RTOL, (b, l, h, mx, rel)
    assert tr.tr_device_flags(dw.ctx) == 0
    # the same graphs after a reset give the same loop again
    dw.reset()
    ol2 = OracleLoop(w, n_rot=3)
    for i in range(4):
        graphs[i % dw.n_rot].replay()
        compare_step(ol2.step(i), dw.snapshot(), dw.ctx.max_new)
    dw.close()


# ------------------------------------------------------------------ the step from a given top-k: ordering and bad input
def _topk_step_fixture(tr, V=500, k=8, seed=3):
    parent, rank = tr.tr_template_from_branching((4, 2, 1), 15)
    ctx = tr.tr_init(V, k, parent, rank)
    rng = np.random.default_rng(seed)
    M = rng.integers(0, V, size=(V, k), dtype=np.int32)
    tr.tr_matrix_import(ctx, 0, M)
    logits = rng.standard_normal((15, V)).astype(np.float32)
    return ctx, parent, rank, M, logits, rng


def test_verify_update_topk_directly_behind_the_kernels_that_write_its_inputs(tr):
    """tr_verify_update_topk launches only the accept/update/retrieve kernel (with programmatic dependent launch): the
    tree and the top-k it reads may come from the kernel directly in front of it - a device copy, or tr_build_tree
    inside one CUDA graph - and must be read only after that kernel has finished."""
    ctx, parent, rank, M, logits, rng = _topk_step_fixture(tr)
    V, k = M.shape
    out_struct, out = tr.make_step_out(ctx)
    O = orc.argtopk(logits, k)
    d_O = torch.from_numpy(O.astype(np.int32)).cuda()
    stale = torch.full((1, 15), 7, dtype=torch.int32, device="cuda")
    d_tree = stale.clone()
    for trial in range(20):
        root = int(rng.integers(0, V))
        S = orc.bfs_tree(M.astype(np.int64), parent, rank, root)
        d_S = torch.from_numpy(S.astype(np.int32)).cuda().reshape(1, 15)
        tr.tr_matrix_import(ctx, 0, M)
        d_tree.copy_(stale)
        out["topk_idx"].zero_()
        torch.cuda.synchronize()
        # device copies of both inputs, then the call, back to back on one stream
        out["topk_idx"].copy_(d_O.reshape(1, 15, k))
        d_tree.copy_(d_S)
        tr.tr_verify_update_topk(ctx, d_tree, out_struct)
        torch.cuda.synchronize()
        Mo = M.astype(np.int64).copy()
        n_new, acc, toks, nroot = orc.accept(S, O[:, 0], parent)
        orc.update_matrix(Mo, S, O)
        assert out["n_new"].item() == n_new and out["next_root"].item() == nroot
        assert (out["next_tree"].cpu().numpy()[0] == orc.bfs_tree(Mo, parent, rank, nroot)).all()
        assert (tr.tr_matrix_export(ctx, 0) == Mo).all()
    # tr_build_tree and the step in one graph, nothing in between
    d_root = torch.zeros(1, dtype=torch.int32, device="cuda")
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    out["topk_idx"].copy_(d_O.reshape(1, 15, k))
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            tr.tr_build_tree(ctx, d_root, d_tree, s)
            tr.tr_verify_update_topk(ctx, d_tree, out_struct, s)
    for trial in range(20):
        root = int(rng.integers(0, V))
        tr.tr_matrix_import(ctx, 0, M)
        d_root.fill_(root)
        d_tree.copy_(stale)
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        Mo = M.astype(np.int64).copy()
        S = orc.bfs_tree(Mo, parent, rank, root)
        n_new, acc, toks, nroot = orc.accept(S, O[:, 0], parent)
        orc.update_matrix(Mo, S, O)
        assert out["n_new"].item() == n_new and out["next_root"].item() == nroot
        assert (out["next_tree"].cpu().numpy()[0] == orc.bfs_tree(Mo, parent, rank, nroot)).all()
        assert (tr.tr_matrix_export(ctx, 0) == Mo).all()
    assert tr.tr_device_flags(ctx) == 0
    tr.tr_destroy(ctx)


def test_verify_update_topk_rejects_indices_outside_the_vocabulary(tr):
    """A top-k index outside [0, V) handed to tr_verify_update_topk must not reach the matrix (its entries are later
    used as row numbers): the flag is raised, the entry counts as token 0, nothing faults."""
    ctx, parent, rank, M, logits, rng = _topk_step_fixture(tr)
    V, k = M.shape
    out_struct, out = tr.make_step_out(ctx)
    O = orc.argtopk(logits, k)
    bad = O.astype(np.int32).copy()
    bad[0, 0] = V + 12345          # the root's argmax: would become the next root and a row number
    bad[3, 2] = -4
    bad[7, 7] = 2 ** 31 - 1
    S = orc.bfs_tree(M.astype(np.int64), parent, rank, 11)
    d_tree = torch.from_numpy(S.astype(np.int32)).cuda().reshape(1, 15)
    out["topk_idx"].copy_(torch.from_numpy(bad).cuda().reshape(1, 15, k))
    tr.tr_verify_update_topk(ctx, d_tree, out_struct)
    torch.cuda.synchronize()
    assert tr.tr_device_flags(ctx) & tr.TR_FLAG_BAD_TOKEN
    Mg = tr.tr_matrix_export(ctx, 0)
    assert Mg.min() >= 0 and Mg.max() < V
    fixed = np.where((bad < 0) | (bad >= V), 0, bad).astype(np.int64)
    Mo = M.astype(np.int64).copy()
    n_new, acc, toks, nroot = orc.accept(S, fixed[:, 0], parent)
    orc.update_matrix(Mo, S, fixed)
    assert (Mg == Mo).all()
    assert out["next_root"].item() == nroot and 0 <= nroot < V
    assert (out["next_tree"].cpu().numpy()[0] == orc.bfs_tree(Mo, parent, rank, nroot)).all()
    tr.tr_destroy(ctx)


# ------------------------------------------------------------------ the paper's uncontrolled update and seeded fill
def test_update_rule_cur_every_element_comes_from_an_occurrence(tr):
    """Appendix "Explanation of Three Update Strategies": under the uncontrolled update the row of a repeated token may
    mix its occurrences element by element.  Valid outcomes: every element of M[a] equals that element of O[i] for
    some i with S[i] = a; rows of tokens outside S are untouched; the next tree is the retrieval from the matrix as it
    came out."""
    parent, rank = tr.tr_template_from_branching((4, 2, 1), 15)
    V, k = 300, 8
    ctx = tr.tr_init(V, k, parent, rank)
    tr.tr_set_update_rule(ctx, tr.TR_UPDATE_CUR, tr.TR_UPDATE_ALL_DRAFT)
    out_struct, out = tr.make_step_out(ctx)
    rng = np.random.default_rng(11)
    for trial in range(10):
        M = rng.integers(0, V, size=(V, k), dtype=np.int32)
        tr.tr_matrix_import(ctx, 0, M)
        S = rng.integers(0, 6, size=15).astype(np.int32)            # 15 nodes over 6 tokens: every token repeats
        logits = rng.standard_normal((1, 15, V)).astype(np.float32)
        O = orc.argtopk(logits[0], k)
        tr.tr_verify_update(ctx, torch.from_numpy(logits).cuda(), torch.from_numpy(S).cuda().reshape(1, 15), out_struct)
        torch.cuda.synchronize()
        Mg = tr.tr_matrix_export(ctx, 0)
        for a in range(V):
            occ = [i for i in range(15) if S[i] == a]
            if not occ:
                assert (Mg[a] == M[a]).all()
            else:
                for c in range(k):
                    assert Mg[a, c] in {int(O[i, c]) for i in occ}, (a, c)
        n_new, acc, toks, nroot = orc.accept(S, O[:, 0], parent)
        assert out["n_new"].item() == n_new and out["out_tokens"].cpu().numpy()[0, :n_new].tolist() == toks
        assert (out["next_tree"].cpu().numpy()[0] == orc.bfs_tree(Mg.astype(np.int64), parent, rank, nroot)).all()
    assert tr.tr_device_flags(ctx) == 0
    tr.tr_destroy(ctx)


def test_matrix_fill_seeded_matches_the_documented_hash(tr):
    """tr_matrix_fill(TR_FILL_SEEDED): the integer hash written in the header, restated here with Python integers."""
    parent, rank = tr.tr_template_from_branching((4, 2, 1), 15)
    V, k, B, seed = 1000, 8, 2, 0xC0FFEE1234
    ctx = tr.tr_init(V, k, parent, rank, batch=B)
    tr.tr_matrix_fill(ctx, tr.TR_FILL_SEEDED, seed)
    mask = (1 << 64) - 1
    want = np.empty(B * V * k, dtype=np.int64)
    for i in range(B * V * k):
        z = (seed + 0x9E3779B97F4A7C15 * (i + 1)) & mask
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
        z ^= z >> 31
        want[i] = ((z >> 32) * V) >> 32
    want = want.reshape(B, V, k)
    for b in range(B):
        got = tr.tr_matrix_export(ctx, b)
        assert (got == want[b]).all()
        assert got.min() >= 0 and got.max() < V
    assert len(np.unique(want)) > V // 2                           # spread over the vocabulary
    tr.tr_matrix_fill(ctx, tr.TR_FILL_ZERO)
    assert (tr.tr_matrix_export(ctx, 1) == 0).all()
    with pytest.raises(tr.TrError):
        tr.tr_matrix_fill(ctx, 5)
    tr.tr_destroy(ctx)


# ------------------------------------------------------------------ decoder loop with KV / token commit
def test_decode_loop_with_commit_grows_the_prefix(tr):
    """Steps of: attention at the current (device-resident) prefix length -> verify/update/retrieve -> commit of the
    accepted path.  Cache contents, prefix lengths and emitted tokens must equal the oracle's, bit for bit, and the
    attention output of the last step must match the oracle's attention over the oracle's cache."""
    B, L, Hq, Hkv, D, N, V, k_cand = 2, 2, 4, 2, 128, 15, 500, 8
    w = dataclasses.replace(synth.WORKLOADS["tiny"], vocab=V, ctx=(70, 37), n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv,
                            head_dim=D, boost=5.0)
    steps, cap_rows, cap_tok = 12, 70 + N + 12 * 7 + 8, 12 * 7 + 4
    parent, rank = tr.tr_template_from_branching(w.branching, N)
    ctx = tr.tr_init(V, k_cand, parent, rank, batch=B)
    rng = np.random.default_rng(5)
    bits = lambda shape: synth.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    k_h, v_h = bits((B, L, Hkv, cap_rows, D)), bits((B, L, Hkv, cap_rows, D))
    q_h = bits((B, L, N, Hq, D))
    from paper_2408_08696_b200.harness import bf16_tensor
    dev = torch.device("cuda", 0)
    d_k, d_v, d_q = bf16_tensor(k_h, dev), bf16_tensor(v_h, dev), bf16_tensor(q_h, dev)
    d_o = torch.zeros_like(d_q)
    d_ctx = torch.tensor(list(w.ctx), dtype=torch.int32, device=dev)
    d_tokens = torch.zeros(B, cap_tok, dtype=torch.int32, device=dev)
    d_ntok = torch.zeros(B, dtype=torch.int32, device=dev)
    attn = tr.make_attn_args(ctx, d_q, d_k, d_v, d_o, d_ctx, cap_rows - N)
    cargs = tr.make_commit_args(ctx, d_k, d_v, d_ctx, d_tokens, d_ntok)
    out_struct, out = tr.make_step_out(ctx)
    # integer loop state on both sides
    M = synth.seeded_matrix(w)
    for b in range(B):
        tr.tr_matrix_import(ctx, b, M[b])
    Mo = [m.astype(np.int64) for m in M]
    succ, noise = synth.zipf_successors(w), synth.noise_logits(w, 2)
    roots = synth.root_tokens(w)
    d_tree = torch.zeros(B, N, dtype=torch.int32, device=dev)
    tr.tr_build_tree(ctx, torch.from_numpy(roots).to(dev), d_tree)
    So = [orc.bfs_tree(Mo[b], parent, rank, int(roots[b])) for b in range(B)]
    c_o, tok_o = list(w.ctx), [[] for _ in range(B)]
    for s in range(steps):
        logits = np.stack([synth.step_logits(noise[s % 2, b], So[b], succ, w.boost) for b in range(B)])
        tr.tr_tree_attention(ctx, attn)
        tr.tr_verify_update(ctx, torch.from_numpy(logits).to(dev), d_tree, out_struct)
        tr.tr_commit(ctx, cargs, out["acc_nodes"], out["out_tokens"], out["n_new"])
        d_tree.copy_(out["next_tree"])
        torch.cuda.synchronize()
        if s == steps - 1:                                    # attention of the last step, at the grown prefix
            for b in range(B):
                for l in range(L):
                    ref = orc.tree_attention(synth.bf16_bits_to_f32(q_h[b, l]),
                                             synth.bf16_bits_to_f32(k_h[b, l, :, : c_o[b] + N]),
                                             synth.bf16_bits_to_f32(v_h[b, l, :, : c_o[b] + N]), c_o[b], parent)
                    got = d_o[b, l].float().cpu().numpy()
                    for h in range(Hq):
                        mx, rel = attention_close(got[:, h], ref[:, h])
                        assert mx <= ATOL and rel <= RTOL, (b, l, h, mx, rel)
        for b in range(B):
            rec = orc.verify_update(Mo[b], So[b], logits[b], parent, rank)
            c_o[b], tok_o[b] = orc.commit(k_h[b], v_h[b], c_o[b], tok_o[b], rec["acc_nodes"], rec["out_tokens"])
            So[b] = rec["next_tree"]
        assert d_ctx.cpu().tolist() == c_o
        assert d_ntok.cpu().tolist() == [len(t) for t in tok_o]
    assert tr.tr_device_flags(ctx) == 0
    for b in range(B):
        assert d_tokens[b, : len(tok_o[b])].cpu().tolist() == tok_o[b]
        assert len(tok_o[b]) > steps                           # some drafts were accepted along the way
    assert (d_k.view(torch.int16).cpu().numpy().view(np.uint16) == k_h).all()
    assert (d_v.view(torch.int16).cpu().numpy().view(np.uint16) == v_h).all()
    # a cache without room for another tree: flagged, sequence left untouched
    d_ctx[0] = cap_rows - N
    before = d_ctx.clone()
    tr.tr_commit(ctx, cargs, out["acc_nodes"], out["out_tokens"], out["n_new"])
    assert tr.tr_device_flags(ctx) & tr.TR_FLAG_CACHE_FULL
    assert d_ctx[0].item() == before[0].item()
    tr.tr_destroy(ctx)


# ------------------------------------------------------------------ whole step, host-buffer entry point
@pytest.mark.parametrize("ctxs,L", [((100,), 2), ((100, 37, 64), 5)])
def test_step_host_matches_device_calls(harness, tr, ctxs, L):
    """The host-buffer entry point (copies pipelined over two layer groups, one strided copy per sequence and group
    for the tree K/V rows): one sequence, and three sequences with different prefix lengths over five layers."""
    w = dataclasses.replace(synth.WORKLOADS["tiny"], ctx=ctxs)
    dw = harness.DeviceWorkload(w, n_layers=L)
    ol = OracleLoop(w)
    B, N, V, Hq, Hkv, D = w.batch, w.n_nodes, w.vocab, w.n_q_heads, w.n_kv_heads, w.head_dim
    q, k, v = synth.attention_inputs(w, L)
    h_q = torch.from_numpy(q.view(np.int16)).pin_memory()
    tk = np.stack([k[b, :, :, c:c + N] for b, c in enumerate(w.ctx)])
    tv = np.stack([v[b, :, :, c:c + N] for b, c in enumerate(w.ctx)])
    h_tk = torch.from_numpy(np.ascontiguousarray(tk).view(np.int16)).pin_memory()
    h_tv = torch.from_numpy(np.ascontiguousarray(tv).view(np.int16)).pin_memory()
    for b, c in enumerate(w.ctx):       # the call itself must place the tree rows
        dw.k[b, :, :, c:c + N] = 0
        dw.v[b, :, :, c:c + N] = 0
    logits = np.stack([synth.step_logits(ol.noise[0, b], ol.S[b], ol.succ, w.boost) for b in range(B)])
    h_logits = torch.from_numpy(logits).pin_memory()
    h_ctx = np.array(w.ctx, dtype=np.int32)
    h_out = torch.zeros(B, L, N, Hq, D, dtype=torch.bfloat16).pin_memory()
    h_n_new = torch.zeros(B, dtype=torch.int32).pin_memory()
    h_tokens = torch.zeros(B, dw.ctx.max_new, dtype=torch.int32).pin_memory()
    h_next = torch.zeros(B, N, dtype=torch.int32).pin_memory()
    io = tr.tr_host_io()
    io.h_q, io.h_tree_k, io.h_tree_v = h_q.data_ptr(), h_tk.data_ptr(), h_tv.data_ptr()
    io.h_logits, io.h_ctx_len = h_logits.data_ptr(), h_ctx.ctypes.data
    io.d_logits_staging, io.d_tree = dw.d_logits[0].data_ptr(), dw.d_tree.data_ptr()
    io.h_out, io.h_n_new, io.h_out_tokens, io.h_next_tree = (h_out.data_ptr(), h_n_new.data_ptr(),
                                                             h_tokens.data_ptr(), h_next.data_ptr())
    dw.q.zero_()
    tr.tr_step_host(dw.ctx, dw.attn, dw.out_struct, io)
    recs = ol.step(0)
    compare_step(recs, dw.snapshot(), dw.ctx.max_new)
    for b in range(B):
        assert h_n_new[b].item() == recs[b]["n_new"]
        assert h_tokens[b, : recs[b]["n_new"]].tolist() == recs[b]["out_tokens"]
        assert (h_next[b].numpy() == recs[b]["next_tree"]).all()
        for l in range(L):
            ref = oracle_attention(w, q, k, v, b, l, dw.parent)
            for h in range(Hq):
                mx, rel = attention_close(h_out[b, l, :, h].float().numpy(), ref[:, h])
                assert mx <= ATOL and rel <= RTOL
    assert tr.tr_device_flags(dw.ctx) == 0
    dw.close()
