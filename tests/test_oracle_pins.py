"""Pins for the CPU oracle: each check uses something other than the oracle's
own formula - values the paper prints, closed forms, brute force, a library
routine on a special case - so that a wrong sign, index or dropped term fails."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import tr_oracle as orc
from paper_2408_08696_b200 import synth


def _read_golden(path):
    rows = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = line.split(":", 1)
        rows[key.strip()] = [int(x) for x in val.split()]
    return rows


# ---------------------------------------------------------------- template
def test_template_level_histograms(golden_dir):
    for line in open(os.path.join(golden_dir, "template_levels.txt")):
        if line.startswith("#") or not line.strip():
            continue
        parts = [p.split(":")[1].split() for p in line.split("|")]
        b, max_nodes, levels = [int(x) for x in parts[0]], int(parts[1][0]), [int(x) for x in parts[2]]
        parent, rank = orc.template_from_branching(b, max_nodes)
        assert len(parent) == max_nodes
        depth = orc.node_depth(parent)
        assert np.bincount(depth).tolist() == levels


def test_template_structure_is_layer_ordered_and_left_heavy():
    parent, rank = orc.template_from_branching((8, 4, 3, 2, 2, 1), 80)
    depth = orc.node_depth(parent)
    assert parent[0] == -1 and rank[0] == 0
    assert all(parent[i] < i for i in range(1, 80))
    assert all(depth[i] <= depth[i + 1] for i in range(79))          # layer order
    assert all(parent[i] <= parent[i + 1] for i in range(1, 79))     # parent by parent
    # siblings: ranks 0,1,2.. in order
    for p in range(80):
        kids = [i for i in range(80) if parent[i] == p]
        assert [rank[i] for i in kids] == list(range(len(kids)))
    # imbalance (Sec. 3.2): earlier siblings never have fewer children than later ones
    nchild = np.bincount(parent[1:], minlength=80)
    for p in range(80):
        kids = [i for i in range(80) if parent[i] == p]
        full = [i for i in kids if depth[i] < 4]       # away from the truncated last level
        assert all(nchild[a] >= nchild[b] for a, b in zip(full, full[1:]))
    # paper: maximum acceptance length 6 with 6 layers -> deepest node at depth 5 (+1 bonus token)
    assert depth.max() + 1 == 6
    assert rank.max() < 8


def test_storage_matches_table_2():
    # Table 2 / Sec. 4.1: k=8 costs 1.95 MB (< 2 MB): V*k entries; 8-byte ids give 1.953 MiB,
    # the int32 matrix of this build is half of that.
    V, k = 32000, 8
    M = np.zeros((V, k), dtype=np.int32)
    assert M.size == V * k
    assert abs(V * k * 8 / 2**20 - 1.95) < 0.01
    assert M.nbytes == 1_024_000 and M.nbytes < 2 * 2**20


# ---------------------------------------------------------------- argtopk
def _brute_topk(row, k):
    idx = list(range(len(row)))
    chosen = []
    for _ in range(k):
        best = None
        for i in idx:
            if i in chosen:
                continue
            if best is None or row[i] > row[best]:      # strict: first (lowest) index wins ties
                best = i
        chosen.append(best)
    return chosen


def test_topk_bruteforce_ties():
    rng = np.random.default_rng(1)
    for trial in range(20):
        v = int(rng.integers(8, 60))
        x = rng.integers(-3, 4, size=(5, v)).astype(np.float32)       # heavy ties
        got = orc.argtopk(x, 8)
        for i in range(5):
            assert got[i].tolist() == _brute_topk(x[i].tolist(), 8)


def test_topk_special_values():
    ninf = -np.inf
    x = np.array([[ninf, 0.0, -0.0, 5.0, ninf, 5.0, -1.0, 0.0, 2.0]], dtype=np.float32)
    # 5.0@3, 5.0@5, 2.0@8, zeros (signed zeros compare equal -> index order 1,2,7), -1@6, -inf@0
    assert orc.argtopk(x, 8)[0].tolist() == [3, 5, 8, 1, 2, 7, 6, 0]
    assert orc.argtopk(np.zeros((1, 20), np.float32), 8)[0].tolist() == list(range(8))


def test_topk_column0_is_argmax_and_matches_library_without_ties():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((16, 5000)).astype(np.float32)
    got = orc.argtopk(x, 8)
    assert (got[:, 0] == x.argmax(axis=1)).all()                   # Sec. 2.1: x^0 = argmax
    lib = torch.topk(torch.from_numpy(x), 8, dim=1).indices.numpy()
    assert (got == lib).all()
    vals = np.take_along_axis(x, got, axis=1)
    assert (np.diff(vals, axis=1) <= 0).all()


# ---------------------------------------------------------------- attention
def _causal_path_attention(q_path, k_all, v_all, scale):
    """Plain causal attention of one linear sequence: prefix rows then the path
    rows; query t sees the prefix and path rows 0..t.  Pure Python loops."""
    out = []
    c = k_all.shape[0] - q_path.shape[0]
    for t in range(q_path.shape[0]):
        ks = k_all[: c + t + 1]
        vs = v_all[: c + t + 1]
        s = [float(np.dot(q_path[t], kk)) * scale for kk in ks]
        m = max(s)
        e = [np.exp(si - m) for si in s]
        z = sum(e)
        out.append(sum(ei / z * vi for ei, vi in zip(e, vs)))
    return np.stack(out)


@pytest.mark.parametrize("hq,hkv", [(2, 2), (4, 2)])
def test_tree_attention_equals_per_path_causal(hq, hkv):
    rng = np.random.default_rng(3)
    parent, rank = orc.template_from_branching((3, 2, 1), 9)
    n, d, c = len(parent), 8, 5
    q = rng.standard_normal((n, hq, d))
    k = rng.standard_normal((hkv, c + n, d))
    v = rng.standard_normal((hkv, c + n, d))
    out = orc.tree_attention(q, k, v, c, parent)
    scale = 1 / np.sqrt(d)
    leaves = [i for i in range(n) if i not in set(parent.tolist())]
    covered = set()
    for leaf in leaves:
        path = []
        j = leaf
        while j >= 0:
            path.append(j)
            j = parent[j]
        path = path[::-1]
        for h in range(hq):
            g = h // (hq // hkv)
            k_lin = np.concatenate([k[g, :c], k[g, c + np.array(path)]])
            v_lin = np.concatenate([v[g, :c], v[g, c + np.array(path)]])
            ref = _causal_path_attention(q[path, h], k_lin, v_lin, scale)
            np.testing.assert_allclose(out[path, h], ref, rtol=1e-12, atol=1e-12)
        covered.update(path)
    assert covered == set(range(n))


def test_tree_attention_needs_self_key():
    # Root with no prefix sees only itself: output must be exactly its own value row.
    parent = np.array([-1, 0, 0])
    rng = np.random.default_rng(4)
    q, k, v = rng.standard_normal((3, 1, 4)), rng.standard_normal((1, 3, 4)), rng.standard_normal((1, 3, 4))
    out = orc.tree_attention(q, k, v, 0, parent)
    np.testing.assert_allclose(out[0, 0], v[0, 0], rtol=1e-14)
    # siblings 1 and 2 never see each other: changing node 2's key/value leaves node 1 unchanged
    k2, v2 = k.copy(), v.copy()
    k2[0, 2] += 5.0
    v2[0, 2] -= 7.0
    out2 = orc.tree_attention(q, k2, v2, 0, parent)
    np.testing.assert_array_equal(out[1], out2[1])
    assert not np.allclose(out[2], out2[2])


def test_tree_attention_closed_forms():
    parent, _ = orc.template_from_branching((2, 2), 7)
    n, d, c = 7, 6, 4
    rng = np.random.default_rng(5)
    q = rng.standard_normal((n, 1, d))
    v = rng.standard_normal((1, c + n, d))
    # all keys equal -> uniform weights over the visible set -> mean of visible values
    k = np.tile(rng.standard_normal((1, 1, d)), (1, c + n, 1))
    out = orc.tree_attention(q, k, v, c, parent)
    anc = orc.ancestor_mask(parent)
    for i in range(n):
        vis = list(range(c)) + [c + j for j in range(n) if anc[i, j]]
        np.testing.assert_allclose(out[i, 0], v[0, vis].mean(axis=0), rtol=1e-12)
    # one dominating key (a prefix row aligned with every query) -> that value row
    k = np.zeros((1, c + n, d))
    q = np.ones((n, 1, d))
    k[0, 2] = 1000.0
    out = orc.tree_attention(q, k, v, c, parent)
    np.testing.assert_allclose(out[:, 0], np.tile(v[0, 2], (n, 1)), rtol=1e-9)


def test_tree_attention_single_node_is_library_decode():
    rng = np.random.default_rng(6)
    d, c, h = 16, 33, 3
    q = rng.standard_normal((1, h, d)).astype(np.float32)
    k = rng.standard_normal((h, c + 1, d)).astype(np.float32)
    v = rng.standard_normal((h, c + 1, d)).astype(np.float32)
    out = orc.tree_attention(q, k, v, c, np.array([-1]))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).permute(1, 0, 2), torch.from_numpy(k), torch.from_numpy(v))
    np.testing.assert_allclose(out[0], ref[:, 0].numpy(), rtol=2e-5, atol=2e-6)


def test_tree_attention_gqa_head_mapping():
    rng = np.random.default_rng(7)
    parent, _ = orc.template_from_branching((2, 1), 4)
    q = rng.standard_normal((4, 4, 8))
    k, v = rng.standard_normal((2, 7, 8)), rng.standard_normal((2, 7, 8))
    out = orc.tree_attention(q, k, v, 3, parent)
    for h in range(4):
        one = orc.tree_attention(q[:, h:h + 1], k[h // 2:h // 2 + 1], v[h // 2:h // 2 + 1], 3, parent)
        np.testing.assert_allclose(out[:, h], one[:, 0], rtol=1e-13)


# ---------------------------------------------------------------- accept
def _brute_accept(S, argmax, parent):
    n = len(S)
    best_len, best_leaf = 0, 0
    for leaf in range(n):
        path, j = [], leaf
        while j >= 0:
            path.append(j)
            j = parent[j]
        path = path[::-1]
        ok = all(S[c] == argmax[parent[c]] for c in path[1:])
        if ok and len(path) - 1 > best_len:
            best_len, best_leaf = len(path) - 1, leaf
    return best_len + 1, best_leaf


def test_accept_bruteforce_including_duplicates():
    rng = np.random.default_rng(8)
    parent, _ = orc.template_from_branching((4, 2, 1), 15)
    for trial in range(300):
        S = rng.integers(0, 3, size=15)
        am = rng.integers(0, 3, size=15)
        n_new, acc, toks, nxt = orc.accept(S, am, parent)
        bn, bleaf = _brute_accept(S, am, parent)
        assert n_new == bn and acc[-1] == bleaf and acc[0] == 0
        assert 1 <= n_new <= orc.node_depth(parent).max() + 1
        assert toks[-1] == am[acc[-1]] == nxt
        assert toks[:-1] == [S[c] for c in acc[1:]]


def test_accept_nothing_matches_gives_one_token():
    parent, _ = orc.template_from_branching((4, 2, 1), 15)
    S = np.arange(15) + 100
    am = np.arange(15)
    assert orc.accept(S, am, parent) == (1, [0], [0], 0)      # AR step: MAT counts the bonus token


def _toy_logits(path_tokens, V, salt):
    """Deterministic toy model: logits are a pure function of the token path."""
    h = salt
    for t in path_tokens:
        h = (h * 1000003 + int(t) + 12345) % (2**61 - 1)
    return np.random.default_rng(h).standard_normal(V).astype(np.float32)


@pytest.mark.parametrize("init", ["zero", "random"])
def test_losslessness_against_greedy_decoding(init):
    """Sec. 1 / Sec. 2.2: speculative decoding with verification emits exactly the
    greedy sequence, whatever the matrix and template hold."""
    V, k, steps = 50, 4, 25
    parent, rank = orc.template_from_branching((3, 2, 1), 10)
    rng = np.random.default_rng(9)
    M = np.zeros((V, k), dtype=np.int64) if init == "zero" else rng.integers(0, V, size=(V, k))
    prefix = [7]
    ar = list(prefix)
    for _ in range(steps * 4 + 4):
        ar.append(int(np.argmax(_toy_logits(ar, V, 5))))
    seq = list(prefix)
    S = orc.bfs_tree(M, parent, rank, seq[-1])
    mats = []
    for _ in range(steps):
        logits = np.zeros((len(parent), V), dtype=np.float32)
        for i in range(len(parent)):
            path, j = [], i
            while j > 0:
                path.append(int(S[j]))
                j = parent[j]
            logits[i] = _toy_logits(seq + path[::-1], V, 5)
        r = orc.verify_update(M, S, logits, parent, rank)
        assert S[0] == seq[-1]
        seq += r["out_tokens"]
        assert r["next_tree"][0] == seq[-1]
        S = r["next_tree"]
        mats.append(r["n_new"])
        assert ((M >= 0) & (M < V)).all()
    assert seq == ar[: len(seq)]
    assert max(mats) > 1            # recycling does accept drafts on this toy model


# ---------------------------------------------------------------- update
def test_update_last_writer_matches_appendix_example(golden_dir):
    g = _read_golden(os.path.join(golden_dir, "update_last_example.txt"))
    S = np.array(g["S"])
    O = np.array([g["O%d" % i] for i in range(5)])
    M = np.full((20, 4), -1, dtype=np.int64)
    orc.update_matrix(M, S, O)
    assert M[10].tolist() == g["M[a] last"] != g["M[a] first"]
    assert M[11].tolist() == g["M[b]"] and M[12].tolist() == g["M[c]"] and M[13].tolist() == g["M[d]"]
    untouched = [i for i in range(20) if i not in (10, 11, 12, 13)]
    assert (M[untouched] == -1).all()
    # "First": positions of each token's first occurrence
    M1 = np.full((20, 4), -1, dtype=np.int64)
    orc.update_matrix(M1, S, O, rule="first")
    assert M1[10].tolist() == g["M[a] first"] and M1[13].tolist() == g["M[d]"] and (M1[untouched] == -1).all()
    # only a subset of the nodes (the "only accepted" setting): others keep their old rows
    M2 = np.full((20, 4), -1, dtype=np.int64)
    orc.update_matrix(M2, S, O, nodes=[0, 2])
    assert M2[10].tolist() == g["M[a] first"] and M2[12].tolist() == g["M[c]"] and (M2[[11, 13]] == -1).all()


def test_update_covers_root_and_rejected_nodes():
    # Sec. 3.3 / Sec. 5.2 "Effect of Rejected Tokens": every node of S gets its row, not only accepted ones.
    parent, rank = orc.template_from_branching((2, 1), 4)
    V, k = 30, 2
    M = np.zeros((V, k), dtype=np.int64)
    S = np.array([5, 6, 7, 8])
    logits = np.full((4, V), -1.0, dtype=np.float32)
    for i in range(4):
        logits[i, 20 + i] = 3.0
        logits[i, 10 + i] = 2.0
    r = orc.verify_update(M, S, logits, parent, rank)
    assert r["n_new"] == 1                                    # nothing accepted
    for i, t in enumerate(S):
        assert M[t].tolist() == [20 + i, 10 + i]


# ---------------------------------------------------------------- BFS
def test_bfs_matches_section_3_2_walkthrough(golden_dir):
    g = _read_golden(os.path.join(golden_dir, "bfs_walkthrough.txt"))
    M = np.zeros((11, 3), dtype=np.int64)
    for t in (1, 2, 3):
        M[t] = g["M[%d]" % t]
    S = orc.bfs_tree(M, np.array(g["parent"]), np.array(g["rank"]), g["root"][0])
    assert S.tolist() == g["S"]


def _algorithm_1_layer_by_layer(M, parent, rank, root):
    """Algorithm 1 as printed, with the depth counter advancing once per iteration: the current layer L starts as
    (root); xs = M[L] holds all candidates of the layer; the template picks from the flattened xs the entries
    (position of the parent inside L) * k + rank for each child; S collects the layers in order."""
    n, k = len(parent), M.shape[1]
    depth = orc.node_depth(parent)
    S, L, layer_nodes, d = [], np.asarray([root], dtype=np.int64), [0], 0
    while len(S) < n:
        S.extend(int(t) for t in L)
        xs = M[L]
        nxt = [i for i in range(n) if depth[i] == d + 1]
        pos = {node: p for p, node in enumerate(layer_nodes)}
        index = [pos[parent[i]] * k + rank[i] for i in nxt]
        L = xs.reshape(-1)[index] if index else np.zeros(0, dtype=np.int64)
        layer_nodes, d = nxt, d + 1
        if not nxt:
            break
    return S


@pytest.mark.parametrize("b,n", [((8, 4, 3, 2, 2, 1), 80), ((4, 2, 1), 15), ((2,) * 6, 127), ((1,) * 9, 10), ((16,), 17)])
def test_bfs_equals_algorithm_1_layer_by_layer(b, n):
    parent, rank = orc.template_from_branching(b, n)
    rng = np.random.default_rng(n)
    V, k = 300, 16
    M = rng.integers(0, V, size=(V, k))
    for root in (0, 7, V - 1):
        assert orc.bfs_tree(M, parent, rank, root).tolist() == _algorithm_1_layer_by_layer(M, parent, rank, root)


def test_bfs_node_count_parent_structure_and_zero_matrix():
    parent, rank = orc.template_from_branching((8, 4, 3, 2, 2, 1), 80)
    rng = np.random.default_rng(10)
    V, k = 500, 8
    M = rng.integers(0, V, size=(V, k))
    S = orc.bfs_tree(M, parent, rank, 17)
    assert len(S) == 80 and S[0] == 17
    for i in range(1, 80):                                    # per-node statement of Algorithm 1
        assert S[i] == M[S[parent[i]], rank[i]]
    Z = orc.bfs_tree(np.zeros((V, k), dtype=np.int64), parent, rank, 17)
    assert Z[0] == 17 and (Z[1:] == 0).all()                  # Sec. 3.1: zero init -> no valid candidates yet


# ---------------------------------------------------------------- generators
def test_synth_is_seeded_and_shaped():
    w = synth.WORKLOADS["tiny"]
    a, b = synth.noise_logits(w, 2), synth.noise_logits(w, 2)
    assert a.shape == (2, 1, 15, 1000) and (a == b).all()
    succ = synth.zipf_successors(w)
    assert succ.min() >= 0 and succ.max() < w.vocab
    assert (succ < 10).mean() > 0.3                            # Zipf(1.1): mass on the first ranks
    q, k, v = synth.attention_inputs(w)
    assert q.shape == (1, 1, 15, 4, 64) and k.shape == (1, 1, 4, 143, 64)
    pool = synth.normal_pool(w.seed)
    qs, ks, vs = synth.attention_slice(w, pool, 0, 0, 2)
    assert (ks == k[0, 0, 2]).all() and (vs == v[0, 0, 2]).all() and (qs == q[0, 0]).all()
    x = np.array([1.0, 1.00390625, -2.5, 3.1415926], dtype=np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert (synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x)) == ref).all()
    lg = synth.step_logits(a[0, 0], np.zeros(15, dtype=np.int64), succ, 4.0)
    assert np.count_nonzero(lg != a[0, 0]) == 15
    assert len(synth.WORKLOADS["llama2-70b-b8"].ctx) == 8


# ---------------------------------------------------------------- commit of the accepted path
def test_commit_hand_example_and_gather_property():
    # tree rows sit at 3..8 of a 10-row cache (prefix C = 3, N = 6); accepted path = nodes 0, 2, 5
    k = np.arange(10, dtype=np.float64)[None, :, None] * np.ones((2, 1, 4)) + np.array([0.0, 100.0])[:, None, None]
    v = -k.copy()
    k0, v0 = k.copy(), v.copy()
    c, toks = orc.commit(k, v, 3, [9, 9, 9], [0, 2, 5], [41, 42, 43])
    assert c == 6 and toks == [9, 9, 9, 41, 42, 43]
    assert k[0, :, 0].tolist() == [0, 1, 2, 3, 5, 8, 6, 7, 8, 9]          # rows 3,4,5 <- old rows 3,5,8
    assert (k[:, 3:6] == k0[:, [3, 5, 8]]).all() and (v[:, 3:6] == v0[:, [3, 5, 8]]).all()
    assert (k[:, :3] == k0[:, :3]).all() and (k[:, 6:] == k0[:, 6:]).all()  # nothing else moves
    # overlapping case: a later destination is an earlier source (path 0, 1, 2 after 0, 2, ... is impossible; use 0,2,3)
    k = k0.copy(); v = v0.copy()
    orc.commit(k, v, 3, [], [0, 2, 3], [1, 2, 3])
    assert k[0, 3:6, 0].tolist() == [3, 5, 6]


# ---------------------------------------------------------------------------
# Output layer + argtopk (Sec. 2.1: p = M(x), x^0..x^{k-1} = argtopk(p))
# ---------------------------------------------------------------------------
def test_lm_head_bruteforce_small_integers():
    """Pure-Python integer dot products and a (-value, index) sort on a tiny case full of ties."""
    r = np.random.default_rng(5)
    rows, H, V, k = 4, 6, 9, 5
    hid = r.integers(-2, 3, size=(rows, H))
    wt = r.integers(-2, 3, size=(V, H))
    idx, logits = orc.lm_head_topk(hid, wt, k)
    for i in range(rows):
        dots = [sum(int(hid[i, h]) * int(wt[v, h]) for h in range(H)) for v in range(V)]
        assert [float(d) for d in dots] == list(logits[i])
        want = sorted(range(V), key=lambda v: (-dots[v], v))[:k]
        assert list(idx[i]) == want
    # a transposed weight or a sum over the wrong axis cannot pass: V != H here and wt is not symmetric


def test_lm_head_one_hot_rows_select_weight_columns():
    """hidden = e_h picks column h of the weight: the top-k is then the top-k of that column."""
    r = np.random.default_rng(6)
    V, H, k = 50, 8, 4
    wt = r.standard_normal((V, H)).astype(np.float32)
    hid = np.zeros((H, H), dtype=np.float32)
    hid[np.arange(H), np.arange(H)] = 1.0
    idx, logits = orc.lm_head_topk(hid, wt, k)
    for h in range(H):
        assert np.array_equal(logits[h], wt[:, h].astype(np.float64))
        want = sorted(range(V), key=lambda v: (-float(wt[v, h]), v))[:k]
        assert list(idx[h]) == want


def test_lm_head_vocabulary_permutation_and_positive_scaling():
    """Permuting the vocabulary rows of the weight permutes the indices; a positive scale of the hidden states
    leaves them unchanged (tie-free random values)."""
    r = np.random.default_rng(7)
    rows, V, H, k = 5, 64, 16, 6
    hid = r.standard_normal((rows, H)).astype(np.float32)
    wt = r.standard_normal((V, H)).astype(np.float32)
    idx, _ = orc.lm_head_topk(hid, wt, k)
    perm = r.permutation(V)
    idx_p, _ = orc.lm_head_topk(hid, wt[perm], k)
    assert np.array_equal(perm[idx_p], idx)
    idx_s, _ = orc.lm_head_topk(hid * 4.0, wt, k)
    assert np.array_equal(idx_s, idx)


def test_lm_head_synthetic_inputs():
    w = synth.WORKLOADS["tiny"]
    h1, w1 = synth.lm_head_inputs(w)
    h2, w2 = synth.lm_head_inputs(w)
    assert np.array_equal(h1, h2) and np.array_equal(w1, w2)
    assert h1.shape == (w.batch * w.n_nodes, w.n_q_heads * w.head_dim) and w1.shape == (w.vocab, h1.shape[1])
    hi, wi = synth.lm_head_inputs(w, kind="small-int")
    fi, fw = synth.bf16_bits_to_f32(hi), synth.bf16_bits_to_f32(wi)
    assert np.array_equal(fi, np.round(fi)) and np.abs(fi).max() <= 2 and np.abs(fw).max() <= 3
    # small-integer inputs: the logits are exact integers, identical in float32 and float64
    _, logits = orc.lm_head_topk(fi, fw, w.k)
    assert np.array_equal(logits, np.round(logits)) and np.array_equal(logits.astype(np.float32).astype(np.float64), logits)


# ---------------------------------------------------------------------------
# Temperature sampling (Sec. 5.3): the draw as a Gumbel-max, then greedy-style matching
# ---------------------------------------------------------------------------
def test_sample_tokens_without_noise_is_the_argmax_and_noise_can_overturn_it():
    r = np.random.default_rng(11)
    logits = r.standard_normal((9, 40)).astype(np.float32)
    logits[3, 7] = logits[3, 21] = logits[3].max() + 1      # a tie: the lower index wins
    zero = np.zeros_like(logits)
    for inv_t in (1.0, 0.25, 3.0):
        assert np.array_equal(orc.sample_tokens(logits, zero, inv_t), orc.argtopk(logits, 1)[:, 0])
    # hand case: logits (2, 1, 0) at T = 0.5 -> scaled (4, 2, 0); noise (0, 3, 0) makes index 1 the draw (5 > 4)
    lg = np.array([[2.0, 1.0, 0.0]], dtype=np.float32)
    assert orc.sample_tokens(lg, np.array([[0.0, 3.0, 0.0]], dtype=np.float32), 2.0)[0] == 1
    assert orc.sample_tokens(lg, np.array([[0.0, 1.5, 0.0]], dtype=np.float32), 2.0)[0] == 0


def test_sample_tokens_follow_the_softmax_at_temperature():
    """Gumbel-max theorem: the frequencies of many draws match softmax(logits / T)."""
    r = np.random.default_rng(12)
    logits = np.array([1.5, 0.3, -0.2, 2.0, 0.0, -1.0], dtype=np.float32)
    for T in (0.5, 1.0):
        n = 60000
        u = r.random((n, logits.size))
        g = (-np.log(-np.log(u))).astype(np.float32)
        draws = orc.sample_tokens(np.broadcast_to(logits, (n, logits.size)), g, 1.0 / T)
        freq = np.bincount(draws, minlength=logits.size) / n
        p = np.exp(logits.astype(np.float64) / T)
        p /= p.sum()
        assert np.abs(freq - p).max() < 4 * np.sqrt(0.25 / n) + 1e-3      # four standard errors of a proportion


def test_sampled_verification_equals_token_by_token_sampling():
    """Losslessness under sampling: TR with 'sample, then match' emits exactly the tokens that token-by-token
    decoding with the same per-position draws emits (toy model: logits depend on the last token only, the draw at a
    position uses that position's noise row)."""
    r = np.random.default_rng(13)
    V, k, steps = 50, 4, 20
    parent, rank = orc.template_from_branching((3, 2, 1), 12)
    table = r.standard_normal((V, V)).astype(np.float32) * 2      # next-token logits given the last token
    M = r.integers(0, V, size=(V, k)).astype(np.int64)
    root = 5
    # one noise row per absolute position, so both decoders see the same randomness
    noise = (-np.log(-np.log(r.random((400, V))))).astype(np.float32)
    inv_t = 1.0 / 0.7
    # token-by-token
    ref = [root]
    for pos in range(300):
        ref.append(int(orc.sample_tokens(table[ref[-1]][None], noise[pos][None], inv_t)[0]))
    # TR: node i of the tree sits at position pos + depth(i); its draw uses that position's noise row
    depth = orc.node_depth(parent)
    out = [root]
    S = orc.bfs_tree(M, parent, rank, root)
    for _ in range(steps):
        pos = len(out) - 1
        logits = table[S]                                          # [N, V]
        g = noise[pos + np.asarray(depth)]
        rec = orc.verify_update_sampled(M, S, logits, g, inv_t, parent, rank)
        out.extend(rec["out_tokens"])
        S = rec["next_tree"]
    assert out == ref[:len(out)]
    assert len(out) - 1 > steps        # some drafts were accepted
