"""CPU oracle for one Token Recycling verify-and-recycle step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA path is checked against.  It shares no code with the CUDA path and is
imported only by the tests, by the smoke check and by the benchmark's
``cpu_baseline`` / ``--impl reference`` legs.  The product path never calls it.

Everything is written in the paper's order and notation:

  V      vocabulary size                       (Sec. 3.1)
  k      candidates stored per token           (Sec. 3.1)
  M      adjacency matrix, int [V, k]          (Sec. 3.1)
  Tree   static template: parent[i], rank[i]   (Sec. 3.2, Appendix "Draft Tree
         Algorithm and Structure", Algorithm 1)
  S      merged sequence = tree tokens in layer (BFS) order, root first
                                               (Sec. 3.3, Algorithm 1)
  O      per-node argtopk of the output distribution (Appendix "Explanation of
         Three Update Strategies")

Floating point: attention is evaluated in float64 from the given inputs.
Top-k only compares float32 values, so it is exact.

Pin status (tests/test_oracle_pins.py): every function below is pinned by a
test that does not re-use its own formula; see each docstring.  The whole step
has no printed numeric example in the paper, so `step` is pinned only through
its parts and through the losslessness property (Sec. 1, Sec. 2.2).
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------
# Static tree template (Sec. 3.2 "static and imbalanced"; Appendix tree figure)
# --------------------------------------------------------------------------
def template_from_branching(b, max_nodes):
    """Build a static, left-heavy tree template in layer order.

    The paper's own tree is given only as a figure; the workload definition
    used here generates one by rule: a node at depth d whose rank among its
    siblings is r gets max(0, b[d] - r) children, children are appended parent
    by parent with rank ascending, and the list is cut at `max_nodes`.  Depths
    past the end of `b` re-use its last entry.  The rule reproduces the
    properties Sec. 3.2 states: earlier nodes in a layer have more children and
    reach deeper, and the number on a node is the column of M it is drawn from.

    Returns (parent, rank): parent[0] = -1, rank[0] = 0.
    Pinned by: node counts and per-level histograms worked out by hand
    (1,8,10,20,25,16 for b=(8,4,3,2,2,1) cut at 80; 1,4,3,2,2,2,1 for
    b=(4,2,1) cut at 15).
    """
    b = list(b)
    parent, rank, depth = [-1], [0], [0]
    head = 0
    while head < len(parent) and len(parent) < max_nodes:
        d = depth[head]
        bd = b[min(d, len(b) - 1)]
        for r in range(max(0, bd - rank[head])):
            if len(parent) >= max_nodes:
                break
            parent.append(head)
            rank.append(r)
            depth.append(d + 1)
        head += 1
    return np.asarray(parent, dtype=np.int64), np.asarray(rank, dtype=np.int64)


def node_depth(parent):
    """Depth of every node (root = 0)."""
    depth = np.zeros(len(parent), dtype=np.int64)
    for i in range(1, len(parent)):
        depth[i] = depth[parent[i]] + 1
    return depth


def ancestor_mask(parent):
    """anc[i, j] is True iff j == i or j is an ancestor of i (Sec. 2.2: a node
    attends to the nodes on its own root path, never to siblings)."""
    n = len(parent)
    anc = np.zeros((n, n), dtype=bool)
    for i in range(n):
        j = i
        while j >= 0:
            anc[i, j] = True
            j = parent[j]
    return anc


# --------------------------------------------------------------------------
# Tree attention (Sec. 2.2 "Tree Attention")
# --------------------------------------------------------------------------
def tree_attention(q, k, v, ctx_len, parent, scale=None):
    """Masked attention of the tree's queries over prefix + tree keys.

    q : [N, Hq, D]        queries of the N tree nodes
    k : [Hkv, C + N, D]   keys; rows 0..C-1 are the prefix, rows C..C+N-1 the
    v : [Hkv, C + N, D]   tree nodes in the same order as q
    Node i sees every prefix row and tree row j iff j is i or an ancestor of i.
    Query head h uses KV head h // (Hq // Hkv).
    Returns float64 [N, Hq, D].

    Pinned by: equality with plain causal attention run separately over
    prefix + each root-to-leaf path; closed forms (equal keys -> mean of the
    visible values; one dominating key -> that value row); N = 1 against a
    library attention routine.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    n, hq, d = q.shape
    hkv = k.shape[0]
    c = int(ctx_len)
    group = hq // hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    anc = ancestor_mask(parent)
    visible = np.concatenate([np.ones((n, c), dtype=bool), anc], axis=1)  # [N, C+N]
    out = np.zeros((n, hq, d), dtype=np.float64)
    for h in range(hq):
        g = h // group
        s = (q[:, h, :] @ k[g, : c + n, :].T) * scale        # [N, C+N]
        s = np.where(visible, s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)                                         # masked -> exactly 0
        p = p / p.sum(axis=1, keepdims=True)
        out[:, h, :] = p @ v[g, : c + n, :]
    return out


# --------------------------------------------------------------------------
# argtopk (Sec. 2.1)
# --------------------------------------------------------------------------
def argtopk(logits, k):
    """Indices of the k largest entries of every row, largest first; equal
    values are ordered by lower index first (the argmax convention the paper's
    appendix on identical probabilities describes, applied at every rank).
    Column 0 is therefore the argmax (Sec. 2.1: x^0 = x).

    Definition written out: sort the whole row, keep the first k.
    Pinned by: pure-Python brute force on tie-heavy rows, hand cases with
    -inf / signed zeros, agreement with a library top-k on tie-free rows.
    """
    logits = np.asarray(logits, dtype=np.float32)
    n, v = logits.shape
    out = np.zeros((n, k), dtype=np.int64)
    for i in range(n):
        # stable sort of the negated row: descending value, ascending index on ties
        order = np.argsort(-logits[i], kind="stable")
        out[i] = order[:k]
    return out


# --------------------------------------------------------------------------
# Output distribution from the last hidden states (Sec. 2.1: p = M(x); Sec. 5
# notes that the model forward dominates a step).  The last linear layer of the
# model followed directly by argtopk, so that the logits need not be stored.
# --------------------------------------------------------------------------
def lm_head_logits(hidden, weight):
    """logits[i, v] = sum_h hidden[i, h] * weight[v, h], in float64 from the
    given (bf16-valued) inputs; `weight` is [V, hidden] as a linear layer
    stores it.  Definition written out with a library matrix product.
    Pinned by: pure-Python integer dot products on a tiny case, one-hot hidden
    rows (the logits are then a column of the weight), vocabulary permutation.
    """
    hidden = np.asarray(hidden, dtype=np.float64)
    weight = np.asarray(weight, dtype=np.float64)
    return hidden @ weight.T


def lm_head_topk(hidden, weight, k):
    """argtopk of the float32-rounded logits of every row (the comparison is
    made in the kernel's precision, float32; the paper fixes none).  Returns
    (indices [n, k], logits float64 [n, V])."""
    logits = lm_head_logits(hidden, weight)
    return argtopk(logits.astype(np.float32), k), logits


# --------------------------------------------------------------------------
# Verification (Sec. 2.2 "Guess and Verify", Sec. 3.3)
# --------------------------------------------------------------------------
def accept(S, argmax, parent):
    """Longest correct path of the draft tree.

    A tree node c is correct iff its parent is correct and its token equals the
    model's greedy token after the parent, S[c] == argmax[parent[c]]; the root
    (last confirmed token) is correct by definition.  The deepest correct node
    wins, the lowest layer-order index among equally deep ones.  The step emits
    the accepted draft tokens plus one more greedy token taken at the last
    accepted node, so between 1 and depth_max + 1 tokens.

    Returns (n_new, acc_nodes, out_tokens, next_root).
    Pinned by: brute force over all root-to-node paths; losslessness against
    token-by-token greedy decoding of a toy model.
    """
    S = np.asarray(S)
    n = len(S)
    depth = node_depth(parent)
    valid = np.zeros(n, dtype=bool)
    valid[0] = True
    for c in range(1, n):
        valid[c] = valid[parent[c]] and (S[c] == argmax[parent[c]])
    best = 0
    for c in range(n):
        if valid[c] and depth[c] > depth[best]:
            best = c
    path = []
    c = best
    while c >= 0:
        path.append(c)
        c = parent[c]
    acc_nodes = path[::-1]
    out_tokens = [int(S[c]) for c in acc_nodes[1:]] + [int(argmax[best])]
    return len(out_tokens), acc_nodes, out_tokens, int(argmax[best])


# --------------------------------------------------------------------------
# Matrix update (Sec. 3.3; Appendix "Explanation of Three Update Strategies")
# --------------------------------------------------------------------------
def update_matrix(M, S, O, rule="last", nodes=None):
    """M[S[i]] <- O[i] for every node of the merged sequence, root and rejected
    nodes included, applied in increasing i: a token that occurs several times
    keeps the row of its last occurrence (the appendix's "Last" strategy, which
    is one of the outcomes the uncontrolled parallel update may produce).
    rule="first" is the appendix's "First" strategy (positions of each token's
    first occurrence); `nodes` restricts the update to a subset of the nodes
    (the "only accepted" setting of Sec. 5.2, Table 4).
    In place; also returns M.
    Pinned by: the appendix's worked example S = [a, b, c, a, d] for both rules.
    """
    idx = list(range(len(S))) if nodes is None else sorted(int(i) for i in nodes)
    if rule == "last":
        for i in idx:
            M[S[i], :] = O[i, :]
    elif rule == "first":
        for i in reversed(idx):      # going backwards, the first occurrence is written last
            M[S[i], :] = O[i, :]
    else:
        raise ValueError(rule)
    return M


# --------------------------------------------------------------------------
# Draft tree retrieval (Sec. 3.2, Algorithm 1)
# --------------------------------------------------------------------------
def bfs_tree(M, parent, rank, root):
    """Merged sequence S for the next step (Sec. 3.2): the root is the last
    confirmed token, and every other template node holds the candidate that its
    parent's token has in the column the template names,

        S[0] = root,   S[i] = M[S[parent[i]], rank[i]]   for i = 1 .. N-1,

    taken in layer order, so a parent's token is known before its children's.
    This is what Algorithm 1's layer-by-layer loop produces (its flat index
    into xs = M[L] is (position of the parent in the layer) * k + rank); the
    tests check that layered form against this definition.
    Pinned by: the two-layer walk-through of Sec. 3.2 on symbolic tokens; the
    layer-by-layer form of Algorithm 1 written out in the test; node count;
    all-zero matrix -> all drafts are token 0.
    """
    parent = np.asarray(parent)
    rank = np.asarray(rank)
    S = np.zeros(len(parent), dtype=np.int64)
    S[0] = root
    for i in range(1, len(parent)):
        S[i] = M[S[parent[i]], rank[i]]
    return S


# --------------------------------------------------------------------------
# One whole step
# --------------------------------------------------------------------------
def verify_update(M, S, logits, parent, rank, rule="last", only_accepted=False):
    """argtopk -> accept -> update M -> next tree from the updated M, rooted at
    the last confirmed token (the retrieve / verify / update cycle of Sec. 3 and
    Sec. 5.4).  M is modified in place.
    Returns dict(topk, n_new, acc_nodes, out_tokens, next_root, next_tree).
    """
    k = M.shape[1]
    O = argtopk(logits, k)
    n_new, acc_nodes, out_tokens, next_root = accept(S, O[:, 0], parent)
    update_matrix(M, S, O, rule=rule, nodes=acc_nodes if only_accepted else None)
    nxt = bfs_tree(M, parent, rank, next_root)
    return dict(topk=O, n_new=n_new, acc_nodes=acc_nodes, out_tokens=out_tokens,
                next_root=next_root, next_tree=nxt)


# --------------------------------------------------------------------------
# Verification under temperature sampling (Sec. 5.3 "Temperature Sampling").
# The paper reports that TR keeps working at temperatures 0.3 - 1.0 and explains
# the slight loss by sampled tokens falling outside the stored top-k; it does not
# spell the acceptance rule out.  Reading used here ("sample, then match"): every
# node draws ONE token from its output distribution at temperature T, and a draft
# child is correct iff it equals the token drawn at its parent - greedy
# verification with the argmax replaced by the draw, which emits exactly the
# tokens that token-by-token sampling with the same draws would.  The draw is
# written as a Gumbel-max so that it is an argmax of per-element float32
# arithmetic (no summation order): x = argmax_v ( logits[v] / T + g[v] ),
# g = -log(-log(u)), u uniform; the noise g is an INPUT (the caller's generator).
# --------------------------------------------------------------------------
def sample_tokens(logits, gumbel, inv_temperature):
    """Token drawn at every node: argmax_v of z[v] = fl32(fl32(logits[v] * inv_temperature) + gumbel[v]), lowest
    index among equal z (float32 multiply, then float32 add: two roundings, the decision precision of the kernel).
    With gumbel == 0 this is the greedy argmax for any inv_temperature > 0.
    Pinned by: gumbel = 0 gives argtopk's column 0; empirical frequencies of many draws against softmax(logits / T)
    (the Gumbel-max theorem); a hand case where the noise overturns the argmax.
    """
    logits = np.asarray(logits, dtype=np.float32)
    gumbel = np.asarray(gumbel, dtype=np.float32)
    z = (logits * np.float32(inv_temperature)).astype(np.float32) + gumbel
    return argtopk(z.astype(np.float32), 1)[:, 0]


def verify_update_sampled(M, S, logits, gumbel, inv_temperature, parent, rank, rule="last", only_accepted=False):
    """verify_update with the draw of sample_tokens in place of the argmax for acceptance and for the extra token;
    the matrix still stores argtopk(logits) of every node (the candidates are the model's top-k, whatever was
    drawn - which is why, in the paper's words, draws outside the top-k cost acceptance at high temperature).
    M is modified in place.  Returns verify_update's dict plus `sampled`.
    """
    k = M.shape[1]
    O = argtopk(logits, k)
    x = sample_tokens(logits, gumbel, inv_temperature)
    n_new, acc_nodes, out_tokens, next_root = accept(S, x, parent)
    update_matrix(M, S, O, rule=rule, nodes=acc_nodes if only_accepted else None)
    nxt = bfs_tree(M, parent, rank, next_root)
    return dict(topk=O, sampled=x, n_new=n_new, acc_nodes=acc_nodes, out_tokens=out_tokens,
                next_root=next_root, next_tree=nxt)


# --------------------------------------------------------------------------
# Commit of the accepted path (Sec. 5.4: besides the matrix, a step advances the token list and the KV cache)
# --------------------------------------------------------------------------
def commit(k, v, ctx_len, tokens, acc_nodes, out_tokens):
    """After verification the accepted nodes (root first) are the tokens whose keys and values now belong to the
    prefix: their cache rows are gathered, in path order, right behind the old prefix; the step's new tokens
    (accepted drafts + the extra greedy token) are appended to the text; the prefix grows by their count.

    k, v : [..., rows, D] caches with the tree's rows at ctx_len .. ctx_len + N - 1 (modified in place)
    Returns (new ctx_len, new token list).
    Pinned by: a hand-worked example; the gathered rows equal the rows of the accepted path taken from a copy.
    """
    n = len(acc_nodes)
    src_k = k[..., [ctx_len + a for a in acc_nodes], :].copy()
    src_v = v[..., [ctx_len + a for a in acc_nodes], :].copy()
    k[..., ctx_len:ctx_len + n, :] = src_k
    v[..., ctx_len:ctx_len + n, :] = src_v
    return ctx_len + n, list(tokens) + [int(t) for t in out_tokens]
