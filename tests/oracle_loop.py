"""Checker-side driver: runs the multi-step toy-model loop and attention with the CPU oracle on the same seeded
inputs the device harness uploads."""
import numpy as np

from oracle import tr_oracle as orc
from paper_2408_08696_b200 import synth


class OracleLoop:
    def __init__(self, w, n_rot=4, zero_matrix=False, rule="last", only_accepted=False):
        self.w = w
        self.rule, self.only_accepted = rule, only_accepted
        self.parent, self.rank = orc.template_from_branching(w.branching, w.n_nodes)
        self.M = [np.zeros((w.vocab, w.k), dtype=np.int64) if zero_matrix else m.astype(np.int64)
                  for m in synth.seeded_matrix(w)]
        self.succ = synth.zipf_successors(w)
        self.noise = synth.noise_logits(w, n_rot)
        self.n_rot = n_rot
        roots = synth.root_tokens(w)
        self.S = [orc.bfs_tree(self.M[b], self.parent, self.rank, int(roots[b])) for b in range(w.batch)]

    def step(self, i):
        r = i % self.n_rot
        recs = []
        for b in range(self.w.batch):
            logits = synth.step_logits(self.noise[r, b], self.S[b], self.succ, self.w.boost)
            rec = orc.verify_update(self.M[b], self.S[b], logits, self.parent, self.rank, rule=self.rule,
                                    only_accepted=self.only_accepted)
            self.S[b] = rec["next_tree"]
            recs.append(rec)
        return recs


def compare_step(recs, snap, max_new):
    """Bit-exact comparison of one step's integer outputs (device snapshot vs oracle records)."""
    for b, rec in enumerate(recs):
        assert (snap["topk_idx"][b] == rec["topk"]).all(), "topk differs (seq %d)" % b
        assert snap["n_new"][b] == rec["n_new"]
        n = rec["n_new"]
        assert snap["acc_nodes"][b, :n].tolist() == rec["acc_nodes"]
        assert (snap["acc_nodes"][b, n:] == -1).all()
        assert snap["out_tokens"][b, :n].tolist() == rec["out_tokens"]
        assert (snap["out_tokens"][b, n:] == -1).all()
        assert snap["next_root"][b] == rec["next_root"]
        assert (snap["tree"][b] == rec["next_tree"]).all(), "next tree differs (seq %d)" % b


def oracle_attention(w, q_bits, k_bits, v_bits, b, l, parent, heads=None):
    """float64 tree attention of sequence b, layer l from bf16 bit patterns; returns [N, Hq, D]."""
    q = synth.bf16_bits_to_f32(q_bits[b, l]).astype(np.float64)
    k = synth.bf16_bits_to_f32(k_bits[b, l]).astype(np.float64)
    v = synth.bf16_bits_to_f32(v_bits[b, l]).astype(np.float64)
    c = w.ctx[b]
    return orc.tree_attention(q, k[:, : c + w.n_nodes], v[:, : c + w.n_nodes], c, parent)


def attention_close(got_f32, ref_f64):
    """The tolerance of the build's target: max |diff| <= 2e-2 and relative L2 error <= 1e-2."""
    diff = np.abs(got_f32.astype(np.float64) - ref_f64)
    rel = np.linalg.norm(got_f32.astype(np.float64) - ref_f64) / max(np.linalg.norm(ref_f64), 1e-30)
    return diff.max(), rel
