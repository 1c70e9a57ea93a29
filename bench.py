#!/usr/bin/env python
"""Benchmark of the Token Recycling verify-and-recycle step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload llama2-7b]

One step = toy-model logits patch (harness) -> tree attention over all layers (one launch) -> fused
argmax/top-k -> accept + matrix update + next-tree retrieval, replayed as one CUDA graph per step with all
state resident on the device.  Prints ONE JSON line (rank 0).  With N > 1 every rank runs an independent
replica on its own GPU (the step has no exchange between GPUs); the job's time is the slowest rank's.
`--impl reference` times the CPU oracle (the checker the tests use) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "us per TR verify-and-recycle step"
UNIT = "us/step"


def load_peaks():
    """(HBM GB/s, sustained dense bf16 TFLOP/s, where they come from)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return (float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", 1400.0)),
                "measured (MEASURED_PEAKS.json: copy bandwidth, sustained cuBLAS bf16)")
    return 6650.0, 1400.0, "fallback (earlier measurement on this pool)"


def attention_flops(w, n_layers):
    """4 N Hq (C_b + N) D per sequence and layer: the two products over the prefix and the whole tree block."""
    return sum(4 * w.n_nodes * w.n_q_heads * (c + w.n_nodes) * w.head_dim for c in w.ctx) * n_layers


def algorithmic_bytes(w, n_layers):
    """Bytes the method must move per step: K/V once, Q and O once, logits once, 2N matrix rows."""
    N, D = w.n_nodes, w.head_dim
    kv = sum(2 * w.n_kv_heads * (c + N) * D * 2 for c in w.ctx) * n_layers
    qo = 2 * w.batch * N * w.n_q_heads * D * 2 * n_layers
    logits = w.batch * N * w.vocab * 4
    matrix = w.batch * 2 * N * w.k * 4 + w.batch * N * w.k * 4       # rows written + rows gathered + top-k out
    return {"attention": kv + qo, "logits": logits, "matrix": matrix, "total": kv + qo + logits + matrix}


class ClockSampler:
    """nvidia-smi in query mode (read-only) every 25 ms; `stop(t0, t1)` keeps the samples taken between the two host
    times, i.e. during the timed region."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    BAD = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            pass

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        import datetime
        sm, mx, reasons, n_all = [], [], set(), 0
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                clk, cmax = float(f[1]), float(f[2])
            except ValueError:
                continue
            n_all += 1
            if ts < t0 - 0.03 or ts > t1 + 0.03:      # a sample describes the ~25 ms before its time stamp
                continue
            sm.append(clk); mx.append(cmax)
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "samples_outside_region": n_all - len(sm),
                "reasons": sorted(reasons), "sampled": "every 25 ms during the timed blocks"}


# ---------------------------------------------------------------------------------------------------
class OracleSampler:
    """Times the CPU oracle, as it stands, on a bounded sample of one step of workload `w`: `n_units` of the
    (sequence, layer, kv-head) attention units, scaled to all of them, plus one full top-k / accept / update /
    retrieve pass per sequence."""

    def __init__(self, w):
        from oracle import tr_oracle as orc
        from paper_2408_08696_b200 import synth
        self.orc, self.synth, self.w = orc, synth, w
        try:
            from threadpoolctl import threadpool_info
            self.threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        except Exception:
            self.threads = 1
        self.parent, self.rank = orc.template_from_branching(w.branching, w.n_nodes)
        self.pool = synth.normal_pool(w.seed)
        self.rng = np.random.default_rng(7)
        self.units_total = w.batch * w.n_layers * w.n_kv_heads
        self.M = synth.seeded_matrix(w)[0].astype(np.int64)
        self.succ = synth.zipf_successors(w)
        self.noise = synth.noise_logits(w, 1)[0]
        self.S = orc.bfs_tree(self.M, self.parent, self.rank, int(synth.root_tokens(w)[0]))

    def step_us(self, n_units):
        w, orc, synth = self.w, self.orc, self.synth
        group = w.n_q_heads // w.n_kv_heads
        n_units = min(n_units, self.units_total)
        t_attn = 0.0
        for _ in range(n_units):
            b = int(self.rng.integers(0, w.batch))
            l, g = int(self.rng.integers(0, w.n_layers)), int(self.rng.integers(0, w.n_kv_heads))
            qs, ks, vs = synth.attention_slice(w, self.pool, b, l, g)
            qf = synth.bf16_bits_to_f32(qs[:, g * group:(g + 1) * group])
            kf, vf = synth.bf16_bits_to_f32(ks)[None], synth.bf16_bits_to_f32(vs)[None]
            t0 = time.perf_counter()
            orc.tree_attention(qf, kf, vf, w.ctx[b], self.parent)
            t_attn += time.perf_counter() - t0
        logits = synth.step_logits(self.noise[0], self.S, self.succ, w.boost)
        t0 = time.perf_counter()
        rec = orc.verify_update(self.M, self.S, logits, self.parent, self.rank)
        t_int = (time.perf_counter() - t0) * w.batch
        self.S = rec["next_tree"]
        return (t_attn / n_units * self.units_total + t_int) * 1e6

    def describe(self, n_units, steps):
        return ("%d step(s); per step %d of %d (sequence, layer, kv-head) attention units timed and scaled to all, "
                "plus one full top-k/accept/update/retrieve pass per sequence"
                % (steps, min(n_units, self.units_total), self.units_total))


def run_reference(args, w):
    """The oracle as the reference arm: K steps, each a bounded sample scaled to a whole step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSampler(w)
    n_units = 32
    vals = [smp.step_us(n_units) for _ in range(args.warmup + args.steps)][args.warmup:]
    v = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": v / 1000.0, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "note": "CPU oracle on host cores; each step is a bounded sample scaled up"},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": smp.threads, "kind": "oracle",
                         "sample": smp.describe(n_units, args.steps)},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------------
def measure_lm_head(torch, tr, dw, w, dev, reps=20):
    """The output layer fused with argtopk (not part of the timed step, whose logits come from the toy model): one
    pass over a random bf16 weight [V, hidden] for the step's batch * N rows; graphs of 4 calls, `reps` calls in all.
    The weight (hundreds of MB) is larger than L2, so every replay streams it from HBM."""
    H = w.n_q_heads * w.head_dim
    rows = w.batch * w.n_nodes
    g = torch.Generator(device=dev).manual_seed(w.seed & 0x7FFFFFFF)
    d_h = torch.randn(rows, H, device=dev, generator=g).to(torch.bfloat16)
    d_w = torch.randn(w.vocab, H, device=dev, generator=g).to(torch.bfloat16)
    idx = torch.zeros(rows, w.k, dtype=torch.int32, device=dev)
    s = torch.cuda.Stream(dev)
    graph = torch.cuda.CUDAGraph()
    tr.tr_lm_head_topk(dw.ctx, d_h, d_w, idx)
    torch.cuda.synchronize()
    per_graph = 4                                              # calls per graph, like the steps of a round graph
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            for _ in range(per_graph):
                tr.tr_lm_head_topk(dw.ctx, d_h, d_w, idx, stream=s)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_rep = max(1, reps // per_graph)
    e0.record()
    for _ in range(n_rep):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / (n_rep * per_graph) * 1000.0
    groups = (rows + 127) // 128                               # row groups: the CTAs of a vocabulary slice share it via L2
    byts = w.vocab * H * 2 + rows * H * 2 + rows * w.k * 4      # algorithmic: the weight ONCE, hidden states, output
    return {"us": us, "bound": "hbm", "achieved": byts / us / 1e3, "unit": "GB/s", "algorithmic_bytes": byts,
            "row_groups": groups, "weight_bytes_through_sms": groups * w.vocab * H * 2,
            "rows": rows, "hidden": H, "vocab": w.vocab, "gpu_launches": 2,
            "device_flags": tr.tr_device_flags(dw.ctx)}


def measure_sampled_verify(torch, tr, dw, w, dev, reps=20):
    """Verification under temperature sampling on the step's logits (not part of the timed step, which is greedy):
    tr_verify_update_sampled as a CUDA graph replayed `reps` times on its own copy of the loop state, beside the
    greedy tr_verify_update timed the same way.  Two passes over the logits and one over the noise."""
    from paper_2408_08696_b200 import synth
    rows = w.batch * w.n_nodes
    gen = torch.Generator(device=dev).manual_seed((w.seed + 7) & 0x7FFFFFFF)
    u = torch.rand(w.batch, w.n_nodes, w.vocab, device=dev, generator=gen).clamp_(1e-20, 1.0 - 2.0 ** -24)
    d_g = -torch.log(-torch.log(u))
    d_tree = dw.d_tree.clone()
    out_struct, out = tr.make_step_out(dw.ctx)
    out_struct.d_next_tree = d_tree.data_ptr()
    M0 = [tr.tr_matrix_export(dw.ctx, b) for b in range(w.batch)]      # the measurement must not disturb the loop
    res = {}
    for name in ("sampled", "greedy"):
        s = torch.cuda.Stream(dev)
        graph = torch.cuda.CUDAGraph()

        def call(stream=None):
            if name == "sampled":
                tr.tr_verify_update_sampled(dw.ctx, dw.d_logits[0], d_g, 1.0 / 0.7, d_tree, out_struct, stream=stream)
            else:
                tr.tr_verify_update(dw.ctx, dw.d_logits[0], d_tree, out_struct, stream)
        call()
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            with torch.cuda.graph(graph, stream=s):
                call(s)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        res[name] = e0.elapsed_time(e1) / reps * 1000.0
    for b in range(w.batch):
        tr.tr_matrix_import(dw.ctx, b, M0[b])
    byts = rows * w.vocab * 4 * 3
    return {"us": res["sampled"], "greedy_verify_update_us": res["greedy"], "algorithmic_bytes": byts,
            "achieved": byts / res["sampled"] / 1e3, "unit": "GB/s", "temperature": 0.7, "gpu_launches": 2,
            "device_flags": tr.tr_device_flags(dw.ctx)}


def check_parity(torch, tr, harness, dw, w, graphs, round_graph):
    """Outside the timed region: the very graphs that were timed, replayed from the initial state, against the CPU
    oracle - every integer output of 4 single-step replays, then one whole-round replay (n_rot steps in one graph):
    last step's integer outputs, the matrices, and a seeded sample of 8 attention heads."""
    from oracle import tr_oracle as orc
    from paper_2408_08696_b200 import synth
    from tests.oracle_loop import OracleLoop, attention_close, compare_step
    res = {"single_step_replays": 4, "round_replay_steps": dw.n_rot, "attention_heads": 8}
    try:
        dw.reset()
        ol = OracleLoop(w, n_rot=dw.n_rot)
        for i in range(4):
            graphs[i].replay()
            compare_step(ol.step(i), dw.snapshot(), dw.ctx.max_new)
        dw.reset()
        ol = OracleLoop(w, n_rot=dw.n_rot)
        dw.o.zero_()
        round_graph.replay()
        recs = [ol.step(i) for i in range(dw.n_rot)][-1]
        compare_step(recs, dw.snapshot(), dw.ctx.max_new)
        for b in range(w.batch):
            assert (tr.tr_matrix_export(dw.ctx, b) == ol.M[b]).all(), "matrix differs"
        import dataclasses
        pool = synth.normal_pool(w.seed)
        rng = np.random.default_rng(99)
        group = w.n_q_heads // w.n_kv_heads
        ws = dataclasses.replace(w, n_layers=dw.L)                # the slices are cut for the layer count in use
        worst = [0.0, 0.0]
        for _ in range(8):
            b, l, h = int(rng.integers(0, w.batch)), int(rng.integers(0, dw.L)), int(rng.integers(0, w.n_q_heads))
            qs, ks, vs = synth.attention_slice(ws, pool, b, l, h // group)
            ref = orc.tree_attention(synth.bf16_bits_to_f32(qs[:, h:h + 1]), synth.bf16_bits_to_f32(ks)[None],
                                     synth.bf16_bits_to_f32(vs)[None], w.ctx[b], dw.parent)
            mx, rel = attention_close(dw.o[b, l, :, h].float().cpu().numpy(), ref[:, 0])
            assert mx <= 2e-2 and rel <= 1e-2, ("attention", b, l, h, mx, rel)
            worst = [max(worst[0], mx), max(worst[1], rel)]
        assert tr.tr_device_flags(dw.ctx) == 0
        res.update(ok=True, attention_max_abs=worst[0], attention_rel_l2=worst[1])
    except AssertionError as e:
        res.update(ok=False, error=str(e)[:200])
    return res


def ensure_built():
    """The product path needs the CUDA library (there is no fallback).  Local rank 0 builds it if it is missing or
    older than its sources; the other ranks of the node wait for the files."""
    from paper_2408_08696_b200 import build
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        build.build()
        return
    deadline = time.time() + 600
    while time.time() < deadline and not (os.path.exists(build.LIB_TR) and os.path.exists(build.LIB_SYNTH)):
        time.sleep(1.0)
    time.sleep(2.0)  # (a library that is being rewritten: let rank 0's linker finish)


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    ensure_built()
    from paper_2408_08696_b200 import binding as tr
    from paper_2408_08696_b200 import harness, replicas, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the step has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    K, W = args.steps, max(args.warmup, 3)

    # rotating logits buffers larger than L2 in total, so that every step's logits come from HBM like its K/V
    n_rot = harness.rotation_larger_than_l2(w)
    dw = harness.DeviceWorkload(w, n_layers=args.layers or None, device=local_rank, n_rot=n_rot)
    graphs = dw.capture_graphs()          # one step per graph
    round_graph = dw.capture_round()      # n_rot steps in one graph

    def run_steps(n):
        """n steps: whole rounds as one graph launch each, the rest as single-step graphs."""
        q, r = divmod(n, n_rot)
        for _ in range(q):
            round_graph.replay()
        for i in range(r):
            graphs[i].replay()

    if args.profile:
        run_steps(W + K)
        torch.cuda.synchronize()
        dw.close()
        return
    stream = torch.cuda.current_stream()
    run_steps(W)
    torch.cuda.synchronize()
    # a first estimate of the step time sizes the number of timed blocks
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    run_steps(K)
    e1.record(stream)
    torch.cuda.synchronize()
    est_ms = max(e0.elapsed_time(e1), 1e-3)
    n_blocks = int(min(400, max(5, np.ceil(args.min_timed_ms / est_ms))))
    if world > 1:  # every rank must run the same number of blocks
        t = torch.tensor([n_blocks], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        n_blocks = int(t.item())

    # ---- timed region: n_blocks blocks of exactly K steps; each block is bracketed by a barrier and a device
    #      synchronisation on both sides and timed on the device (two events on the launching stream); the clocks
    #      are sampled while the blocks run.  value = median block (per block: slowest rank).
    for attempt in range(2):
        sampler = ClockSampler(local_rank) if rank == 0 else None
        if sampler:
            time.sleep(0.25)              # let nvidia-smi come up before the region starts
        block_ms = []
        t_begin = time.time()
        for _ in range(n_blocks):
            replicas.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            run_steps(K)
            e1.record(stream)
            torch.cuda.synchronize()
            replicas.barrier()
            block_ms.append(e0.elapsed_time(e1))
        t_end = time.time()
        clocks = sampler.stop(t_begin, t_end) if sampler else None
        if not clocks or not (set(clocks["reasons"]) & set(ClockSampler.BAD)):
            break
        clocks["note"] = "first attempt saw %s and was measured again" % clocks["reasons"]
    block_ms = replicas.max_over_ranks_vec(block_ms, device=dev if world > 1 else "cpu")
    med_ms = float(np.median(block_ms))
    agg = replicas.aggregate(med_ms, K, device="cpu", reduce=False)
    flags = tr.tr_device_flags(dw.ctx)
    # acceptance statistic of the toy model (a sanity figure, not a result): 64 untimed steps, n_new read each step
    n_new_sum, n_stat = 0, 64
    for i in range(n_stat):
        graphs[i % n_rot].replay()
        n_new_sum += int(dw.out["n_new"].sum().item())

    # ---- dominant kernel (tree attention) alone: event pair around every launch, same stream
    time.sleep(0.3)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for i in range(K):
        r = i % n_rot
        tr.trs_patch_logits(dw.d_logits[r], dw.d_noise[r], dw.d_tree, dw.d_prev_col[r], dw.d_succ, w.boost)
        ev[i][0].record(stream)
        tr.tr_tree_attention(dw.ctx, dw.attn)
        ev[i][1].record(stream)
        tr.tr_verify_update(dw.ctx, dw.d_logits[r], dw.d_tree, dw.out_struct)
    torch.cuda.synchronize()
    attn_eager_ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
    # ... and as a run of back-to-back launches (a graph of 8 attention launches, replayed until >= K launches, one
    # event pair around the run): the event pair around a single eager launch also times the front end's idle gaps
    # before and after it, a run times launches and the boundaries between them.  This is the roofline's duration.
    per_graph = 8
    ga = torch.cuda.CUDAGraph()
    sa = torch.cuda.Stream(dev)
    with torch.cuda.stream(sa):
        with torch.cuda.graph(ga, stream=sa):
            for _ in range(per_graph):
                tr.tr_tree_attention(dw.ctx, dw.attn, sa)
    n_rep = max(1, -(-K // per_graph))
    ga.replay()
    torch.cuda.synchronize()
    time.sleep(0.3)
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record(stream)
    for _ in range(n_rep):
        ga.replay()
    b1.record(stream)
    torch.cuda.synchronize()
    attn_ms = b0.elapsed_time(b1) / (n_rep * per_graph)
    # per-layer launches (one call per layer, as a real model's forward would issue them), for the record
    per_layer_ms = None
    if dw.L > 1:
        args_l = [tr.make_attn_args(dw.ctx, dw.q[:, l:l + 1], dw.k[:, l:l + 1], dw.v[:, l:l + 1], dw.o[:, l:l + 1],
                                    dw.d_ctx_len, w.max_ctx, prefix_stable=True) for l in range(dw.L)]
        # (prefix_stable: nothing writes the prefix lengths or the prefix K/V between these launches)
        gl = torch.cuda.CUDAGraph()
        s2 = torch.cuda.Stream(dev)
        with torch.cuda.stream(s2):
            with torch.cuda.graph(gl, stream=s2):
                for a in args_l:
                    tr.tr_tree_attention(dw.ctx, a, s2)
        torch.cuda.synchronize()
        for _ in range(3):
            gl.replay()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for _ in range(20):
            gl.replay()
        a1.record(stream)
        torch.cuda.synchronize()
        per_layer_ms = a0.elapsed_time(a1) / 20

    # ---- end to end through the host-buffer entry point: pinned inputs in, results out, every step
    B, N, V, Hq, Hkv, D, L = w.batch, w.n_nodes, w.vocab, w.n_q_heads, w.n_kv_heads, w.head_dim, dw.L
    h_q = dw.q.cpu().pin_memory()
    h_tk = torch.stack([dw.k[b, :, :, c:c + N] for b, c in enumerate(w.ctx)]).cpu().contiguous().pin_memory()
    h_tv = torch.stack([dw.v[b, :, :, c:c + N] for b, c in enumerate(w.ctx)]).cpu().contiguous().pin_memory()
    h_logits = [dw.d_noise[r].cpu().pin_memory() for r in range(min(4, n_rot))]
    h_ctx = np.array(w.ctx, dtype=np.int32)
    h_out = torch.zeros(B, L, N, Hq, D, dtype=torch.bfloat16).pin_memory()
    h_n_new = torch.zeros(B, dtype=torch.int32).pin_memory()
    h_tok = torch.zeros(B, dw.ctx.max_new, dtype=torch.int32).pin_memory()
    h_next = torch.zeros(B, N, dtype=torch.int32).pin_memory()
    d_stage = torch.empty(B, N, V, dtype=torch.float32, device=dev)
    io = tr.tr_host_io()
    io.h_q, io.h_tree_k, io.h_tree_v = h_q.data_ptr(), h_tk.data_ptr(), h_tv.data_ptr()
    io.h_ctx_len, io.d_logits_staging, io.d_tree = h_ctx.ctypes.data, d_stage.data_ptr(), dw.d_tree.data_ptr()
    io.h_out, io.h_n_new, io.h_out_tokens, io.h_next_tree = (h_out.data_ptr(), h_n_new.data_ptr(), h_tok.data_ptr(),
                                                             h_next.data_ptr())
    h2d = h_q.numel() * 2 + h_tk.numel() * 2 + h_tv.numel() * 2 + h_logits[0].numel() * 4 + h_ctx.nbytes
    d2h = h_out.numel() * 2 + h_n_new.numel() * 4 + h_tok.numel() * 4 + h_next.numel() * 4
    Ke = max(3, min(K, 20))
    for i in range(2):
        io.h_logits = h_logits[i % len(h_logits)].data_ptr()
        tr.tr_step_host(dw.ctx, dw.attn, dw.out_struct, io)
    replicas.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(Ke):
        io.h_logits = h_logits[i % len(h_logits)].data_ptr()
        tr.tr_step_host(dw.ctx, dw.attn, dw.out_struct, io)      # synchronises the stream itself
    e2e_ms = (time.perf_counter() - t0) * 1000.0
    e2e = replicas.aggregate(e2e_ms, Ke, device=dev if world > 1 else "cpu")

    lm = measure_lm_head(torch, tr, dw, w, dev) if rank == 0 else None
    sampled_verify = measure_sampled_verify(torch, tr, dw, w, dev) if rank == 0 else None
    parity = check_parity(torch, tr, harness, dw, w, graphs, round_graph) if rank == 0 else None

    if rank == 0:
        hbm_peak, tf_peak, peak_src = load_peaks()
        ab = algorithmic_bytes(w, dw.L)
        fl = attention_flops(w, dw.L)
        attn_gbs = ab["attention"] / (attn_ms * 1e-3) / 1e9
        attn_tfs = fl / (attn_ms * 1e-3) / 1e12
        step_gbs = ab["total"] / (agg["ms_per_step"] * 1e-3) / 1e9
        hbm = {"achieved": attn_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": attn_gbs / hbm_peak}
        tensor = {"achieved": attn_tfs, "peak": tf_peak, "unit": "TFLOP/s", "frac": attn_tfs / tf_peak,
                  "flops_per_launch": fl, "peak_kind": "sustained dense bf16 (the launch runs inside a long step)"}
        bound = "tensor" if tensor["frac"] > hbm["frac"] else "hbm"
        top = tensor if bound == "tensor" else hbm
        smp = OracleSampler(w)
        cpu_units, cpu_steps = 2048, 3                       # roughly 15-20 s of host work at the 7B shape
        cpu_us = float(np.mean([smp.step_us(cpu_units) for _ in range(cpu_steps)]))
        cpu_desc, cpu_threads = smp.describe(cpu_units, cpu_steps), smp.threads
        kv_mb = ab["attention"] / 1e6
        l2_note = ("inputs larger than L2: %.0f MB of K/V and %d rotating logits buffers (%.0f MB) per round"
                   % (kv_mb, n_rot, n_rot * ab["logits"] / 1e6)) if ab["attention"] > harness.L2_BYTES else \
                  "inputs fit in L2 (%.1f MB per step): a correctness-sized workload, not flushed" % (ab["total"] / 1e6)
        line = {
            "metric": METRIC, "value": agg["us_per_step_job"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": agg["ms_per_step"], "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "vocab": V, "k": w.k, "tree_nodes": N, "layers": L, "q_heads": Hq,
                       "kv_heads": Hkv, "head_dim": D, "context": list(w.ctx), "batch": B,
                       "attention_launch": "all layers in one launch",
                       "graphs": "%d consecutive steps per CUDA graph launch, remaining steps one graph each" % n_rot,
                       "l2": l2_note, "parallelism": "replicas only" if world > 1 else "1 gpu"},
            "timing": {"blocks": len(block_ms), "steps_per_block": K, "value_is": "median block",
                       "block_us_per_step_min": 1000.0 * min(block_ms) / K,
                       "block_us_per_step_max": 1000.0 * max(block_ms) / K,
                       "timed_device_ms": float(sum(block_ms))},
            "steps_per_s": agg["steps_per_s"],
            "step_hbm": {"algorithmic_bytes": ab["total"], "achieved_gbs": step_gbs,
                         "frac_of_measured": step_gbs / hbm_peak, "frac_of_8tbs": step_gbs / 8000.0},
            "roofline": {"kernel": "tree attention (all layers)", "bound": bound, "achieved": top["achieved"],
                         "peak": top["peak"], "unit": top["unit"], "frac": top["frac"], "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": ab["attention"], "avg_launch_ms": attn_ms,
                         "avg_launch_ms_is": "mean over %d back-to-back launches (graphs of %d), one event pair" % (n_rep * per_graph, per_graph),
                         "eager_event_pair_ms": attn_eager_ms,
                         "traffic": NCU_TRAFFIC_BYTES.get(w.name), "hbm": hbm, "tensor": tensor},
            "attention_per_layer_launches_ms": per_layer_ms,
            "cpu_baseline": {"value": cpu_us, "unit": UNIT, "cores": cpu_threads, "kind": "oracle", "sample": cpu_desc},
            "e2e": {"value": e2e["us_per_step_job"], "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": Ke},
            "gpu_launches": dw.kernels_per_step() * K,
            "clocks": clocks,
            "mean_new_tokens_per_step": n_new_sum / (B * n_stat),
            "parity_checked": bool(parity and parity.get("ok")), "parity": parity,
            "next_rows": {"lm_head_topk": dict(lm, frac=lm["achieved"] / hbm_peak, peak=hbm_peak),
                          "verify_update_sampled": sampled_verify},
            "device_flags": flags,
        }
        print(json.dumps(line), flush=True)
    dw.close()
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (read + write) of one attention launch from the committed ncu captures (see profiles/), per workload.
NCU_TRAFFIC_BYTES = {
    # profiles/tr_attn_tc_kernel_llama2-7b_16layers.md: (300.07 MB read + 4.93 MB written) per 16-layer launch,
    # scaled to the 32 layers of one benchmark launch (traffic is proportional to the layers processed)
    "llama2-7b": 2 * (300_067_584 + 4_926_464),
    # profiles/tr_attn_pair_kernel_llama3-8b_12layers.md: (414.64 MB read + 3.81 MB written) per 12-layer launch,
    # scaled to 32 layers
    "llama3-8b": int(round(32 / 12 * (414_638_080 + 3_806_208))),
    # profiles/tr_attn_tc_kernel_llama2-13b_4layers.md: (345.53 MB read + 3.08 MB written) per 4-layer launch, 40 layers
    "llama2-13b": 10 * (345_531_392 + 3_084_032),
    # profiles/tr_attn_pair_kernel_llama2-70b-b8_4layers.md: (365.11 MB read + 4.73 MB written) per 4-layer launch, 80 layers
    "llama2-70b-b8": 20 * (365_111_040 + 4_734_720),
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling small cases)")
    ap.add_argument("--min-timed-ms", type=float, default=50.0,
                    help="the K-step block is repeated until the timed blocks add up to this much device time (>= 5 blocks)")
    ap.add_argument("--profile", action="store_true",
                    help="only warm up and replay the step graph K times (for ncu); prints no bench line")
    ap.add_argument("--lm-head-only", action="store_true",
                    help="only time the output layer fused with argtopk (for ncu); prints its figures, no bench line")
    args = ap.parse_args()
    from paper_2408_08696_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.lm_head_only:
        import torch
        ensure_built()
        from paper_2408_08696_b200 import binding as tr
        from paper_2408_08696_b200 import harness
        dw = harness.DeviceWorkload(w, with_attention=False)
        print(json.dumps({"lm_head_topk": measure_lm_head(torch, tr, dw, w, dw.dev, reps=5), "workload": w.name}))
        dw.close()
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
