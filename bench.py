#!/usr/bin/env python
"""Benchmark of the Talon hot path: draft-and-verify steps per second on synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl talon|reference]

A *step* is one pass of the whole path over one batch: tree reset, D_max expansion-layer calls
(Algorithm 2; layers after the budget is spent read nothing), tree finalisation, tree attention of
the N tree tokens against the prefix KV cache, target argmax and the greedy accept walk.  The draft
and target model forwards are not part of the path: their outputs (fp32 logits, bf16 Q/K/V) are
seeded synthetic tensors, resident in HBM before the timed region starts.

The timed region is K back-to-back ``talon_step`` calls that rotate over enough distinct input sets
that the bytes touched between two uses of a set exceed the L2 capacity several times over, so
every step reads its inputs from HBM.  It is bracketed by a barrier and a device synchronisation on
both sides, timed with CUDA events, and reported as the maximum over ranks.  With more than one
GPU every rank runs its own replicas (sequences are independent: no data-path collective).

Rank 0 prints one JSON line.  Beside the contract's keys it carries ``roofline`` (the dominant
kernel's algorithmic bytes over its event-timed launches of the timed region, against the measured
copy bandwidth), ``cpu_baseline`` (the fp64 CPU oracle timed on a bounded sample), ``e2e`` (the same
step through ``talon_step_host`` with pinned host buffers), ``graph_replay`` (the step captured in a
CUDA graph), ``kernels`` (per-kernel time from a separate bracketed pass) and ``tree_shapes``.
``--impl reference`` times the CPU oracle alone, on host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "draft+verify steps/sec"
UNIT = "steps/s"
L2_BYTES = 126 * 1024 * 1024
ROTATION_FACTOR = 3.0            # bytes between two uses of an input set, in units of L2
TIMED_EVERY = 32                 # the dominant kernel is event-bracketed on every 32nd timed step


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------
class ClockSampler:
    """Polls nvidia-smi for SM clock and throttle reasons of one GPU while work is running."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 50):
        self.samples = []            # (t, sm, max_sm, power, [reasons])
        self.proc = None
        self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", str(period_ms), "-i", str(gpu_index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm, mx = float(parts[0]), float(parts[1])
                power = float(parts[2]) if parts[2].replace(".", "", 1).isdigit() else float("nan")
            except ValueError:
                continue
            reasons = [n for n, p in zip(names, parts[3:7]) if p.lower().startswith("active")]
            self.samples.append((time.time(), sm, mx, power, reasons))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=5)

    def summary(self, t0: float, t1: float):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        if len(inside) < 3:          # a short timed region sees few samples: take the whole busy span
            inside = list(self.samples)
            window = "warm-up to end of run"
        if not inside:
            return None
        reasons = sorted({r for s in inside for r in s[4]})
        return {"sm_mhz": statistics.median(s[1] for s in inside), "sm_max_mhz": inside[0][2],
                "reasons": reasons, "samples": len(inside), "window": window,
                "power_w_max": max((s[3] for s in inside if s[3] == s[3]), default=None)}


# --------------------------------------------------------------------------------------------
# the oracle as a timed CPU baseline (the only place outside tests/ and smoke that runs it)
# --------------------------------------------------------------------------------------------
class OracleStep:
    """One draft-and-verify step of one sequence through the CPU oracle, inputs prepared up front."""

    def __init__(self, cfg, seed: int, seq_id: int, heads):
        from oracle import talon_oracle as O
        from paper_2601_07353_b200 import synth
        self.O, self.cfg, self.heads = O, cfg, list(heads)
        self.p = O.Params(cfg.budget, cfg.topk, cfg.topk, cfg.mu, cfg.max_depth)
        self.root = synth.root_token(cfg, seed, seq_id)
        self.L = synth.prefix_len(cfg, seed, seq_id)
        self.rows = {}
        gen = lambda path: synth.draft_logits_row(cfg, seed, seq_id, path)

        def cached(path):
            key = tuple(path)
            if key not in self.rows:
                self.rows[key] = gen(path)
            return self.rows[key]
        self.logits_fn = cached
        tree = O.expand(self.root, cached, self.p)        # untimed pass: fills the row cache
        n, N = tree.n_nodes, cfg.budget
        self.target = np.zeros((N, cfg.vocab), np.float32)
        for i in range(n):
            self.target[i] = synth.target_logits_row(cfg, seed, seq_id, O.path_tokens(tree, i))
        Hq, Hkv, Dh, g = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.group
        kvs = sorted({h // g for h in self.heads})
        q = synth.qkv_block(seed, synth.STREAM_Q, seq_id, N * Hq * Dh).reshape(N, Hq, Dh)
        kt = synth.qkv_block(seed, synth.STREAM_KT, seq_id, N * Hkv * Dh).reshape(N, Hkv, Dh)
        vt = synth.qkv_block(seed, synth.STREAM_VT, seq_id, N * Hkv * Dh).reshape(N, Hkv, Dh)
        kp = np.zeros((self.L, Hkv, Dh), np.float32)
        vp = np.zeros((self.L, Hkv, Dh), np.float32)
        step = 4096
        for t0 in range(0, self.L, step):
            t1 = min(self.L, t0 + step)
            cnt, off = (t1 - t0) * Hkv * Dh, t0 * Hkv * Dh
            kp[t0:t1] = synth.qkv_block(seed, synth.STREAM_K, seq_id, cnt, None, off).reshape(-1, Hkv, Dh)
            vp[t0:t1] = synth.qkv_block(seed, synth.STREAM_V, seq_id, cnt, None, off).reshape(-1, Hkv, Dh)
        self.q, self.kt, self.vt, self.kp, self.vp, self.kvs = q, kt, vt, kp, vp, kvs

    def run(self):
        """Returns (seconds for expansion + finalise + accept, seconds for attention on self.heads)."""
        O, cfg = self.O, self.cfg
        t0 = time.perf_counter()
        tree = O.expand(self.root, self.logits_fn, self.p)
        O.finalize(tree, self.L)
        tt = O.target_argmax(self.target, tree.n_nodes)
        O.accept(tree, tt)
        t1 = time.perf_counter()
        g = cfg.group
        for h in self.heads:
            kv = h // g
            O.tree_attention(self.q[:, h:h + 1], self.kp[:, kv:kv + 1], self.vp[:, kv:kv + 1],
                             self.kt[:, kv:kv + 1], self.vt[:, kv:kv + 1], tree, 1.0 / math.sqrt(cfg.head_dim))
        t2 = time.perf_counter()
        return t1 - t0, t2 - t1


def oracle_sample_plan(cfg):
    """Which part of a step the oracle is timed on, so that one sample stays within seconds."""
    all_heads = cfg.n_q_heads * (cfg.prefix_max + cfg.budget) <= 32 * 4200
    heads = list(range(cfg.n_q_heads)) if all_heads else [0, cfg.n_q_heads // 2, cfg.n_q_heads - 1]
    return heads


def time_oracle(cfg, seed: int, steps: int, warmup: int, budget_s: float):
    """Times the oracle on sequence 0 of the workload.  Returns a dict with steps/s of a whole batch
    (sequence time x batch; attention scaled from the sampled heads to all heads)."""
    try:
        from threadpoolctl import threadpool_limits
        limiter = threadpool_limits(limits=1)
    except Exception:                                     # pragma: no cover
        limiter = None
    heads = oracle_sample_plan(cfg)
    st = OracleStep(cfg, seed, 0, heads)
    for _ in range(warmup):
        st.run()
    times = []
    t_start = time.perf_counter()
    for i in range(steps):
        a, b = st.run()
        times.append(a + b * cfg.n_q_heads / len(heads))
        if time.perf_counter() - t_start > budget_s and i + 1 >= 1:
            break
    if limiter is not None:
        limiter.restore_original_limits()
    per_seq = sum(times) / len(times)
    per_step = per_seq * cfg.batch
    sample = (f"{len(times)} oracle steps of sequence 0 ({'all' if len(heads) == cfg.n_q_heads else len(heads)} "
              f"of {cfg.n_q_heads} attention heads{'' if len(heads) == cfg.n_q_heads else ', scaled to all'}; "
              f"x batch {cfg.batch})")
    return dict(value=1.0 / per_step, unit=UNIT, cores=1, kind="oracle", sample=sample,
                ms_per_step=per_step * 1e3, steps_timed=len(times))


def workload_text(cfg) -> str:
    pl = f"{cfg.prefix_min}" if cfg.prefix_min == cfg.prefix_max else f"U[{cfg.prefix_min},{cfg.prefix_max}]"
    return (f"{cfg.name}: batch {cfg.batch}, vocab {cfg.vocab}, budget N={cfg.budget} (root included), D_max "
            f"{cfg.max_depth}, K {cfg.topk}, mu {cfg.mu}, {cfg.n_q_heads}/{cfg.n_kv_heads} heads, Dh {cfg.head_dim}, "
            f"prefix {pl}, spike mix '{cfg.spike}', T {cfg.temp}")


# --------------------------------------------------------------------------------------------
# reference arm: the oracle on host cores
# --------------------------------------------------------------------------------------------
def run_reference(args, cfg):
    from paper_2601_07353_b200 import dist
    info = dist.env_rank_info()
    if not info.is_main:
        return 0
    r = time_oracle(cfg, args.seed, args.steps, args.warmup, budget_s=150.0)
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": r["steps_timed"], "warmup": args.warmup, "ms_per_step": r["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_text(cfg)},
        "cpu_baseline": {"value": r["value"], "unit": UNIT, "cores": r["cores"], "kind": "oracle",
                         "sample": r["sample"]},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# --------------------------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------------------------
def set_bytes(cfg, wl) -> int:
    """HBM bytes one step touches in one input set (upper bound: every draft row counted)."""
    t = wl.draft.numel() * 4 + wl.target.numel() * 4
    for x in (wl.q, wl.k_prefix, wl.v_prefix, wl.k_tree, wl.v_tree, wl.out):
        t += x.numel() * 2
    return t


def run_talon(args, cfg):
    import torch
    from paper_2601_07353_b200 import dist, roofline, synth, talon, workload

    info = dist.env_rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    dev_index = info.local_rank % torch.cuda.device_count()
    torch.cuda.set_device(dev_index)
    dev = torch.device("cuda", dev_index)
    dist.init(info, "nccl")
    peaks = roofline.load_peaks(ROOT)

    B, N, V, D = cfg.batch, cfg.budget, cfg.vocab, cfg.max_depth
    t = workload.make_talon(cfg, device=dev_index)
    # how many input sets: bytes between two uses of a set must exceed L2 several times
    probe = workload.build_workload(cfg, t, args.seed, dist.rank_sequence_ids(info, 1, B)[0])
    per_set = set_bytes(cfg, probe)
    n_sets = max(1, math.ceil(ROTATION_FACTOR * L2_BYTES / per_set)) if args.sets is None else args.sets
    free_b, _ = torch.cuda.mem_get_info(dev)
    n_sets = max(1, min(n_sets, int(0.6 * free_b // per_set) + 1))
    ids = dist.rank_sequence_ids(info, n_sets, B)
    sets = [probe] + [workload.build_workload(cfg, t, args.seed, ids[s]) for s in range(1, n_sets)]
    torch.cuda.synchronize()
    assert t.poll_status() == talon.OK

    # ---- per-step algorithmic work, from the trees the sets produce ----
    exp_b = arg_b = att_b = att_f = 0
    shapes = []
    att_flops_set = []
    for wl in sets:
        f_before = att_f
        lo = wl.tree.layer_off.cpu().numpy()
        nn = wl.tree.n_nodes.cpu().numpy()
        pl = wl.prefix_len.cpu().numpy()
        for b in range(B):
            rows = roofline.expanded_rows(lo[b], N, D)
            exp_b += roofline.expand_bytes(rows, V)
            arg_b += roofline.argmax_bytes(int(nn[b]), V)
            att_b += roofline.attention_bytes(int(pl[b]), int(nn[b]), cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, N)
            att_f += roofline.attention_flops(int(pl[b]), int(nn[b]), cfg.n_q_heads, cfg.head_dim)
            shapes.append((int(nn[b]), int(np.max(wl.tree.depth[b].cpu().numpy())), rows))
        att_flops_set.append(att_f - f_before)
    per_step = {k: v / n_sets for k, v in dict(expand_rows=exp_b, target_argmax=arg_b, tree_attention=att_b).items()}
    att_flops_step = att_f / n_sets

    sampler = ClockSampler(dev_index) if info.is_main else None
    step = lambda i: workload.run_step_fused(t, sets[i % n_sets])
    # Everything below runs on a stream of its own: talon_step replays a captured graph of its
    # launches from the second call with the same arguments, which the legacy default stream cannot do.
    torch.cuda.synchronize()
    main_stream = torch.cuda.Stream(dev)
    torch.cuda.set_stream(main_stream)

    # ---- warm-up (every input set at least twice, so that each set's step has been captured),
    # then an untimed pass with every kernel bracketed: which kernel dominates ----
    warm = max(args.warmup, 3, 2 * n_sets)
    for i in range(warm):
        step(i)
    torch.cuda.synchronize()
    t.timing_enable(64 * (2 * D + 8))
    prof_steps = args.prof_steps
    for i in range(prof_steps):
        step(i)
    kt = t.timing_read()
    kernels = {k: {"ms_per_step": ms / prof_steps, "launches_per_step": n / prof_steps} for k, (ms, n) in kt.items() if n}
    streaming = [k for k in ("expand_rows", "tree_attention", "target_argmax") if k in kernels]
    dominant = max(streaming, key=lambda k: kernels[k]["ms_per_step"])
    t.timing_enable(0)

    # ---- the timed region: K steps, the dominant kernel bracketed by events on the launch stream ----
    K = args.steps
    # the dominant kernel is bracketed on every TIMED_EVERY-th step of the timed region only, so
    # that the event records do not slow the headline down
    sampled = [i for i in range(K) if i % TIMED_EVERY == 0]
    t.timing_enable(int(len(sampled) * kernels[dominant]["launches_per_step"]) + 8, [dominant])
    launches0 = t.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    dist.barrier(info)
    wall0 = time.time()
    ev0.record()
    for i in range(K):
        t.timing_pause(i % TIMED_EVERY != 0)
        step(i)
    ev1.record()
    torch.cuda.synchronize()
    dist.barrier(info)
    wall1 = time.time()
    seconds = ev0.elapsed_time(ev1) * 1e-3
    gpu_launches = t.launch_count() - launches0
    dom_ms, dom_n = t.timing_read()[dominant]
    t.timing_enable(0)
    assert t.poll_status() == talon.OK
    seconds_max = dist.max_over_ranks(seconds, info, dev)
    value = dist.whole_job_rate(K, seconds_max, info)

    # ---- the same steps as one CUDA graph replay each (no library entry, no launch gaps from the host) ----
    graph_info = None
    if not args.no_graph:
        try:
            graphs = []
            side = torch.cuda.Stream(dev)
            with torch.cuda.stream(side):
                for s in range(n_sets):
                    gph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(gph, stream=side):
                        workload.run_step_fused(t, sets[s])
                    graphs.append(gph)
            torch.cuda.synchronize()
            for i in range(3 * n_sets):
                graphs[i % n_sets].replay()
            torch.cuda.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record()
            for i in range(K):
                graphs[i % n_sets].replay()
            g1.record()
            torch.cuda.synchronize()
            gs = dist.max_over_ranks(g0.elapsed_time(g1) * 1e-3, info, dev)
            graph_info = {"value": dist.whole_job_rate(K, gs, info), "unit": UNIT, "ms_per_step": gs / K * 1e3}
            del graphs
        except Exception as e:                           # graph capture is an extra, never the headline
            graph_info = {"error": str(e).splitlines()[0][:200]}
            torch.cuda.synchronize()

    # ---- the sampling verification (the paper's temperature-1 setting) on the same trees: an extra, not the headline ----
    sampling = None
    if not args.no_sampling:
        Ks = min(K, 64)
        dev_t = sets[0].target.device
        uas = [torch.from_numpy(np.stack([synth.verify_uniforms(args.seed, sid, N, 0)[0] for sid in wl.seq_ids])).to(dev_t)
               for wl in sets]
        uss = [torch.tensor([synth.verify_uniforms(args.seed, sid, N, 0)[1] for sid in wl.seq_ids], dtype=torch.float64,
                            device=dev_t) for wl in sets]
        s_tok = torch.zeros(B, dtype=torch.int32, device=dev_t)

        def sample_step(i):
            wl = sets[i % n_sets]
            t.accept_sample(wl.tree, wl.target, 1.0, uas[i % n_sets], uss[i % n_sets], wl.accept_len, wl.accept_nodes, s_tok)

        for i in range(3):
            sample_step(i)
        torch.cuda.synchronize()
        t.timing_enable(2 * Ks + 8, ["target_softmax_stats", "accept_sample"])
        for i in range(Ks):
            sample_step(i)
        st = t.timing_read()
        t.timing_enable(0)
        assert t.poll_status() == talon.OK
        sm_ms, sm_n = st["target_softmax_stats"]
        wk_ms, wk_n = st["accept_sample"]
        if sm_n and wk_n:
            gbs = per_step["target_argmax"] / (sm_ms / sm_n * 1e-3) / 1e9
            sampling = {"temperature": 1.0, "calls": Ks,
                        "target_softmax_stats": {"ms_per_call": sm_ms / sm_n, "algorithmic_gbs": gbs,
                                                 "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]},
                        "accept_sample": {"ms_per_call": wk_ms / wk_n}}

    # ---- end to end: host buffers in, host results out, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        pin = lambda x: x.cpu().pin_memory()
        hi32 = lambda *s: torch.zeros(*s, dtype=torch.int32).pin_memory()
        n_host = max(1, min(n_sets, int((8 << 30) // per_set)))
        host = []
        for wl in sets[:n_host]:
            host.append((pin(wl.root_tok), pin(wl.prefix_len), pin(wl.draft), pin(wl.target), pin(wl.q),
                         pin(wl.k_prefix), pin(wl.v_prefix), pin(wl.k_tree), pin(wl.v_tree)))
        out_h = torch.zeros(B, N, cfg.n_q_heads, cfg.head_dim, dtype=torch.bfloat16).pin_memory()
        res = (hi32(B), hi32(B, N), hi32(B, N), hi32(B, N), hi32(B, N), hi32(B), hi32(B, D + 1), hi32(B))
        h2d = sum(x.numel() * x.element_size() for x in host[0]) + 8 * B
        d2h = out_h.numel() * 2 + sum(x.numel() * 4 for x in res)
        Ke = max(3, min(K, int(20.0 / max(1e-4, h2d / 20e9))))       # keep this leg within ~20 s
        scale = 1.0 / math.sqrt(cfg.head_dim)
        for i in range(3):
            assert t.step_host(*host[i % n_host], scale, out_h, *res) == talon.OK
        torch.cuda.synchronize()
        dist.barrier(info)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0 = time.perf_counter()
        e0.record()
        for i in range(Ke):
            t.step_host(*host[i % n_host], scale, out_h, *res)
        e1.record()
        torch.cuda.synchronize()
        w1 = time.perf_counter()
        dist.barrier(info)
        es = dist.max_over_ranks(max(e0.elapsed_time(e1) * 1e-3, 0.0), info, dev)
        e2e = {"value": dist.whole_job_rate(Ke, es, info), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": Ke, "ms_per_step": es / Ke * 1e3,
               "host_wall_ms_per_step": (w1 - w0) / Ke * 1e3,
               "api": "talon_step_host (pinned host buffers in, host results out)"}
        del host

    if sampler is not None:
        sampler.stop()
    clocks = sampler.summary(wall0, wall1) if sampler is not None else None

    # ---- roofline of the dominant kernel over the timed region ----
    per_set_bytes = []
    for wl in sets:
        lo = wl.tree.layer_off.cpu().numpy(); nn = wl.tree.n_nodes.cpu().numpy(); pl = wl.prefix_len.cpu().numpy()
        tot = 0
        for b in range(B):
            if dominant == "expand_rows":
                tot += roofline.expand_bytes(roofline.expanded_rows(lo[b], N, D), V)
            elif dominant == "target_argmax":
                tot += roofline.argmax_bytes(int(nn[b]), V)
            else:
                tot += roofline.attention_bytes(int(pl[b]), int(nn[b]), cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, N)
        per_set_bytes.append(tot)
    dom_bytes_total = float(sum(per_set_bytes[i % n_sets] for i in sampled))      # the bracketed steps' bytes
    dom_flops_total = float(sum(att_flops_set[i % n_sets] for i in sampled))
    roof = None
    if dom_n > 0 and dom_ms > 0:
        timed_frac = dom_n / max(1.0, len(sampled) * kernels[dominant]["launches_per_step"])
        achieved = dom_bytes_total * timed_frac / (dom_ms * 1e-3) / 1e9
        intensity = att_flops_step / max(1.0, per_step["tree_attention"])
        ridge = peaks["bf16_tflops_sustained"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
        bound = "hbm"
        ratio = roofline.captured_traffic_ratio(dominant)
        roof = {"kernel": dominant, "bound": bound, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_source": f"of {peaks['source']}",
                "traffic": None if ratio is None else ratio * dom_bytes_total * timed_frac / dom_n,
                "traffic_source": None if ratio is None else "ncu capture of an earlier run, same kernel source: DRAM bytes per algorithmic byte x this run's bytes per launch",
                "launches_timed": int(dom_n), "timed_steps": f"1 step in {TIMED_EVERY} of the timed region", "avg_launch_us": dom_ms / dom_n * 1e3,
                "algorithmic_bytes_per_launch": dom_bytes_total * timed_frac / dom_n}
        if dominant == "tree_attention" and intensity > ridge:
            tf = dom_flops_total * timed_frac / (dom_ms * 1e-3) / 1e12
            roof.update({"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                         "frac": tf / peaks["bf16_tflops_sustained"]})
    # secondary figures from the bracketed pass (event pairs around every kernel; launch gaps included)
    for k in ("expand_rows", "target_argmax", "tree_attention"):
        if k in kernels and kernels[k]["ms_per_step"] > 0:
            kernels[k]["algorithmic_gbs"] = per_step[k] / (kernels[k]["ms_per_step"] * 1e-3) / 1e9
            kernels[k]["frac_of_hbm_peak"] = kernels[k]["algorithmic_gbs"] / peaks["hbm_gbs"]
            kernels[k]["frac_of_nominal_8tbs"] = kernels[k]["algorithmic_gbs"] / 8000.0
    if "tree_attention" in kernels:
        kernels["tree_attention"]["tflops"] = att_flops_step / (kernels["tree_attention"]["ms_per_step"] * 1e-3) / 1e12

    cpu = None
    if info.is_main and info.world == 1 and not args.no_cpu_baseline:
        r = time_oracle(cfg, args.seed, 10, 0, budget_s=15.0)
        cpu = {"value": r["value"], "unit": UNIT, "cores": r["cores"], "kind": "oracle", "sample": r["sample"]}

    if info.is_main:
        nn = [s[0] for s in shapes]; dp = [s[1] for s in shapes]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": info.world, "steps": K, "warmup": warm,
            "ms_per_step": seconds_max / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32 logits, f64 path scores, bf16 attention (f32 accumulate)", "data": "synthetic",
            "config": {"workload": workload_text(cfg),
                       "l2": f"inputs larger than L2: steps rotate over {n_sets} input sets of {per_set / 1e6:.1f} MB "
                             f"({n_sets * per_set / 1e6:.0f} MB vs 126 MB L2)",
                       "step": f"talon_step: reset + {D} expand-layer calls + build + tree attention + accept "
                               "(the library replays its own captured graph of these launches; steps whose "
                               "dominant kernel is bracketed by events are launched one by one)",
                       "sequences_per_rank": B, "input_sets": n_sets},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(gpu_launches), "roofline": roof, "cpu_baseline": cpu,
            "graph_replay": graph_info, "kernels": kernels, "sampling_verify": sampling,
            "tree_shapes": {"n_nodes_min": min(nn), "n_nodes_max": max(nn), "max_depth_min": min(dp), "max_depth_max": max(dp),
                            "expanded_rows_per_seq_mean": float(np.mean([s[2] for s in shapes]))},
            "sequence_steps_per_s": value * B,
        }
        print(json.dumps(line))
    t.close()
    dist.shutdown()
    return 0


# --------------------------------------------------------------------------------------------
# the paper's own on-path experiment: single-layer tree-expansion latency on Zipf rows
# --------------------------------------------------------------------------------------------
def run_zipf_micro(args):
    """Latency of one expansion layer (the K children of the root as frontier, batch 1) on rows with
    P(rank r) ~ r^-alpha, for the paper's vocabularies and exponents: 20 warm-up runs, mean of 100,
    as in the appendix's tree-construction micro-benchmark.  Extra mode; prints its own JSON line."""
    import torch
    from paper_2601_07353_b200 import roofline, synth, talon

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = roofline.load_peaks(ROOT)
    N, K, D = 60, 10, 8
    results = []
    for V in (32000, 128256, 151936):
        t = talon.Talon(batch_max=1, vocab=V, budget=N, root_topk=K, cand_topk=K, max_depth=D, mu=0.03,
                        n_q_heads=32, n_kv_heads=8, head_dim=128, device=0)
        tree = t.alloc_tree(1)
        root = torch.zeros(1, dtype=torch.int32, device=dev)
        plen = torch.zeros(1, dtype=torch.int32, device=dev)
        draft = torch.zeros(1, N, V, dtype=torch.float32, device=dev)
        for alpha in (0.7, 1.35, 5.0):
            for i in range(K + 1):                    # the root's row and the rows of its K children
                draft[0, i] = synth.zipf_logits_row(V, alpha, args.seed, i, device=dev)
            e0 = [torch.cuda.Event(enable_timing=True) for _ in range(120)]
            e1 = [torch.cuda.Event(enable_timing=True) for _ in range(120)]
            for it in range(120):
                t.reset(tree, root, plen)
                t.expand_layer(tree, draft)           # root layer (Top-K): untimed
                e0[it].record()
                t.expand_layer(tree, draft)           # the timed layer: K frontier rows, gate, truncation
                e1[it].record()
            torch.cuda.synchronize()
            assert t.poll_status() == talon.OK
            lo = tree.layer_off[0].cpu().tolist()
            rows = lo[2] - lo[1]
            us = [a.elapsed_time(b) * 1e3 for a, b in zip(e0[20:], e1[20:])]
            mean = sum(us) / len(us)
            results.append({"vocab": V, "alpha": alpha, "frontier_rows": rows, "nodes_added": lo[3] - lo[2],
                            "us_mean": mean, "us_min": min(us),
                            "algorithmic_gbs": 4.0 * V * rows / (mean * 1e-6) / 1e9})
        t.close()
    print(json.dumps({"metric": "single-layer tree-expansion latency (Zipf rows, warm caches)", "unit": "us",
                      "higher_is_better": False, "n_gpus": 1, "data": "synthetic",
                      "config": {"workload": "batch 1, budget 60, K 10, frontier = the root's children; "
                                             "20 warm-up runs, mean of 100, events around the launch"},
                      "peak_hbm_gbs": peaks["hbm_gbs"], "results": results}))
    return 0


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", choices=["talon", "reference"], default="talon")
    ap.add_argument("--config", default="llama8b")
    ap.add_argument("--seed", type=int, default=None)
    ap.add_argument("--sets", type=int, default=None, help="input sets to rotate over (default: enough to defeat L2)")
    ap.add_argument("--prof-steps", type=int, default=32, help="steps of the untimed per-kernel pass")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sampling", action="store_true", help="skip the sampling-verification extra")
    ap.add_argument("--zipf-micro", action="store_true",
                    help="instead of the step benchmark: single-layer expansion latency on Zipf rows")
    args = ap.parse_args(argv)
    from paper_2601_07353_b200 import synth
    if args.seed is None:
        args.seed = synth.DEFAULT_SEED
    if args.zipf_micro:
        return run_zipf_micro(args)
    cfg = synth.CONFIGS[args.config]
    if args.impl == "reference":
        args.steps = 10 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        return run_reference(args, cfg)
    args.steps = 2000 if args.steps is None else args.steps
    args.warmup = 20 if args.warmup is None else args.warmup
    return run_talon(args, cfg)


if __name__ == "__main__":
    sys.exit(main())
