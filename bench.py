#!/usr/bin/env python
"""Benchmark of the speculative decode round (draft k steps -> verify k+1 -> accept/rollback).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config NAME] [--k K]

A step is one round over the synthetic workload (default: the 0.5B-class parallel hybrid, batch 1,
512-token prompt, seeded geometric accept pattern with per-token success 0.68).  Rank 0 prints one
JSON line.  With N > 1 every rank runs an independent replica (sequences are independent; there is
no collective on the data path) and the value is the sum over replicas divided by the slowest; without a
launcher around it (no RANK in the environment) `--gpus N` starts the N ranks itself.
The default single-GPU run also reports plain autoregressive decoding (k = 0), the other draft lengths, and
the other workloads (3B-class at batch 1 and 8, the sequential hybrid, batch-64 long context) under `by_config`.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import hs_inputs as hi  # noqa: E402

METRIC = "decode tokens/s at k=2 (seeded accept)"
UNIT = "tokens/s"
ALPHA = 0.68
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the projection kernel from the ncu capture summarised in
# profiles/gemv_kernel_cfg2.md: mean over the four projections of a layer of a verify pass, caches left alone (None: the
# kernel changed after the counters were taken)
GEMV_DRAM_BYTES_PER_LAUNCH = 11.60e6


# ------------------------------------------------------------------------------------------------
# algorithmic bytes of one step: every used weight once, recurrent state read + written once,
# KV rows read once + T rows appended, logits written (snapshot copies beyond the first are overhead)
# ------------------------------------------------------------------------------------------------
def step_bytes(s, draft: bool, T: int, kv_len: float, batch: int = 1) -> float:
    w = 0.0          # weight bytes, shared by the batch
    per_seq = 0.0
    for l in range(s.L):
        t = s.layer_type(l)
        if draft and t == hi.LAYER_ATT:
            continue
        attn_rows = (s.qh + 2 * s.kvh) * s.hd
        mlp = 3 * s.ff * s.d
        if t == hi.LAYER_PAR:
            rows = 2 * s.d_inner + 2 * s.N + s.H + (0 if draft else attn_rows)
            w += 2 * (rows * s.d + s.d * s.d_inner + (0 if draft else s.d * s.qh * s.hd) + mlp)
            w += 4 * (2 * s.d + s.convd * 5 + 3 * s.H + s.d_inner)
            per_seq += 2 * 4 * s.H * s.P * s.N + 2 * 4 * 3 * s.convd
        elif t == hi.LAYER_GDN:
            rows = 2 * s.gh * s.gdk + 2 * s.gh * s.gdv + 2 * s.gh
            w += 2 * (rows * s.d + s.d * s.gh * s.gdv + mlp) + 4 * (2 * s.d + s.convd * 5 + s.gdv)
            per_seq += 2 * 4 * s.gh * s.gdv * s.gdk + 2 * 4 * 3 * s.convd
        else:
            w += 2 * (attn_rows * s.d + s.d * s.qh * s.hd + mlp) + 4 * 2 * s.d
        if not draft and t != hi.LAYER_GDN:
            per_seq += 2 * 2 * s.kvh * s.hd * (kv_len + T)          # K and V rows read + appended
    w += 2 * s.V * s.d + 4 * s.d                                      # LM head + final norm
    per_seq += T * (2 * s.d + 4 * s.V)                                # embedding rows, logits
    return w + batch * per_seq


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx, self.rows, self.proc = gpu_index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm = [float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) < 9:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ------------------------------------------------------------------------------------------------
def oracle_seq_with_context(model, s, ctx_len, seq=0, seed=3):
    """An oracle sequence that holds ctx_len consumed tokens: the seeded synthetic context of the parity tests
    (recurrent state, conv window, KV rows) is written into it, since consuming a long prompt on the CPU would take
    minutes before the first timed round."""
    q = model.new_seq()
    for l in range(s.L):
        t = s.layer_type(l)
        if t != hi.LAYER_ATT:
            (q.ssm() if t == hi.LAYER_PAR else q.gdn())[l] = hi.injected_state(s, l, seq, hi.CTX_SSM if t == hi.LAYER_PAR else hi.CTX_GDN, seed)
            q.conv()[l] = hi.injected_state(s, l, seq, hi.CTX_CONV, seed)
        if t != hi.LAYER_GDN and ctx_len > 0:
            q.k()[l, :ctx_len] = hi.injected_kv(s, l, seq, ctx_len, hi.CTX_K, seed)
            q.v()[l, :ctx_len] = hi.injected_kv(s, l, seq, ctx_len, hi.CTX_V, seed)
    q.set(ctx_len, int(hi.make_prompt(s.V, 1, seq=1000 + seq)[0]))
    return q


def cpu_oracle_rate(s, blob, table, k, budget_s=15.0, max_rounds=24):
    """tokens/s of the oracle, as it stands, on the host cores, on a bounded sample of the workload: the same
    model, draft length, accept pattern and context length, fewer rounds."""
    import oracle
    model = oracle.Model(s, blob, table, s.prompt_len + (max_rounds + 2) * (k + 1) + 8)
    q = oracle_seq_with_context(model, s, s.prompt_len)
    forced = hi.forced_accept(k, max_rounds + 1)
    q.round(k, forced_n=int(forced[0]))                  # warm-up round
    t0 = time.perf_counter(); toks = 0; r = 0
    while r < max_rounds and (time.perf_counter() - t0 < budget_s or r < 2):
        res = q.round(k, forced_n=int(forced[r + 1]))
        toks += res["n"] + 1; r += 1
    dt = time.perf_counter() - t0
    return toks / dt, r, dt, s.prompt_len


def run_reference(args):
    """The reference arm of this build is the CPU oracle, timed as it stands on the host cores: the same workload
    (model shape, draft length, accept pattern, context length), each step one round."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    s = hi.CONFIGS[args.config]
    if args.prompt_len is not None:
        s = s.replace(prompt_len=args.prompt_len)
    blob, table = hi.make_weights(s, 0, "unit")
    import oracle
    k, plen = args.k, s.prompt_len
    B = s.batch if args.batch is None else args.batch
    model = oracle.Model(s, blob, table, plen + (args.steps + args.warmup + 2) * (k + 1) + 8)
    q = oracle_seq_with_context(model, s, plen)
    forced = hi.forced_accept(k, args.steps + args.warmup)
    for r in range(args.warmup):
        q.round(k, forced_n=int(forced[r]))
    t0 = time.perf_counter(); toks = 0
    for r in range(args.steps):
        toks += q.round(k, forced_n=int(forced[args.warmup + r]))["n"] + 1
    dt = time.perf_counter() - t0
    val = toks / dt
    cores = len(os.sched_getaffinity(0))
    sample = "%s shape, one sequence, %d-token injected context, %d rounds at k=%d, forced accept pattern" % (s.name, plen, args.steps, k)
    print(json.dumps({
        "impl": "reference", "metric": METRIC.replace("k=2", "k=%d" % k), "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": s.name, "k": k, "batch": B, "prompt_len": plen, "alpha": ALPHA,
                   "sampled": "one sequence of the batch" if B > 1 else "the whole batch"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def free_port():
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_replicas(args, argv):
    """`python bench.py --gpus N` outside a launcher: start the N ranks here (one process per GPU, rendezvous on
    127.0.0.1); rank 0 prints the JSON line.  Returns the largest exit code."""
    port = free_port()
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + argv, env=env))
    return max(p.wait() for p in procs)


class Legs:
    """Timed rounds on one engine.  A leg = W warm-up + K timed rounds at one draft length from a restored context,
    everything enqueued without host reads (graph replay), timed with CUDA events on the library's stream."""

    def __init__(self, torch, dev, world, steps, warm):
        self.torch, self.dev, self.world, self.steps, self.warm = torch, dev, world, steps, warm

    def barrier(self):
        self.torch.cuda.synchronize(self.dev)
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
            self.torch.cuda.synchronize(self.dev)

    def timed(self, eng, B, k, restore, ctx_mean):
        torch, steps, warm = self.torch, self.steps, self.warm
        restore()
        forced = np.stack([hi.forced_accept(k, warm + steps, seq=b) for b in range(B)], axis=1)   # [rounds][B]
        f_dev = torch.from_numpy(np.ascontiguousarray(forced)).to(self.dev)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
        for r in range(warm):
            eng.draft(k); eng.verify(k); eng.accept_rollback(f_dev[r], wait=False)
        self.barrier()
        l0 = eng.launch_count()
        for r in range(steps):
            e = ev[r]
            e[0].record(eng.stream)
            eng.draft(k)
            e[1].record(eng.stream)
            eng.verify(k)
            e[2].record(eng.stream)
            eng.accept_rollback(f_dev[warm + r], wait=False)
            e[3].record(eng.stream)
        self.barrier()
        total_ms = ev[0][0].elapsed_time(ev[-1][3])
        d_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / steps
        v_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / steps
        a_ms = sum(e[2].elapsed_time(e[3]) for e in ev) / steps
        toks = int((forced[warm:] + 1).sum())
        assert eng.device_status() == 0
        kv_mid = ctx_mean + float((forced + 1).sum(axis=0).mean()) * (warm + steps / 2) / (warm + steps)
        return dict(total_ms=total_ms, draft_ms=d_ms, verify_ms=v_ms, accept_ms=a_ms, tokens=toks,
                    launches=eng.launch_count() - l0, kv_mid=kv_mid)

    def report(self, s, B, k, r, peak):
        """Step-level figures of one leg: latencies, tokens/s and algorithmic bytes / event time against the peak."""
        db, vb = step_bytes(s, True, 1, 0, B), step_bytes(s, False, k + 1, r["kv_mid"], B)
        d_step_ms = r["draft_ms"] / max(k, 1)
        out = {"tokens_per_s": self.world * r["tokens"] / (r["total_ms"] * 1e-3), "ms_per_round": r["total_ms"] / self.steps,
               "draft_step_ms": d_step_ms if k else None, "verify_step_ms": r["verify_ms"], "accept_ms": r["accept_ms"],
               "draft_step_GBps": db / (d_step_ms * 1e-3) / 1e9 if k else None,
               "verify_step_GBps": vb / (r["verify_ms"] * 1e-3) / 1e9,
               "draft_frac_of_measured_peak": db / (d_step_ms * 1e-3) / 1e9 / peak if k else None,
               "verify_frac_of_measured_peak": vb / (r["verify_ms"] * 1e-3) / 1e9 / peak,
               "draft_bytes": db, "verify_bytes": vb, "mean_context": r["kv_mid"]}
        return out


def inject_random_context(torch, eng, s, B, lens, seed=3):
    """Contexts too long to prefill inside a benchmark run are injected: the recurrent state, the conv windows and
    the KV cache are filled on the device with seeded random values (uniform +-0.5 state, N(0,1) conv inputs and
    KV rows, the value distributions of the parity tests' injected contexts), and every sequence is declared to
    hold lens[b] tokens.  Returns the function that restores kv_len / pending before a leg."""
    g = torch.Generator(device=eng.device).manual_seed(seed)

    def fill(t, kind):
        n = t.numel() - eng.GUARD
        step = 1 << 30
        for o in range(0, n, step):
            m = min(step, n - o)
            if kind == "bf16":
                t[o:o + m].view(torch.bfloat16).normal_(generator=g)
            elif kind == "state":
                t[o:o + m].view(torch.float32).uniform_(-0.5, 0.5, generator=g)
            else:
                t[o:o + m].view(torch.float32).normal_(generator=g)
    with torch.cuda.stream(eng.stream):
        fill(eng.t_kv, "bf16"); fill(eng.t_snap, "state"); fill(eng.t_conv, "conv")
    eng.stream.synchronize()
    pend = [int(hi.make_prompt(s.V, 1, seq=1000 + b)[0]) for b in range(B)]

    def restore():
        for b in range(B):
            eng.set_context(b, int(lens[b]), pend[b])
        eng.set_batch(B)
    return restore


def run_ours(args):
    import torch
    from paper_2605_01106_b200 import binding as hs
    from paper_2605_01106_b200.replicas import reduce_max_sum
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    if local_rank >= torch.cuda.device_count():
        raise SystemExit("rank %d has no GPU: %d visible" % (local_rank, torch.cuda.device_count()))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    s = hi.CONFIGS[args.config]
    if args.prompt_len is not None:
        s = s.replace(prompt_len=args.prompt_len)
    B = s.batch if args.batch is None else args.batch
    # draft lengths of the headline workload: the requested one first; k = 0 is plain autoregressive decoding with
    # the full model (one verify pass per token), the denominator of the paper's speed-up (Eq. 1)
    ks = [args.k] + [k for k in (0,) + tuple(s.ks) if k != args.k and args.all_k and world == 1]
    max_k = max(max(ks), 1)
    steps, warm = args.steps, max(args.warmup, 3)
    legs = Legs(torch, dev, world, steps, warm)
    peak, peak_src = measured_peak()
    inject = s.prompt_len > 1024 or B > 4              # long or many prompts: injected context instead of hs_prefill
    blob, table = hi.make_weights(s, 0, "unit")
    lens = hi.context_lengths(B, 4096, 16384) if (s.name == "cfg5_b64" and args.prompt_len is None) else np.full(B, s.prompt_len, np.int32)
    cap = int(lens.max()) + (steps + warm + 4) * (max_k + 1) * 2 + 64
    eng = hs.Engine(s, blob, max_batch=B, max_k=max_k, kv_capacity=cap, flags=hs.HS_FLAG_GRAPHS, device=str(dev))
    if args.attn_geometry:
        ck, tl = (int(x) for x in args.attn_geometry.split("x"))
        eng.set_attn_geometry(ck, tl)
    if inject:
        fresh_context = inject_random_context(torch, eng, s, B, lens)
    else:
        prompts = [hi.make_prompt(s.V, s.prompt_len, seq=b) for b in range(B)]

        def fresh_context():
            eng.reset()
            eng.prefill(prompts)

    def max_over_ranks(ms):
        return reduce_max_sum(ms, 0.0, world, dev)[0]

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    results = {k: legs.timed(eng, B, k, fresh_context, float(lens.mean())) for k in ks}
    clocks = sampler.stop() if rank == 0 else None
    main = results[args.k]
    total_ms = max_over_ranks(main["total_ms"])
    value = world * main["tokens"] / (total_ms * 1e-3)

    # ---- end to end through the host-buffer entry point (H2D of the accept pattern, D2H of results)
    k = args.k
    fresh_context()
    forced = np.stack([hi.forced_accept(k, warm + steps, seq=b) for b in range(B)], axis=1).astype(np.int32)
    pinned = torch.from_numpy(np.ascontiguousarray(forced)).pin_memory().numpy()
    for r in range(warm):
        eng.round_host(k, forced_n=pinned[r])
    legs.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(eng.stream)
    toks_e2e = 0
    for r in range(steps):
        n, em = eng.round_host(k, forced_n=pinned[warm + r])
        toks_e2e += int(n.sum()) + B
    e1.record(eng.stream)
    legs.barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1))
    e2e_val = world * toks_e2e / (e2e_ms * 1e-3)

    # ---- dominant kernel (projection family): live event timing of every launch
    fresh_context()
    f_dev = torch.from_numpy(np.ascontiguousarray(forced)).to(dev)
    eng.profile(True)
    for r in range(min(steps, 10)):
        eng.draft(k); eng.verify(k); eng.accept_rollback(f_dev[r])
    prof = eng.profile_read()
    eng.profile(False)
    g_ms, g_n, g_bytes = prof["gemv"]
    traffic = GEMV_DRAM_BYTES_PER_LAUNCH
    # Duration of the projection kernels inside the timed region.  The kernels of a step overlap (a kernel's
    # prologue runs while its predecessors finish), so a launch has no duration of its own inside the replayed
    # graph.  Bracketing every launch with events serialises the step and adds the cost of the event records, so
    # the bracketed times are only used as weights: the device time of the timed rounds (graph replay, events on
    # the library's stream) is split between the kernel families in proportion to them.
    # achieved = algorithmic bytes of a launch / that in-situ duration.
    prof_rounds = min(steps, 10)
    tot_iso = sum(v[0] for v in prof.values())
    share = g_ms / tot_iso if tot_iso > 0 else 0.0
    round_ms = main["total_ms"] / steps
    n_per_round = g_n / prof_rounds if prof_rounds else 0
    in_situ_us = 1e3 * round_ms * share / n_per_round if n_per_round else 0.0
    bytes_per_launch = g_bytes / max(g_n, 1)
    achieved = bytes_per_launch / (in_situ_us * 1e-6) / 1e9 if in_situ_us else 0.0
    achieved_iso = bytes_per_launch / (g_ms / g_n * 1e-3) / 1e9 if g_n else 0.0
    roofline = {"bound": "hbm", "kernel": "projection kernels (all projections of a round)", "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src, "traffic": traffic,
                "launches_per_round": n_per_round, "avg_launch_us": in_situ_us,
                "algorithmic_bytes_per_launch": bytes_per_launch,
                "isolated": {"avg_launch_us": 1e3 * g_ms / max(g_n, 1), "GBps": achieved_iso,
                             "note": "every launch bracketed by two events: no overlap with neighbours, event cost included"},
                "time_share": {kk: v[0] / tot_iso for kk, v in prof.items()} if tot_iso > 0 else {},
                "time_share_note": "in parallel hybrid blocks the verify attention runs inside the fused mixer launch "
                                   "and is counted under 'mixer'"}
    eng.close()
    del eng
    torch.cuda.empty_cache()

    # ---- the other workloads (rank 0, single GPU): each from an injected context, one clock record per leg
    by_config = {}
    if world == 1 and args.by_config and args.config == "cfg2_0p5b":
        # (workload, batch, draft lengths, extra flags): the batched workloads also with rollback by replay
        # (HS_FLAG_REPLAY: an update log instead of k + 1 state snapshots per verify pass)
        # k = 0 is plain autoregressive decoding with the full model: the denominator of Eq. 1 on that workload.
        # The batch-64 workload is quoted at k = 4; k = 1..3 are added because there the 4 * (k + 1) query rows per KV
        # head still fit one 16-row tensor-core tile of the verify attention.
        plan = [("cfg3_3b", 1, (0, 2, 4), 0), ("cfg3_3b", 8, (0, 4), 0), ("cfg3_3b", 8, (4,), hs.HS_FLAG_REPLAY),
                ("cfg4_seq", 1, (0, 2, 4), 0), ("cfg5_b64", 64, (0, 1, 2, 3, 4), 0), ("cfg5_b64", 64, (4,), hs.HS_FLAG_REPLAY)]
        ar_rate = {}
        blobs = {"cfg2_0p5b": blob}
        for name, nb, kset, xflags in plan:
            sc = hi.CONFIGS[name]
            arch = lambda c: (c.arch, c.L, c.d, c.V, c.H, c.P, c.N, c.qh, c.kvh, c.hd, c.ff, c.gh, c.gdk, c.gdv)
            if name not in blobs:
                same = [n for n in blobs if arch(hi.CONFIGS[n]) == arch(sc)]
                if same:
                    blobs[name] = blobs[same[0]]           # same architecture: the same seeded weights
                else:
                    blobs = {n: b for n, b in blobs.items() if b.nbytes < (2 << 30)}     # keep host memory bounded
                    blobs[name] = hi.make_weights(sc, 0, "unit")[0]
            lens_c = hi.context_lengths(nb, 4096, 16384) if name == "cfg5_b64" else np.full(nb, sc.prompt_len, np.int32)
            mk = max(kset)
            cap_c = int(lens_c.max()) + (steps + warm + 4) * (mk + 1) + 64
            e = hs.Engine(sc, blobs[name], max_batch=nb, max_k=mk, kv_capacity=cap_c, flags=hs.HS_FLAG_GRAPHS | xflags, device=str(dev))
            restore = inject_random_context(torch, e, sc, nb, lens_c)
            entry = {"batch": nb, "context": "injected, lengths %d..%d (mean %.0f)" % (lens_c.min(), lens_c.max(), lens_c.mean()),
                     "rollback": "replay log" if xflags & hs.HS_FLAG_REPLAY else "state snapshots"}
            unit = 4.0 * nb * sum((sc.H * sc.P * sc.N if sc.layer_type(l) == hi.LAYER_PAR else sc.gh * sc.gdv * sc.gdk)
                                  for l in range(sc.L) if sc.layer_type(l) != hi.LAYER_ATT)        # bytes of all recurrent states
            for kk in kset:
                smp = ClockSampler(local_rank); smp.start()
                r = legs.timed(e, nb, kk, restore, float(lens_c.mean()))
                rep = legs.report(sc, nb, kk, r, peak)
                rep["clocks"] = smp.stop()
                # recurrent-state bytes one round really moves in its verify + rollback: snapshots: read 1, write k + 1;
                # replay: read 1 in verify, read 1 + write 1 in the replay kernel (the algorithmic figure counts 2)
                rep["state_traffic_bytes_per_round"] = unit * (3 if xflags & hs.HS_FLAG_REPLAY else kk + 2)
                if kk == 0:
                    ar_rate[(name, nb)] = rep["tokens_per_s"]
                if (name, nb) in ar_rate:
                    rep["speedup_vs_autoregressive"] = rep["tokens_per_s"] / ar_rate[(name, nb)]
                entry["k%d" % kk] = rep
            by_config["%s@b%d%s" % (name, nb, "+replay" if xflags & hs.HS_FLAG_REPLAY else "")] = entry
            e.close()
            del e
            torch.cuda.empty_cache()

    if rank != 0:
        return
    step_roof = {str(kk): legs.report(s, B, kk, r, peak) for kk, r in results.items()}
    if "0" in step_roof:
        ar = step_roof["0"]["tokens_per_s"]
        for kk, v in step_roof.items():
            v["speedup_vs_autoregressive"] = v["tokens_per_s"] / ar
    out = {
        "metric": METRIC.replace("k=2", "k=%d" % args.k), "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warm,
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": s.name, "k": args.k, "batch": B, "prompt_len": s.prompt_len, "alpha": ALPHA,
                   "context": "injected" if inject else "prefilled",
                   "weights": "bf16", "state": "f32", "kv": "bf16", "cuda_graphs": True,
                   "l2": "inputs larger than L2 (every step streams %.2f GB of weights)" % (step_bytes(s, True, 1, 0, B) / 1e9),
                   "parallelism": "replicas x%d (no collective)" % world},
        "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": 4 * B, "d2h_bytes_per_step": 4 * B * (k + 2),
                "ms_per_step": e2e_ms / steps},
        "gpu_launches": int(main["launches"]),
        "roofline": roofline,
        "by_k": step_roof,
        "by_k_note": "k = 0 is plain autoregressive decoding with the full model (one verify pass per token)",
        "by_config": by_config,
    }
    if world == 1 and not args.no_cpu:
        val, rounds, dt, plen = cpu_oracle_rate(s, blob, table, args.k)
        out["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                               "sample": "%s shape, one sequence, %d-token injected context, %d rounds at k=%d (%.1f s), forced accept pattern"
                                         % (s.name, plen, rounds, args.k, dt)}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg2_0p5b", choices=sorted(hi.CONFIGS))
    ap.add_argument("--k", type=int, default=2)
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--prompt-len", type=int, default=None, help="override the workload's prompt length (profiling runs)")
    ap.add_argument("--all-k", dest="all_k", action="store_true", default=True)
    ap.add_argument("--one-k", dest="all_k", action="store_false")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--attn-geometry", default=None, help="CHUNKxTILES: fix the KV split of the verify attention (profiling runs)")
    ap.add_argument("--no-configs", dest="by_config", action="store_false", default=True,
                    help="skip the legs on the other workloads (profiling and quick runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(spawn_replicas(args, sys.argv[1:]))     # no launcher around us: start the N ranks here
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
