#!/usr/bin/env python
"""Benchmark of the DART drafting step (dart_draft_step + dart_build_tree) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch of synthetic input: feature FC,
draft decoder layer, LM head with fused log-softmax/top-k, N-gram tree pruning.  Prints ONE
JSON line (rank 0).  With N > 1 every rank runs an independent replica of the step on its
own GPU (the path has no exchange step: "replicas only", weak scaling); the timed region is
bracketed by barriers and the time is the max over ranks.

--impl reference times the CPU oracle (oracle/) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "draft_steps_per_second"
UNIT = "steps/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200",
                                          "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[1])); smax.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7), ("sw_power_cap", 8)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def run_reference(args):
    """The oracle, as it stands, on the host cores.  A full fp64 step takes ~12 s at the Qwen3-14B
    shape, so each timed step is a bounded sample of it: every matrix product of the step is run
    by the oracle's own `linear` on the first `frac` of that matrix's output rows (inputs are the
    step's real activations), attention, top-k and the tree run in full.  `value` counts the
    fraction of a step each sample covers."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import parity
    from oracle import forward as ofw, tree as otree
    from paper_2601_19278_b200 import synthetic as syn
    w = syn.WORKLOADS[args.workload]
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    rows = syn.make_ngram_rows(w.vocab, min(w.ngram_rows, 200_000), w.ngram_mode)
    tri, bi = otree.tables_from_rows(rows)
    npw, npi = parity.np_weights(wt), parity.np_inputs(inp)
    cfg = parity.oracle_cfg(w)
    t0 = time.perf_counter()
    full = ofw.draft_forward(cfg, npw, npi, keep_intermediates=True)      # untimed: activations + full-step time
    t_full = time.perf_counter() - t0
    frac = min(1.0, 120.0 / ((args.steps + args.warmup) * t_full))
    feats = ofw.bf16_to_f64(npi["feats"])
    seq = npi["seq_lens"]

    def part(x, name):
        r = max(16, int(npw[name].shape[0] * frac))
        return ofw.linear(x, npw[name][:r])

    def one_step():
        part(feats, "w_fc")
        for n in ("w_q", "w_k", "w_v"):
            part(full["z"], n)
        for b in range(w.batch):
            P = int(seq[b])
            k_all = np.concatenate([ofw.bf16_to_f64(npi["k_cache"][b, :, :P]), full["k_new"][b].transpose(1, 0, 2)], axis=1)
            v_all = np.concatenate([ofw.bf16_to_f64(npi["v_cache"][b, :, :P]), full["v_new"][b].transpose(1, 0, 2)], axis=1)
            ofw.attention_rows(full["q"][b], k_all, v_all, P)
        part(full["attn"], "w_o")
        ofw.silu(part(full["n2"], "w_gate")) * part(full["n2"], "w_up")
        r = max(16, int(npw["w_down"].shape[0] * frac))
        ofw.linear(full["u"], npw["w_down"][:r])
        logits = part(full["n3"], "w_lm")
        for b in range(w.batch):
            c = [ofw.topk_candidates(logits[b, rr], w.topk, 1e-10) for rr in range(w.K)]
            ids = np.stack([x["ids"] for x in c]); sl = np.stack([x["slogit"] for x in c]).astype(np.float32)
            otree.build_tree(ids, sl, tuple(inp["ctx_tail"].numpy()[b]), tri, bi, beam=w.beam, budget=w.tree_budget)

    for _ in range(args.warmup):
        one_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_step()
    dt = time.perf_counter() - t0
    value = frac * args.steps / dt
    cores = _blas_threads()
    sample = (f"each of the {args.steps} timed steps = {frac:.4f} of a full step of workload {w.name}: every matrix product on the "
              f"first {frac:.4f} of its output rows, attention/top-k/tree in full; one untimed full fp64 step took {t_full:.1f} s")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / (args.steps * frac), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": w.name},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(args):
    import torch
    from paper_2601_19278_b200 import replicas, runner, synthetic as syn

    world, rank, local = replicas.env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    replicas.init(world, "nccl", dev)

    w = syn.WORKLOADS[args.workload]
    if args.vocab:
        w = syn.small_variant(w, vocab=args.vocab, name=f"{w.name} with vocab cut to {args.vocab}")
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w, n_fresh=syn.draw_fresh_counts(w) if args.ragged_fresh else None)
    rows = syn.make_ngram_rows(w.vocab, args.ngram_rows or w.ngram_rows, w.ngram_mode)
    ses = runner.DraftSession(w, wt, rows, device=f"cuda:{local}", want_logits=False,
                              ngram_layout={"hash": 0, "trie": 1}[args.ngram_layout])
    ses.load_inputs(inp)
    stream = torch.cuda.current_stream()
    any_fresh = int(np.max(inp["n_fresh"])) > 0
    n_launch = ses.draft.launch_count(w.batch, 1 if any_fresh else 0)
    hbm_peak, peak_kind = _peaks()
    bytes_step = syn.algorithmic_bytes(w, inp["seq_lens"].numpy())
    lm_bytes = 2 * w.vocab * w.hidden

    def barrier():
        replicas.barrier(world, torch.cuda.synchronize)

    def step(i):
        ses.step(step_counter=i)
        ses.tree()

    # ---- device-resident timing
    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    # the dominant kernel is bracketed with events on every LM_EVERY-th timed step only: an event record between
    # two kernels takes away the overlap of one kernel's start with its predecessor's tail (~20 us per step)
    lm_steps = [i for i in range(args.steps) if i % LM_EVERY == 0]
    lm_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in lm_steps]
    for a, b in lm_ev:                       # torch creates the CUDA event lazily, on its first record
        a.record(stream)
        b.record(stream)
    torch.cuda.synchronize()
    ev[0].record(stream)
    for i in range(args.steps):
        if i % LM_EVERY == 0:
            ses.draft.set_profile_events(6, lm_ev[i // LM_EVERY][0], lm_ev[i // LM_EVERY][1])
        step(args.warmup + i)
        ev[i + 1].record(stream)
    barrier()
    total_ms = ev[0].elapsed_time(ev[-1])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    lm_ms = [a.elapsed_time(b) for a, b in lm_ev]
    lm_in_region = len(lm_ms)
    # short runs bracket too few launches inside the timed region for a stable average: the same loop goes on, with
    # every launch bracketed, until ten have been timed (these steps are outside the timed region)
    extra = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(max(0, 10 - lm_in_region))]
    for j, (a, b) in enumerate(extra):
        a.record(stream); b.record(stream)
        ses.draft.set_profile_events(6, a, b)
        step(args.warmup + args.steps + j)
    torch.cuda.synchronize()
    lm_ms += [a.elapsed_time(b) for a, b in extra]
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end through the C ABI with host buffers: dart_draft_step_host takes the step's small inputs from
    # one pinned host buffer (one copy in), runs the forward pass and the tree, and leaves the tree in another (one
    # copy out) before it returns.
    in_host, in_dev, out_host, out_dev, _ = ses.pack_io()
    h2d, d2h = in_host.numel(), out_host.numel()
    e2e_step = ses.host_step(in_host, in_dev, out_host, out_dev, stream=stream)

    for i in range(args.warmup):
        e2e_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        e2e_step(i)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    # ---- per-stage device times (outside both timed regions; each stage bracketed by events on its own steps)
    stage_names = ["fc", "qkv_rope", "attention", "o_proj", "gate_up", "down", "lm_head", "topk_merge", "tree"]
    stages_us = {}
    if rank == 0:
        for sidx, sname in enumerate(stage_names):
            if sidx == 0 and not any_fresh:
                continue
            ts = []
            for i in range(12):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); b.record(stream)
                stream.synchronize()
                ses.draft.set_profile_events(sidx, a, b)
                step(i)
                stream.synchronize()
                ts.append(1e3 * a.elapsed_time(b))
            stages_us[sname] = statistics.median(ts)

    total_ms, e2e_ms = replicas.max_over_ranks([total_ms, e2e_ms], world, dev)
    assert ses.draft.device_status() == 0
    gpu_tree = ses.tree_outputs() if rank == 0 else None

    if rank == 0:
        ms_per_step = total_ms / args.steps
        value = replicas.job_steps_per_second(world, args.steps, total_ms)
        lm_avg_ms = sum(lm_ms) / len(lm_ms)
        achieved = lm_bytes / (lm_avg_ms * 1e-3) / 1e9
        step_gbs = bytes_step / (ms_per_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{w.name}: batch {w.batch}, hidden {w.hidden}, {w.n_q_heads}q/{w.n_kv_heads}kv x{w.head_dim}, "
                                   f"mlp {w.mlp_inter}, vocab {w.vocab}, prefix {w.prefix}, K={w.K}, n_fresh={inp['n_fresh']}, "
                                   f"topk {w.topk}, beam {w.beam}, budget {w.tree_budget}, ngram_rows {len(rows['next'])}, T={w.temperature}",
                       "parallelism": "replicas only" if world > 1 else "1 GPU",
                       "l2": f"inputs larger than L2: {bytes_step / 1e9:.3f} GB of weights+KV streamed per step",
                       "feature_fc_in_path": any_fresh,
                       "ngram": f"{args.ngram_layout} layout, {ses.draft.ngram_bytes() / 1e6:.1f} MB in HBM"},
            "latency_us": {"p50": 1e3 * statistics.median(per_step), "p10": 1e3 * float(np.percentile(per_step, 10)),
                           "p90": 1e3 * float(np.percentile(per_step, 90)), "min": 1e3 * min(per_step), "max": 1e3 * max(per_step)},
            "stages_us": stages_us,
            "step_bytes": bytes_step, "step_gbs": step_gbs,
            "step_frac_of_hbm_peak": step_gbs / hbm_peak, "step_frac_of_8tbs": step_gbs / 8000.0,
            "roofline": {"bound": "hbm", "kernel": "lm_head_dense_kernel" if w.batch * w.K > 32 else "lm_head_umma_kernel", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                         "frac": achieved / hbm_peak, "peak_kind": f"of {peak_kind}",
                         "traffic": args.lm_traffic if args.lm_traffic is not None else lm_bytes * LM_READ_RATIO + LM_WRITE_BYTES,
                         "traffic_source": "ncu capture of a vocab-32768 launch (profiles/lm_head_umma_kernel_C3_vocab32768.txt), reads "
                                           "scaled by the bytes streamed, writes taken as measured",
                         "bytes_per_launch": lm_bytes, "us_per_launch": 1e3 * lm_avg_ms, "launches_timed": len(lm_ms),
                         "launches_in_timed_region": lm_in_region},
            "e2e": {"value": replicas.job_steps_per_second(world, args.steps, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps},
            "gpu_launches": args.steps * n_launch,
            "clocks": clocks,
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w, wt, inp, rows, gpu_tree)
        print(json.dumps(line))
    ses.close()
    replicas.finish(world)


def run_prefill(args):
    """Draft-side prefill (dart_draft_prefill): time to build the draft layer's KV cache for --prefill-rows new
    prefix rows of one sequence.  The work is two dense projections per row (feature FC and k/v), so its bound is
    the tensor pipe: 2 * rows * (3h*h + 2h*2*Hkv*dh) flop against the measured bf16 peak."""
    import torch
    from paper_2601_19278_b200 import replicas, runner, synthetic as syn
    world, rank, local = replicas.env()
    torch.cuda.set_device(local)
    w = syn.WORKLOADS[args.workload]
    n = args.prefill_rows
    assert 0 < n <= w.prefix, "the rows must fit the workload's cache"
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    inp["seq_lens"] = torch.zeros(w.batch, dtype=torch.int32)
    ses = runner.DraftSession(w, wt, None, device=f"cuda:{local}")
    ses.load_inputs(inp)
    g = torch.Generator().manual_seed(5)
    feats = torch.randn(n, 3 * w.hidden, generator=g).to(torch.bfloat16).to(ses.dev)
    tokens = torch.randint(0, w.vocab, (n,), generator=g, dtype=torch.int32).to(ses.dev)
    counts = [n] + [0] * (w.batch - 1)
    stream = torch.cuda.current_stream()
    for _ in range(max(args.warmup, 3)):
        ses.prefill(feats, tokens, counts)
    torch.cuda.synchronize()
    steps = min(args.steps, 20)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        ses.prefill(feats, tokens, counts)
    e1.record(stream)
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    ms = e0.elapsed_time(e1) / steps
    flop = 2.0 * n * (3 * w.hidden * w.hidden + 2 * w.hidden * 2 * w.n_kv_heads * w.head_dim)
    peak, sustained = 1590.0, None
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    kind = "fallback"
    if os.path.exists(pk):
        d = json.load(open(pk))
        if "bf16_tflops" in d:
            peak, kind = float(d["bf16_tflops"]), "measured"
        sustained = d.get("bf16_tflops_sustained")
    if rank == 0:
        print(json.dumps({
            "metric": "draft_prefill_rows_per_second", "value": n / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1, "steps": steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{w.name}: draft-side prefill of {n} rows of one sequence (hidden {w.hidden}, {w.n_kv_heads} kv heads x {w.head_dim})"},
            "roofline": {"bound": "tensor", "achieved": flop / (ms * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                         "frac": flop / (ms * 1e-3) / 1e12 / peak, "peak_kind": f"of {kind} (burst; sustained {sustained})",
                         "traffic": None, "kernel": "umma_dense_kernel (two launches per pass: feature FC, k/v projection)"},
        }))
    ses.close()


def run_train_attn(args):
    """Forward attention under the prefix-shared training mask (dart_train_attention_fwd) for one packed row of
    --train-attn-prompt clean positions with the workload's heads and K = draft length.  Compute-bound: the flop
    count is 4 * head_dim per visible (query, key) pair and query head -- the mask's own work, nothing for the
    hidden part -- against the measured bf16 peak."""
    import torch
    from paper_2601_19278_b200 import binding, replicas, synthetic as syn
    world, rank, local = replicas.env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    w = syn.WORKLOADS[args.workload]
    Lp, d, Hq, Hkv, dh, B = args.train_attn_prompt, w.K, w.n_q_heads, w.n_kv_heads, w.head_dim, 1
    L = Lp * (1 + d)
    g = torch.Generator().manual_seed(11)
    q = torch.randn(B, Hq, L, dh, generator=g).to(torch.bfloat16).to(dev)
    k = torch.randn(B, Hkv, L, dh, generator=g).to(torch.bfloat16).to(dev)
    v = torch.randn(B, Hkv, L, dh, generator=g).to(torch.bfloat16).to(dev)
    out = torch.empty_like(q)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    call = lambda: binding.train_attention_fwd(q, k, v, [Lp] * B, Lp, d, out, status)
    for _ in range(max(args.warmup, 3)):
        call()
    torch.cuda.synchronize()
    steps = min(args.steps, 20)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        call()
    e1.record(stream)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ms = e0.elapsed_time(e1) / steps
    pairs = Lp * (Lp + 1) // 2 + d * Lp * (Lp + 1) // 2 + Lp * d * (d + 1) // 2      # clean causal + blocks x prefix + inside blocks
    flop = 4.0 * dh * pairs * Hq * B
    peak, sustained, kind = 1590.0, None, "fallback"
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        dd = json.load(open(pk))
        if "bf16_tflops" in dd:
            peak, kind = float(dd["bf16_tflops"]), "measured"
        sustained = dd.get("bf16_tflops_sustained")
    if rank == 0:
        print(json.dumps({
            "metric": "train_attention_fwd_rows_per_second", "value": B * L / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1, "steps": steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{w.name} heads ({Hq}q/{Hkv}kv x{dh}): one packed training row, {Lp} clean positions + {Lp} blocks of {d} masked positions = {L} slots; inputs larger than L2: {q.numel() * 2 * 2 / 1e6 + k.numel() * 4 / 1e6:.0f} MB"},
            "roofline": {"bound": "tensor", "achieved": flop / (ms * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                         "frac": flop / (ms * 1e-3) / 1e12 / peak, "peak_kind": f"of {kind} (burst; sustained {sustained})",
                         "traffic": None, "kernel": "train_attn_kernel", "flop_visible_pairs": flop},
        }))


def _blas_threads():
    """Threads of the BLAS pool that numpy's matmul (the oracle's contractions) runs on."""
    try:
        from threadpoolctl import threadpool_info
        n = [int(i["num_threads"]) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def _tree_paths(tokens, parents, n_nodes):
    """Root-to-node token paths of one draft tree (what a verification pass would accept prefixes of)."""
    paths = set()
    for x in range(1, int(n_nodes)):
        path, y = [], x
        while y > 0:
            path.append(int(tokens[y])); y = int(parents[y])
        paths.add(tuple(reversed(path)))
    return paths


def cpu_baseline(w, wt, inp, rows, gpu_tree=None):
    """The oracle, as it stands, timed on this machine's host cores on one full step of the same workload: the forward
    pass (numpy fp64, contractions on the BLAS pool), the candidate selection and Algorithm 1, each timed apart (the
    paper's CPU figure for the pruning alone is about 2 ms).  For the workloads that one core finishes in seconds the
    step is timed again with the BLAS pool held to one thread.  Also reported, not gated: how far the GPU's tree (from
    its own candidates) agrees with the oracle's tree from the oracle's candidates -- the Jaccard index of their
    root-to-node token paths."""
    import torch
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import parity
    from oracle import forward as ofw, tree as otree
    tri, bi = otree.tables_from_rows(rows)
    npw, npi = parity.np_weights(wt), parity.np_inputs(inp)

    def one_step():
        t0 = time.perf_counter()
        ref = ofw.draft_forward(parity.oracle_cfg(w), npw, npi)
        t1 = time.perf_counter()
        cands = []
        for b in range(w.batch):
            c = [ofw.topk_candidates(ref["logits"][b, r], w.topk, 1e-10) for r in range(w.K)]
            cands.append((np.stack([x["ids"] for x in c]), np.stack([x["slogit"] for x in c]).astype(np.float32)))
        t2 = time.perf_counter()
        trees = [otree.build_tree(ids, sl, tuple(inp["ctx_tail"].numpy()[b]), tri, bi, beam=w.beam, budget=w.tree_budget)
                 for b, (ids, sl) in enumerate(cands)]
        t3 = time.perf_counter()
        return trees, (t1 - t0, t2 - t1, t3 - t2)

    threads = _blas_threads()
    trees, (tf, tk, tt) = one_step()
    out = {"value": 1.0 / (tf + tk + tt), "unit": UNIT, "cores": threads, "kind": "oracle",
           "sample": f"1 full step of workload {w.name}: forward (numpy fp64, BLAS pool of {threads} threads), top-k, tree",
           "forward_s": tf, "topk_s": tk, "tree_s": tt}
    if w.name in ("C1", "C2", "C3") and w.temperature == 0:
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1, user_api="blas"):
                _, (tf1, tk1, tt1) = one_step()
            out["one_thread"] = {"value": 1.0 / (tf1 + tk1 + tt1), "forward_s": tf1, "topk_s": tk1, "tree_s": tt1}
        except Exception as e:          # threadpoolctl missing: say so instead of guessing
            out["one_thread"] = {"unavailable": repr(e)}
    if gpu_tree is not None and w.temperature == 0:
        j = []
        for b in range(w.batch):
            a = _tree_paths(gpu_tree["tokens"][b], gpu_tree["parents"][b], gpu_tree["n_nodes"][b])
            o = _tree_paths(trees[b]["tokens"], trees[b]["parents"], trees[b]["n_nodes"])
            j.append(len(a & o) / max(1, len(a | o)))
        out["tree_path_jaccard_vs_oracle_end_to_end"] = float(np.mean(j))
    return out


# DRAM traffic of one LM-head launch, from the committed ncu capture of the vocab-32768 case of the same
# kernel: dram__bytes_read / algorithmic bytes, and dram__bytes_write (per-CTA results, independent of vocab).
LM_READ_RATIO = 335.78e6 / 335.544e6
LM_WRITE_BYTES = 4.0e6
LM_EVERY = 8      # timed steps between two event-bracketed LM-head launches


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--vocab", type=int, default=0,
                    help="override the workload's vocabulary (a smaller case of the same kernels, for ncu captures)")
    ap.add_argument("--prefill-rows", type=int, default=0,
                    help="time dart_draft_prefill on this many new prefix rows instead of the drafting step")
    ap.add_argument("--train-attn-prompt", type=int, default=0,
                    help="time dart_train_attention_fwd on one packed training row of this many clean positions instead of the drafting step")
    ap.add_argument("--ragged-fresh", action="store_true",
                    help="per-sequence fresh-row counts (a steady-state call after a verification that accepted a different "
                         "number of tokens per sequence) instead of the workload's uniform count")
    ap.add_argument("--ngram-layout", default="hash", choices=["hash", "trie"],
                    help="device layout of the N-gram: open-addressing hash table, or child lists (Appendix C's trie)")
    ap.add_argument("--ngram-rows", type=int, default=0, help="generate this many N-gram rows instead of the workload's count")
    ap.add_argument("--lm-traffic", type=float, default=None,
                    help="DRAM bytes per LM-head launch from the committed ncu capture (profiles/), reported as roofline.traffic")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.prefill_rows > 0 and args.impl == "ours":
        run_prefill(args)
    elif args.train_attn_prompt > 0 and args.impl == "ours":
        run_train_attn(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
