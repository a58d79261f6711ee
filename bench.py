#!/usr/bin/env python
"""Benchmark of the PrefixKV hot path on B200.

One step = one pass of the whole path over one batch of the LLaVA-1.5-7B-shaped
workload (batch 1, 32 layers, 32 heads, head_dim 128, bf16, 640 prompt tokens,
20 % budget): score -> sort/cumulative/search -> compact, then T = 128 decode
steps of ragged attention.  Throughput is generated tokens per second of that
step, B * T / step time (the paper's table divides batch * generated tokens by
latency the same way; here only attention is in the step, not a whole model).

Prints ONE JSON line.  `python bench.py --impl reference` times the CPU oracle
on a bounded sample of the same workload instead.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llava7b_b1")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-workloads", action="store_true",
                    help="skip the short runs of the other configurations (the `workloads` key)")
    ap.add_argument("--workload-steps", type=int, default=2)
    return ap.parse_args()


def rank_launch_command(gpus, argv, port=None, script=None):
    """Command line that starts this script as `gpus` ranks on this node (one per GPU, NCCL for
    the barrier and the max over ranks only): `python bench.py --gpus N` run by hand, with no
    launcher around it, re-executes itself through torch.distributed.run."""
    import socket
    if port is None:
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(gpus),
            "--master-addr", "127.0.0.1", "--master-port", str(port),
            os.path.abspath(__file__ if script is None else script)] + list(argv)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


# Which kernel a decode call takes: the library's rule (launch_decode_heads in csrc/decode_heads.cu)
# restated, for the kernel's name, the launch count and the traffic figure below.
DECODE_KERNELS = {
    "heads": ("decode_heads_kernel", "decode_heads.cu", "decode_heads_kernel(const __grid_constant__ HeadMaps maps", 1),
    "stream": ("decode_stream_kernel + its merge kernel", "decode_stream.cu", "decode_stream_kernel(const DecodeArgs a)", 2),
}


def decode_path(w, sms):
    nact = w.B * w.L
    cap_rows = w.B * (min(w.budget_rows(), w.L * w.N) + w.L * w.T)       # as Session sizes the cache
    heads = w.D in (64, 128) and nact <= 256 and nact * w.H >= 4 * sms and cap_rows // nact <= 1024
    return "heads" if heads else "stream"


# DRAM bytes (read + write) of one launch of the workload's decode kernel from an ncu capture (its
# summary is kept under profiles/), keyed by workload and kernel, with the hash of the kernel's source
# the counters were taken on: once that function changes the figure is stale and `traffic` reads null.
DECODE_TRAFFIC = {("llava7b_b1", "heads"): (107.22e6, "4b1d941c9d9fc8cf")}


def decode_traffic(workload, path):
    """The captured figure, or None when the kernel's source (the function itself, from its
    signature to its closing brace) is no longer what the counters were taken on."""
    import hashlib
    ent = DECODE_TRAFFIC.get((workload, path))
    if ent is None:
        return None
    _, fname, signature, _ = DECODE_KERNELS[path]
    src = os.path.join(ROOT, "paper_2412_03409_b200", "csrc", fname)
    try:
        with open(src) as f:
            text = f.read()
        start = text.index(signature)
        end = text.index("\n}\n", start)
    except (OSError, ValueError):
        return None
    digest = hashlib.sha256(text[start:end].encode()).hexdigest()[:16]
    return ent[0] if digest == ent[1] else None


# ---------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append((time.perf_counter(), ln.strip()))

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.proc = None

    def window(self, t0=None, t1=None):
        """Summary of the samples received in [t0, t1] (host clock), all of them if none fall there."""
        if self.proc is None:
            return None
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [ln for ts, ln in self.lines if t0 is None or t0 <= ts <= t1]
        for ln in inside or [ln for _, ln in self.lines]:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------
# CPU oracle timing (bounded sample)
# ---------------------------------------------------------------------------
def time_oracle_sample(w, score_layers=1, decode_steps=(0,)):
    """Times the oracle, single-threaded, on a slice of the workload and scales to the
    whole step.  Returns (tok/s estimate, description, seconds spent)."""
    import numpy as np
    import torch

    import oracle
    from paper_2412_03409_b200 import workloads as wl

    oracle.build()
    f32 = lambda t: t.detach().float().cpu().numpy()
    t_begin = time.perf_counter()
    sub = wl.scaled(w, L=score_layers)
    q, k, v = wl.make_prompt(sub, "cpu", samples=[0])
    scale = wl.layer_scale(w)
    t0 = time.perf_counter()
    sc = [oracle.score_layer(f32(q[0, l]), f32(k[0, l]), float(scale[l])) for l in range(score_layers)]
    t_score = (time.perf_counter() - t0) * (w.L / score_layers)
    scores = np.stack([sc[l % score_layers] for l in range(w.L)])
    t0 = time.perf_counter()
    order, cum, res = oracle.select_sample(scores, w.budget_rows(), w.tol)
    t_select = time.perf_counter() - t0
    t0 = time.perf_counter()
    caches = []
    for l in range(score_layers):
        kept = oracle.retained_positions(order[l], res.len[l])
        caches.append((oracle.gather_rows(f32(k[0, l]), kept), oracle.gather_rows(f32(v[0, l]), kept)))
    t_compact = (time.perf_counter() - t0) * (w.L / score_layers)
    rows0 = float(np.mean([c[0].shape[0] for c in caches]))
    qd, kn, vn = wl.make_decode_inputs(sub, 0, "cpu", samples=[0])
    t0 = time.perf_counter()
    for _ in decode_steps:
        for l in range(score_layers):
            kc = np.concatenate([caches[l][0], f32(kn[0, l])[None]])
            vc = np.concatenate([caches[l][1], f32(vn[0, l])[None]])
            oracle.decode_attn(f32(qd[0, l]), kc, vc, float(scale[l]))
    per_row = (time.perf_counter() - t0) / (len(decode_steps) * score_layers * (rows0 + 1))
    mean_rows = float(res.len.mean())
    t_decode = sum(per_row * (mean_rows + t + 1) * w.L for t in range(w.T))
    total = w.B * (t_score + t_select + t_compact + t_decode)
    desc = ("sample 0: score+compact+decode of %d of %d layers (all heads), selection of all layers; "
            "scaled by layer count, decode by rows x %d steps, x batch %d; single thread"
            % (score_layers, w.L, w.T, w.B))
    return w.B * w.T / total, desc, time.perf_counter() - t_begin


def base_config(w):
    return {"workload": w.name, "batch": w.B, "layers": w.L, "heads": w.H, "head_dim": w.D,
            "prompt_len": w.N, "budget_rows": w.budget_rows(), "decode_steps": w.T}


def run_reference(args):
    """The oracle, as it stands, on one host core: every step times a bounded sample of the
    workload (one layer's scoring, compaction and decode, the whole selection) and scales it to
    the whole step, so `ms_per_step` is an extrapolation and says so."""
    from paper_2412_03409_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.WORKLOADS[args.workload]
    vals, desc, spent = [], "", 0.0
    for i in range(args.warmup + args.steps):
        v, desc, sec = time_oracle_sample(w)
        if i >= args.warmup:
            vals.append(v)
            spent += sec
    value = statistics.mean(vals)
    cfg = base_config(w)
    cfg["timing"] = ("each step times a sample (%.2f s of CPU work) and scales it to the whole step: "
                     "ms_per_step is extrapolated, not elapsed" % (spent / max(1, len(vals))))
    line = {"impl": "reference", "metric": "tok/s", "value": value, "unit": "tok/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.B * w.T / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": cfg,
            "cpu_baseline": {"value": value, "unit": "tok/s", "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
def measure_workload(w, steps, warmup, dev, rank, world, sampler=None, with_lse=False):
    """Times `steps` passes of the whole path over workload `w` on this rank's samples.
    Returns per-prompt-batch stage times (ms), algorithmic byte counts and, on request, the
    scoring time when the caller supplies the log-sum-exp."""
    import torch

    from paper_2412_03409_b200 import sharding, workloads as wl
    from paper_2412_03409_b200.session import Session

    scale = wl.layer_scale(w)
    budget = w.budget_rows()
    # Inputs larger than L2: R independent prompts (replicas) are run interleaved, each as its own
    # batch-B call, so that between two calls on one prompt's data at least 256 MiB of other
    # prompts' K/V has passed through the 126 MB L2.  No flush kernel sits in the timed region.
    retained_bytes = 2 * w.B * budget * w.row_bytes
    R = max(1, min(8, 1 + -(-(256 << 20) // retained_bytes))) if retained_bytes < (256 << 20) else 1
    # Ranks hold different samples of the same workload (batch sharding, no exchange).
    reps = []
    for samples in sharding.samples_for_rank(rank, world, w.B, R):
        q, k, v = wl.make_prompt(w, dev, samples=samples)
        s = Session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=w.T, max_budget_rows=budget,
                    device=dev)
        s.budget.fill_(budget)
        reps.append((s, q, k, v))
    n_pool = 8
    pool = [wl.make_decode_inputs(w, t, dev, samples=list(range(w.B))) for t in range(n_pool)]
    stream = torch.cuda.current_stream()

    def step(events):
        """One pass of the whole path for each of the R prompts; one CUDA-event pair per stage."""
        def timed(fn, tag):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            events.append((tag, a, b))
        timed(lambda: [ss.score(qq, kk) for ss, qq, kk, vv in reps], "score")
        timed(lambda: [ss.search(None, tol=w.tol) for ss, qq, kk, vv in reps], "search")
        timed(lambda: [ss.compact(kk, vv) for ss, qq, kk, vv in reps], "compact")

        def decode_all():
            for t in range(w.T):
                qd, kn, vn = pool[t % n_pool]
                for ss, _, _, _ in reps:
                    ss.decode(qd, kn, vn)
        timed(decode_all, "decode")

    def barrier():
        import torch.distributed as dist
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        step([])
    barrier()
    all_events = []
    wall0 = time.perf_counter()
    for _ in range(steps):
        ev = []
        step(ev)
        all_events.append(ev)
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.window(wall0, wall0 + wall) if sampler is not None else None
    for ss, _, _, _ in reps:
        assert ss.status.cpu().tolist() == [0] * w.B, "device status raised"

    # per prompt batch: each stage's event time divided by the R prompts it covered
    stage_ms = {"score": 0.0, "search": 0.0, "compact": 0.0, "decode": 0.0}
    for ev in all_events:
        for tag, a, b in ev:
            stage_ms[tag] += a.elapsed_time(b)
    for kx in stage_ms:
        stage_ms[kx] /= steps * R

    s0 = reps[0][0]
    # algorithmic bytes of the decode steps (rows actually attended, K and V, plus the append)
    lens = (s0.cache.len.cpu().to(torch.int64) - w.T)      # retained rows after compaction
    retained = int(lens.sum())
    nseg = w.B * w.L
    io_small = 4 * nseg * w.H * w.D * w.esize             # q, k_new, v_new read + out written
    dec_bytes = sum(2 * (retained + nseg * (t + 1)) * w.row_bytes + 2 * nseg * w.row_bytes + io_small
                    for t in range(w.T))
    res = {"stage_ms": stage_ms, "R": R, "wall_ms_per_prompt": 1e3 * wall / (steps * R), "clocks": clocks,
           "dec_bytes": dec_bytes, "compact_bytes": 2 * 2 * retained * w.row_bytes, "budget": budget,
           "causal_flop": 2.0 * w.D * w.N * (w.N + 1) / 2 * w.H * w.L * w.B, "score_lse_ms": None,
           "reps": reps, "pool": pool}

    # Scoring when the caller's prefill attention kept its log-sum-exp (pass 1 is skipped): timed
    # over the same interleaved prompts, outside the step.  The lse comes from plain torch, untimed.
    if with_lse and w.N <= 4096:
        lses = []
        for ss, qq, kk, vv in reps:
            lse = torch.empty((w.B, w.L, w.H, w.N), dtype=torch.float32, device=dev)
            mask = torch.ones(w.N, w.N, dtype=torch.bool, device=dev).tril()
            for b in range(w.B):
                for l in range(w.L):
                    lg = torch.einsum("hmd,hnd->hmn", qq[b, l].float(), kk[b, l].float()) * float(scale[l])
                    lse[b, l] = torch.logsumexp(lg.masked_fill(~mask, float("-inf")), dim=-1)
            lses.append(lse)
        for _ in range(3):
            for (ss, qq, kk, vv), lse in zip(reps, lses):
                ss.score(qq, kk, lse=lse)
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_rep = 5
        ea.record(stream)
        for _ in range(n_rep):
            for (ss, qq, kk, vv), lse in zip(reps, lses):
                ss.score(qq, kk, lse=lse)
        eb.record(stream)
        torch.cuda.synchronize()
        res["score_lse_ms"] = ea.elapsed_time(eb) / (n_rep * R)
        del lses
    return res


def workload_summary(w, m, hbm_peak, tf_peak, sms):
    """The figures of one configuration that the targets are stated on."""
    st = m["stage_ms"]
    dec_gbs = m["dec_bytes"] / (st["decode"] * 1e-3) / 1e9
    compress_ms = st["score"] + st["search"] + st["compact"]
    return {"decode_gbs": dec_gbs, "decode_frac_of_measured_copy": dec_gbs / hbm_peak,
            "decode_pct_of_8tbs": 100 * dec_gbs / NOMINAL_HBM_GBS, "decode_us_per_call": 1e3 * st["decode"] / w.T,
            "compress_ms_per_prompt": compress_ms / w.B, "stages_ms": st,
            "score_tensor_util_vs_burst": m["causal_flop"] * 2 / (st["score"] * 1e-3) / (tf_peak * 1e12),
            "tok_s": w.B * w.T / (sum(st.values()) * 1e-3), "prompts_interleaved": m["R"], "clocks": m["clocks"],
            "decode_kernel": DECODE_KERNELS[decode_path(w, sms)][0]}


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2412_03409_b200 import api, sharding, workloads as wl

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # run by hand without a launcher: start the ranks ourselves
        sys.exit(subprocess.call(rank_launch_command(args.gpus, sys.argv[1:])))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = wl.WORKLOADS[args.workload]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()                 # nvidia-smi needs a moment to come up: start before warm-up
    m = measure_workload(w, args.steps, args.warmup, dev, rank, world, sampler if rank == 0 else None,
                         with_lse=True)
    stage_ms, R, budget = m["stage_ms"], m["R"], m["budget"]
    s, q, k, v = m["reps"][0]
    pool = m["pool"]
    step_ms = sum(stage_ms.values())
    step_ms_max = sharding.max_over_ranks(step_ms, dev)
    dec_bytes = m["dec_bytes"]
    dec_gbs = dec_bytes / (stage_ms["decode"] * 1e-3) / 1e9
    compress_ms = stage_ms["score"] + stage_ms["search"] + stage_ms["compact"]
    hbm_peak, tf_peak, peak_kind = measured_peaks()
    score_lse_ms = m["score_lse_ms"]

    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(torch, api, w, s, q, k, v, pool, budget, dev, max(2, min(args.steps, 20)))
        e2e["ms"] = sharding.max_over_ranks(e2e["ms"], dev)
    del m["reps"], s, q, k, v
    torch.cuda.empty_cache()

    # The other configurations, a few steps each (rank 0 of a one-GPU run only): the figures the
    # bandwidth and latency targets are stated on, measured in this same process.
    others = {}
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    if world == 1 and not args.no_workloads and args.workload == "llava7b_b1":
        others[w.name] = workload_summary(w, m, hbm_peak, tf_peak, sms)
        for name in wl.ORDER:
            if name == w.name:
                continue
            wo = wl.WORKLOADS[name]
            mo = measure_workload(wo, args.workload_steps, 3, dev, 0, 1, sampler)
            del mo["reps"], mo["pool"]
            others[name] = workload_summary(wo, mo, hbm_peak, tf_peak, sms)
            torch.cuda.empty_cache()
    clocks = m["clocks"]
    sampler.stop()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    value = world * w.B * w.T / (step_ms_max * 1e-3)
    path = decode_path(w, sms)
    line = {
        "metric": "tok/s", "value": value, "unit": "tok/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms_max, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.esize == 2 else "f32",
        "data": "synthetic",
        "config": {**base_config(w),
                   "parallelism": "batch-sharded x%d, no collective" % world,
                   "prompts_interleaved": R,
                   "l2": "inputs larger than L2: %d independent prompts interleaved call by call, so "
                         ">= 256 MiB of other K/V passes between two calls on one prompt" % R,
                   "timing": "one CUDA-event pair per stage over all %d prompts; ms_per_step and "
                             "stages_ms are per prompt; wall %.2f ms per prompt"
                             % (R, m["wall_ms_per_prompt"])},
        "stages_ms": stage_ms,
        "decode_attn": {"gbs": dec_gbs, "pct_of_8tbs": 100 * dec_gbs / NOMINAL_HBM_GBS,
                        "pct_of_measured_copy": 100 * dec_gbs / hbm_peak,
                        "tok_s_decode_only": w.B * w.T / (stage_ms["decode"] * 1e-3)},
        "compress": {"ms_per_prompt": compress_ms / w.B,
                     "ms_per_prompt_given_lse": None if score_lse_ms is None else
                     (score_lse_ms + stage_ms["search"] + stage_ms["compact"]) / w.B,
                     "compact_gbs": m["compact_bytes"] / (stage_ms["compact"] * 1e-3) / 1e9,
                     "score_tensor_util_vs_burst": m["causal_flop"] * 2 / (stage_ms["score"] * 1e-3) / (tf_peak * 1e12),
                     "target_ms_strict": m["causal_flop"] / (0.5 * tf_peak * 1e12) * 1e3},
        "roofline": {"bound": "hbm", "kernel": DECODE_KERNELS[path][0] + " (one decode call, launch gaps included)",
                     "achieved": dec_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": dec_gbs / hbm_peak,
                     "peak_kind": "of " + peak_kind, "traffic": decode_traffic(w.name, path),
                     "bytes_per_launch": dec_bytes / w.T, "us_per_launch": 1e3 * stage_ms["decode"] / w.T},
        "gpu_launches": args.steps * R * LAUNCHES_PER_STEP(w, path),
        "clocks": clocks,
    }
    if others:
        line["workloads"] = others
    if e2e is not None:
        line["e2e"] = {"value": world * w.B * w.T / (e2e["ms"] * 1e-3), "unit": "tok/s",
                       "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                       "note": "host pinned Q,K,V and per-token q,k,v copied in, outputs copied out and "
                               "synchronised per token; the next prompt uploads on a copy stream, one piece "
                               "per token, while this one decodes; wall clock over the steps, no L2 flush"}
    if world == 1 and not args.no_cpu_baseline:
        v_cpu, desc, spent = time_oracle_sample(w, score_layers=min(w.L, 16), decode_steps=(0, 1, 2, 3))
        line["cpu_baseline"] = {"value": v_cpu, "unit": "tok/s", "cores": 1, "kind": "oracle",
                                "sample": desc, "seconds": spent}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def LAUNCHES_PER_STEP(w, path):
    # score: lse + column sums + head mean; search: sort/scan + bisection;
    # compact: plan + gather; decode: one kernel per token, or stream + merge
    return 3 + 2 + 2 + DECODE_KERNELS[path][3] * w.T


def run_e2e(torch, api, w, s, q, k, v, pool, budget, dev, steps):
    """Same path with host buffers: every step's prompt tensors start in pinned host memory and every
    token's q, k, v are copied in and its output copied out, with a host synchronisation per token
    (the result is needed before the next token).  The way a serving loop would run it: the next
    prompt's upload goes through a copy stream into a second set of device buffers, piece by piece
    between the tokens of the current prompt; a token's three inputs travel as one copy."""
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    hpool = [torch.stack([x.cpu() for x in p]).pin_memory() for p in pool]      # [3, B, L, H, D] per token
    dbuf = [tuple(torch.empty_like(t) for t in (q, k, v)) for _ in range(2)]
    dtok = torch.empty_like(hpool[0], device=dev)
    hout = torch.empty(s.out.shape, dtype=s.out.dtype).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv)) + w.T * hpool[0].numel() * hpool[0].element_size()
    d2h = w.T * hout.numel() * hout.element_size()
    main = torch.cuda.current_stream()
    copy = torch.cuda.Stream(device=dev)
    ready = [torch.cuda.Event() for _ in range(2)]
    free = [torch.cuda.Event() for _ in range(2)]

    # The upload of the next prompt is cut into one piece per token of the current prompt (a run of
    # (layer, head) slices of Q, K or V, 3.75 MB here), handed to the copy stream right behind the
    # token's own inputs: all host-to-device copies go through one engine in the order they were
    # submitted, so a token's small copy queued behind a 160 MB one waited milliseconds for it,
    # while a piece of this size crosses the link in the time the token takes to compute, come
    # back and be followed by the next.
    def pieces(i):
        flat = [(d_.flatten(0, 2), h_.flatten(0, 2)) for d_, h_ in zip(dbuf[i % 2], (hq, hk, hv))]  # [B*L*H, N, D] each
        rows = flat[0][0].shape[0]
        per = -(-len(flat) * rows // w.T)
        out = []
        for t in range(w.T):
            todo = []
            for r in range(t * per, min((t + 1) * per, len(flat) * rows)):
                todo.append((r // rows, r % rows))
            runs = []
            for which, r in todo:                       # consecutive rows of one tensor travel as one copy
                if runs and runs[-1][0] == which and runs[-1][2] == r:
                    runs[-1][2] = r + 1
                else:
                    runs.append([which, r, r + 1])
            out.append([(flat[which][0][a:b], flat[which][1][a:b]) for which, a, b in runs])
        return out

    def send(todo):
        with torch.cuda.stream(copy):
            for d_, h_ in todo:
                d_.copy_(h_, non_blocking=True)

    def run(n):
        for e in free:
            e.record(main)
        copy.wait_event(free[0])
        for todo in pieces(0):
            send(todo)
        ready[0].record(copy)
        for i in range(n):
            nxt = pieces(i + 1) if i + 1 < n else []
            if nxt:
                copy.wait_event(free[(i + 1) % 2])  # the buffers' previous prompt has been compacted
            dq, dk, dv = dbuf[i % 2]
            main.wait_event(ready[i % 2])
            s.score(dq, dk)
            s.search(None, tol=w.tol)
            s.compact(dk, dv)
            free[i % 2].record(main)
            for t in range(w.T):
                dtok.copy_(hpool[t % len(hpool)], non_blocking=True)
                # (right behind the token's inputs, so that they cross the link while the token is computed)
                if nxt:
                    send(nxt[t])
                s.decode(dtok[0], dtok[1], dtok[2])
                hout.copy_(s.out, non_blocking=True)
                main.synchronize()                # the token's result is needed on the host
            if nxt:
                ready[(i + 1) % 2].record(copy)

    run(1)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    run(steps)
    torch.cuda.synchronize()
    return {"ms": 1e3 * (time.perf_counter() - t0) / steps, "h2d": h2d, "d2h": d2h}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
