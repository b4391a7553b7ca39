"""Throughput of the instance-shrinking batch generator on the image-classification shape.

One step = one pass of the whole hot path over one candidate pool: Assistant score ->
Bernoulli shrink -> ordered batch list (aa_score_shrink), per-instance Boss loss of the
accepted batch (aa_instance_loss), labels + one Assistant SGD step (aa_assistant_step_scored: the
parameters are those the pool was screened with, so the step takes the screen's pre-activations).
Pool: 65,536 candidates x 3072 bf16 features (403 MB, larger than L2; pools rotate),
100-class fp32 logits, gamma 0.1, lr 0.05.  Prints ONE JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--legs a,b,...]

The line's headline is the whole step; beside it (single GPU, each with its own roofline entry,
none of them depending on --steps):
  roofline            the screening kernel alone, launches back to back over the rotating pools
  stages              per-stage CUDA events inside whole steps (a fixed number of extra steps)
  instance_loss_rows  per-sentence loss on the translation shape (25,000 x 32,000 bf16 logits)
  csr                 bag-of-words screen: one 16,384-sentence pool, and 64 pools in one launch
  mlp                 two-layer Assistant shape (262,144 x 3072 bf16, hidden 256): tensor-core screen,
                      1000-class loss, two-layer step
  conv                convolutional Assistant: feature kernel (ALU roofline) and the linear layer's screen on its features
  sweep               fused screen of 2^22 x 512 fp32, shrink+compact of 2^24 stored scores,
                      loss of 16,384 x 131,072 bf16 logits
  pipeline            the same step as the two-stream Assistant / Boss schedule
  e2e                 the step through the host-buffer entry point (pinned host memory)
  cpu_baseline        the CPU oracle, one core and all cores

N > 1 is launched with torch.distributed.run, one rank per GPU; every rank screens its own
pools with its own Assistant (the path shards by instance, no data-path collective), and the
reported value is all ranks' candidates over the slowest rank's device time.
--impl reference times the CPU oracle (as it stands) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidates screened/sec (score+shrink+compact -> instance loss -> Assistant step)"
UNIT = "candidates/s"
ALL_LEGS = ("stages", "loss", "csr", "mlp", "conv", "sweep", "pipeline", "e2e", "cpu")

# Kernel-alone timings: REPS launches back to back between two events, LOOPS such loops, median and best loop.
REPS = 24
LOOPS = 5
STAGE_STEPS = 56   # whole steps with per-stage events (a multiple of the rotating pools)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--pools", type=int, default=8, help="distinct resident pools rotated through the steps")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--cpu-steps", type=int, default=40, help="oracle steps timed for cpu_baseline")
    ap.add_argument("--pool-rows", type=int, default=None, help="override the pool size (testing only)")
    ap.add_argument("--pipeline-steps", type=int, default=300, help="steps of the two-stream Assistant/Boss schedule")
    ap.add_argument("--pipeline-depth", type=int, default=2, help="Boss queue depth k of that schedule")
    ap.add_argument("--legs", default=",".join(ALL_LEGS),
                    help="comma-separated secondary measurements to run (single GPU only): " + ", ".join(ALL_LEGS))
    ap.add_argument("--small", action="store_true", help="shrink the secondary workloads (profiling / testing only)")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            rec = json.load(f)
        return {"hbm": float(rec["hbm_gbs"]), "burst": float(rec["bf16_tflops"]),
                "sustained": float(rec["bf16_tflops_sustained"]), "kind": "measured"}
    except Exception:
        return {"hbm": 6650.0, "burst": 1590.0, "sustained": 1400.0, "kind": "fallback"}


NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0


def hbm_roofline(bytes_per_launch, ms, best_ms, launches, peaks, kernel=None, **extra):
    ach = bytes_per_launch / (ms * 1e-3) / 1e9
    r = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm"], "unit": "GB/s", "frac": ach / peaks["hbm"],
         "peak_kind": f"of {peaks['kind']}", "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
         "algorithmic_bytes_per_launch": bytes_per_launch, "avg_launch_ms": ms, "best_launch_ms": best_ms,
         "launches_timed": launches}
    if kernel:
        r["kernel"] = kernel
    r.update(extra)
    return r


def tensor_roofline(flops_per_launch, ms, best_ms, launches, peaks, kernel=None, **extra):
    ach = flops_per_launch / (ms * 1e-3) / 1e12
    r = {"bound": "tensor", "achieved": ach, "peak": peaks["burst"], "unit": "TFLOP/s", "frac": ach / peaks["burst"],
         "peak_kind": f"of {peaks['kind']} (cuBLAS bf16 burst: the kernel is timed alone)",
         "frac_of_sustained": ach / peaks["sustained"], "frac_of_nominal_2250": ach / NOMINAL_BF16_TFLOPS,
         "flops_per_launch": flops_per_launch, "avg_launch_ms": ms, "best_launch_ms": best_ms, "launches_timed": launches}
    if kernel:
        r["kernel"] = kernel
    r.update(extra)
    return r


TRAFFIC_PROFILE = os.path.join(ROOT, "profiles", "score_shrink_tma_bf16_d3072.txt")
TRAFFIC_SOURCES = ("score_shrink_tma.cu", "scan_tail.cuh", "async_copy.cuh", "aa_internal.cuh")


def kernel_source_digest():
    """SHA-256 over the sources of the dominant kernel, as recorded beside its ncu counters."""
    import hashlib

    h = hashlib.sha256()
    for name in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, "paper_1905_03381_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def ncu_traffic_bytes(candidates: int):
    """DRAM bytes per launch of the dominant kernel, scaled from the committed ncu summary by the candidates
    one launch screens; None when the summary is missing or the kernel's sources changed since the capture."""
    try:
        rec = {}
        with open(TRAFFIC_PROFILE) as f:
            for line in f:
                if ":" in line and not line.startswith("#"):
                    k, v = line.split(":", 1)
                    rec[k.strip()] = v.strip()
        if rec.get("source_sha256") != kernel_source_digest():
            return None
        return float(rec["dram_bytes_per_candidate"]) * candidates
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


def back_to_back(torch, launch, reps=REPS, loops=LOOPS, warm=3):
    """Times launch(i) for i = 0, 1, ...: `loops` loops of `reps` calls, one event pair around each loop, on the current
    stream.  Returns (median loop's ms per call, best loop's ms per call, calls timed)."""
    i = 0
    for _ in range(warm):
        launch(i); i += 1
    torch.cuda.synchronize()
    per_call = []
    for _ in range(loops):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            launch(i); i += 1
        e1.record()
        torch.cuda.synchronize()
        per_call.append(e0.elapsed_time(e1) / reps)
    per_call.sort()
    return per_call[len(per_call) // 2], per_call[0], reps * loops


# --------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline and --impl reference)
# --------------------------------------------------------------------------

def oracle_step_seconds(cfg, x_host, w0, logits_host, labels_host, steps: int):
    """Times `steps` whole steps of the oracle, as it stands, single-threaded.  Returns (seconds, candidates, final (w, b))."""
    import numpy as np

    from oracle import aa_oracle as O

    w, b = w0.copy(), np.float32(0.0)
    n = x_host.shape[0]
    t0 = time.perf_counter()
    for step in range(steps):
        scr = O.screen_linear_dense(x_host, w, b, cfg.gamma, cfg.philox_seed, step)
        Bidx = scr["B"]
        m = len(Bidx)
        f = O.row_loss(logits_host[:m], labels_host[:m]).astype(np.float32)
        w, b, _ = O.assistant_step_linear_dense(x_host, f, w, b, cfg.lr, row_idx=Bidx)
    return time.perf_counter() - t0, n * steps, (w, b)


def oracle_step_seconds_all_cores(cfg, x_host, w0, logits_host, labels_host, steps: int, threads: int):
    """The same oracle functions run row-parallel: the pool, the batch's logit rows and the batch's gradient are cut into
    one contiguous slice per thread (the rows are independent; the oracle's C routines run outside the interpreter
    lock).  The slices' mean gradients are combined by their row counts.  Returns (seconds, candidates, final (w, b))."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor

    from oracle import aa_oracle as O

    n = x_host.shape[0]
    w, b = w0.copy(), np.float32(0.0)

    def cuts(total):
        edges = np.linspace(0, total, threads + 1).astype(np.int64)
        return [(int(a), int(e)) for a, e in zip(edges[:-1], edges[1:]) if e > a]

    with ThreadPoolExecutor(max_workers=threads) as pool:
        t0 = time.perf_counter()
        for step in range(steps):
            parts = list(pool.map(lambda ae: O.screen_linear_dense(x_host[ae[0]:ae[1]], w, b, cfg.gamma, cfg.philox_seed, step,
                                                                   id_base=ae[0])["B"].astype(np.int64) + ae[0], cuts(n)))
            Bidx = np.concatenate(parts).astype(np.int32)
            m = len(Bidx)
            f = np.concatenate(list(pool.map(lambda ae: O.row_loss(logits_host[ae[0]:ae[1]], labels_host[ae[0]:ae[1]]),
                                             cuts(m)))).astype(np.float32) if m else np.zeros(0, np.float32)
            if m:
                z = O.labels(f, O.batch_mean(f))

                def grad(ae):
                    rows = Bidx[ae[0]:ae[1]]
                    s = O.score_dense(x_host, w, b, row_idx=rows)
                    gw, gb = O.linear_grad_dense(x_host, s, z[ae[0]:ae[1]], row_idx=rows)
                    return gw * (ae[1] - ae[0]), gb * (ae[1] - ae[0])

                gs = list(pool.map(grad, cuts(m)))
                gw = sum(g[0] for g in gs) / m
                gb = sum(g[1] for g in gs) / m
                w = O.sgd(w, gw, cfg.lr)
                b = O.sgd(np.array([b], np.float32), np.array([gb]), cfg.lr)[0]
        return time.perf_counter() - t0, n * steps, (w, b)


def run_reference(args, cfg):
    """The reference arm: the CPU oracle on this machine's host cores, bounded sample per step."""
    import torch

    from oracle import aa_oracle as O
    from paper_1905_03381_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    O.build()
    sample_rows = min(cfg.n, 8192)
    x = W.to_oracle(W.uniform01((sample_rows, cfg.d), 100, torch.bfloat16, "cpu"))
    w0 = W.linear_assistant(cfg.d, 2, "cpu")[0].numpy()
    logits = W.normal((sample_rows, cfg.classes), 3.0, 200, torch.float32, "cpu").numpy()
    labels = W.randint(0, cfg.classes, (sample_rows,), 300, "cpu").numpy()
    for _ in range(min(args.warmup, 2)):
        oracle_step_seconds(cfg, x, w0, logits, labels, 1)
    steps = max(1, min(args.steps, 16))
    sec, cand, _ = oracle_step_seconds(cfg, x, w0, logits, labels, steps)
    value = cand / sec
    sample = f"{sample_rows} of {cfg.n} candidates per step, {steps} steps"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": min(args.warmup, 2), "ms_per_step": 1e3 * sec / steps * (cfg.n / sample_rows),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, args, reference=True),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(cfg, args, reference=False):
    return {
        "workload": "image-classification shape: pool 65,536 x 3072 bf16 features U[0,1), linear Assistant, "
                    "100-class fp32 logits N(0,3), mix 0.1, SGD lr 0.05 every step",
        "pool_rows": cfg.n, "d": cfg.d, "classes": cfg.classes, "mix": cfg.gamma, "lr": cfg.lr,
        "pools_rotated": None if reference else args.pools,
        "l2_policy": "inputs larger than L2: each pool is 403 MB and pools rotate",
        "kernel_timing": None if reference else
            f"kernels alone: {LOOPS} loops of {REPS} launches back to back, one CUDA event pair per loop, median loop; "
            f"stages: per-stage CUDA events in {STAGE_STEPS} extra whole steps; neither depends on --steps",
        "parallelism": f"instance-sharded x{args.gpus}, one Assistant per GPU, no data-path collective",
    }


# --------------------------------------------------------------------------
# secondary legs (single GPU)
# --------------------------------------------------------------------------

def leg_translation_loss(torch, B, W, dev, peaks, small):
    """Second half of the metric: per-instance-loss rows/s on the translation shape (25,000 token rows x 32,000-word bf16
    logits = 1.6 GB per call, larger than L2; per-sentence sums)."""
    t2 = W.TranslationShape()
    rows2 = 4096 if small else t2.token_budget
    lg2 = t2.token_logits(rows2, dev)
    ids2 = t2.token_ids(rows2, dev)
    off2 = torch.from_numpy(W.ragged_offsets(rows2, t2.len_lo, t2.len_hi, 9)).to(dev)
    sent_loss = torch.zeros(off2.numel() - 1, dtype=torch.float32, device=dev)
    aa2 = B.AutoAssist(max_rows=rows2, max_d=8, device=dev)
    g2 = B.logits_desc(lg2)
    n0 = aa2.aa_launch_count()
    ms2, best2, calls = back_to_back(torch, lambda i: aa2.aa_instance_loss(g2, ids2, sent_loss, offsets=off2))
    launches = aa2.aa_launch_count() - n0
    assert aa2.aa_device_status() == B.AA_OK
    bytes2 = rows2 * t2.vocab * 2 + rows2 * 8 + off2.numel() * 4 + sent_loss.numel() * 4
    out = {"workload": f"translation shape: {rows2} token rows x {t2.vocab} bf16 logits N(0,4), "
                       f"{sent_loss.numel()} sentences of 8..128 tokens, summed per sentence",
           "value": rows2 / (ms2 * 1e-3), "unit": "token rows/s", "ms_per_call": ms2,
           "launches_per_call": launches // (calls + 3),
           "roofline": hbm_roofline(bytes2, ms2, best2, calls, peaks, kernel="row_loss_cta_kernel + segment_sum_kernel")}
    aa2.close()
    return out


def leg_csr(torch, B, W, dev, peaks, small):
    """Bag-of-words screen (translation shape): one 16,384-sentence pool per launch (16 distinct pools rotate: 144 MB,
    larger than L2), and 64 pools' worth of sentences in one launch (570 MB)."""
    t = W.TranslationShape()
    w, b = t.assistant(dev)
    asst = B.linear_assistant(w, b)

    def pool(n, seed):
        g = torch.Generator(device=dev).manual_seed(seed)
        lengths = torch.randint(t.len_lo, t.len_hi + 1, (n,), generator=g, device=dev, dtype=torch.int64)
        indptr = torch.zeros(n + 1, dtype=torch.int64, device=dev)
        indptr[1:] = torch.cumsum(lengths, 0)
        nnz = int(indptr[-1].item())
        col = torch.randint(0, t.buckets, (nnz,), generator=g, device=dev, dtype=torch.int32)
        val = torch.ones(nnz, dtype=torch.float32, device=dev)
        return indptr.to(torch.int32), col, val, nnz

    out = {}
    n_big = t.n * (4 if small else 64)
    aa = B.AutoAssist(max_rows=n_big, max_d=t.buckets, device=dev)
    out_idx = torch.zeros(n_big, dtype=torch.int32, device=dev)
    cnt = torch.zeros(1, dtype=torch.int32, device=dev)

    pools = [pool(t.n, 500 + k) for k in range(4 if small else 16)]
    feats = [B.csr_features(p[0], p[1], p[2], t.buckets, nnz=p[3]) for p in pools]
    ms, best, calls = back_to_back(torch, lambda i: aa.aa_score_shrink(feats[i % len(feats)], asst, t.gamma, t.philox_seed, i,
                                                                       out_idx, cnt))
    nnz_mean = sum(p[3] for p in pools) / len(pools)
    bytes1 = 8 * nnz_mean + 4 * (t.n + 1) + 4 * int(cnt.item())
    out["single_pool"] = {"workload": f"{t.n} sentences of 8..128 hashed tokens, 2^18 buckets, mix {t.gamma}; {len(pools)} pools rotate",
                          "value": t.n / (ms * 1e-3), "unit": UNIT, "ms_per_call": ms,
                          "roofline": hbm_roofline(bytes1, ms, best, calls, peaks, kernel="score_shrink_csr_kernel",
                                                   note="8.9 MB per launch: bounded by launch latency, not by HBM")}
    del pools, feats
    ip, col, val, nnz = pool(n_big, 600)
    big = B.csr_features(ip, col, val, t.buckets, nnz=nnz)
    ms, best, calls = back_to_back(torch, lambda i: aa.aa_score_shrink(big, asst, t.gamma, t.philox_seed, i, out_idx, cnt),
                                   reps=8, loops=5)
    bytes_big = 8 * nnz + 4 * (n_big + 1) + 4 * int(cnt.item())
    out["batched"] = {"workload": f"{n_big} sentences ({n_big // t.n} pools) in one launch, {nnz} non-zeros",
                      "value": n_big / (ms * 1e-3), "unit": UNIT, "ms_per_call": ms,
                      "roofline": hbm_roofline(bytes_big, ms, best, calls, peaks, kernel="score_shrink_csr_kernel")}
    assert aa.aa_device_status() == B.AA_OK
    aa.close()
    return out


def leg_mlp(torch, B, W, dev, peaks, small):
    """Two-layer Assistant shape: pool 262,144 x 3072 bf16 N(0,1), 3072 -> 256 (ReLU) -> 1, 1000-class fp32 logits,
    SGD lr 0.01 on both layers.  Screen alone (tensor roofline), loss alone, step alone on the screen's batch list, and
    whole steps."""
    import numpy as np
    cfg = W.MlpShape()
    if small:
        cfg.n = 32768
    x = cfg.pool(dev)
    W1, b1, w2, b2 = cfg.assistant(dev)
    W1b = W1.to(torch.bfloat16).contiguous()
    logits = cfg.logits(cfg.n, dev)
    labels = cfg.labels(cfg.n, dev)
    aa = B.AutoAssist(max_rows=cfg.n, max_d=cfg.d, max_hidden=cfg.hidden, device=dev)
    asst = B.mlp_assistant(W1, W1b, b1, w2, b2)
    out_idx = torch.zeros(cfg.n, dtype=torch.int32, device=dev)
    cnt = torch.zeros(1, dtype=torch.int32, device=dev)
    loss = torch.zeros(cfg.n, dtype=torch.float32, device=dev)
    feat, batch = B.dense_features(x), B.dense_features(x, row_idx=out_idx)
    lg = B.logits_desc(logits)

    ms_s, best_s, calls_s = back_to_back(torch, lambda i: aa.aa_score_shrink(feat, asst, cfg.gamma, cfg.philox_seed, i, out_idx, cnt),
                                         reps=10, loops=5)
    m = int(cnt.item())
    ms_l, best_l, calls_l = back_to_back(torch, lambda i: aa.aa_instance_loss(lg, labels, loss, count_dev=cnt), reps=10, loops=5)
    ms_a, best_a, calls_a = back_to_back(torch, lambda i: aa.aa_assistant_step(batch, loss, asst, cfg.lr, count_dev=cnt),
                                         reps=10, loops=5)

    score = torch.zeros(cfg.n, dtype=torch.float32, device=dev)
    marks = []

    def step(i):
        # the update takes the scores the screening wrote and the gates it left in the context's workspace
        aa.aa_score_shrink(feat, asst, cfg.gamma, cfg.philox_seed, 100 + i, out_idx, cnt, score)
        aa.aa_instance_loss(lg, labels, loss, count_dev=cnt)
        if marks is not None and len(marks) < 2 * 12:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            aa.aa_assistant_step_scored(batch, loss, score, asst, cfg.lr, count_dev=cnt)
            e1.record()
            marks.extend((e0, e1))
        else:
            aa.aa_assistant_step_scored(batch, loss, score, asst, cfg.lr, count_dev=cnt)

    for i in range(12):                                   # the update alone, inside whole steps (it needs a fresh screening)
        step(i)
    torch.cuda.synchronize()
    ms_sc = float(np.median([marks[2 * j].elapsed_time(marks[2 * j + 1]) for j in range(len(marks) // 2)]))
    ms_w, best_w, calls_w = back_to_back(torch, step, reps=10, loops=3)
    assert aa.aa_device_status() == B.AA_OK
    flops = 2.0 * cfg.n * cfg.d * cfg.hidden
    out = {
        "workload": f"MLP Assistant shape: pool {cfg.n} x {cfg.d} bf16 N(0,1), {cfg.d}->{cfg.hidden} (ReLU)->1, "
                    f"{cfg.classes}-class fp32 logits N(0,3), mix {cfg.gamma}, SGD lr {cfg.lr} on both layers; pool 1.6 GB > L2",
        "accepted": m,
        "score_shrink": {"value": cfg.n / (ms_s * 1e-3), "unit": UNIT, "ms_per_call": ms_s,
                         "roofline": tensor_roofline(flops, ms_s, best_s, calls_s, peaks, kernel="mlp_score_shrink_kernel",
                                                     hbm_GBs=cfg.n * cfg.d * 2 / (ms_s * 1e-3) / 1e9,
                                                     hbm_frac=cfg.n * cfg.d * 2 / (ms_s * 1e-3) / 1e9 / peaks["hbm"])},
        "instance_loss": {"value": m / (ms_l * 1e-3), "unit": "rows/s", "ms_per_call": ms_l,
                          "roofline": hbm_roofline(m * (cfg.classes * 4 + 8), ms_l, best_l, calls_l, peaks,
                                                   kernel="row_loss_group_kernel")},
        "assistant_step": {"ms_per_call": ms_a, "rows": m,
                           "roofline": tensor_roofline(2 * 2.0 * m * cfg.d * cfg.hidden, ms_a, best_a, calls_a, peaks,
                                                       kernel="mlp_residual_kernel + mlp_w1_grad_kernel (+ updates)")},
        "assistant_step_scored": {"ms_per_call": ms_sc, "how": "CUDA events around the call inside 12 whole steps (median); one "
                                  "contraction (the W1 gradient), the forward pass is the screening's",
                                  "useful_TFLOPs": 2.0 * m * cfg.d * cfg.hidden / (ms_sc * 1e-3) / 1e12},
        "whole_step": {"value": cfg.n / (ms_w * 1e-3), "unit": UNIT, "ms_per_step": ms_w, "steps_timed": calls_w},
    }
    aa.close()
    return out


def leg_conv(torch, B, W, dev, peaks, small, clocks_mhz):
    """Convolutional Assistant (Boss's 3 x 3 convolution with 16 channels -> rectifier -> 4 x 4 average pooling -> linear
    layer) on a 65,536-image pool: the feature kernel alone (a small contraction on the warp-level matrix instructions), then the screen of
    the linear layer on the 1024 features per instance."""
    cfg = W.ConvShape()
    if small:
        cfg.n = 8192
    x = cfg.pool_images(0, dev)
    weight, bias = cfg.conv(dev)
    w, b = cfg.assistant(dev)
    asst = B.linear_assistant(w, b)
    F = cfg.features
    phi = torch.zeros((cfg.n, F), dtype=torch.float32, device=dev)
    aa = B.AutoAssist(max_rows=cfg.n, max_d=max(cfg.d, F), device=dev)
    images, cv = B.dense_features(x), B.conv_layer(weight, bias, cfg.height, cfg.width, cfg.pool)
    out_idx = torch.zeros(cfg.n, dtype=torch.int32, device=dev)
    cnt = torch.zeros(1, dtype=torch.int32, device=dev)
    ms_c, best_c, calls_c = back_to_back(torch, lambda i: aa.aa_conv_pool_features(images, cv, phi), reps=6, loops=5)
    feat = B.dense_features(phi)
    ms_s, best_s, calls_s = back_to_back(torch, lambda i: aa.aa_score_shrink(feat, asst, cfg.gamma, cfg.philox_seed, i, out_idx, cnt),
                                         reps=12, loops=5)
    assert aa.aa_device_status() == B.AA_OK
    flops = 2.0 * cfg.n * cfg.c_out * cfg.height * cfg.width * cfg.c_in * cfg.ksize * cfg.ksize
    sm_mhz = clocks_mhz or 1965.0
    alu_peak = 148 * 128 * 2 * sm_mhz * 1e6 / 1e12          # fp32 lanes x 2 flop per multiply-add x SM clock
    ach = flops / (ms_c * 1e-3) / 1e12
    # The bf16 kernel multiplies on the warp-level matrix instructions: taps padded to whole 16-tap steps, channels to whole
    # 8-channel tiles, fp32 taps as three bf16 terms.  ncu counts 8 tensor-pipe cycles per m16n8k16 per SM sub-partition,
    # i.e. 4096 flop / 8 cycles x 4 sub-partitions x 148 SMs x clock for this instruction path.
    taps = cfg.c_in * cfg.ksize * cfg.ksize
    issued = 2.0 * cfg.n * cfg.height * cfg.width * (-(-taps // 16) * 16) * (-(-cfg.c_out // 8) * 8) * 3
    mma_peak = 148 * 4 * (4096 / 8.0) * sm_mhz * 1e6 / 1e12
    ach_issued = issued / (ms_c * 1e-3) / 1e12
    out = {
        "workload": f"{cfg.n} images of {cfg.c_in} x {cfg.height} x {cfg.width} bf16 U[0,1), {cfg.c_out} channels of "
                    f"{cfg.ksize} x {cfg.ksize} taps, {cfg.pool} x {cfg.pool} average pooling -> {F} fp32 features per instance",
        "features": {"value": cfg.n / (ms_c * 1e-3), "unit": UNIT, "ms_per_call": ms_c,
                     "roofline": {"bound": "tensor", "kernel": "conv_pool_mma_kernel", "achieved": ach_issued, "peak": mma_peak,
                                  "unit": "TFLOP/s", "frac": ach_issued / mma_peak,
                                  "peak_kind": f"mma.sync m16n8k16 bf16 path: 148 SMs x 4 sub-partitions x 512 flop per cycle x "
                                               f"{sm_mhz:.0f} MHz (8 tensor-pipe cycles per instruction, from ncu); issued flops "
                                               f"= 3 bf16 terms of the fp32 taps, taps padded to 16s, channels to 8s",
                                  "flops_per_launch": issued, "useful_flops_per_launch": flops, "useful_TFLOPs": ach,
                                  "useful_over_fp32_alu_peak": ach / alu_peak, "fp32_alu_peak_TFLOPs": alu_peak,
                                  "avg_launch_ms": ms_c, "best_launch_ms": best_c, "launches_timed": calls_c,
                                  "hbm_GBs": cfg.n * (cfg.d * 2 + F * 4) / (ms_c * 1e-3) / 1e9,
                                  "hbm_frac": cfg.n * (cfg.d * 2 + F * 4) / (ms_c * 1e-3) / 1e9 / peaks["hbm"]}},
        "linear_layer_screen": {"value": cfg.n / (ms_s * 1e-3), "unit": UNIT, "ms_per_call": ms_s, "accepted": int(cnt.item()),
                                "roofline": hbm_roofline(cfg.n * F * 4 + F * 4 + 4 * int(cnt.item()), ms_s, best_s, calls_s, peaks,
                                                         kernel="score_shrink_tma_kernel<float>")},
    }
    aa.close()
    return out


def leg_sweep(torch, B, W, dev, peaks, small):
    """Scaling-sweep points: fused screen of a 2^22 x 512 fp32 pool (8.6 GB), shrink+compact of 2^24 stored scores (three
    score arrays rotate: 201 MB, larger than L2), per-row loss of 16,384 x 131,072 bf16 logits (4.3 GB)."""
    out = {}
    sw = W.SweepShape()
    n1 = (1 << 18) if small else (1 << 22)
    n2 = (1 << 20) if small else (1 << 24)
    aa = B.AutoAssist(max_rows=n2, max_d=sw.d, device=dev)
    w, b = sw.assistant(dev)
    asst = B.linear_assistant(w, b)
    out_idx = torch.zeros(n2, dtype=torch.int32, device=dev)
    cnt = torch.zeros(1, dtype=torch.int32, device=dev)
    for mix in (0.05, 0.5):
        x = torch.randn((n1, sw.d), device=dev, dtype=torch.float32, generator=torch.Generator(device=dev).manual_seed(14))
        feat = B.dense_features(x)
        ms, best, calls = back_to_back(torch, lambda i: aa.aa_score_shrink(feat, asst, mix, 0, i, out_idx, cnt), reps=8, loops=5)
        m = int(cnt.item())
        out[f"fused_screen_mix{mix}"] = {
            "workload": f"{n1} x {sw.d} fp32 N(0,1), linear Assistant, mix {mix}", "value": n1 / (ms * 1e-3), "unit": UNIT,
            "ms_per_call": ms, "accepted": m,
            "roofline": hbm_roofline(n1 * sw.d * 4 + sw.d * 4 + 4 * m, ms, best, calls, peaks, kernel="score_shrink_tma_kernel<float>")}
        del x, feat
    scores = [W.normal((n2,), 2.0, 700 + k, torch.float32, dev) for k in range(3)]
    for mix in (0.05, 0.5):
        ms, best, calls = back_to_back(torch, lambda i: aa.aa_shrink_compact(scores[i % 3], mix, 0, i, out_idx, cnt), reps=12, loops=5)
        m = int(cnt.item())
        out[f"shrink_compact_mix{mix}"] = {
            "workload": f"{n2} stored scores N(0,2), mix {mix}", "value": n2 / (ms * 1e-3), "unit": UNIT, "ms_per_call": ms,
            "accepted": m,
            "roofline": hbm_roofline(4 * n2 + 4 * m, ms, best, calls, peaks, kernel="shrink_from_scores_kernel",
                                     note="Philox + sigmoid (about 130 instructions per candidate) and the look-back latency "
                                          "bound this kernel, not its 4 + 4p bytes per candidate")}
    assert aa.aa_device_status() == B.AA_OK
    del scores, out_idx
    aa.close()
    rows, vocab = (2048, 131072) if small else (16384, 131072)
    lg = W.sweep_logits(rows, vocab, dev)
    ids = W.randint(0, vocab, (rows,), 16, dev)
    ell = torch.zeros(rows, dtype=torch.float32, device=dev)
    aa2 = B.AutoAssist(max_rows=rows, max_d=8, device=dev)
    g = B.logits_desc(lg)
    ms, best, calls = back_to_back(torch, lambda i: aa2.aa_instance_loss(g, ids, ell), reps=8, loops=5)
    assert aa2.aa_device_status() == B.AA_OK
    out["instance_loss"] = {"workload": f"{rows} x {vocab} bf16 logits N(0,4), per row", "value": rows / (ms * 1e-3),
                            "unit": "rows/s", "ms_per_call": ms,
                            "roofline": hbm_roofline(rows * (vocab * 2 + 8), ms, best, calls, peaks, kernel="row_loss_cta_kernel")}
    aa2.close()
    return out


# --------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------

def run_b200(args, cfg):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_1905_03381_b200 import binding as B, build as lib_build, sharding, workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        lib_build.build()
    if world > 1:
        dist.barrier()
    legs = set(x for x in args.legs.split(",") if x) if world == 1 else set()
    if world > 1:
        legs = {"e2e"}
    unknown = legs - set(ALL_LEGS)
    if unknown:
        raise SystemExit(f"unknown --legs entries: {sorted(unknown)}")
    peaks = measured_peaks()

    plan = sharding.plan(rank, world, args.pools, cfg.n)
    pools = [cfg.pool(pid, dev) for pid in plan.pool_ids]
    logits = [cfg.logits(pid, dev) for pid in plan.pool_ids]
    labels = [cfg.labels(pid, dev) for pid in plan.pool_ids]
    w, b = cfg.assistant(dev)
    aa = B.AutoAssist(max_rows=cfg.n, max_d=cfg.d, device=dev)
    asst = B.linear_assistant(w, b)
    out_idx = torch.zeros(cfg.n, dtype=torch.int32, device=dev)
    # one device count per step, so that the mean batch size of the timed steps is known without a host read
    warm = max(args.warmup, 3)
    n_slots = warm + max(args.steps, STAGE_STEPS + 1, REPS * LOOPS + 3)
    counts = torch.zeros(n_slots, dtype=torch.int32, device=dev)
    count_of = [counts[j:j + 1] for j in range(n_slots)]
    loss = torch.zeros(cfg.n, dtype=torch.float32, device=dev)
    score = torch.zeros(cfg.n, dtype=torch.float32, device=dev)    # pre-activations of the pool, screen -> step (same parameters)
    feats = [B.dense_features(p, id_base=base) for p, base in zip(pools, plan.id_bases)]
    batch_feats = [B.dense_features(p, row_idx=out_idx, id_base=base) for p, base in zip(pools, plan.id_bases)]
    lg = [B.logits_desc(l) for l in logits]
    npool = len(pools)

    def step(i, events=None, slot=None):
        k = i % npool
        out_count = count_of[(i if slot is None else slot) % n_slots]
        if events is not None:
            events[0].record()
        aa.aa_score_shrink(feats[k], asst, cfg.gamma, cfg.philox_seed, i, out_idx, out_count, score)
        if events is not None:
            events[1].record()
        aa.aa_instance_loss(lg[k], labels[k], loss, count_dev=out_count)
        if events is not None:
            events[2].record()
        # sequential schedule: the parameters are those the pool was just screened with, so the step takes the screen's scores
        aa.aa_assistant_step_scored(batch_feats[k], loss, score, asst, cfg.lr, count_dev=out_count)
        if events is not None:
            events[3].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(warm):
        step(i)
    barrier()
    assert aa.aa_device_status() == B.AA_OK

    # ---- the metric: K whole steps between two events, nothing else in the timed region
    K = args.steps
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = aa.aa_launch_count()
    barrier()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(K):
        step(warm + i)
    t_end.record()
    barrier()
    elapsed_ms = t_start.elapsed_time(t_end)
    launches = aa.aa_launch_count() - launches0
    status = aa.aa_device_status()
    assert status == B.AA_OK, B.status_string(status)
    timed = counts[[(warm + i) % n_slots for i in range(K)]].cpu().numpy().astype(np.int64)
    accepted = float(timed.mean())            # mean batch size M over the timed steps
    agg = sharding.aggregate(dist if world > 1 else None, dev, elapsed_ms, cfg.n * K)

    # ---- the dominant kernel alone: screening launches back to back over the rotating pools (the Assistant stays as the
    # timed steps left it; the Philox step number advances), independent of --steps
    counts.zero_()
    ms_scr, best_scr, calls_scr = back_to_back(
        torch, lambda i: aa.aa_score_shrink(feats[i % npool], asst, cfg.gamma, cfg.philox_seed, 10_000 + i, out_idx,
                                            count_of[i % n_slots], score))
    m_scr = float(counts[3:3 + calls_scr].float().mean().item())
    if rank == 0:
        time.sleep(0.2)
        sampler.stop()
    alg_bytes = cfg.n * cfg.d * 2 + cfg.d * 4 + m_scr * 4 + 4
    roofline = hbm_roofline(alg_bytes, ms_scr, best_scr, calls_scr, peaks, kernel="score_shrink_tma_kernel<bf16, 32>",
                            traffic=ncu_traffic_bytes(cfg.n), accepted_mean=m_scr,
                            timing=f"{LOOPS} loops of {REPS} launches back to back over {npool} rotating pools; median loop")
    screen = {"value": cfg.n / (ms_scr * 1e-3), "unit": UNIT, "what": "score + shrink + compact alone (steps S1-S3), N / t",
              "ms_per_call": ms_scr}

    # ---- per-stage events inside whole steps: a fixed number of extra steps, an event before and after every call
    stages = None
    if "stages" in legs or world > 1:
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(STAGE_STEPS)]
        for i in range(STAGE_STEPS):
            step(20_000 + i, ev[i], slot=i)
        torch.cuda.synchronize()
        m_st = float(counts[:STAGE_STEPS].float().mean().item())
        score_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / STAGE_STEPS
        loss_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / STAGE_STEPS
        asst_ms = sum(e[2].elapsed_time(e[3]) for e in ev) / STAGE_STEPS
        sb = cfg.n * cfg.d * 2 + cfg.d * 4 + m_st * 4 + 4
        stages = {
            "steps": STAGE_STEPS, "accepted_mean": m_st,
            "note": "event to event inside whole steps: includes the event records and the gap to the next launch",
            "score_shrink": {"ms": score_ms, "GB/s": sb / (score_ms * 1e-3) / 1e9, "frac": sb / (score_ms * 1e-3) / 1e9 / peaks["hbm"]},
            "instance_loss": {"ms": loss_ms, "GB/s": m_st * (cfg.classes * 4 + 8) / (loss_ms * 1e-3) / 1e9,
                              "rows_per_s": m_st / (loss_ms * 1e-3)},
            "assistant_step": {"ms": asst_ms, "GB/s": (m_st * (cfg.d * 2 + 8) + 2 * cfg.d * 4) / (asst_ms * 1e-3) / 1e9,
                               "frac": (m_st * (cfg.d * 2 + 8) + 2 * cfg.d * 4) / (asst_ms * 1e-3) / 1e9 / peaks["hbm"]},
        }
        # the loss and the step alone, back to back, on the batch list of a screen under the initial Assistant
        # (weights near zero: about gamma + (1 - gamma) / 2 of the pool, the mean batch of the steps above)
        w_init, b_init = cfg.assistant(dev)
        cl = count_of[STAGE_STEPS]
        aa.aa_score_shrink(feats[0], B.linear_assistant(w_init, b_init), cfg.gamma, cfg.philox_seed, 30_000, out_idx, cl, score)
        m_last = int(cl.item())
        ms_l, best_l, calls_l = back_to_back(torch, lambda i: aa.aa_instance_loss(lg[i % npool], labels[i % npool], loss, count_dev=cl))
        ms_a, best_a, calls_a = back_to_back(torch, lambda i: aa.aa_assistant_step_scored(batch_feats[i % npool], loss, score, asst, cfg.lr,
                                                                                      count_dev=cl))
        ms_r, best_r, calls_r = back_to_back(torch, lambda i: aa.aa_assistant_step(batch_feats[i % npool], loss, asst, cfg.lr, count_dev=cl))
        stages["instance_loss_alone"] = {"rows": m_last, "roofline": hbm_roofline(m_last * (cfg.classes * 4 + 8), ms_l, best_l, calls_l, peaks,
                                                                                  kernel="row_loss_short_kernel")}
        stages["assistant_step_alone"] = {"rows": m_last, "roofline": hbm_roofline(m_last * (cfg.d * 2 + 12) + 2 * cfg.d * 4, ms_a, best_a,
                                                                                   calls_a, peaks, kernel="linear_grad_scored_kernel")}
        stages["assistant_step_recomputing_alone"] = {
            "rows": m_last, "what": "aa_assistant_step: the pre-activations are recomputed (any schedule)",
            "roofline": hbm_roofline(m_last * (cfg.d * 2 + 8) + 2 * cfg.d * 4, ms_r, best_r, calls_r, peaks, kernel="linear_grad_mma_kernel")}
        assert aa.aa_device_status() == B.AA_OK

    # ---- the same three stages as the two-stream schedule with a Boss queue of depth k (screening runs ahead of the
    # losses and updates it no longer waits for); reported beside the sequential figure, which stays the metric
    pipeline = None
    if "pipeline" in legs and args.pipeline_steps > 0:
        from paper_1905_03381_b200.pipeline import StreamPipeline

        pipe = StreamPipeline(args.pipeline_depth, max_rows=cfg.n, max_d=cfg.d, capacity=cfg.n, device=dev)
        gathered = {}

        def features(j, row_idx):
            kk = j % npool
            if row_idx is None:
                return feats[kk]
            key = (kk, row_idx.data_ptr())
            if key not in gathered:
                gathered[key] = B.dense_features(pools[kk], row_idx=row_idx, id_base=plan.id_bases[kk])
            return gathered[key]

        def boss(t, ctx, idx, count_dev, out_loss):
            ctx.aa_instance_loss(lg[t % npool], labels[t % npool], out_loss, count_dev=count_dev)

        P = args.pipeline_steps
        pipe.run(warm, features, boss, asst, cfg.gamma, cfg.philox_seed, cfg.lr, first_step=5000)
        torch.cuda.synchronize()
        n0 = pipe.launch_count()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record()
        pipe.run(P, features, boss, asst, cfg.gamma, cfg.philox_seed, cfg.lr, first_step=6000)
        p1.record()
        torch.cuda.synchronize()
        pst = pipe.device_status()
        assert pst == B.AA_OK, B.status_string(pst)
        pms = p0.elapsed_time(p1) / P
        pipeline = {"schedule": "Assistant stream: screen pool t+k, update on batch t; Boss stream: losses of batch t; "
                                "batch j screened with the parameters after max(0, j-k) updates",
                    "depth": args.pipeline_depth, "steps": P, "ms_per_step": pms, "value": cfg.n / (pms * 1e-3), "unit": UNIT,
                    "gpu_launches": int(pipe.launch_count() - n0)}
        pipe.close()
        del pipe

    # ---- end to end through the host-buffer entry point (pinned host inputs, results read back)
    e2e = None
    if "e2e" in legs and args.e2e_steps > 0:
        xh = pools[0].cpu().pin_memory()
        lh = logits[0].cpu().pin_memory()
        yh = labels[0].cpu().pin_memory()
        idx_h = torch.zeros(cfg.n, dtype=torch.int32).pin_memory()
        cnt_h = torch.zeros(1, dtype=torch.int32).pin_memory()
        loss_h = torch.zeros(cfg.n, dtype=torch.float32).pin_memory()
        hf, hl, staging, sbytes = aa.host_step_plan(xh, lh)
        for i in range(3):
            aa.aa_step_host(hf, asst, cfg.gamma, cfg.philox_seed, i, hl, yh, cfg.lr, idx_h, cnt_h, loss_h, staging, sbytes)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        d2h = 0
        for i in range(args.e2e_steps):
            aa.aa_step_host(hf, asst, cfg.gamma, cfg.philox_seed, 1000 + i, hl, yh, cfg.lr, idx_h, cnt_h, loss_h, staging, sbytes)
            d2h += 4 + 8 * int(cnt_h.item())
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        e2e_agg = sharding.aggregate(dist if world > 1 else None, dev, e2e_ms, cfg.n * args.e2e_steps)
        h2d = xh.numel() * xh.element_size() + lh.numel() * lh.element_size() + yh.numel() * yh.element_size()
        e2e = {"value": e2e_agg["units"] / (e2e_agg["ms"] * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h // args.e2e_steps, "steps": args.e2e_steps,
               "ms_per_step": e2e_agg["ms"] / args.e2e_steps}
        del xh, lh, yh, staging

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- CPU oracle on this machine's host cores: one core, and the same functions row-parallel over all cores
    cpu = cpu_all = None
    if "cpu" in legs and args.cpu_steps > 0:
        from oracle import aa_oracle as O
        O.build()
        xs = W.to_oracle(pools[0])
        w0 = cfg.assistant("cpu")[0].numpy()
        lh_np, yh_np = logits[0].cpu().numpy(), labels[0].cpu().numpy()
        sec, cand, _ = oracle_step_seconds(cfg, xs, w0, lh_np, yh_np, args.cpu_steps)
        cpu = {"value": cand / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"{args.cpu_steps} whole steps on one full pool of {cfg.n} candidates ({sec:.1f} s)"}
        try:
            cores = len(os.sched_getaffinity(0))
        except AttributeError:
            cores = os.cpu_count() or 1
        threads = max(1, min(cores, 64))
        sec2, cand2, _ = oracle_step_seconds_all_cores(cfg, xs, w0, lh_np, yh_np, args.cpu_steps, threads)
        cpu_all = {"value": cand2 / sec2, "unit": UNIT, "cores": threads, "cores_available": cores, "kind": "oracle, row-parallel",
                   "sample": f"{args.cpu_steps} whole steps on one full pool of {cfg.n} candidates, rows cut into {threads} "
                             f"slices, one thread each ({sec2:.1f} s)"}
        del xs

    # ---- secondary workloads, each alone on the GPU (the image pools are released first)
    del pools, logits, labels, feats, batch_feats, lg
    aa.close()
    torch.cuda.empty_cache()
    loss_rows = leg_translation_loss(torch, B, W, dev, peaks, args.small) if "loss" in legs else None
    torch.cuda.empty_cache()
    csr = leg_csr(torch, B, W, dev, peaks, args.small) if "csr" in legs else None
    torch.cuda.empty_cache()
    mlp = leg_mlp(torch, B, W, dev, peaks, args.small) if "mlp" in legs else None
    torch.cuda.empty_cache()
    conv = leg_conv(torch, B, W, dev, peaks, args.small, sampler.summary().get("sm_mhz")) if "conv" in legs else None
    torch.cuda.empty_cache()
    sweep = leg_sweep(torch, B, W, dev, peaks, args.small) if "sweep" in legs else None

    line = {
        "metric": METRIC, "value": agg["units"] / (agg["ms"] * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": warm, "ms_per_step": agg["ms"] / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(cfg, args),
        "roofline": roofline, "screen": screen, "stages": stages, "instance_loss_rows": loss_rows, "csr": csr, "mlp": mlp, "conv": conv,
        "sweep": sweep, "pipeline": pipeline, "cpu_baseline": cpu, "cpu_all_cores": cpu_all, "e2e": e2e,
        "gpu_launches": int(launches), "accepted_mean": accepted, "accepted_min": int(timed.min()),
        "accepted_max": int(timed.max()), "clocks": sampler.summary(),
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    args = parse_args()
    from paper_1905_03381_b200 import workloads as W

    cfg = W.ImageShape()
    if args.pool_rows:
        cfg.n = args.pool_rows
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_b200(args, cfg)


if __name__ == "__main__":
    main()
