"""Throughput of the instance-shrinking batch generator on the image-classification shape.

One step = one pass of the whole hot path over one candidate pool: Assistant score ->
Bernoulli shrink -> ordered batch list (aa_score_shrink), per-instance Boss loss of the
accepted batch (aa_instance_loss), labels + one Assistant SGD step (aa_assistant_step).
Pool: 65,536 candidates x 3072 bf16 features (403 MB, larger than L2; pools rotate),
100-class fp32 logits, gamma 0.1, lr 0.05.  Prints ONE JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

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


# Per-stage CUDA events are recorded on every EVENT_EVERY-th timed step: an event between two kernels keeps the
# second from being scheduled while the first drains, which is how the steps without events run.
EVENT_EVERY = 7   # co-prime with the number of rotating pools, so the sample covers every pool


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--pools", type=int, default=8, help="distinct resident pools rotated through the steps")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--cpu-steps", type=int, default=40, help="oracle steps timed for cpu_baseline (0 = skip)")
    ap.add_argument("--pool-rows", type=int, default=None, help="override the pool size (testing only)")
    ap.add_argument("--workload", default="image", choices=["image", "mlp"],
                    help="image = the benchmark workload; mlp = the two-layer (tensor-core) Assistant shape")
    ap.add_argument("--pipeline-steps", type=int, default=300,
                    help="steps of the two-stream Assistant/Boss schedule timed after the main region (0 = skip)")
    ap.add_argument("--pipeline-depth", type=int, default=2, help="Boss queue depth k of that schedule")
    ap.add_argument("--loss-reps", type=int, default=20,
                    help="timed calls of the per-sentence loss on the translation shape (0 = skip)")
    return ap.parse_args()


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


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


# --------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)
# --------------------------------------------------------------------------

def oracle_step_seconds(cfg, x_host, w0, logits_host, labels_host, steps: int):
    """Times `steps` whole steps of the oracle, as it stands, single-threaded.  Returns (seconds, candidates)."""
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
    return time.perf_counter() - t0, n * steps


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
    sec, cand = oracle_step_seconds(cfg, x, w0, logits, labels, steps)
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
        "stage_events": None if reference else f"per-stage CUDA events on every {EVENT_EVERY}th timed step",
        "parallelism": f"instance-sharded x{args.gpus}, one Assistant per GPU, no data-path collective",
    }


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

    plan = sharding.plan(rank, world, args.pools, cfg.n)
    pools = [cfg.pool(pid, dev) for pid in plan.pool_ids]
    logits = [cfg.logits(pid, dev) for pid in plan.pool_ids]
    labels = [cfg.labels(pid, dev) for pid in plan.pool_ids]
    w, b = cfg.assistant(dev)
    aa = B.AutoAssist(max_rows=cfg.n, max_d=cfg.d, device=dev)
    asst = B.linear_assistant(w, b)
    out_idx = torch.zeros(cfg.n, dtype=torch.int32, device=dev)
    # one device count per step, so that the mean batch size of the timed steps is known without a host read
    n_slots = max(args.warmup, 3) + args.steps
    counts = torch.zeros(n_slots, dtype=torch.int32, device=dev)
    count_of = [counts[j:j + 1] for j in range(n_slots)]
    loss = torch.zeros(cfg.n, dtype=torch.float32, device=dev)
    feats = [B.dense_features(p, id_base=base) for p, base in zip(pools, plan.id_bases)]
    batch_feats = [B.dense_features(p, row_idx=out_idx, id_base=base) for p, base in zip(pools, plan.id_bases)]
    lg = [B.logits_desc(l) for l in logits]
    npool = len(pools)

    def step(i, events=None):
        k = i % npool
        out_count = count_of[i % n_slots]
        if events is not None:
            events[0].record()
        aa.aa_score_shrink(feats[k], asst, cfg.gamma, cfg.philox_seed, i, out_idx, out_count)
        if events is not None:
            events[1].record()
        aa.aa_instance_loss(lg[k], labels[k], loss, count_dev=out_count)
        if events is not None:
            events[2].record()
        aa.aa_assistant_step(batch_feats[k], loss, asst, cfg.lr, count_dev=out_count)
        if events is not None:
            events[3].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    assert aa.aa_device_status() == B.AA_OK

    # ---- device-resident throughput: K steps between two events, kernels timed per call as well
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = aa.aa_launch_count()
    barrier()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(K):
        step(args.warmup + i, ev[i] if i % EVENT_EVERY == 0 else None)   # per-stage events on a sample of the steps
    t_end.record()
    barrier()
    elapsed_ms = t_start.elapsed_time(t_end)
    launches = aa.aa_launch_count() - launches0
    if rank == 0:
        time.sleep(0.2)
        sampler.stop()
    status = aa.aa_device_status()
    assert status == B.AA_OK, B.status_string(status)
    timed = counts[[(args.warmup + i) % n_slots for i in range(K)]].cpu().numpy().astype(np.int64)
    accepted = float(timed.mean())            # mean batch size M over the timed steps
    sampled = [ev[i] for i in range(K) if i % EVENT_EVERY == 0]
    score_ms = sum(e[0].elapsed_time(e[1]) for e in sampled) / len(sampled)
    loss_ms = sum(e[1].elapsed_time(e[2]) for e in sampled) / len(sampled)
    asst_ms = sum(e[2].elapsed_time(e[3]) for e in sampled) / len(sampled)

    agg = sharding.aggregate(dist if world > 1 else None, dev, elapsed_ms, cfg.n * K)

    # ---- the same three stages as the two-stream schedule with a Boss queue of depth k (screening runs ahead of the
    # losses and updates it no longer waits for); reported beside the sequential figure, which stays the metric
    pipeline = None
    if args.pipeline_steps > 0 and world == 1:
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
        pipe.run(max(args.warmup, 3), features, boss, asst, cfg.gamma, cfg.philox_seed, cfg.lr, first_step=5000)
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

    # ---- second half of the metric: per-instance-loss rows/s on the translation shape
    # (25,000 token rows x 32,000-word bf16 logits = 1.6 GB per call, larger than L2; per-sentence sums)
    loss_rows = None
    if args.loss_reps > 0 and rank == 0:
        t2 = W.TranslationShape()
        rows2 = t2.token_budget
        lg2 = t2.token_logits(rows2, dev)
        ids2 = t2.token_ids(rows2, dev)
        off2 = torch.from_numpy(W.ragged_offsets(rows2, t2.len_lo, t2.len_hi, 9)).to(dev)
        sent_loss = torch.zeros(off2.numel() - 1, dtype=torch.float32, device=dev)
        aa2 = B.AutoAssist(max_rows=rows2, max_d=8, device=dev)
        g2 = B.logits_desc(lg2)
        for _ in range(3):
            aa2.aa_instance_loss(g2, ids2, sent_loss, offsets=off2)
        torch.cuda.synchronize()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = aa2.aa_launch_count()
        l0.record()
        for _ in range(args.loss_reps):
            aa2.aa_instance_loss(g2, ids2, sent_loss, offsets=off2)
        l1.record()
        torch.cuda.synchronize()
        assert aa2.aa_device_status() == B.AA_OK
        ms2 = l0.elapsed_time(l1) / args.loss_reps
        bytes2 = rows2 * t2.vocab * 2 + rows2 * 8 + off2.numel() * 4 + sent_loss.numel() * 4
        peak2, kind2 = measured_peak_gbs()
        loss_rows = {"workload": f"translation shape: {rows2} token rows x {t2.vocab} bf16 logits N(0,4), "
                                 f"{sent_loss.numel()} sentences of 8..128 tokens, summed per sentence",
                     "value": rows2 / (ms2 * 1e-3), "unit": "token rows/s", "ms_per_call": ms2,
                     "launches_per_call": (aa2.aa_launch_count() - n0) // args.loss_reps,
                     "roofline": {"bound": "hbm", "achieved": bytes2 / (ms2 * 1e-3) / 1e9, "peak": peak2, "unit": "GB/s",
                                  "frac": bytes2 / (ms2 * 1e-3) / 1e9 / peak2, "peak_kind": f"of {kind2}",
                                  "algorithmic_bytes_per_launch": bytes2}}
        aa2.close()
        del lg2, ids2, aa2

    # ---- end to end through the host-buffer entry point (pinned host inputs, results read back)
    e2e = None
    if args.e2e_steps > 0:
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

    peak, peak_kind = measured_peak_gbs()
    alg_bytes = cfg.n * cfg.d * 2 + cfg.d * 4 + accepted * 4 + 4
    achieved = alg_bytes / (score_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "score_shrink_tma_kernel<bf16, 32>", "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": ncu_traffic_bytes(cfg.n),
                "launches_timed": len(sampled),
                "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_ms": score_ms,
                "frac_of_nominal_8TBs": achieved / 8000.0}
    loss_bytes = accepted * (cfg.classes * 4 + 8)
    asst_bytes = accepted * (cfg.d * 2 + 8) + 2 * cfg.d * 4
    stages = {
        "score_shrink": {"ms": score_ms, "GB/s": achieved},
        "instance_loss": {"ms": loss_ms, "GB/s": loss_bytes / (loss_ms * 1e-3) / 1e9, "rows_per_s": accepted / (loss_ms * 1e-3)},
        "assistant_step": {"ms": asst_ms, "GB/s": asst_bytes / (asst_ms * 1e-3) / 1e9},
    }

    cpu = None
    if world == 1 and args.cpu_steps > 0:
        from oracle import aa_oracle as O
        O.build()
        xs = W.to_oracle(pools[0])
        w0 = cfg.assistant("cpu")[0].numpy()
        sec, cand = oracle_step_seconds(cfg, xs, w0, logits[0].cpu().numpy(), labels[0].cpu().numpy(), args.cpu_steps)
        cpu = {"value": cand / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"{args.cpu_steps} whole steps on one full pool of {cfg.n} candidates ({sec:.1f} s)"}

    line = {
        "metric": METRIC, "value": agg["units"] / (agg["ms"] * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": agg["ms"] / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(cfg, args),
        "roofline": roofline, "stages": stages, "instance_loss_rows": loss_rows, "pipeline": pipeline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
        "accepted_mean": accepted, "accepted_min": int(timed.min()), "accepted_max": int(timed.max()), "clocks": sampler.summary(),
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def measured_peak_tflops(sustained: bool):
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            rec = json.load(f)
        return float(rec["bf16_tflops_sustained" if sustained else "bf16_tflops"]), "measured"
    except Exception:
        return (1400.0 if sustained else 1590.0), "fallback"


def run_mlp(args):
    """Secondary workload (--workload mlp): the two-layer Assistant shape, whose scoring is a dense bf16 contraction.
    One step = MLP score+shrink+compact, 1000-class instance loss, MLP Assistant step on the accepted rows."""
    import torch

    from paper_1905_03381_b200 import binding as B, build as lib_build, workloads as W

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    lib_build.build()
    cfg = W.MlpShape()
    if args.pool_rows:
        cfg.n = args.pool_rows
    x = cfg.pool(dev)
    W1, b1, w2, b2 = cfg.assistant(dev)
    W1b = W1.to(torch.bfloat16).contiguous()
    logits = cfg.logits(cfg.n, dev)
    labels = cfg.labels(cfg.n, dev)
    aa = B.AutoAssist(max_rows=cfg.n, max_d=cfg.d, max_hidden=cfg.hidden, device=dev)
    asst = B.mlp_assistant(W1, W1b, b1, w2, b2)
    out_idx = torch.zeros(cfg.n, dtype=torch.int32, device=dev)
    K = args.steps
    warm = max(args.warmup, 3)
    counts = torch.zeros(warm + K, dtype=torch.int32, device=dev)
    loss = torch.zeros(cfg.n, dtype=torch.float32, device=dev)
    feat, batch = B.dense_features(x), B.dense_features(x, row_idx=out_idx)
    lg = B.logits_desc(logits)

    def step(i, ev=None):
        cnt = counts[i:i + 1]
        if ev: ev[0].record()
        aa.aa_score_shrink(feat, asst, cfg.gamma, cfg.philox_seed, i, out_idx, cnt)
        if ev: ev[1].record()
        aa.aa_instance_loss(lg, labels, loss, count_dev=cnt)
        if ev: ev[2].record()
        aa.aa_assistant_step(batch, loss, asst, cfg.lr, count_dev=cnt)
        if ev: ev[3].record()

    for i in range(warm):
        step(i)
    torch.cuda.synchronize()
    assert aa.aa_device_status() == B.AA_OK
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    n0 = aa.aa_launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(K):
        step(warm + i, evs[i])
    t1.record()
    torch.cuda.synchronize()
    time.sleep(0.2)
    sampler.stop()
    assert aa.aa_device_status() == B.AA_OK
    ms = t0.elapsed_time(t1) / K
    score_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / K
    loss_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / K
    asst_ms = sum(e[2].elapsed_time(e[3]) for e in evs) / K
    m_mean = float(counts[warm:].float().mean().item())
    flops = 2.0 * cfg.n * cfg.d * cfg.hidden
    peak, kind = measured_peak_tflops(sustained=True)
    hbm, hkind = measured_peak_gbs()
    line = {
        "metric": METRIC, "value": cfg.n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": warm,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"MLP Assistant shape: pool {cfg.n} x {cfg.d} bf16 N(0,1), {cfg.d}->{cfg.hidden} (ReLU)->1, "
                               f"{cfg.classes}-class fp32 logits N(0,3), mix {cfg.gamma}, SGD lr {cfg.lr} on both layers",
                   "l2_policy": "inputs larger than L2 (pool 1.6 GB)"},
        "roofline": {"bound": "tensor", "kernel": "mlp_score_shrink_kernel", "achieved": flops / (score_ms * 1e-3) / 1e12,
                     "peak": peak, "unit": "TFLOP/s", "frac": flops / (score_ms * 1e-3) / 1e12 / peak,
                     "peak_kind": f"of {kind} (sustained cuBLAS bf16)", "traffic": None, "avg_launch_ms": score_ms,
                     "hbm_GBs": cfg.n * cfg.d * 2 / (score_ms * 1e-3) / 1e9, "hbm_frac": cfg.n * cfg.d * 2 / (score_ms * 1e-3) / 1e9 / hbm},
        "stages": {"score_shrink": {"ms": score_ms}, "instance_loss": {"ms": loss_ms, "rows_per_s": m_mean / (loss_ms * 1e-3),
                   "GB/s": m_mean * (cfg.classes * 4 + 8) / (loss_ms * 1e-3) / 1e9},
                   "assistant_step": {"ms": asst_ms, "TFLOP/s": 2 * 2.0 * m_mean * cfg.d * cfg.hidden / (asst_ms * 1e-3) / 1e12}},
        "accepted_mean": m_mean, "gpu_launches": int(aa.aa_launch_count() - n0), "clocks": sampler.summary(),
    }
    print(json.dumps(line), flush=True)
    aa.close()


def main():
    args = parse_args()
    from paper_1905_03381_b200 import workloads as W

    if args.workload == "mlp":
        if args.impl == "reference" or args.gpus != 1:
            raise SystemExit("--workload mlp is a single-GPU measurement of the library only")
        run_mlp(args)
        return
    cfg = W.ImageShape()
    if args.pool_rows:
        cfg.n = args.pool_rows
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_b200(args, cfg)


if __name__ == "__main__":
    main()
