"""Benchmark of the adaptive speculative-decoding iteration on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 7b]

A step is one whole iteration of Algorithm 1 (predict length -> draft -> verify -> accept).  The
metric is decode tokens per second at batch 1, timed on the device over exactly K steps after W
warm-up steps (prefill excluded), on seeded synthetic weights and prompts of the named shape.
With N > 1 (launched by torchrun, one rank per GPU) every rank decodes its own replica: the path
has no exchange step, so there is no collective on it; ranks meet only at the timing barriers.

`--impl reference` times the CPU oracle, as it stands, on the host cores over a bounded sample.
Rank 0 prints one JSON line.
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

METRIC = "decode tokens/sec at batch 1 (device-timed)"
UNIT = "tokens/s"
# measured dram__bytes_read+write over algorithmic bytes of k_pass (None once the kernel changed since the capture)
TRAFFIC_PER_ALGORITHMIC_BYTE = 1.006


def load_peaks():
    """Measured HBM copy bandwidth (GB/s) of this machine's B200s, else the stated fallback."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ----------------------------------------------------------------------------- algorithmic bytes

def verify_weight_bytes(sh) -> int:
    """bf16 bytes of every weight a verify pass reads once: L layers + LM head."""
    d, f, v = sh.d_model, sh.d_ffn, sh.vocab
    return 2 * (sh.n_layers * (4 * d * d + 3 * d * f) + v * d)


def draft_step_bytes(sh) -> int:
    """bf16 bytes of one draft-head step: fc + one layer + LM head."""
    d, f, v = sh.d_model, sh.d_ffn, sh.vocab
    return 2 * (2 * d * d + 4 * d * d + 3 * d * f + v * d)


def kv_bytes_per_token(sh) -> int:
    return 2 * 2 * sh.n_layers * sh.d_model


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()   # our own child, by handle
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ----------------------------------------------------------------------------- multi-rank plumbing

def dist_setup(n_gpus: int):
    """(rank, world, local_rank, dist or None).  One process per GPU under torchrun."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world == 1:
        return 0, 1, 0, None
    import torch.distributed as dist
    backend = os.environ.get("ADA_BENCH_BACKEND", "nccl")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend)
    return rank, world, local, dist


def aggregate(dist, local_ms: float, local_units: float, device=None):
    """Whole-job figures: max over ranks of the elapsed time, sum over ranks of the units."""
    if dist is None:
        return local_ms, local_units
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ----------------------------------------------------------------------------- ragged batch of 8 (context)

def batch8_sample(weights, dev, peak, iters: int = 30):
    """The 7B shape with 8 sequences of ragged prompt lengths (uniform in [128, 2048]) and per-sequence draft
    lengths: device time of `iters` iterations through the multi-row path, with the algorithmic bytes of an iteration
    (verify weights once + the cached positions of all sequences + one draft-head weight pass per draft step that
    any sequence takes) against the HBM peak.  Reported beside the batch-1 metric, not part of it."""
    import torch
    import synth_inputs as si
    from paper_2412_18910_b200 import Engine
    sh8 = si.SHAPES["7b_b8"]
    eng = Engine(sh8, weights, max_batch=sh8.batch, kv_capacity=sh8.kv_capacity, device=str(dev))
    prompts = si.make_prompts(sh8)
    for b, pr in enumerate(prompts):
        eng.ada_prefill(b, torch.from_numpy(pr).to(dev), None)
    for _ in range(5):
        eng.ada_step()
    c0 = eng.ada_get_counters()
    lens0 = eng.ada_debug_buffer(3, torch.int32, (sh8.batch, 8))[:, 0].cpu().to(torch.int64)   # committed tokens per sequence
    # per iteration the library itself writes the draft lengths used and the tokens emitted into rows of these arrays
    nused = torch.zeros(iters, sh8.batch, dtype=torch.int32, device=dev)
    nemit = torch.zeros(iters, sh8.batch, dtype=torch.int32, device=dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    e0.record(eng.stream)
    for i in range(iters):
        eng.ada_step(None, nemit[i], nused[i], None)
    e1.record(eng.stream)
    torch.cuda.synchronize(dev)
    c1 = eng.ada_get_counters()
    ms = e0.elapsed_time(e1)
    # cached positions read by the verify pass of iteration t: len - 1 per sequence, len growing by the tokens emitted;
    # draft steps that ran in it: the longest draft length of the iteration
    ne = nemit.cpu().to(torch.int64)
    before = torch.cumsum(ne, dim=0) - ne
    ctx_total = int(((lens0 - 1).unsqueeze(0) + before).sum())
    steps_total = int(nused.cpu().max(dim=1).values.sum())
    kv = ctx_total * kv_bytes_per_token(sh8)
    dkv = ctx_total * 2 * 2 * sh8.d_model          # the draft head's one-layer cache, read by its first step
    bytes_total = iters * verify_weight_bytes(sh8) + kv + steps_total * draft_step_bytes(sh8) + dkv
    gbs = bytes_total / (ms * 1e-3) / 1e9
    out = {"workload": "7b shape, 8 sequences, prompts %s, predictor-chosen draft lengths" % [len(p) for p in prompts],
           "iterations": iters, "ms_per_iteration": ms / iters,
           "tokens_per_s": (c1["n_tokens"] - c0["n_tokens"]) / (ms * 1e-3),
           "mean_draft_len": (c1["n_draft"] - c0["n_draft"]) / max(1, c1["n_target"] - c0["n_target"]),
           "bytes_per_iteration": bytes_total / iters, "kv_bytes_per_iteration": kv / iters,
           "draft_steps_per_iteration": steps_total / iters, "gbs": gbs, "frac_of_measured": gbs / peak,
           "status": c1["status"]}
    eng.close()
    return out


# ----------------------------------------------------------------------------- teacher-forced sweep (context)

def teacher_forced_sweep(weights, dev, peak, iters: int = 64, verify_samples: int = 16):
    """The 7B shape after a 1024-token prompt with drafts forced to the model's own greedy continuation, so that every
    draft is accepted (tau = n + 1), for each forced draft length n = 1..n_max, every sweep from the same prefilled
    state: `iters` whole iterations (ada_step) timed on the device, then `verify_samples` iterations through the
    separate calls with events around the verify launch (latency and bytes per second against n)."""
    import torch
    import synth_inputs as si
    from paper_2412_18910_b200 import Engine
    sh = si.SHAPES["7b_tf"]
    eng = Engine(sh, weights, max_batch=1, kv_capacity=sh.kv_capacity, device=str(dev))
    d_prompt = torch.from_numpy(si.make_prompts(sh)[0]).to(dev)
    nmax = sh.n_max
    need = iters * (nmax + 1) + nmax + 2
    # the greedy continuation, by plain autoregressive steps of the library itself (bit-identical to what it accepts)
    eng.ada_prefill(0, d_prompt, eng.d_first)
    eng.ada_force_n([0])
    stream = torch.zeros(need + nmax + 1, dtype=torch.int32, device=dev)
    stream[0:1] = eng.d_first
    for i in range(1, need):
        eng.ada_step(eng.d_emitted, None, None, None)
        stream[i: i + 1] = eng.d_emitted[0, 0:1]
    rows = []
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for n in range(1, nmax + 1):
        eng.ada_prefill(0, d_prompt, None)
        eng.ada_force_n([n])
        c0 = eng.ada_get_counters()
        off = 1
        for w in range(2):      # warm-up iterations (graph capture for this configuration)
            eng.ada_force_draft(stream[off: off + nmax].view(1, nmax))
            eng.ada_step()
            off += n + 1
        eng.ada_prefill(0, d_prompt, None)
        off = 1
        c0 = eng.ada_get_counters()
        torch.cuda.synchronize(dev)
        ea.record(eng.stream)
        for _ in range(iters):
            eng.ada_force_draft(stream[off: off + nmax].view(1, nmax))
            eng.ada_step()
            off += n + 1
        eb.record(eng.stream)
        torch.cuda.synchronize(dev)
        c1 = eng.ada_get_counters()
        ms = ea.elapsed_time(eb)
        tokens = c1["n_tokens"] - c0["n_tokens"]
        accepted_all = tokens == iters * (n + 1) and (c1["n_waste"] - c0["n_waste"]) == 0
        # verify launch alone, at the contexts the sweep starts from
        eng.ada_prefill(0, d_prompt, None)
        off = 1
        vms, ctxs = [], []
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(verify_samples)]
        ctx = len(d_prompt)
        for i in range(verify_samples):
            eng.ada_force_draft(stream[off: off + nmax].view(1, nmax))
            eng.ada_ldlp_predict(eng.d_n)
            eng.ada_draft(eng.d_n, eng.d_draft)
            evs[i][0].record(eng.stream)
            eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)
            evs[i][1].record(eng.stream)
            eng.ada_accept()
            ctxs.append(ctx + 1)
            ctx += n + 1
            off += n + 1
        torch.cuda.synchronize(dev)
        vms = sorted(a.elapsed_time(b) for a, b in evs)
        v_ms = vms[len(vms) // 2]
        vb = verify_weight_bytes(sh) + (sum(ctxs) / len(ctxs)) * kv_bytes_per_token(sh)
        rows.append({"n": n, "rows": n + 1, "tau": tokens / iters, "all_accepted": bool(accepted_all),
                     "ms_per_iteration": round(ms / iters, 4), "tokens_per_s": round(tokens / (ms * 1e-3), 1),
                     "verify_ms": round(v_ms, 4), "verify_gbs": round(vb / (v_ms * 1e-3) / 1e9, 1),
                     "verify_frac_of_measured": round(vb / (v_ms * 1e-3) / 1e9 / peak, 4)})
    status = eng.ada_get_counters()["status"]
    eng.ada_force_n(None)
    eng.ada_force_draft(None)
    eng.close()
    return {"workload": "7b shape, prompt 1024, drafts teacher-forced to the greedy continuation, draft length forced to n, "
                        "%d iterations per n from the same prefilled state" % iters,
            "verify_timing": "median of %d verify launches (CUDA events) at contexts from 1025 on" % verify_samples,
            "by_n": rows, "status": status}


# ----------------------------------------------------------------------------- the CPU oracle arm

def oracle_sample(sh, weights, prompt, iters: int, warm: int, prefill_tokens: int = 32):
    """Times `iters` oracle iterations (after `warm`) on a short prefix of the prompt.  Returns
    (tokens per second, ms per step, threads, description)."""
    import oracle
    m = oracle.Model(sh, weights)
    seq = m.new_seq(prefill_tokens + (iters + warm + 2) * (sh.n_max + 1) + 4)
    seq.prefill(prompt[:prefill_tokens])
    for _ in range(warm):
        seq.step(-1)
    toks, t0 = 0, time.perf_counter()
    for _ in range(iters):
        toks += len(seq.step(-1)["emitted"])
    dt = time.perf_counter() - t0
    desc = "%d iterations (predictor-chosen lengths) after a %d-token prefill of the same prompt" % (iters, prefill_tokens)
    return toks / dt, 1e3 * dt / iters, oracle.num_threads(), desc


# ----------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="7b", choices=["tiny", "7b", "13b"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-batch8", action="store_true", help="skip the ragged batch-of-8 sample (7b workload only)")
    ap.add_argument("--no-teacher-forced", action="store_true", help="skip the teacher-forced sweep n = 1..n_max (7b workload only)")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (a reduced case for profiler captures)")
    ap.add_argument("--profile-only", action="store_true", help="prefill, a few verify passes, exit (for ncu)")
    ap.add_argument("--profile-batch8", action="store_true",
                    help="with --profile-only: the ragged batch of 8 (multi-row path) instead of batch 1: the 8 prompts, then "
                         "--steps iterations through the separate calls")
    args = ap.parse_args()

    import numpy as np
    import synth_inputs as si

    sh = si.SHAPES[args.workload]
    if args.layers > 0:
        sh = si.scaled(sh, n_layers=args.layers, name="%s-%dlayers" % (sh.name, args.layers))
    K, W = max(1, args.steps), max(0, args.warmup)
    config = {"workload": "%s shape: %d layers, d=%d, %d heads x %d, ffn %d, vocab %d, n_max %d; batch 1, prompt %d "
                          "uniform-random ids, predictor-chosen draft lengths, greedy"
                          % (sh.name, sh.n_layers, sh.d_model, sh.n_heads, sh.head_dim, sh.d_ffn, sh.vocab, sh.n_max,
                             sh.prompt_len),
              "kv_capacity": sh.kv_capacity, "seed": si.DEFAULT_SEED,
              "l2": "inputs larger than L2 (weights %.1f GB per verify pass)" % (verify_weight_bytes(sh) / 1e9)}

    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        if rank != 0:
            return 0
        weights = si.make_weights(sh)
        prompt = si.make_prompts(sh)[0]
        # bounded sample: the oracle needs about a second per 7B iteration
        iters = min(K, 12 if sh.name != "tiny" else 256)
        warm = min(W, 2)
        tps, ms, threads, desc = oracle_sample(sh, weights, prompt, iters, warm)
        config = dict(config, sample="this arm runs a bounded sample of the workload: " + desc)
        line = {"impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": iters,
                "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic", "config": config,
                "cpu_baseline": {"value": tps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
                "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return 0

    import torch
    from paper_2412_18910_b200 import Engine

    rank, world, local, dist = dist_setup(args.gpus)
    dev = torch.device("cuda:%d" % local)
    torch.cuda.set_device(dev)
    weights = si.make_weights(sh)
    if args.profile_only and args.profile_batch8:
        sh8 = si.scaled(si.SHAPES["7b_b8"], n_layers=sh.n_layers, name="7b_b8-%dlayers" % sh.n_layers)
        eng = Engine(sh8, weights, max_batch=sh8.batch, kv_capacity=sh8.kv_capacity, device=str(dev))
        for b, pr in enumerate(si.make_prompts(sh8)):
            eng.ada_prefill(b, torch.from_numpy(pr).to(dev), None)
        for _ in range(max(1, K)):
            eng.ada_ldlp_predict(eng.d_n)
            eng.ada_draft(eng.d_n, eng.d_draft)
            eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)
            eng.ada_accept()
        torch.cuda.synchronize(dev)
        print(json.dumps({"profile_only": True, "batch": sh8.batch, "status": eng.ada_get_counters()["status"]}))
        eng.close()
        return 0
    prompt = si.uniform_ids(si.DEFAULT_SEED + rank, "prompt0", sh.prompt_len, sh.vocab)
    eng = Engine(sh, weights, max_batch=1, kv_capacity=sh.kv_capacity, device=str(dev))
    per_episode = max(1, (sh.kv_capacity - sh.prompt_len - sh.n_max - 4) // (sh.n_max + 1))
    if args.profile_only:
        d_prompt = torch.from_numpy(prompt).to(dev)
        eng.ada_prefill(0, d_prompt, None)
        eng.ada_ldlp_predict(eng.d_n)
        eng.ada_draft(eng.d_n, eng.d_draft)
        for _ in range(max(1, K)):
            eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)
        torch.cuda.synchronize(dev)
        print(json.dumps({"profile_only": True, "status": eng.ada_get_counters()["status"]}))
        eng.close()
        return 0

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()

    # ---- device-timed leg: K steps, inputs resident, no host round trip between steps
    d_prompt = torch.from_numpy(prompt).to(dev)
    eng.ada_prefill(0, d_prompt, None)
    for _ in range(max(W, 3)):
        eng.ada_step()
    sampler = ClockSampler(local)
    sampler.start()
    c0 = eng.ada_get_counters()
    total_ms, done = 0.0, 0
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    used_in_episode = max(W, 3)
    while done < K:
        todo = min(K - done, per_episode - used_in_episode)
        if todo <= 0:                      # cache nearly full: start again from the prompt (not timed)
            eng.ada_prefill(0, d_prompt, None)
            used_in_episode = 0
            continue
        barrier()
        ev0.record(eng.stream)
        for _ in range(todo):
            eng.ada_step()
        ev1.record(eng.stream)
        barrier()
        total_ms += ev0.elapsed_time(ev1)
        done += todo
        used_in_episode += todo
    c1 = eng.ada_get_counters()
    clocks = sampler.stop()
    if c1["status"] != 0:     # a device-side error (a wait that gave up, a full cache) invalidates the timing
        raise RuntimeError("device status word %d after the timed region" % c1["status"])
    tokens = c1["n_tokens"] - c0["n_tokens"]
    launches = c1["launches"] - c0["launches"]
    n_draft = c1["n_draft"] - c0["n_draft"]
    n_target = c1["n_target"] - c0["n_target"]
    job_ms, job_tokens = aggregate(dist, total_ms, float(tokens), dev)
    value = job_tokens / (job_ms * 1e-3)

    # ---- end-to-end leg: prompt from pinned host memory, prefill, K steps each followed by a
    # device->host read of what it emitted (a serving loop must see tokens to stop on a terminator)
    h_prompt = torch.from_numpy(prompt).pin_memory()
    h_out = torch.zeros(sh.n_max + 3, dtype=torch.int32).pin_memory()
    d_out = torch.zeros(sh.n_max + 3, dtype=torch.int32, device=dev)
    Ke = min(K, per_episode)
    barrier()
    t0 = time.perf_counter()
    d_p2 = torch.empty_like(d_prompt)
    d_p2.copy_(h_prompt, non_blocking=True)
    eng.ada_prefill(0, d_p2, d_out[sh.n_max + 2:])
    e_tokens = 0
    for _ in range(Ke):
        eng.ada_step(d_out[: sh.n_max + 1], d_out[sh.n_max + 1: sh.n_max + 2])
        h_out.copy_(d_out, non_blocking=True)
        torch.cuda.synchronize(dev)
        e_tokens += int(h_out[sh.n_max + 1])
    e2e_ms = (time.perf_counter() - t0) * 1e3
    status_e2e = eng.ada_get_counters()["status"]
    if status_e2e != 0:
        raise RuntimeError("device status word %d after the end-to-end leg" % status_e2e)
    e_ms, e_tok = aggregate(dist, e2e_ms, float(e_tokens), dev)
    e2e = {"value": e_tok / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": prompt.nbytes / Ke,
           "d2h_bytes_per_step": h_out.numel() * 4, "steps": Ke,
           "note": "request latency: pinned-host prompt copy + prompt pass + steps with a host read-back each; with few "
                   "steps the prompt pass (see prefill.ms) is a large share of it"}

    # ---- prompt pass (Algorithm 1's first verify, k = 0): device time of ada_prefill on the resident prompt
    pa, pb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pre_ms = []
    for _ in range(3):
        torch.cuda.synchronize(dev)
        pa.record(eng.stream)
        eng.ada_prefill(0, d_prompt, None)
        pb.record(eng.stream)
        torch.cuda.synchronize(dev)
        pre_ms.append(pa.elapsed_time(pb))
    prefill = {"prompt_len": int(sh.prompt_len), "ms": min(pre_ms), "prompt_tokens_per_s": sh.prompt_len / (min(pre_ms) * 1e-3),
               "note": "128-row chunks through the multi-row tensor-core GEMM; not part of the decode metric"}

    # ---- roofline leg: the dominant kernel (skinny GEMM) and the whole verify pass, timed with
    # events on the library's stream at the context length the timed region ended at
    peak, peak_kind = load_peaks()
    eng.ada_prefill(0, d_prompt, None)
    eng.ada_ldlp_predict(eng.d_n)
    n_now = int(eng.d_n.cpu()[0])
    eng.ada_draft(eng.d_n, eng.d_draft)
    reps = 8
    for _ in range(2):
        eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)     # same rows again: nothing is committed
    torch.cuda.synchronize(dev)
    eng.ada_profile(True)
    va, vb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    va.record(eng.stream)
    for _ in range(reps):
        eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)
    vb.record(eng.stream)
    prof = eng.ada_get_profile()
    eng.ada_profile(False)
    verify_ms_prof = va.elapsed_time(vb) / reps
    va.record(eng.stream)
    for _ in range(reps):
        eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)
    vb.record(eng.stream)
    torch.cuda.synchronize(dev)
    verify_ms = va.elapsed_time(vb) / reps
    ctx_len = sh.prompt_len + 1
    vbytes = verify_weight_bytes(sh) + ctx_len * kv_bytes_per_token(sh)
    # verify latency as a function of the context length (cache bytes grow with it): 9 rows after prompts of
    # 1024, 2048 and 4000 tokens, median of 9 ada_verify calls each
    by_ctx = []
    for ctx in (1024, 2048, 4000):
        if ctx + sh.n_max + 2 > sh.kv_capacity:
            continue
        d_long = torch.from_numpy(si.uniform_ids(si.DEFAULT_SEED + rank, "ctx%d" % ctx, ctx, sh.vocab)).to(dev)
        eng.ada_prefill(0, d_long, None)
        eng.d_n.fill_(min(8, sh.n_max))
        eng.ada_draft(eng.d_n, eng.d_draft)
        eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(9)]
        for a_, b_ in pairs:
            a_.record(eng.stream)
            eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)
            b_.record(eng.stream)
        torch.cuda.synchronize(dev)
        ms_c = statistics.median(a_.elapsed_time(b_) for a_, b_ in pairs)
        cb = verify_weight_bytes(sh) + (ctx + 1) * kv_bytes_per_token(sh)
        by_ctx.append({"ctx": ctx + 1, "rows": min(8, sh.n_max) + 1, "ms": round(ms_c, 4), "bytes": cb,
                       "gbs": round(cb / (ms_c * 1e-3) / 1e9, 1), "frac_of_measured": round(cb / (ms_c * 1e-3) / 1e9 / peak, 4)})
    # the dominant kernel: the persistent pass kernel, one launch per verify pass (weights + KV read once)
    launch_ms = prof["gemm_ms"] / max(1, prof["gemm_launches"])
    pass_gbs = vbytes / (launch_ms * 1e-3) / 1e9 if launch_ms > 0 else None
    roofline = {"bound": "hbm", "kernel": "k_pass (target verify pass: embedding, all layers, LM head and greedy choice in one persistent launch)",
                "achieved": pass_gbs, "peak": peak, "unit": "GB/s",
                "frac": (pass_gbs / peak) if pass_gbs else None, "peak_kind": "of " + peak_kind,
                # dram bytes of one launch: not counted in this run; the counters of an ncu capture of the 4-layer case
                # of the same shape, scaled by the bytes processed (traffic grows in proportion to the layers)
                "traffic": (vbytes * TRAFFIC_PER_ALGORITHMIC_BYTE) if (sh.name == "7b" and TRAFFIC_PER_ALGORITHMIC_BYTE) else None,
                "traffic_kind": "scaled from an ncu capture of the 4-layer case" if (sh.name == "7b" and TRAFFIC_PER_ALGORITHMIC_BYTE) else None,
                "launches_timed": prof["gemm_launches"], "avg_launch_us": 1e3 * launch_ms,
                "bytes_per_launch": vbytes, "frac_of_8000": (pass_gbs / 8000.0) if pass_gbs else None,
                "verify_pass": {"rows": n_now + 1, "ctx": ctx_len, "ms": verify_ms, "bytes": vbytes,
                                "weight_bytes": verify_weight_bytes(sh), "kv_bytes": ctx_len * kv_bytes_per_token(sh),
                                "gbs": vbytes / (verify_ms * 1e-3) / 1e9,
                                "frac_of_measured": vbytes / (verify_ms * 1e-3) / 1e9 / peak,
                                "frac_of_8000": vbytes / (verify_ms * 1e-3) / 1e9 / 8000.0},
                "verify_by_ctx": by_ctx}
    # one draft-head step (fc, its layer, the LM head; a persistent launch each): a full-length draft at the same context
    eng.ada_prefill(0, d_prompt, None)
    eng.d_n.fill_(sh.n_max)
    eng.ada_draft(eng.d_n, eng.d_draft)
    eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target)      # rows are not committed: the next draft starts from the same state
    eng.ada_profile(True)
    eng.ada_draft(eng.d_n, eng.d_draft)
    dprof = eng.ada_get_profile()
    eng.ada_profile(False)
    if dprof["gemm_launches"] > 0:
        d_us = 1e3 * dprof["gemm_ms"] / dprof["gemm_launches"]
        dbytes = draft_step_bytes(sh) + ctx_len * 2 * 2 * sh.d_model
        roofline["draft_step"] = {"launches_timed": dprof["gemm_launches"], "avg_launch_us": d_us, "bytes_per_launch": dbytes,
                                  "gbs": dbytes / (d_us * 1e-6) / 1e9, "frac_of_measured": dbytes / (d_us * 1e-6) / 1e9 / peak}
    status_roof = eng.ada_get_counters()["status"]
    if status_roof != 0:
        raise RuntimeError("device status word %d after the roofline leg" % status_roof)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(W, 3),
            "ms_per_step": job_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 weights, fp16 KV cache, f32 accumulate", "data": "synthetic", "config": config, "status": 0,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "tau": tokens / max(1, n_target), "mean_draft_len": n_draft / max(1, n_target), "prefill": prefill}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        tps, ms, threads, desc = oracle_sample(sh, weights, prompt, 10 if sh.name != "tiny" else 64, 1)
        line["cpu_baseline"] = {"value": tps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}
    eng.close()
    if rank == 0 and world == 1 and sh.name == "7b" and not args.layers and not args.no_batch8:
        line["batch8"] = batch8_sample(weights, dev, peak)
        if not args.no_teacher_forced:
            line["teacher_forced"] = teacher_forced_sweep(weights, dev, peak)
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
