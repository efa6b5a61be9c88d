#!/usr/bin/env python
"""Benchmark of the Q-Delta hot path on B200.

A step is one chunkwise forward (saving what the backward needs) plus one chunkwise backward over
one batch of synthetic input of the headline configuration (bf16, B=8, H=16, T=2048,
d_k=d_v=128, chunk 64); the decode step is timed separately on its own configuration and reported
under "decode".  One process per GPU; with N > 1 every rank runs its own batch (weak scaling, no
collective on the data path).  Prints ONE JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

`--impl reference` times the fp64 CPU oracle (the only "reference implementation" this method has
here) on a bounded sample of the same workload.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time
from dataclasses import replace

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "Q-Delta chunkwise fwd+bwd tokens/s (bf16, d=128) and % of roofline on 1 B200"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ---- algorithmic work per token-head (one head's share of one token), bf16 storage ---------------
def path_bytes_per_token_head(dk, dv):
    fwd = 2 * (2 * dk + dv) + 6 + 2 * dv                       # read q,k,v + 3 coefficients, write o
    bwd = 2 * (2 * dk + 2 * dv) + 6 + 2 * (2 * dk + dv) + 12   # read q,k,v,dO + coeffs, write dq,dk,dv + 3 fp32
    return fwd, bwd


def path_flops_per_token_head(dk, dv, C):
    s = 2.0 * C * C * dk / C          # one C x C x d product, per token
    b = 2.0 * C * dk * dv / C         # one C x d x d product, per token
    return 5 * s + 3 * b, 11 * s + 6 * b


def stage_bytes_per_token_head(dk, dv, C):
    """Compulsory HBM bytes of each kernel of the present decomposition, per token-head: bf16
    intermediates stored in their consumer's operand orientation, one bf16 state per chunk."""
    st = 2.0 * dk * dv / C            # one bf16 state per chunk, per token
    qkv = 2 * (2 * dk + dv)
    return {
        # read q,k,v + 3 coefficients; write diag(gamma)Q, P, W~^T, U~^T, g and the inverse for backward
        "prep": qkv + 6 + 2 * dk + 2 * C + 2 * dk + 2 * dv + 4 + 2 * C,
        # read diag(gamma)Q, P, W~^T, U~^T, K, g; write o, entry states, Delta^T
        "chain_fwd": 2 * dk + 2 * C + 2 * dk + 2 * dv + 2 * dk + 4 + 2 * dv + st + 2 * dv,
        # read W~^T, dO, diag(gamma)Q, K, P, g; write dDelta^T and the exit-state gradients
        "chain_bwd": 2 * dk + 2 * dv + 2 * dk + 2 * dk + 2 * C + 4 + 2 * dv + st,
        # read q,k,v,dO, both per-chunk states, Delta^T, dDelta^T, inverse, P, coefficients, g; write 6 gradients
        "chunk_bwd": qkv + 2 * dv + 2 * st + 4 * dv + 4 * C + 6 + 4 + qkv + 12,
    }


# dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu capture summarised in
# profiles/tc_kernels_dram_traffic_cfg2.md (full-size cfg2); other workloads: not captured
NCU_TRAFFIC_BYTES = {"cfg2": {"prep": 421.9e6, "chain_fwd": 532.8e6, "chain_bwd": 469.2e6, "chunk_bwd": 926.2e6}}


class ClockSampler(threading.Thread):
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.stop_flag = index, [], threading.Event()

    def run(self):
        while not self.stop_flag.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                f = [x.strip() for x in out.strip().split(",")]
                if len(f) >= 6:
                    self.samples.append(f)
            except Exception:
                pass
            self.stop_flag.wait(0.2)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        sm = sorted(float(s[0]) for s in self.samples)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i].lower().startswith("active") for s in self.samples)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(self.samples[0][1]), "reasons": reasons,
                "samples": len(sm)}


def oracle_sample(cfg, nseq, steps=1, warmup=0):
    """Time the fp64 oracle (forward + reverse pass) on the first `nseq` sequences of cfg."""
    from paper_2606_08804_b200 import inputs as gen
    from oracle import recurrence as orc
    sub = replace(cfg, B=1, H=nseq)
    d = gen.make_chunk_inputs(sub)

    def run():
        orc.forward(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"])
        orc.backward(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"], d["dO"], d["dhT"])
    for _ in range(warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(steps):
        run()
    dt = (time.perf_counter() - t0) / steps
    tokens = nseq * cfg.T / cfg.H            # a token carries all H heads
    return tokens / dt, dt, orc.max_threads()


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    nseq = max(1, min(cfg.B * cfg.H, 4 * cores))
    val, dt, thr = oracle_sample(cfg, nseq, steps=args.steps, warmup=min(args.warmup, 1))
    sample = "first %d of %d (batch, head) sequences of %s, forward + reverse pass, fp64" % (nseq, cfg.B * cfg.H, cfg.name)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_name(cfg):
    return "%s: bf16 fwd+bwd B=%d H=%d T=%d dk=%d dv=%d chunk=%d" % (cfg.name, cfg.B, cfg.H, cfg.T, cfg.dk, cfg.dv, cfg.chunk)


def run_ours(args, cfg):
    import torch
    from paper_2606_08804_b200 import binding as qd
    from paper_2606_08804_b200 import inputs as gen
    from paper_2606_08804_b200 import sharding

    rank, world, local = sharding.rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    qd.load()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- inputs: pinned host copies and device copies ------------------------------------------
    d = gen.make_chunk_inputs(cfg, seed=sharding.rank_seed(cfg.seed, rank))
    bf, f32 = torch.bfloat16, torch.float32
    host, dev = {}, {}
    for n in ("q", "k", "v", "beta", "alpha", "lam", "dO"):
        host[n] = torch.from_numpy(d[n]).to(bf).pin_memory()
    for n in ("h0", "dhT"):
        host[n] = torch.from_numpy(d[n]).pin_memory()
    for n, t in host.items():
        dev[n] = t.to("cuda", non_blocking=True)
    del d
    B, T, H, dk, dv = cfg.B, cfg.T, cfg.H, cfg.dk, cfg.dv
    shape = qd.make_shape(dev["q"], dev["v"], cfg.chunk)
    ws = qd.alloc_workspace(shape, True, "cuda")
    o = torch.empty((B, T, H, dv), dtype=bf, device="cuda")
    hT = torch.empty((B, H, dk, dv), dtype=f32, device="cuda")
    grads = {}

    def step():
        qd.chunk_fwd(dev["q"], dev["k"], dev["v"], dev["beta"], dev["alpha"], dev["lam"], dev["h0"],
                     chunk=cfg.chunk, save_for_bwd=True, workspace=ws, o=o, hT=hT)
        qd.chunk_bwd(dev["q"], dev["k"], dev["v"], dev["beta"], dev["alpha"], dev["lam"], dev["h0"],
                     dev["dO"], dev["dhT"], chunk=cfg.chunk, workspace=ws, reuse_fwd=True, out=grads)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    assert qd.workspace_status(ws) == 0, "device-side status word is set"

    # ---- timed region: K steps, CUDA events on the launching stream -------------------------------
    # The four kernels of a step are launched so that each may set itself up while the one before it drains
    # (programmatic dependent launch).  Events between the launches would serialise them again, so the per-kernel
    # durations behind `roofline` come from a second pass over the same K steps, right after the timed one.
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    qd.profile_enable(False)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    qd.profile_read(reset=True)
    qd.profile_enable(True)
    for _ in range(args.steps):
        step()
    barrier()
    qd.profile_enable(False)
    stages = qd.profile_read(reset=True)
    # the timed region lasts milliseconds, nvidia-smi answers in ~0.1 s: keep the same step loop running
    # (untimed) for a second or so, so that the clock samples are taken under this load
    t_probe = time.perf_counter()
    while time.perf_counter() - t_probe < 1.5:
        for _ in range(20):
            step()
        torch.cuda.synchronize()
    sampler.stop_flag.set()
    sampler.join()
    ms, tokens_total = sharding.aggregate(ms, B * T * args.steps, "cuda")   # slowest rank, all ranks' tokens
    ms_step = ms / args.steps
    tokens_step = tokens_total // args.steps
    value = sharding.throughput(tokens_total, ms)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ------------
    out_host = {"o": torch.empty_like(o, device="cpu").pin_memory(), "hT": torch.empty_like(hT, device="cpu").pin_memory()}
    for n, t in grads.items():
        out_host[n] = torch.empty_like(t, device="cpu").pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = sum(t.numel() * t.element_size() for t in out_host.values())

    # Three streams, two sets of device buffers: the upload of step i+1 and the download of step i-1 run while
    # step i computes (PCIe is full duplex).  Every step still uploads all of its inputs and downloads all of
    # its results inside the timed region.
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    dev2 = [dev, {n: torch.empty_like(t) for n, t in dev.items()}]
    o2, hT2, g2 = [o, torch.empty_like(o)], [hT, torch.empty_like(hT)], [grads, {}]
    qd.chunk_bwd(dev["q"], dev["k"], dev["v"], dev["beta"], dev["alpha"], dev["lam"], dev["h0"],
                 dev["dO"], dev["dhT"], chunk=cfg.chunk, workspace=ws, reuse_fwd=True, out=g2[1])   # allocate set 1
    torch.cuda.synchronize()
    ev = lambda: torch.cuda.Event()
    in_done, cmp_done, out_done = {}, {}, {}

    def e2e_step(i):
        k = i & 1
        with torch.cuda.stream(s_in):
            if i - 2 in cmp_done:
                s_in.wait_event(cmp_done[i - 2])          # the inputs of step i-2 are no longer needed
            for n, t in host.items():
                dev2[k][n].copy_(t, non_blocking=True)
            in_done[i] = ev(); in_done[i].record(s_in)
        with torch.cuda.stream(s_cmp):
            s_cmp.wait_event(in_done[i])
            if i - 2 in out_done:
                s_cmp.wait_event(out_done[i - 2])         # the results of step i-2 have left the device
            d = dev2[k]
            qd.chunk_fwd(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"],
                         chunk=cfg.chunk, save_for_bwd=True, workspace=ws, o=o2[k], hT=hT2[k])
            qd.chunk_bwd(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"],
                         d["dO"], d["dhT"], chunk=cfg.chunk, workspace=ws, reuse_fwd=True, out=g2[k])
            cmp_done[i] = ev(); cmp_done[i].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(cmp_done[i])
            out_host["o"].copy_(o2[k], non_blocking=True)
            out_host["hT"].copy_(hT2[k], non_blocking=True)
            for n, t in g2[k].items():
                out_host[n].copy_(t, non_blocking=True)
            out_done[i] = ev(); out_done[i].record(s_out)

    e2e_steps = 0 if args.no_extras else max(4, min(args.steps, 10))
    for i in range(2 if e2e_steps else 0):
        e2e_step(i)
    barrier()
    in_done.clear(); cmp_done.clear(); out_done.clear()
    e0.record(s_in)
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record(s_out)
    barrier()
    ems = e0.elapsed_time(e1) if e2e_steps else float("nan")
    ems, _ = sharding.aggregate(ems, 0, "cuda")
    e2e_value = tokens_step / (ems / e2e_steps * 1e-3) if e2e_steps else None

    # ---- roofline of the dominant kernel and of the whole path -----------------------------------
    pk, pk_kind = peaks()
    th = B * T * H                                     # token-heads one launch processes
    sb = stage_bytes_per_token_head(dk, dv, cfg.chunk)
    chunk_stages = {n: v for n, v in stages.items() if n in sb and v[1] > 0}
    dom = max(chunk_stages, key=lambda n: chunk_stages[n][0])
    dom_ms = chunk_stages[dom][0] / chunk_stages[dom][1]
    ach = sb[dom] * th / (dom_ms * 1e-3) / 1e9
    roofline = {"kernel": dom, "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": ach / pk["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES.get(cfg.name, {}).get(dom), "peak_kind": "of " + pk_kind,
                "ms_per_launch": dom_ms, "algorithmic_bytes_per_launch": sb[dom] * th}
    fb, bb = path_bytes_per_token_head(dk, dv)
    ff, fbw = path_flops_per_token_head(dk, dv, cfg.chunk)
    state_io = 4 * dk * dv * 4 * B * H
    t_bytes = ((fb + bb) * th + state_io) / (pk["hbm_gbs"] * 1e9)
    t_flops = (ff + fbw) * th / (pk["bf16_tflops"] * 1e12)
    per_rank_ms = ms_step
    path = {"bytes_per_step": (fb + bb) * th + state_io, "flops_per_step": (ff + fbw) * th,
            "roofline_ms": max(t_bytes, t_flops) * 1e3, "frac": max(t_bytes, t_flops) * 1e3 / per_rank_ms,
            "peak_kind": "of " + pk_kind,
            "roofline_ms_nominal": max(((fb + bb) * th + state_io) / 8.0e12, (ff + fbw) * th / 2.25e15) * 1e3,
            "frac_nominal": max(((fb + bb) * th + state_io) / 8.0e12, (ff + fbw) * th / 2.25e15) * 1e3 / per_rank_ms,
            "stage_ms_per_launch": {n: v[0] / v[1] for n, v in chunk_stages.items()}}
    launches = int(sum(v[1] for v in stages.values()))

    # ---- decode step (separate configuration), in place over a long run of steps ------------------
    decode = bench_decode(args, qd, gen, torch, pk, pk_kind) if (rank == 0 and not args.no_extras) else None

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "l2": "inputs larger than L2 (no flush)",
                       "clock_sampling": "nvidia-smi during the timed steps and 1.5 s more of the same step loop",
                       "kernel_timing": "per-kernel CUDA events in a second pass over the same K steps (events between "
                                        "launches would serialise the overlapped launches of the timed pass)",
                       "tokens_per_step": tokens_step, "parallelism": "batch sharded over %d rank(s), no collective" % world},
            "clocks": sampler.summary(),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "pipelining": "upload, compute and download of consecutive steps overlap on three streams"},
            "gpu_launches": launches, "roofline": roofline, "roofline_path": path, "decode": decode}
    if rank == 0:
        if world == 1 and not args.no_extras:
            cores = os.cpu_count() or 1
            nseq = max(1, min(B * H, 8 * cores))
            reps = 4
            v, dt, thr = oracle_sample(cfg, nseq, steps=reps)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": thr, "kind": "oracle",
                                    "sample": "first %d of %d (batch, head) sequences, fwd + reverse pass, fp64, %d passes of %.1f s"
                                              % (nseq, B * H, reps, dt)}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def bench_decode(args, qd, gen, torch, pk, pk_kind):
    cfg = gen.CONFIGS["cfg4"]
    bf = torch.bfloat16
    state = torch.from_numpy(gen.make_decode_state(cfg)).cuda()
    pool = 8
    tok = gen.make_decode_tokens(cfg, 0, pool)
    tok = {n: torch.from_numpy(a).to("cuda", bf) for n, a in tok.items()}
    o = torch.empty((cfg.B, cfg.H, cfg.dv), dtype=bf, device="cuda")
    nsteps = args.decode_steps

    def one(i):
        j = i % pool
        qd.recurrent_step(tok["q"][j], tok["k"][j], tok["v"][j], tok["beta"][j], tok["alpha"][j], tok["lam"][j],
                          state, o)
    for i in range(10):
        one(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(nsteps):
        one(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / nsteps
    nstates = cfg.B * cfg.H
    bytes_step = nstates * (2 * cfg.dk * cfg.dv * 4 + 2 * (2 * cfg.dk + cfg.dv) + 6 + 2 * cfg.dv)
    gbs = bytes_step / (ms * 1e-3) / 1e9
    return {"workload": "cfg4: batch=%d H=%d dk=%d dv=%d fp32 state in place, bf16 tokens" % (cfg.B, cfg.H, cfg.dk, cfg.dv),
            "steps": nsteps, "us_per_step": ms * 1e3, "tokens_per_s": cfg.B / (ms * 1e-3),
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / pk["hbm_gbs"], "peak_kind": "of " + pk_kind,
                         "algorithmic_bytes_per_launch": bytes_step, "state_larger_than_l2": True}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--only", default="all", choices=["all", "decode"],
                    help="'decode': time only the decode step (small runs for profiler captures)")
    ap.add_argument("--decode-steps", type=int, default=200)
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg3", "small"],
                    help="cfg2: headline (default); cfg3: long context; small: B=2 of cfg2 for profiler captures")
    ap.add_argument("--no-extras", action="store_true", help="skip the end-to-end, decode and CPU-baseline legs")
    args = ap.parse_args()
    from paper_2606_08804_b200 import inputs as gen
    cfg = gen.CONFIGS["cfg3" if args.workload == "cfg3" else "cfg2"]
    if args.workload == "small":
        cfg = replace(cfg, B=2)
    if args.only == "decode":
        import torch
        from paper_2606_08804_b200 import binding as qd
        pk, pk_kind = peaks()
        print(json.dumps({"decode": bench_decode(args, qd, gen, torch, pk, pk_kind)}))
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
