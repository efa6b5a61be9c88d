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


# dram__bytes_read.sum + dram__bytes_write.sum of one launch: NOT measured by this run (a profiler cannot run inside the
# timed program); constants from the ncu capture summarised in profiles/tc_kernels_fullsize_counters_cfg2.md (full-size
# cfg2).  Other workloads: not captured.
NCU_TRAFFIC_BYTES = {"cfg2": {"prep": 421.7e6, "chain_fwd": 532.6e6, "chain_bwd": 470.2e6, "chunk_bwd": 922.1e6}}
NCU_TRAFFIC_SOURCE = "constant from profiles/tc_kernels_fullsize_counters_cfg2.md (ncu, one launch each); not measured by this run"
# which pass of the path a kernel belongs to (its share of the algorithmic bytes of SURVEY section 8(d))
STAGE_PASS = {"prep": "fwd", "chain_fwd": "fwd", "chain_bwd": "bwd", "chunk_bwd": "bwd"}


def path_roofline(cfg, pk, fwd=True, bwd=True):
    """Roofline time of the path on one GPU: max(algorithmic bytes / HBM, algorithmic FLOPs / bf16 peak), both for the
    measured peaks of this machine and for the nominal 8 TB/s and 2.25 PFLOP/s."""
    th = cfg.B * cfg.T * cfg.H
    fb, bb = path_bytes_per_token_head(cfg.dk, cfg.dv)
    ff, fbw = path_flops_per_token_head(cfg.dk, cfg.dv, cfg.chunk)
    nstates = (2 if fwd else 0) + (2 if bwd else 0)            # h0, hT / dhT, dh0: fp32 [dk x dv] per sequence
    nbytes = ((fb if fwd else 0) + (bb if bwd else 0)) * th + nstates * cfg.dk * cfg.dv * 4 * cfg.B * cfg.H
    flops = ((ff if fwd else 0) + (fbw if bwd else 0)) * th
    t_meas = max(nbytes / (pk["hbm_gbs"] * 1e9), flops / (pk["bf16_tflops"] * 1e12))
    t_nom = max(nbytes / 8.0e12, flops / 2.25e15)
    return {"bytes_per_step": nbytes, "flops_per_step": flops, "roofline_ms": t_meas * 1e3, "roofline_ms_nominal": t_nom * 1e3,
            "bound": "hbm" if nbytes / (pk["hbm_gbs"] * 1e9) >= flops / (pk["bf16_tflops"] * 1e12) else "tensor"}


def region_stats(times_ms, steps, mhz):
    """Median / min / max of repeated K-step regions (ms per step) and the clock-normalised figure."""
    per = sorted(t / steps for t in times_ms)
    med = per[len(per) // 2]
    out = {"regions": len(per), "steps_per_region": steps, "ms_per_step_median": med, "ms_per_step_min": per[0],
           "ms_per_step_max": per[-1], "spread": (per[-1] - per[0]) / med}
    if mhz:
        out["ms_x_mhz_median"] = med * mhz          # time x median SM clock: compares runs taken at different clocks
    return out


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


def workload_name(cfg, backward=True):
    return "%s: bf16 %s B=%d H=%d T=%d dk=%d dv=%d chunk=%d" % (cfg.name, "fwd+bwd" if backward else "fwd", cfg.B, cfg.H, cfg.T,
                                                                 cfg.dk, cfg.dv, cfg.chunk)


class Workload:
    """Device-resident inputs, outputs and workspace of one chunkwise configuration, and its step."""

    def __init__(self, torch, qd, gen, cfg, seed, backward=True, drop=(), fused=False):
        d = gen.make_chunk_inputs(cfg, seed=seed)
        bf = torch.bfloat16
        self.host, self.dev = {}, {}
        for n in ("q", "k", "v", "beta", "alpha", "lam", "dO"):
            if d.get(n) is not None:
                self.host[n] = torch.from_numpy(d[n]).to(bf).pin_memory()
        for n in ("h0", "dhT"):
            if d.get(n) is not None:
                self.host[n] = torch.from_numpy(d[n]).pin_memory()
        for n, t in self.host.items():
            self.dev[n] = t.to("cuda", non_blocking=True)
        for n in ("q", "k", "v", "beta", "alpha", "lam", "dO", "h0", "dhT"):
            self.dev.setdefault(n, None)
        for n in drop:                                  # variant runs: the optional input is absent (NULL)
            self.dev[n] = None
        self.cfg, self.qd, self.backward = cfg, qd, backward
        # fused=True: the same tensors read as un-normalised q, k and as gate logits (in-kernel L2 normalisation and
        # sigmoid); the values differ from the plain run, the work per token does not
        self.kw = dict(logits=True, norm_qk=True) if fused else {}
        B, T, H, dk, dv = cfg.B, cfg.T, cfg.H, cfg.dk, cfg.dv
        self.shape = qd.make_shape(self.dev["q"], self.dev["v"], cfg.chunk)
        self.ws = qd.alloc_workspace(self.shape, backward, "cuda")
        self.o = torch.empty((B, T, H, dv), dtype=bf, device="cuda")
        self.hT = torch.empty((B, H, dk, dv), dtype=torch.float32, device="cuda")
        self.grads = {}

    def step(self):
        d, qd, cfg = self.dev, self.qd, self.cfg
        qd.chunk_fwd(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"], chunk=cfg.chunk,
                     save_for_bwd=self.backward, workspace=self.ws, o=self.o, hT=self.hT, **self.kw)
        if self.backward:
            qd.chunk_bwd(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"], d["dO"], d["dhT"],
                         chunk=cfg.chunk, workspace=self.ws, reuse_fwd=True, out=self.grads, **self.kw)


def time_regions(torch, step, steps, regions, barrier):
    """`regions` back-to-back regions of exactly `steps` steps, each bracketed by CUDA events on the launching stream."""
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(regions)]
    barrier()
    for e0, e1 in evs:
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
    barrier()
    return [e0.elapsed_time(e1) for e0, e1 in evs]


def extra_workload(torch, qd, gen, cfg, pk, pk_kind, backward, steps, regions, drop=(), fused=False):
    """A further configuration timed like the headline one (rank 0, one GPU): ms per step, tokens/s, roofline fraction."""
    w = Workload(torch, qd, gen, cfg, cfg.seed, backward=backward, drop=drop, fused=fused)
    for _ in range(3):
        w.step()
    torch.cuda.synchronize()
    assert qd.workspace_status(w.ws) == 0, "device-side status word is set"
    times = time_regions(torch, w.step, steps, regions, torch.cuda.synchronize)
    st = region_stats(times, steps, None)
    qd.profile_read(reset=True)
    qd.profile_enable(True)                 # per-kernel durations, in a pass of their own (they serialise the launches)
    for _ in range(min(steps, 5)):
        w.step()
    torch.cuda.synchronize()
    qd.profile_enable(False)
    stage_ms = {n: v[0] / v[1] for n, v in qd.profile_read(reset=True).items() if v[1] > 0}
    rl = path_roofline(cfg, pk, fwd=True, bwd=backward)
    ms = st["ms_per_step_median"]
    out = {"workload": workload_name(cfg, backward), "ms_per_step": ms, "tokens_per_s": cfg.B * cfg.T / (ms * 1e-3),
           "roofline_ms": rl["roofline_ms"], "frac": rl["roofline_ms"] / ms, "frac_nominal": rl["roofline_ms_nominal"] / ms,
           "peak_kind": "of " + pk_kind, "regions": st, "stage_ms_per_launch": stage_ms}
    if drop:
        out["absent_inputs"] = list(drop)
    del w
    torch.cuda.empty_cache()
    return out


def torch_preprocessing_ms(torch, gen, cfg, steps=10):
    """What the stages QD_NORM_QK | QD_COEF_LOGITS fuse cost when a caller runs them as separate PyTorch operations around
    the plain call: forward (normalise q and k, three sigmoids) and backward (through the normalisation and the
    sigmoids), bf16 tensors of the same shape.  Context for `fused_preprocessing`, not part of the library."""
    bf = torch.bfloat16
    B, T, H, dk = cfg.B, cfg.T, cfg.H, cfg.dk
    g = torch.Generator(device="cuda").manual_seed(0)
    q, k, dqh, dkh = (torch.randn((B, T, H, dk), device="cuda", generator=g).to(bf) for _ in range(4))
    zb, za, zl, db, da, dl = (torch.randn((B, T, H), device="cuda", generator=g).to(bf) for _ in range(6))

    def step():
        outs = []
        for x, dxh in ((q, dqh), (k, dkh)):
            xf = x.float()
            r = torch.rsqrt((xf * xf).sum(-1, keepdim=True) + 1e-6)
            xh = xf * r
            outs.append(xh.to(bf))                                   # forward: the normalised rows the kernel is given
            d = dxh.float()
            outs.append((r * (d - xh * (xh * d).sum(-1, keepdim=True))).to(bf))   # backward through the normalisation
        for z, dgate in ((zb, db), (za, da), (zl, dl)):
            s_ = torch.sigmoid(z.float())
            outs.append(s_.to(bf))
            outs.append(dgate.float() * s_ * (1 - s_))
        return outs
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


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
    w = Workload(torch, qd, gen, cfg, sharding.rank_seed(cfg.seed, rank), backward=True)
    host, dev, ws, o, hT, grads, step = w.host, w.dev, w.ws, w.o, w.hT, w.grads, w.step
    B, T, H, dk, dv = cfg.B, cfg.T, cfg.H, cfg.dk, cfg.dv
    assert qd.chunk_path(w.shape) == "tensor_core"
    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    barrier()
    assert qd.workspace_status(ws) == 0, "device-side status word is set"

    # ---- timed regions: each is exactly K steps between two CUDA events on the launching stream; `regions` of them
    # run back to back so that the figure is the sustained one (power cap, clocks settled), the median is reported.
    # The four kernels of a step are launched so that each may set itself up while the one before it drains; events
    # between the launches would serialise them, so the per-kernel durations come from a separate pass afterwards.
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    qd.profile_enable(False)
    times = time_regions(torch, step, args.steps, max(1, args.regions), barrier)
    qd.profile_read(reset=True)
    qd.profile_enable(True)
    for _ in range(args.steps):
        step()
    barrier()
    qd.profile_enable(False)
    stages = qd.profile_read(reset=True)
    # nvidia-smi answers in ~0.1 s: keep the same step loop running (untimed) a little longer so that enough clock
    # samples are taken under this load
    t_probe = time.perf_counter()
    while not args.no_clock_probe and time.perf_counter() - t_probe < 1.0:
        for _ in range(20):
            step()
        torch.cuda.synchronize()
    sampler.stop_flag.set()
    sampler.join()
    clocks = sampler.summary()
    med_ms = sorted(times)[len(times) // 2]
    ms, tokens_total = sharding.aggregate(med_ms, B * T * args.steps, "cuda")   # slowest rank, all ranks' tokens
    ms_step = ms / args.steps
    tokens_step = tokens_total // args.steps
    value = sharding.throughput(tokens_total, ms)
    regions = region_stats(times, args.steps, clocks.get("sm_mhz"))

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
    e2e_steps = 0 if args.no_extras else max(4, min(args.steps, 10))
    e2e_value = None
    if e2e_steps:
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

        for i in range(2):
            e2e_step(i)
        barrier()
        in_done.clear(); cmp_done.clear(); out_done.clear()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s_in)
        for i in range(e2e_steps):
            e2e_step(i)
        e1.record(s_out)
        barrier()
        ems = e0.elapsed_time(e1)
        ems, _ = sharding.aggregate(ems, 0, "cuda")
        e2e_value = tokens_step / (ems / e2e_steps * 1e-3)
        del dev2, o2, hT2, g2

    # ---- roofline: the whole path (what the target is stated on) and the dominant kernel ----------------------
    pk, pk_kind = peaks()
    th = B * T * H                                     # token-heads one launch processes
    rl = path_roofline(cfg, pk)
    chunk_stages = {n: v for n, v in stages.items() if n in STAGE_PASS and v[1] > 0}
    stage_ms = {n: v[0] / v[1] for n, v in chunk_stages.items()}
    path = dict(rl, frac=rl["roofline_ms"] / ms_step, frac_nominal=rl["roofline_ms_nominal"] / ms_step,
                peak_kind="of " + pk_kind, stage_ms_per_launch=stage_ms,
                note="whole fwd+bwd step against max(algorithmic bytes / HBM, algorithmic FLOPs / bf16 peak); "
                     "target 0.50")
    dom = max(stage_ms, key=lambda n: stage_ms[n])
    fb, bb = path_bytes_per_token_head(dk, dv)
    # algorithmic bytes of the pass the dominant kernel belongs to (forward 1030 B, backward 1810 B per token-head at
    # d = 128, plus that pass's two fp32 states per sequence); the kernels of a pass share them, so each kernel's
    # fraction is an upper bound on what the pass reaches
    pass_bytes = (fb if STAGE_PASS[dom] == "fwd" else bb) * th + 2 * dk * dv * 4 * B * H
    ach = pass_bytes / (stage_ms[dom] * 1e-3) / 1e9
    sb = stage_bytes_per_token_head(dk, dv, cfg.chunk)
    roofline = {"kernel": dom, "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": ach / pk["hbm_gbs"], "peak_kind": "of " + pk_kind, "ms_per_launch": stage_ms[dom],
                "algorithmic_bytes_per_launch": pass_bytes,
                "algorithmic_bytes_are": "the %s pass's bytes of the path (inputs read once, outputs written once), not "
                                         "the intermediates this decomposition stages" % STAGE_PASS[dom],
                "traffic": NCU_TRAFFIC_BYTES.get(cfg.name, {}).get(dom),
                "traffic_source": NCU_TRAFFIC_SOURCE if cfg.name in NCU_TRAFFIC_BYTES else None,
                # what this kernel would take if it moved only its own staged bytes at the HBM peak
                "stage_floor": {n: {"bytes_per_launch": sb[n] * th, "ms_at_peak": sb[n] * th / (pk["hbm_gbs"] * 1e6),
                                    "achieved_gbs_of_staged_bytes": sb[n] * th / (stage_ms[n] * 1e-3) / 1e9}
                                for n in stage_ms}}
    launches = int(sum(v[1] for v in stages.values()))

    extras = {}
    if rank == 0 and world == 1 and not args.no_extras:
        del w, host, dev, ws, o, hT, grads, out_host
        torch.cuda.empty_cache()
        # forward only at the headline shape (configuration 1) and the long-context configuration 3
        extras["forward_only"] = extra_workload(torch, qd, gen, gen.CONFIGS["cfg1"], pk, pk_kind, False, 20, 5)
        if cfg.name != "cfg3":
            extras["long_context"] = extra_workload(torch, qd, gen, gen.CONFIGS["cfg3"], pk, pk_kind, True, 5, 5)
        # the update rule's special cases as absent inputs: lambda = NULL is the gated delta rule (Eq. 3), alpha = NULL
        # drops the forget gate, both together give DeltaNet (Eq. 2)
        base = ms_step
        var = {}
        for name, drop in (("lambda_absent", ("lam",)), ("alpha_absent", ("alpha",)), ("both_absent", ("lam", "alpha"))):
            r = extra_workload(torch, qd, gen, cfg, pk, pk_kind, True, 20, 3, drop=drop)
            var[name] = {"ms_per_step": r["ms_per_step"], "speedup_vs_full_rule": base / r["ms_per_step"],
                         "stage_ms_per_launch": r["stage_ms_per_launch"]}
        extras["variants"] = var
        # pre-processing fused into the kernels: L2 normalisation of q, k and sigmoid gates (with their backward)
        r = extra_workload(torch, qd, gen, cfg, pk, pk_kind, True, 20, 3, fused=True)
        extras["fused_preprocessing"] = {"flags": "QD_NORM_QK | QD_COEF_LOGITS", "ms_per_step": r["ms_per_step"],
                                         "overhead_ms_vs_plain": r["ms_per_step"] - base,
                                         "stage_ms_per_launch": r["stage_ms_per_launch"],
                                         "same_stages_as_torch_ops_ms": torch_preprocessing_ms(torch, gen, cfg)}

    # ---- decode step (separate configuration), in place over a long run of steps ------------------
    decode = bench_decode(args, qd, gen, torch, pk, pk_kind) if (rank == 0 and not args.no_extras) else None

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "l2": "inputs larger than L2 (no flush)",
                       "timing": "median of %d back-to-back regions of exactly %d steps, CUDA events on the launching "
                                 "stream, max over ranks" % (len(times), args.steps),
                       "clock_sampling": "nvidia-smi during the timed regions and 1 s more of the same step loop",
                       "kernel_timing": "per-kernel CUDA events in a separate pass over K steps (events between "
                                        "launches would serialise the overlapped launches of the timed regions)",
                       "tokens_per_step": tokens_step, "parallelism": "batch sharded over %d rank(s), no collective" % world},
            "clocks": clocks, "regions": regions,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "pipelining": "upload, compute and download of consecutive steps overlap on three streams"},
            "gpu_launches": launches, "roofline": roofline, "roofline_path": path,
            "decode": decode}
    line.update(extras)
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
    # multi-token step (S tokens per call share one read and one write of the state)
    multi = {}
    for S in (2, 4, 8):
        tk = gen.make_decode_tokens(cfg, 100, S)
        tk = {n: torch.from_numpy(np.ascontiguousarray(np.moveaxis(a, 0, 1))).to("cuda", bf) for n, a in tk.items()}
        oS = torch.empty((cfg.B, S, cfg.H, cfg.dv), dtype=bf, device="cuda")
        calls = max(50, nsteps // S)
        for _ in range(5):
            qd.recurrent_steps(tk["q"], tk["k"], tk["v"], tk["beta"], tk["alpha"], tk["lam"], state, oS)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(calls):
            qd.recurrent_steps(tk["q"], tk["k"], tk["v"], tk["beta"], tk["alpha"], tk["lam"], state, oS)
        e1.record()
        torch.cuda.synchronize()
        msS = e0.elapsed_time(e1) / calls
        bytesS = nstates * (2 * cfg.dk * cfg.dv * 4 + S * (2 * (2 * cfg.dk + cfg.dv) + 6 + 2 * cfg.dv))
        multi["S=%d" % S] = {"us_per_call": msS * 1e3, "tokens_per_s": cfg.B * S / (msS * 1e-3),
                             "achieved_gbs": bytesS / (msS * 1e-3) / 1e9, "frac": bytesS / (msS * 1e-3) / 1e9 / pk["hbm_gbs"]}
    # reduced-precision option: the same step with the state stored in bf16 (QD_STATE_BF16), one token per call
    st16 = state.to(bf)
    tk1 = {n: t[:, :1].contiguous() for n, t in tk.items()}          # one token of the last multi-token set
    o1 = torch.empty((cfg.B, 1, cfg.H, cfg.dv), dtype=bf, device="cuda")
    for _ in range(5):
        qd.recurrent_steps(tk1["q"], tk1["k"], tk1["v"], tk1["beta"], tk1["alpha"], tk1["lam"], st16, o1)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(nsteps):
        qd.recurrent_steps(tk1["q"], tk1["k"], tk1["v"], tk1["beta"], tk1["alpha"], tk1["lam"], st16, o1)
    e1.record()
    torch.cuda.synchronize()
    ms16 = e0.elapsed_time(e1) / nsteps
    bytes16 = nstates * (2 * cfg.dk * cfg.dv * 2 + 2 * (2 * cfg.dk + cfg.dv) + 6 + 2 * cfg.dv)
    bf16_state = {"us_per_step": ms16 * 1e3, "tokens_per_s": cfg.B / (ms16 * 1e-3), "achieved_gbs": bytes16 / (ms16 * 1e-3) / 1e9,
                  "frac": bytes16 / (ms16 * 1e-3) / 1e9 / pk["hbm_gbs"],
                  "note": "reduced-precision OPTION (state rounded to bf16 once per call); not the configuration's fp32 state"}
    del st16
    # the same loop replayed from one CUDA graph of `pool` steps (no per-step launch cost on the host)
    graph_us = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(pool):
                one(i)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(pool):
                one(i)
        reps = max(1, nsteps // pool)
        g.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        graph_us = e0.elapsed_time(e1) / (reps * pool) * 1e3
    except Exception as exc:                         # graph capture is a convenience of the harness, not of the library
        graph_us = "unavailable: %s" % type(exc).__name__
    return {"workload": "cfg4: batch=%d H=%d dk=%d dv=%d fp32 state in place, bf16 tokens" % (cfg.B, cfg.H, cfg.dk, cfg.dv),
            "steps": nsteps, "us_per_step": ms * 1e3, "tokens_per_s": cfg.B / (ms * 1e-3), "multi_token": multi,
            "us_per_step_cuda_graph": graph_us, "bf16_state_option": bf16_state,
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
    ap.add_argument("--regions", type=int, default=21,
                    help="how many back-to-back regions of --steps steps are timed (the median is reported)")
    ap.add_argument("--decode-steps", type=int, default=1000, help="configuration 4 runs 1000 sequential steps")
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg3", "small"],
                    help="cfg2: headline (default); cfg3: long context; small: B=2 of cfg2 for profiler captures")
    ap.add_argument("--no-extras", action="store_true", help="skip the end-to-end, decode and CPU-baseline legs")
    ap.add_argument("--no-clock-probe", action="store_true",
                    help="do not keep the step loop running for clock samples (short runs for profiler captures)")
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
