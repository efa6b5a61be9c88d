"""GPU-vs-oracle parity of the chunkwise forward and backward (through the C ABI)."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2606_08804_b200 import inputs as gen
import gpu_util as gu

pytestmark = pytest.mark.gpu


def _label(cfg, extra=""):
    return "%s/%s B%d T%d H%d dk%d dv%d %s%s" % (cfg.name, cfg.regime, cfg.B, cfg.T, cfg.H, cfg.dk, cfg.dv, cfg.dtype, extra)


def _fwd_check(cfg, d=None, pairs=None, check_status=True, save=False):
    """Forward through the C ABI against the oracle: `pairs` = the (b, h) sequences the oracle computes (all if None).
    Every sequence is checked for finite values.  save=True runs the call that also keeps what the backward needs."""
    from paper_2606_08804_b200 import binding as qd
    d = gen.make_chunk_inputs(cfg) if d is None else d
    t = gu.dev_inputs(d, cfg.dtype)
    o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], chunk=cfg.chunk,
                             save_for_bwd=save)
    torch.cuda.synchronize()
    if check_status:
        assert qd.workspace_status(ws) == 0
    assert gu.all_finite(o, hT), "non-finite forward output"
    lab = _label(cfg, " save" if save else "")
    if pairs is None:
        ro, rh = gu.oracle_fwd(d)
        eo, eh = gu.check(lab, "o", o, ro, cfg.dtype), gu.check(lab, "hT", hT, rh, cfg.dtype, state=True)
    else:
        ro, rh = gu.oracle_fwd(gu.pick_sequences(d, pairs))
        eo = gu.check(lab, "o", gu.pick_result(o, pairs), ro, cfg.dtype)
        eh = gu.check(lab, "hT", gu.pick_result(hT, pairs, True), rh, cfg.dtype, state=True)
    return eo, eh


def _bwd_check(cfg, d=None, pairs=None, reuse=False, only=None):
    from paper_2606_08804_b200 import binding as qd
    d = gen.make_chunk_inputs(cfg) if d is None else d
    t = gu.dev_inputs(d, cfg.dtype)
    ws = None
    if reuse:
        o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"],
                                 chunk=cfg.chunk, save_for_bwd=True)
    g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"],
                     chunk=cfg.chunk, workspace=ws, reuse_fwd=reuse)
    torch.cuda.synchronize()
    assert gu.all_finite(*g.values()), "non-finite gradient"
    sub = d if pairs is None else gu.pick_sequences(d, pairs)
    ref = gu.oracle_bwd(sub)
    lab = _label(cfg, " reuse" if reuse else " recompute")
    errs = {}
    for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0"):
        if g.get(n) is None or (only and n not in only):
            continue
        got = g[n] if pairs is None else gu.pick_result(g[n], pairs, n == "dh0")
        errs[n] = gu.check(lab, n, got, ref[n], cfg.dtype, state=(n == "dh0"))
    return errs


def test_cfg0_tiny_fp32_forward():
    _fwd_check(gen.CONFIGS["cfg0"])


@pytest.mark.parametrize("regime", gen.REGIMES)
def test_small_fp32_forward_backward_regimes(regime):
    cfg = replace(gen.CONFIGS["cfg0"], B=2, H=2, T=192, h0=True, backward=True, regime=regime, seed=3)
    _fwd_check(cfg)
    _bwd_check(cfg)


@pytest.mark.parametrize("regime", gen.REGIMES)
def test_small_bf16_forward_backward_regimes(regime):
    cfg = replace(gen.CONFIGS["cfg2"], B=2, H=3, T=320, regime=regime, seed=5)
    _fwd_check(cfg)
    _bwd_check(cfg)
    _bwd_check(cfg, reuse=True)


def test_mixed_head_dims_fp32():
    cfg = replace(gen.CONFIGS["cfg0"], B=1, H=2, T=128, dk=128, dv=64, h0=True, backward=True, seed=7)
    _fwd_check(cfg)
    _bwd_check(cfg)
    cfg = replace(cfg, dk=64, dv=128)
    _fwd_check(cfg)
    _bwd_check(cfg)


def test_single_chunk_and_optional_inputs():
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg2"], B=1, H=2, T=64, seed=9)
    d = gen.make_chunk_inputs(cfg)
    _fwd_check(cfg, d)
    _bwd_check(cfg, d)
    # alpha = lambda = h0 = dhT = NULL
    d2 = dict(d, alpha=None, lam=None, h0=None, dhT=None)
    t = gu.dev_inputs(d2, cfg.dtype)
    o, hT, _ = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"])
    ro, rh = gu.oracle_fwd(d2)
    assert gu.rel_err(o, ro) <= 2e-2 and gu.rel_err(hT, rh) <= 2e-2
    g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], None, None, None, t["dO"], None)
    ref = gu.oracle_bwd(d2)
    for n in ("dq", "dk", "dv", "dbeta", "dh0"):
        assert gu.rel_err(g[n], ref[n]) <= 2e-2, n
    assert g["dalpha"] is None and g["dlam"] is None


def test_segment_invariance_on_gpu():
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg1"], B=1, H=2, T=256, regime="alpha_slow", seed=11)
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    o, hT, _ = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"])
    c = lambda x, s: x[:, s].contiguous()
    a, b = slice(0, 128), slice(128, 256)
    o1, h1, _ = qd.chunk_fwd(c(t["q"], a), c(t["k"], a), c(t["v"], a), c(t["beta"], a), c(t["alpha"], a),
                             c(t["lam"], a), t["h0"])
    o2, h2, _ = qd.chunk_fwd(c(t["q"], b), c(t["k"], b), c(t["v"], b), c(t["beta"], b), c(t["alpha"], b),
                             c(t["lam"], b), h1)
    torch.cuda.synchronize()
    assert torch.equal(torch.cat([o1, o2], dim=1), o)
    assert torch.equal(h2, hT)


def test_deterministic_bitwise():
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg2"], B=2, H=2, T=256, seed=13)
    t = gu.dev_inputs(gen.make_chunk_inputs(cfg), cfg.dtype)
    runs = []
    for _ in range(2):
        o, hT, _ = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"])
        g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"])
        torch.cuda.synchronize()
        runs.append([o, hT] + [g[n] for n in sorted(g)])
    for x, y in zip(*runs):
        assert torch.equal(x, y)


def _sample_pairs(cfg, n, seed=0):
    r = np.random.default_rng(seed)
    idx = r.choice(cfg.B * cfg.H, size=min(n, cfg.B * cfg.H), replace=False)
    return [(int(i) // cfg.H, int(i) % cfg.H) for i in idx]


def test_cfg1_cfg2_full_size():
    # config 1 (forward) and config 2 (forward + backward) share inputs; every sequence is run on the
    # GPU in the benchmarked launch configuration, the oracle checks a sample of whole sequences
    cfg = gen.CONFIGS["cfg2"]
    d = gen.make_chunk_inputs(cfg)
    # forward: the oracle checks every one of the 128 sequences, for the plain call and for the saving call the
    # benchmark times; reverse pass: a sample of 16 whole sequences (all sequences are checked for finite values)
    _fwd_check(cfg, d)
    _fwd_check(cfg, d, _sample_pairs(cfg, 32, seed=1), save=True)
    _bwd_check(cfg, d, _sample_pairs(cfg, 16), reuse=True)


def test_cfg3_long_context_full_size():
    cfg = gen.CONFIGS["cfg3"]
    d = gen.make_chunk_inputs(cfg)
    pairs = _sample_pairs(cfg, 4)
    _fwd_check(cfg, d, _sample_pairs(cfg, 8, seed=1))
    _fwd_check(cfg, d, pairs, save=True)
    _bwd_check(cfg, d, pairs, reuse=True)


@pytest.mark.parametrize("regime", gen.REGIMES)
def test_tensor_core_forward_regimes(regime):
    # bf16, d = 128, T a multiple of 128: the tcgen05 kernels run the forward
    cfg = replace(gen.CONFIGS["cfg2"], B=2, H=3, T=384, regime=regime, seed=17)
    _fwd_check(cfg)
    _bwd_check(cfg)
    _bwd_check(cfg, reuse=True)


def test_tensor_core_forward_single_pair_no_h0():
    cfg = replace(gen.CONFIGS["cfg1"], B=1, H=1, T=128, h0=False, seed=19)
    _fwd_check(cfg)


def test_tensor_core_optional_inputs_absent():
    # bf16, d = 128, T a multiple of 128 (the tcgen05 kernels) with alpha = lambda = h0 = dhT = NULL, each alone and
    # all together; backward both with its own forward recomputation and on the forward's saved workspace
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg2"], B=2, H=2, T=256, seed=23)
    d = gen.make_chunk_inputs(cfg)
    variants = [dict(alpha=None), dict(lam=None), dict(h0=None), dict(dhT=None),
                dict(alpha=None, lam=None, h0=None, dhT=None)]
    for drop in variants:
        d2 = dict(d, **drop)
        t = gu.dev_inputs(d2, cfg.dtype)
        ro, rh = gu.oracle_fwd(d2)
        ref = gu.oracle_bwd(d2)
        for reuse in (False, True):
            o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], save_for_bwd=reuse)
            g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"],
                             workspace=ws if reuse else None, reuse_fwd=reuse)
            torch.cuda.synchronize()
            assert qd.workspace_status(ws) == 0
            assert gu.rel_err(o, ro) <= 2e-2 and gu.rel_err(hT, rh) <= 2e-2, drop
            for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0"):
                if g.get(n) is None:            # d alpha / d lambda of an absent input
                    continue
                assert gu.rel_err(g[n], ref[n]) <= 2e-2, (drop, reuse, n)
            assert (g["dalpha"] is None) == (d2["alpha"] is None) and (g["dlam"] is None) == (d2["lam"] is None)


def test_back_to_back_launches_without_host_sync():
    # The kernels of a step are launched so that each may begin while its predecessor drains.  Many steps in a row on
    # one workspace, no host synchronisation in between, alternating two input sets: every step's results must equal
    # the results of the same step run alone.
    from paper_2606_08804_b200 import binding as qd
    cfgs = [replace(gen.CONFIGS["cfg2"], B=2, H=3, T=384, seed=s) for s in (31, 32)]
    ts = [gu.dev_inputs(gen.make_chunk_inputs(c), c.dtype) for c in cfgs]

    def run(t, ws=None, out=None):
        o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], save_for_bwd=True,
                                 workspace=ws)
        g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"],
                         workspace=ws, reuse_fwd=True, out=out)
        return o, hT, g, ws

    alone = []
    for t in ts:
        o, hT, g, _ = run(t)
        torch.cuda.synchronize()
        alone.append([o.clone(), hT.clone()] + [g[n].clone() for n in sorted(g)])
    ws = qd.alloc_workspace(qd.make_shape(ts[0]["q"], ts[0]["v"], 64), True, "cuda")
    got = []
    for i in range(12):
        o, hT, g, _ = run(ts[i & 1], ws)
        got.append([o, hT] + [g[n] for n in sorted(g)])
    torch.cuda.synchronize()
    assert qd.workspace_status(ws) == 0
    for i, res in enumerate(got):
        for x, y in zip(res, alone[i & 1]):
            assert torch.equal(x, y), i


def test_more_chains_than_sms():
    # 256 (batch, head) chains -- the paper's (2048, 16) training batch has 16 x 16 of them -- so the chain kernels run
    # a second wave of CTAs while their neighbours' launches overlap; every sequence is checked by the oracle
    cfg = replace(gen.CONFIGS["cfg2"], B=16, H=16, T=256, seed=41)
    d = gen.make_chunk_inputs(cfg)
    _fwd_check(cfg, d)
    _bwd_check(cfg, d)
    _bwd_check(cfg, d, reuse=True)


@pytest.mark.parametrize("T", [1000, 320, 64, 37, 129])
def test_ragged_sequence_length_tensor_core(T):
    # T not a multiple of the chunk (or of the chunk pair the preparation kernel takes): bf16, d = 128 stays on the
    # tcgen05 kernels; outputs beyond T do not exist, and a guard band behind every output shows that nothing is written there
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg2"], B=2, H=2, T=T, regime="alpha_slow", seed=43 + T)
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    assert qd.chunk_path(qd.make_shape(t["q"], t["v"], 64)) == "tensor_core"
    _fwd_check(cfg, d)
    _bwd_check(cfg, d)
    _bwd_check(cfg, d, reuse=True)


@pytest.mark.parametrize("T", [200, 50])
def test_ragged_sequence_length_fp32(T):
    cfg = replace(gen.CONFIGS["cfg0"], B=2, H=2, T=T, h0=True, backward=True, regime="alpha_slow", seed=47 + T)
    _fwd_check(cfg)
    _bwd_check(cfg)


def test_fp32_long_sequence_holds_the_fp32_bar():
    # the 1e-4 bar at a length where the carried state has gone through 128 chunks
    cfg = replace(gen.CONFIGS["cfg0"], B=1, H=2, T=8192, h0=True, backward=True, regime="alpha_slow", seed=53)
    _fwd_check(cfg)
    _bwd_check(cfg)


@pytest.mark.parametrize("regime", ["trained_like", "alpha_slow"])
def test_decay_gradient_long_slow_decay(regime):
    # d alpha = d log alpha / alpha is the heavy-tailed gradient; slow decay keeps the whole history alive
    cfg = replace(gen.CONFIGS["cfg2"], B=1, H=4, T=2048, regime=regime, seed=59)
    _bwd_check(cfg, reuse=True)


def test_backward_right_behind_the_kernels_that_write_its_inputs():
    # dO and dhT are produced by other kernels on the same stream immediately before a backward that reuses the
    # forward's workspace: stream order alone must make them visible (no host synchronisation in between)
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg2"], B=2, H=3, T=384, regime="alpha_slow", seed=61)
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    ref = gu.oracle_bwd(d)
    dO = torch.zeros_like(t["dO"])
    dhT = torch.zeros_like(t["dhT"])
    half_dO, half_dhT = (t["dO"].float() * 0.5).to(t["dO"].dtype), t["dhT"] * 0.5      # exact in bf16 / fp32
    for rep in range(3):
        dO.zero_(); dhT.zero_()
        o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], save_for_bwd=True)
        torch.cuda.synchronize()
        torch.add(half_dO, half_dO, out=dO)            # the producers ...
        torch.add(half_dhT, half_dhT, out=dhT)
        g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], dO, dhT,
                         workspace=ws, reuse_fwd=True)   # ... and the consumer right behind them
        torch.cuda.synchronize()
        for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0"):
            gu.check(_label(cfg, " behind producers"), n, g[n], ref[n], cfg.dtype, state=(n == "dh0"))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_gradients_of_absent_coefficients_on_request(dtype):
    # alpha = NULL means alpha == 1 and lambda = NULL means lambda == 0; their gradients at those values are still
    # defined and are written when the caller passes buffers for them
    from paper_2606_08804_b200 import binding as qd
    base = gen.CONFIGS["cfg2"] if dtype == "bf16" else replace(gen.CONFIGS["cfg0"], h0=True, backward=True)
    cfg = replace(base, B=2, H=2, T=192, seed=67)
    d = dict(gen.make_chunk_inputs(cfg), alpha=None, lam=None)
    t = gu.dev_inputs(d, cfg.dtype)
    ref = gu.oracle_bwd(d)
    for reuse in (False, True):
        ws = None
        if reuse:
            _, _, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], None, None, t["h0"], save_for_bwd=True)
        out = {"dalpha": torch.full((cfg.B, cfg.T, cfg.H), float("nan"), device="cuda"),
               "dlam": torch.full((cfg.B, cfg.T, cfg.H), float("nan"), device="cuda")}
        g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], None, None, t["h0"], t["dO"], t["dhT"], workspace=ws,
                         reuse_fwd=reuse, out=out)
        torch.cuda.synchronize()
        for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0"):
            gu.check(_label(cfg, " absent coefficients, gradients requested"), n, g[n], ref[n], cfg.dtype, state=(n == "dh0"))


@pytest.mark.parametrize("dtype,T", [("bf16", 300), ("f32", 192)])
def test_gates_from_logits(dtype, T):
    # QD_COEF_LOGITS: beta, alpha, lambda are pre-activation logits (lambda's centred on the -0.8 bias of Appendix B);
    # the kernels apply the sigmoid and return gradients with respect to the logits.  Forward, backward (both modes),
    # and the multi-token decode step.
    from oracle import recurrence as orc
    from paper_2606_08804_b200 import binding as qd
    base = gen.CONFIGS["cfg2"] if dtype == "bf16" else replace(gen.CONFIGS["cfg0"], h0=True, backward=True)
    cfg = replace(base, B=2, H=3, T=T, seed=101)
    d = gen.make_chunk_inputs(cfg)
    r = np.random.default_rng(7)
    rnd = (lambda x: gen.round_bf16(x.astype(np.float32))) if dtype == "bf16" else (lambda x: x.astype(np.float32))
    shp = (cfg.B, cfg.T, cfg.H)
    z = dict(beta=rnd(r.normal(0.0, 1.5, shp)), alpha=rnd(r.normal(3.0, 1.5, shp)), lam=rnd(r.normal(-0.8, 1.0, shp)))
    d = dict(d, **z)
    t = gu.dev_inputs(d, cfg.dtype)
    ro, rh = orc.forward_logits(d["q"], d["k"], d["v"], z["beta"], z["alpha"], z["lam"], d["h0"])
    ref = orc.backward_logits(d["q"], d["k"], d["v"], z["beta"], z["alpha"], z["lam"], d["h0"], d["dO"], d["dhT"])
    lab = _label(cfg, " logits")
    for reuse in (False, True):
        o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], save_for_bwd=reuse, logits=True)
        g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"],
                         workspace=ws if reuse else None, reuse_fwd=reuse, logits=True)
        torch.cuda.synchronize()
        gu.check(lab, "o", o, ro, cfg.dtype)
        gu.check(lab, "hT", hT, rh, cfg.dtype, state=True)
        for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0"):
            gu.check(lab, n, g[n], ref[n], cfg.dtype, state=(n == "dh0"))
    # decode: the first 5 tokens through the multi-token step with logits
    S = 5
    c = lambda x: x[:, :S].contiguous()
    state = t["h0"].clone()
    od = qd.recurrent_steps(c(t["q"]), c(t["k"]), c(t["v"]), c(t["beta"]), c(t["alpha"]), c(t["lam"]), state, logits=True)
    torch.cuda.synchronize()
    ro5, rh5 = orc.forward_logits(d["q"][:, :S], d["k"][:, :S], d["v"][:, :S], z["beta"][:, :S], z["alpha"][:, :S],
                                  z["lam"][:, :S], d["h0"])
    assert gu.rel_err(od, ro5) <= gu.TOL[dtype] and gu.rel_err(state, rh5) <= gu.TOL[dtype]


@pytest.mark.parametrize("dtype,T,logits,drop", [("bf16", 300, False, ()), ("bf16", 256, True, ()), ("bf16", 192, False, ("lam", "alpha")),
                                                 ("f32", 150, False, ()), ("f32", 128, True, ("lam",))])
def test_in_kernel_l2_normalisation(dtype, T, logits, drop):
    # QD_NORM_QK: q and k arrive un-normalised (rows of very different lengths); the kernels normalise them and the
    # backward returns gradients with respect to the un-normalised rows.  Alone, with logit gates, with absent inputs.
    from oracle import recurrence as orc
    from paper_2606_08804_b200 import binding as qd
    base = gen.CONFIGS["cfg2"] if dtype == "bf16" else replace(gen.CONFIGS["cfg0"], h0=True, backward=True)
    cfg = replace(base, B=2, H=3, T=T, regime="alpha_slow", seed=103 + T)
    d = gen.make_chunk_inputs(cfg)
    r = np.random.default_rng(11)
    rnd = (lambda x: gen.round_bf16(x.astype(np.float32))) if dtype == "bf16" else (lambda x: x.astype(np.float32))
    scale = lambda shape: np.exp(r.normal(0.0, 1.0, shape[:-1] + (1,)))          # row lengths over two orders of magnitude
    d["q"] = rnd(d["q"] * scale(d["q"].shape))
    d["k"] = rnd(d["k"] * scale(d["k"].shape))
    if logits:
        shp = (cfg.B, cfg.T, cfg.H)
        d["beta"], d["alpha"], d["lam"] = rnd(r.normal(0.0, 1.5, shp)), rnd(r.normal(3.0, 1.5, shp)), rnd(r.normal(-0.8, 1.0, shp))
    for n in drop:
        d[n] = None
    t = gu.dev_inputs(d, cfg.dtype)
    ro, rh = orc.forward_fused(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"], logits=logits, norm_qk=True)
    ref = orc.backward_fused(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"], d["dO"], d["dhT"],
                             logits=logits, norm_qk=True)
    lab = _label(cfg, " norm_qk%s%s" % (" logits" if logits else "", " without " + "+".join(drop) if drop else ""))
    for reuse in (False, True):
        o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], save_for_bwd=reuse,
                                 logits=logits, norm_qk=True)
        g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"],
                         workspace=ws if reuse else None, reuse_fwd=reuse, logits=logits, norm_qk=True)
        torch.cuda.synchronize()
        assert qd.workspace_status(ws) == 0 if reuse else True
        gu.check(lab, "o", o, ro, cfg.dtype)
        gu.check(lab, "hT", hT, rh, cfg.dtype, state=True)
        for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0"):
            if g.get(n) is not None:
                gu.check(lab, n, g[n], ref[n], cfg.dtype, state=(n == "dh0"))
    S = 4
    c = lambda x: None if x is None else x[:, :S].contiguous()
    state = t["h0"].clone()
    od = qd.recurrent_steps(c(t["q"]), c(t["k"]), c(t["v"]), c(t["beta"]), c(t["alpha"]), c(t["lam"]), state,
                            logits=logits, norm_qk=True)
    torch.cuda.synchronize()
    cut = lambda a: None if a is None else a[:, :S]
    roS, rhS = orc.forward_fused(cut(d["q"]), cut(d["k"]), cut(d["v"]), cut(d["beta"]), cut(d["alpha"]), cut(d["lam"]), d["h0"],
                                 logits=logits, norm_qk=True)
    assert gu.rel_err(od, roS) <= gu.TOL[dtype] and gu.rel_err(state, rhS) <= gu.TOL[dtype]


@pytest.mark.parametrize("case", range(12))
def test_random_shapes_flags_and_absent_inputs(case):
    # seeded sweep over what the entry points accept: any T, either path, absent optional inputs, both pre-processing
    # flags, backward with and without the forward's workspace -- each case against the oracle
    from oracle import recurrence as orc
    from paper_2606_08804_b200 import binding as qd
    r = np.random.default_rng(1000 + case)
    tc = case % 2 == 0                                   # even cases: bf16 d = 128 (tensor cores); odd: fp32 path shapes
    if tc:
        base, dk, dv, dtype = gen.CONFIGS["cfg2"], 128, 128, "bf16"
    else:
        dk, dv = [(64, 64), (128, 64), (64, 128)][case % 3]
        dtype = "f32" if case % 4 == 1 else "bf16"
        base = replace(gen.CONFIGS["cfg0"], h0=True, backward=True, dtype=dtype)
    B, H = int(r.integers(1, 4)), int(r.integers(1, 5))
    T = int(r.integers(1, 400))
    regime = gen.REGIMES[int(r.integers(0, len(gen.REGIMES)))]
    cfg = replace(base, B=B, H=H, T=T, dk=dk, dv=dv, regime=regime, seed=2000 + case)
    d = gen.make_chunk_inputs(cfg)
    logits, norm = bool(r.integers(0, 2)), bool(r.integers(0, 2))
    rnd = (lambda x: gen.round_bf16(x.astype(np.float32))) if dtype == "bf16" else (lambda x: x.astype(np.float32))
    if norm:
        d["q"] = rnd(d["q"] * np.exp(r.normal(0, 0.7, d["q"].shape[:-1] + (1,))))
        d["k"] = rnd(d["k"] * np.exp(r.normal(0, 0.7, d["k"].shape[:-1] + (1,))))
    if logits:
        shp = (B, T, H)
        d["beta"], d["alpha"], d["lam"] = rnd(r.normal(0, 1.5, shp)), rnd(r.normal(3, 1.5, shp)), rnd(r.normal(-0.8, 1, shp))
    for n in ("alpha", "lam", "h0", "dhT"):
        if r.random() < 0.25:
            d[n] = None
    t = gu.dev_inputs(d, cfg.dtype)
    assert qd.chunk_path(qd.make_shape(t["q"], t["v"], 64)) == ("tensor_core" if tc else "fp32")
    ro, rh = orc.forward_fused(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"], logits=logits, norm_qk=norm)
    ref = orc.backward_fused(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"], d["dO"], d["dhT"],
                             logits=logits, norm_qk=norm)
    lab = _label(cfg, " sweep %d logits=%d norm=%d absent=%s" % (case, logits, norm, [n for n in ("alpha", "lam", "h0", "dhT") if d[n] is None]))
    for reuse in (False, True):
        o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], save_for_bwd=reuse,
                                 logits=logits, norm_qk=norm)
        g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"],
                         workspace=ws if reuse else None, reuse_fwd=reuse, logits=logits, norm_qk=norm)
        torch.cuda.synchronize()
        gu.check(lab, "o", o, ro, cfg.dtype)
        gu.check(lab, "hT", hT, rh, cfg.dtype, state=True)
        for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0"):
            if g.get(n) is not None:
                gu.check(lab, n, g[n], ref[n], cfg.dtype, state=(n == "dh0"))


def test_autograd_front_end():
    # torch.autograd wrapper: gradients of a scalar loss on o and hT equal the oracle's reverse pass
    from paper_2606_08804_b200.autograd import qdelta_chunk
    cfg = replace(gen.CONFIGS["cfg2"], B=2, H=2, T=200, regime="alpha_slow", seed=107)
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    leaves = {n: t[n].clone().requires_grad_(True) for n in ("q", "k", "v", "beta", "alpha", "lam", "h0")}
    o, hT = qdelta_chunk(**leaves)
    loss = (o.float() * t["dO"].float()).sum() + (hT * t["dhT"]).sum()
    loss.backward()
    torch.cuda.synchronize()
    ro, rh = gu.oracle_fwd(d)
    ref = gu.oracle_bwd(d)
    lab = _label(cfg, " autograd")
    gu.check(lab, "o", o, ro, cfg.dtype)
    gu.check(lab, "hT", hT, rh, cfg.dtype, state=True)
    for n, gn in (("q", "dq"), ("k", "dk"), ("v", "dv"), ("beta", "dbeta"), ("alpha", "dalpha"), ("lam", "dlam"), ("h0", "dh0")):
        # coefficient gradients come back in the coefficients' dtype (bf16): one more rounding than the raw fp32 ones
        gu.check(lab, gn, leaves[n].grad, ref[gn], cfg.dtype, state=(n == "h0"))
    # without any input requiring grad the forward does not keep a backward-sized workspace
    with torch.no_grad():
        o2, _ = qdelta_chunk(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"])
    assert torch.equal(o2, o.detach())
