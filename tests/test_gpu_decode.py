"""GPU-vs-oracle parity of the recurrent decode step (through the C ABI)."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import recurrence as orc
from paper_2606_08804_b200 import inputs as gen
import gpu_util as gu

pytestmark = pytest.mark.gpu


def _run(cfg, steps, check_at, sample=None, null_coeffs=False):
    from paper_2606_08804_b200 import binding as qd
    t = gu.TDT[cfg.dtype]
    s0 = gen.make_decode_state(cfg)
    state = gu.to_dev(s0, torch.float32)
    Bn, H = cfg.B, cfg.H
    if sample is None:
        sel_b, sel_h = np.meshgrid(np.arange(Bn), np.arange(H), indexing="ij")
        sel_b, sel_h = sel_b.ravel(), sel_h.ravel()
    else:
        r = np.random.default_rng(1)
        idx = r.choice(Bn * H, size=sample, replace=False)
        sel_b, sel_h = idx // H, idx % H
    ref_state = s0[sel_b, sel_h][:, None].astype(np.float64)           # [n,1,dk,dv]
    done = 0
    block = 50
    while done < steps:
        n = min(block, steps - done)
        tok = gen.make_decode_tokens(cfg, done, n)
        if null_coeffs:
            tok["alpha"] = None; tok["lam"] = None
        dev = {k_: gu.to_dev(a, t) for k_, a in tok.items()}
        outs = []
        for i in range(n):
            o = qd.recurrent_step(dev["q"][i], dev["k"][i], dev["v"][i], dev["beta"][i],
                                  None if null_coeffs else dev["alpha"][i],
                                  None if null_coeffs else dev["lam"][i], state)
            outs.append(o)
        torch.cuda.synchronize()
        sub = {k_: (None if a is None else a[:, sel_b, sel_h][:, :, None]) for k_, a in tok.items()}
        ro, ref_state = orc.decode(ref_state, sub["q"], sub["k"], sub["v"], sub["beta"], sub["alpha"], sub["lam"])
        for i in range(n):
            step = done + i + 1
            if step in check_at:
                got = outs[i][sel_b, sel_h][:, None]
                e = gu.rel_err(got, ro[i])
                assert e <= gu.TOL[cfg.dtype], ("o", step, e)
                if i == n - 1:
                    es = gu.rel_err(state[sel_b, sel_h][:, None], ref_state)
                    assert es <= gu.TOL[cfg.dtype], ("state", step, es)
        done += n
    es = gu.rel_err(state[sel_b, sel_h][:, None], ref_state)
    assert es <= gu.TOL[cfg.dtype], ("final state", es)


def test_decode_small_bf16_all_states():
    cfg = replace(gen.CONFIGS["cfg4"], B=3, H=5)
    _run(cfg, 60, set(range(1, 61)))


@pytest.mark.parametrize("dk,dv", [(64, 64), (128, 64), (64, 128)])
def test_decode_fp32_shapes(dk, dv):
    cfg = replace(gen.CONFIGS["cfg4"], B=2, H=3, dk=dk, dv=dv, dtype="f32")
    _run(cfg, 20, set(range(1, 21)))


def test_decode_null_coefficients():
    cfg = replace(gen.CONFIGS["cfg4"], B=2, H=2)
    _run(cfg, 10, set(range(1, 11)), null_coeffs=True)


def test_decode_slow_decay_long():
    cfg = replace(gen.CONFIGS["cfg4"], B=2, H=4, regime="trained_like")
    _run(cfg, 300, {1, 10, 100, 300})


def test_cfg4_full_size_1000_steps_sampled():
    # the benchmarked launch shape (256 x 16 states of 128 x 128); the oracle follows 48 sampled states
    cfg = gen.CONFIGS["cfg4"]
    _run(cfg, 1000, {1, 10, 100, 1000}, sample=48)


def test_decode_matches_chunk_forward_on_gpu():
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg1"], B=2, H=2, T=128, regime="alpha_slow", seed=21)
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    o, hT, _ = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"])
    state = t["h0"].clone()
    outs = []
    for s in range(cfg.T):
        outs.append(qd.recurrent_step(t["q"][:, s].contiguous(), t["k"][:, s].contiguous(), t["v"][:, s].contiguous(),
                                      t["beta"][:, s].contiguous(), t["alpha"][:, s].contiguous(),
                                      t["lam"][:, s].contiguous(), state))
    torch.cuda.synchronize()
    o2 = torch.stack(outs, dim=1)
    den = o.float().abs().max()
    assert ((o2.float() - o.float()).abs().max() / den).item() <= 2e-2
    assert ((state - hT).abs().max() / hT.abs().max()).item() <= 2e-2


@pytest.mark.parametrize("dtype,dk,dv,S", [("bf16", 128, 128, 4), ("bf16", 128, 128, 1), ("bf16", 64, 128, 7), ("f32", 64, 64, 5)])
def test_multi_token_step_is_the_single_step_repeated(dtype, dk, dv, S):
    # S tokens in one call: bit-identical to S single-token calls, and equal to the oracle's recurrence
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg1"], B=3, H=5, T=S, dk=dk, dv=dv, dtype=dtype, regime="alpha_slow", seed=83)
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    st_multi = gu.Guarded((cfg.B, cfg.H, dk, dv), torch.float32, fill=t["h0"])
    o_multi = gu.Guarded((cfg.B, S, cfg.H, dv), gu.TDT[dtype])
    qd.recurrent_steps(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], st_multi.t, o_multi.t)
    st_single = t["h0"].clone()
    outs = []
    for s in range(S):
        c = lambda x: x[:, s].contiguous()
        outs.append(qd.recurrent_step(c(t["q"]), c(t["k"]), c(t["v"]), c(t["beta"]), c(t["alpha"]), c(t["lam"]), st_single))
    torch.cuda.synchronize()
    assert st_multi.intact() and o_multi.intact()
    assert torch.equal(o_multi.t, torch.stack(outs, dim=1))
    assert torch.equal(st_multi.t, st_single)
    ro, rh = gu.oracle_fwd(d)
    assert gu.rel_err(o_multi.t, ro) <= gu.TOL[dtype] and gu.rel_err(st_multi.t, rh) <= gu.TOL[dtype]


def test_prefill_then_multi_token_decode():
    # a prompt through the chunkwise forward (ragged length), its final state handed to the multi-token decode step:
    # together they must equal the recurrence over the whole sequence
    from paper_2606_08804_b200 import binding as qd
    S, Tp = 6, 150
    cfg = replace(gen.CONFIGS["cfg1"], B=2, H=3, T=Tp + 2 * S, regime="trained_like", seed=89)
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    c = lambda x, a, b: x[:, a:b].contiguous()
    names = ("q", "k", "v", "beta", "alpha", "lam")
    pre = [c(t[n], 0, Tp) for n in names]
    o_pre, state, _ = qd.chunk_fwd(*pre, t["h0"])
    outs = [o_pre]
    for j in range(2):
        seg = [c(t[n], Tp + j * S, Tp + (j + 1) * S) for n in names]
        outs.append(qd.recurrent_steps(*seg, state))
    torch.cuda.synchronize()
    ro, rh = gu.oracle_fwd(d)
    assert gu.rel_err(torch.cat(outs, dim=1), ro) <= 2e-2
    assert gu.rel_err(state, rh) <= 2e-2


def test_multi_token_step_null_coefficients_and_argument_errors():
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg1"], B=2, H=2, T=3, seed=97)
    d = dict(gen.make_chunk_inputs(cfg), alpha=None, lam=None)
    t = gu.dev_inputs(d, cfg.dtype)
    state = t["h0"].clone()
    o = qd.recurrent_steps(t["q"], t["k"], t["v"], t["beta"], None, None, state)
    torch.cuda.synchronize()
    ro, rh = gu.oracle_fwd(d)
    assert gu.rel_err(o, ro) <= 2e-2 and gu.rel_err(state, rh) <= 2e-2
    lib = qd.load()
    fake = 0x1000
    assert lib.qdelta_recurrent_steps(1, 0, 1, 64, 64, 0, fake, fake, fake, fake, None, None, fake, fake, 0, None) == 1
    assert lib.qdelta_recurrent_steps(1, 2, 1, 96, 64, 0, fake, fake, fake, fake, None, None, fake, fake, 0, None) == 2
    assert lib.qdelta_recurrent_steps(1, 2, 1, 64, 64, 0, fake, fake, fake, fake, None, None, fake, fake, 64, None) == 1


def test_decode_steps_replayed_from_a_cuda_graph():
    # a fixed run of decode steps captured once in a CUDA graph and replayed: the library enqueues only kernels on the
    # caller's stream (no allocation, no synchronisation), so capture works and a replay equals the eager run
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg4"], B=4, H=3)
    n = 6
    tok = gen.make_decode_tokens(cfg, 0, n)
    dev = {k_: gu.to_dev(a, torch.bfloat16) for k_, a in tok.items()}
    s0 = gu.to_dev(gen.make_decode_state(cfg), torch.float32)
    outs = [torch.empty((cfg.B, cfg.H, cfg.dv), dtype=torch.bfloat16, device="cuda") for _ in range(n)]

    def run(state):
        for i in range(n):
            qd.recurrent_step(dev["q"][i], dev["k"][i], dev["v"][i], dev["beta"][i], dev["alpha"][i], dev["lam"][i],
                              state, outs[i])
    eager_state = s0.clone()
    run(eager_state)
    torch.cuda.synchronize()
    eager_outs = [o.clone() for o in outs]
    state = s0.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run(state)                                   # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run(state)
    for rep in range(2):
        state.copy_(s0)
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(state, eager_state)
        for a, b in zip(outs, eager_outs):
            assert torch.equal(a, b)


@pytest.mark.parametrize("S", [1, 4])
def test_decode_with_bf16_state_storage(S):
    # QD_STATE_BF16: the state lives in bf16 between calls (fp32 inside a call).  Checked against the oracle run with
    # exactly that rounding between calls, and -- in the forgetful regime of the decode configuration, where the gate
    # damps the rounding -- against the plain fp64 oracle within the bf16 bar.
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg4"], B=3, H=4)
    calls = 200 // S
    s0 = gen.round_bf16(gen.make_decode_state(cfg))
    state = gu.Guarded((cfg.B, cfg.H, cfg.dk, cfg.dv), torch.bfloat16, fill=torch.from_numpy(s0).cuda().to(torch.bfloat16))
    ref_r = s0.astype(np.float64)            # oracle state, rounded to bf16 after every call
    ref_x = s0.astype(np.float64)            # oracle state, never rounded
    worst_r = worst_x = 0.0
    for c in range(calls):
        tok = gen.make_decode_tokens(cfg, c * S, S)
        dev = {n: gu.to_dev(np.ascontiguousarray(np.moveaxis(a, 0, 1)), torch.bfloat16) for n, a in tok.items()}
        o = qd.recurrent_steps(dev["q"], dev["k"], dev["v"], dev["beta"], dev["alpha"], dev["lam"], state.t)
        o_r, ref_r = orc.decode(ref_r, tok["q"], tok["k"], tok["v"], tok["beta"], tok["alpha"], tok["lam"])
        ref_r = gen.round_bf16(ref_r.astype(np.float32)).astype(np.float64)
        o_x, ref_x = orc.decode(ref_x, tok["q"], tok["k"], tok["v"], tok["beta"], tok["alpha"], tok["lam"])
        if c % 10 == 9 or c == calls - 1:
            torch.cuda.synchronize()
            worst_r = max(worst_r, gu.rel_err(o, np.moveaxis(o_r, 0, 1)))
            worst_x = max(worst_x, gu.rel_err(o, np.moveaxis(o_x, 0, 1)))
    torch.cuda.synchronize()
    assert state.intact()
    assert worst_r <= 2e-2 and gu.rel_err(state.t.float(), ref_r) <= 2e-2, (worst_r,)
    assert worst_x <= 2e-2 and gu.rel_err(state.t.float(), ref_x) <= 2e-2, (worst_x,)
