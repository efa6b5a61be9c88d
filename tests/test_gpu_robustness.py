"""Bounds and failure handling of the CUDA path, checked without faulting anything.

* Guard bands: every output, state and workspace buffer of a call sits between two 4 KB bands of a fixed byte pattern;
  after the call the bands must be untouched (compute-sanitizer is not available here, so this is the bounds check).
* Bounded waits: a self-test kernel waits, with a short limit, on an mbarrier that nothing arrives on.  It must come
  back with QD_ERR_TIMEOUT having released its tensor memory, and the device must be fully usable afterwards.
"""
import ctypes
from dataclasses import replace

import pytest
import torch

from paper_2606_08804_b200 import inputs as gen
import gpu_util as gu

pytestmark = pytest.mark.gpu

BF, F32 = torch.bfloat16, torch.float32

# two shapes per path; ragged lengths on purpose (the last chunk is partly, or wholly, outside the tensors)
TC_SHAPES = [dict(B=2, H=3, T=384), dict(B=1, H=2, T=200)]
F32_SHAPES = [dict(B=1, H=2, T=128, dk=64, dv=64), dict(B=2, H=1, T=100, dk=128, dv=64)]


def _guarded_call(cfg):
    from paper_2606_08804_b200 import binding as qd
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    dt = gu.TDT[cfg.dtype]
    B, T, H, dk, dv = cfg.B, cfg.T, cfg.H, cfg.dk, cfg.dv
    shape = qd.make_shape(t["q"], t["v"], cfg.chunk)
    G = gu.Guarded
    bands = {
        "o": G((B, T, H, dv), dt), "hT": G((B, H, dk, dv), F32),
        "ws_fwd": G((qd.chunk_workspace_bytes(shape, False),), torch.uint8),
        "ws_bwd": G((qd.chunk_workspace_bytes(shape, True),), torch.uint8),
        "dq": G((B, T, H, dk), dt), "dk": G((B, T, H, dk), dt), "dv": G((B, T, H, dv), dt),
        "dbeta": G((B, T, H), F32), "dalpha": G((B, T, H), F32), "dlam": G((B, T, H), F32),
        "dh0": G((B, H, dk, dv), F32),
    }
    grads = {n: bands[n].t for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0")}
    ref_o, ref_h = gu.oracle_fwd(d)
    ref_g = gu.oracle_bwd(d)

    def intact(where):
        torch.cuda.synchronize()
        bad = [n for n, g in bands.items() if not g.intact()]
        assert not bad, (where, bad)

    # plain forward on a forward-sized workspace
    qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], workspace=bands["ws_fwd"].t,
                 o=bands["o"].t, hT=bands["hT"].t)
    intact("forward")
    assert gu.rel_err(bands["o"].t, ref_o) <= gu.TOL[cfg.dtype]
    # backward that recomputes the forward, then saving forward + backward on its workspace
    for reuse in (False, True):
        if reuse:
            qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], workspace=bands["ws_bwd"].t,
                         o=bands["o"].t, hT=bands["hT"].t, save_for_bwd=True)
            intact("saving forward")
        qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"],
                     workspace=bands["ws_bwd"].t, reuse_fwd=reuse, out=grads)
        intact("backward reuse=%s" % reuse)
        for n in grads:
            assert gu.rel_err(grads[n], ref_g[n]) <= gu.TOL[cfg.dtype], (n, reuse)
    assert gu.rel_err(bands["hT"].t, ref_h) <= gu.TOL[cfg.dtype]
    return t, bands, ref_o


@pytest.mark.parametrize("shp", TC_SHAPES)
def test_guard_bands_tensor_core_path(shp):
    from paper_2606_08804_b200 import binding as qd
    cfg = replace(gen.CONFIGS["cfg2"], regime="alpha_slow", seed=71, **shp)
    t, bands, ref_o = _guarded_call(cfg)
    # the allocation-free forward writes only o and hT
    bands["o"].t.zero_()
    qd.chunk_fwd_static(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], bands["o"].t, bands["hT"].t)
    torch.cuda.synchronize()
    assert bands["o"].intact() and bands["hT"].intact()
    assert gu.rel_err(bands["o"].t, ref_o) <= gu.TOL[cfg.dtype]


@pytest.mark.parametrize("shp", F32_SHAPES)
def test_guard_bands_fp32_path(shp):
    cfg = replace(gen.CONFIGS["cfg0"], h0=True, backward=True, regime="alpha_slow", seed=73, **shp)
    _guarded_call(cfg)


@pytest.mark.parametrize("B,H,dk,dv", [(3, 5, 128, 128), (2, 2, 64, 128)])
def test_guard_bands_decode_step(B, H, dk, dv):
    from paper_2606_08804_b200 import binding as qd
    from oracle import recurrence as orc
    cfg = replace(gen.CONFIGS["cfg4"], B=B, H=H, dk=dk, dv=dv, T=3)
    state0 = gen.make_decode_state(cfg)
    tok = gen.make_decode_tokens(cfg, 0, 3)
    state = gu.Guarded((B, H, dk, dv), F32, fill=torch.from_numpy(state0).cuda())
    o = gu.Guarded((B, H, dv), BF)
    td = {n: torch.from_numpy(a).to("cuda", BF) for n, a in tok.items()}
    outs = []
    for s in range(3):
        qd.recurrent_step(td["q"][s], td["k"][s], td["v"][s], td["beta"][s], td["alpha"][s], td["lam"][s], state.t, o.t)
        torch.cuda.synchronize()
        assert state.intact() and o.intact(), s
        outs.append(o.t.clone())
    ro, rh = orc.decode(state0.astype("float64"), tok["q"], tok["k"], tok["v"], tok["beta"], tok["alpha"], tok["lam"])
    assert gu.rel_err(torch.stack(outs, 0), ro) <= 2e-2
    assert gu.rel_err(state.t, rh) <= 2e-2


def test_bounded_wait_runs_out_and_the_device_stays_usable():
    from paper_2606_08804_b200 import binding as qd
    lib = qd.load()
    fn = lib.qdelta_selftest_timeout
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_void_p, ctypes.c_uint, ctypes.c_void_p]
    out = torch.zeros(2, dtype=torch.int32, device="cuda")
    limit_ns = 200_000                                 # 0.2 ms
    for rep in range(3):                               # three times: the tensor memory it takes must come back each time
        out.zero_()
        assert fn(out.data_ptr(), limit_ns, torch.cuda.current_stream().cuda_stream) == 0
        torch.cuda.synchronize()                       # returns: the kernel gave up by itself
        status, waited = int(out[0].item()), int(out[1].item()) & 0xFFFFFFFF
        assert status == 5 and qd.status_string(status) == "QD_ERR_TIMEOUT"
        assert limit_ns <= waited < 50 * limit_ns, waited      # it waited about as long as it was told to, not seconds
    assert fn(out.data_ptr(), 0, None) == 1            # limits outside (0, 0.1 s] are refused on the host
    # an ordinary forward + backward on the same device right afterwards: status word clear, results right
    cfg = replace(gen.CONFIGS["cfg2"], B=2, H=2, T=256, seed=79)
    d = gen.make_chunk_inputs(cfg)
    t = gu.dev_inputs(d, cfg.dtype)
    o, hT, ws = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], save_for_bwd=True)
    g = qd.chunk_bwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], t["dO"], t["dhT"],
                     workspace=ws, reuse_fwd=True)
    torch.cuda.synchronize()
    assert qd.workspace_status(ws) == 0
    ro, rh = gu.oracle_fwd(d)
    assert gu.rel_err(o, ro) <= 2e-2 and gu.rel_err(hT, rh) <= 2e-2
    ref = gu.oracle_bwd(d)
    assert gu.rel_err(g["dq"], ref["dq"]) <= 2e-2
