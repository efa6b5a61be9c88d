"""The allocation-free forward entry point (`qdelta_chunk_fwd_static`), through the C ABI.

Collected last on purpose: it must pass both alone in a fresh process and after every other GPU test
has used the library.  It is compared with the ordinary entry point on the same inputs, twice in a
row (the second call reuses the built-in scratch array the first one left dirty).
"""
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2606_08804_b200 import inputs as gen

pytestmark = pytest.mark.gpu

CASES = {
    # tensor-core kernels: bf16, d = 128, T a multiple of 128; two sequences per head-batch, several chunks
    "bf16_tc": gen.Config("static_tc", 2, 512, 4, 128, 128, 64, "bf16", True, False, seed=21),
    # fp32 kernels
    "f32": gen.Config("static_f32", 1, 256, 2, 64, 64, 64, "f32", True, False, seed=22),
}


def _to_gpu(d, cfg):
    import torch
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    t = {n: torch.from_numpy(d[n]).to(dt).cuda() for n in ("q", "k", "v", "beta", "alpha", "lam")}
    t["h0"] = torch.from_numpy(d["h0"]).cuda() if d.get("h0") is not None else None
    return t, dt


@pytest.mark.parametrize("case", sorted(CASES))
def test_static_forward_matches_ordinary_entry_point_twice(case):
    import torch
    from paper_2606_08804_b200 import binding as qd
    from gpu_util import TOL, rel_err

    cfg = CASES[case]
    t, dt = _to_gpu(gen.make_chunk_inputs(cfg), cfg)
    o_ref, hT_ref, _ = qd.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], chunk=cfg.chunk)
    torch.cuda.synchronize()

    o = torch.empty_like(o_ref)
    hT = torch.empty_like(hT_ref)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    tol = TOL[cfg.dtype]
    free_before = None
    for call in range(2):
        o.fill_(float("nan"))
        hT.fill_(float("nan"))
        status.fill_(77)
        torch.cuda.synchronize()
        if call == 1:
            free_before = torch.cuda.mem_get_info()[0]
        qd.chunk_fwd_static(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], o, hT, status, chunk=cfg.chunk)
        torch.cuda.synchronize()
        if call == 1:
            # set-up happened in the first call; the second must not change the device's free memory
            assert torch.cuda.mem_get_info()[0] == free_before
        assert int(status.item()) == 0
        e_o = rel_err(o, o_ref.float().cpu().numpy())
        e_h = rel_err(hT, hT_ref.cpu().numpy())
        assert e_o <= tol and e_h <= tol, (case, call, e_o, e_h)


def test_static_forward_matches_oracle():
    import torch
    from oracle import recurrence
    from paper_2606_08804_b200 import binding as qd
    from gpu_util import TOL, rel_err

    cfg = CASES["bf16_tc"]
    d = gen.make_chunk_inputs(cfg)
    t, dt = _to_gpu(d, cfg)
    o = torch.empty((cfg.B, cfg.T, cfg.H, cfg.dv), dtype=dt, device="cuda")
    qd.chunk_fwd_static(t["q"], t["k"], t["v"], t["beta"], t["alpha"], t["lam"], t["h0"], o, None, None, chunk=cfg.chunk)
    torch.cuda.synchronize()
    o_ref, _ = recurrence.forward(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"])
    assert rel_err(o, o_ref) <= TOL[cfg.dtype]
