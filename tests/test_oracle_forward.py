"""Pins of the forward recurrence oracle (CPU only)."""
import os
import numpy as np
import pytest

from oracle import recurrence as orc
from oracle import chunkwise_form as cw
import independent_forms as ind


def _rand(seed, B=1, T=12, H=2, dk=5, dv=4, alpha_lo=0.3):
    r = np.random.default_rng(seed)
    unit = lambda x: x / np.linalg.norm(x, axis=-1, keepdims=True)
    return dict(q=unit(r.standard_normal((B, T, H, dk))), k=unit(r.standard_normal((B, T, H, dk))),
                v=r.standard_normal((B, T, H, dv)), beta=r.uniform(0.05, 1.0, (B, T, H)),
                alpha=r.uniform(alpha_lo, 1.0, (B, T, H)), lam=r.uniform(0.0, 1.0, (B, T, H)),
                h0=0.3 * r.standard_normal((B, H, dk, dv)))


def test_one_step_closed_form():
    # T = 1: h_1 = a h_0 + b k (v - a h_0^T x)^T, o_1 = h_1^T q   (Section 3.3.1, gated rule)
    d = _rand(1, T=1)
    o, hT = orc.forward(**d)
    for hh in range(2):
        q, k, v = d["q"][0, 0, hh], d["k"][0, 0, hh], d["v"][0, 0, hh]
        b, a, l = d["beta"][0, 0, hh], d["alpha"][0, 0, hh], d["lam"][0, 0, hh]
        h0 = d["h0"][0, hh]
        x = k + l * q
        h1 = a * h0 + b * np.outer(k, v - a * h0.T @ x)
        np.testing.assert_allclose(hT[0, hh], h1, rtol=0, atol=1e-14)
        np.testing.assert_allclose(o[0, 0, hh], h1.T @ q, rtol=0, atol=1e-14)


def test_three_printed_forms_agree_and_match_oracle():
    d = _rand(2, T=1)
    d["alpha"][:] = 1.0
    _, hT = orc.forward(**d)
    for hh in range(2):
        q, k, v = d["q"][0, 0, hh], d["k"][0, 0, hh], d["v"][0, 0, hh]
        b, l = d["beta"][0, 0, hh], d["lam"][0, 0, hh]
        S0 = d["h0"][0, hh].T
        s_err = ind.qdelta_error_form(S0, q, k, v, b, l)
        s_lin = ind.qdelta_linear_form(S0, q, k, v, b, l)
        s_gat = ind.qdelta_gated_form(S0, q, k, v, b, 1.0, l)
        np.testing.assert_allclose(s_err, s_lin, atol=1e-14)
        np.testing.assert_allclose(s_err, s_gat, atol=1e-14)
        np.testing.assert_allclose(hT[0, hh].T, s_err, atol=1e-14)
    # gated printed form with alpha != 1
    d = _rand(3, T=1)
    _, hT = orc.forward(**d)
    for hh in range(2):
        S1 = ind.qdelta_gated_form(d["h0"][0, hh].T, d["q"][0, 0, hh], d["k"][0, 0, hh],
                                   d["v"][0, 0, hh], d["beta"][0, 0, hh], d["alpha"][0, 0, hh],
                                   d["lam"][0, 0, hh])
        np.testing.assert_allclose(hT[0, hh].T, S1, atol=1e-14)


@pytest.mark.parametrize("alpha_one", [False, True])
def test_lambda_zero_reduces_to_gated_delta_rule(alpha_one):
    d = _rand(4, T=40, dk=6, dv=5)
    d["lam"][:] = 0.0
    if alpha_one:
        d["alpha"][:] = 1.0          # DeltaNet, Eq. 2
    o, hT = orc.forward(**d)
    o_none, hT_none = orc.forward(d["q"], d["k"], d["v"], d["beta"],
                                  None if alpha_one else d["alpha"], None, d["h0"])
    np.testing.assert_allclose(o, o_none, atol=1e-14)
    for hh in range(2):
        o_ref, S = ind.gated_delta_rule(d["q"][0, :, hh], d["k"][0, :, hh], d["v"][0, :, hh],
                                        d["beta"][0, :, hh], d["alpha"][0, :, hh], d["h0"][0, hh].T)
        np.testing.assert_allclose(o[0, :, hh], o_ref, atol=1e-13)
        np.testing.assert_allclose(hT[0, hh].T, S, atol=1e-13)


def test_beta_zero_pure_decay():
    d = _rand(5, T=20)
    d["beta"][:] = 0.0
    o, hT = orc.forward(**d)
    gam = np.cumprod(d["alpha"], axis=1)
    for hh in range(2):
        np.testing.assert_allclose(hT[0, hh], gam[0, -1, hh] * d["h0"][0, hh], atol=1e-14)
        for t in range(20):
            np.testing.assert_allclose(o[0, t, hh], gam[0, t, hh] * d["h0"][0, hh].T @ d["q"][0, t, hh],
                                       atol=1e-14)


def test_chunk_expansion_bruteforce_and_value_span():
    d = _rand(6, T=7, H=1, dk=4, dv=3)
    args = (d["q"][0, :, 0], d["k"][0, :, 0], d["v"][0, :, 0], d["beta"][0, :, 0],
            d["alpha"][0, :, 0], d["lam"][0, :, 0])
    states = ind.chunk_expansion_bruteforce(d["h0"][0, 0].T, *args)
    for r in range(1, 8):
        sl = {kk: (vv[:, :r] if kk != "h0" else vv) for kk, vv in d.items()}
        o, hT = orc.forward(**sl)
        np.testing.assert_allclose(hT[0, 0].T, states[r - 1], atol=1e-13)
        np.testing.assert_allclose(o[0, r - 1, 0], states[r - 1] @ d["q"][0, r - 1, 0], atol=1e-13)
    # value-span decomposition needs S_0 = 0
    vs = ind.value_span_state(*args)
    d0 = dict(d); d0["h0"] = None
    for r in (1, 3, 7):
        sl = {kk: (vv[:, :r] if vv is not None else None) for kk, vv in d0.items()}
        _, hT = orc.forward(**sl)
        np.testing.assert_allclose(hT[0, 0].T, vs[r - 1], atol=1e-13)


def test_lemma1_identity_and_theorem1_inequality():
    # exact identity in the proof of Lemma 1, here with the forget gate included:
    # v_t - h_t^T x_t = (1 - beta_t a_t)(v_t - alpha_t h_{t-1}^T x_t), a_t = k_t . x_t
    d = _rand(7, T=30, H=1, dk=6, dv=5)
    q, k, v = d["q"][0, :, 0], d["k"][0, :, 0], d["v"][0, :, 0]
    for t in range(1, 31):
        sl = {kk: (vv[:, :t] if kk != "h0" else vv) for kk, vv in d.items()}
        _, h_t = orc.forward(**sl)
        if t == 1:
            h_prev = d["h0"]
        else:
            sl = {kk: (vv[:, :t - 1] if kk != "h0" else vv) for kk, vv in d.items()}
            _, h_prev = orc.forward(**sl)
        b, a, l = d["beta"][0, t - 1, 0], d["alpha"][0, t - 1, 0], d["lam"][0, t - 1, 0]
        x = k[t - 1] + l * q[t - 1]
        at = k[t - 1] @ x
        lhs = v[t - 1] - h_t[0, 0].T @ x
        rhs = (1 - b * at) * (v[t - 1] - a * h_prev[0, 0].T @ x)
        np.testing.assert_allclose(lhs, rhs, atol=1e-13)
    # Theorem 1 (alpha = 1): ||e_t|| <= |1 - beta a| (||e_{t-1}|| + ||r_t||), and the unrolled bound
    d["alpha"][:] = 1.0
    d["h0"] = None
    e_prev = np.zeros(5); v_prev = np.zeros(5); x_prev = np.zeros(6)
    S_prev = np.zeros((5, 6))
    rho, rmax, errs = 0.0, 0.0, []
    for t in range(1, 31):
        sl = {kk: (vv[:, :t] if vv is not None else None) for kk, vv in d.items()}
        _, h_t = orc.forward(**sl)
        S = h_t[0, 0].T
        b, l = d["beta"][0, t - 1, 0], d["lam"][0, t - 1, 0]
        x = k[t - 1] + l * q[t - 1]
        fac = abs(1 - b * (k[t - 1] @ x))
        r_t = (v[t - 1] - v_prev) - S_prev @ (x - x_prev)
        e = v[t - 1] - S @ x
        assert np.linalg.norm(e) <= fac * (np.linalg.norm(e_prev) + np.linalg.norm(r_t)) + 1e-12
        rho = max(rho, fac); rmax = max(rmax, np.linalg.norm(r_t)); errs.append(np.linalg.norm(e))
        e_prev, v_prev, x_prev, S_prev = e, v[t - 1], x, S
    assert rho < 1.0
    for t, en in enumerate(errs, start=1):
        assert en <= (1 - rho ** t) / (1 - rho) * rho * rmax + 1e-12


def test_wy_identity():
    # prod_i (I - beta_i x_i k_i^T) = I - sum_i w^i k_i^T   (extended WY, Section 3.3.2)
    d = _rand(8, T=9, H=1, dk=5, dv=3)
    q, k = d["q"][0, :, 0], d["k"][0, :, 0]
    beta, lam = d["beta"][0, :, 0], d["lam"][0, :, 0]
    W = ind.wy_vectors(q, k, beta, lam)
    P = np.eye(5)
    for i in range(9):
        P = P @ (np.eye(5) - beta[i] * np.outer(k[i] + lam[i] * q[i], k[i]))
    np.testing.assert_allclose(P, np.eye(5) - W.T @ k, atol=1e-13)
    # and the UT-transform matrix form of W used by the chunkwise form (alpha = 1: gamma = 1)
    c = cw._chunk_quantities(q, k, d["v"][0, :, 0], beta, np.ones(9), lam)
    np.testing.assert_allclose(c["W"], W, atol=1e-13)


@pytest.mark.parametrize("chunk", [1, 2, 4, 8, 16, 32])
def test_chunkwise_form_equals_recurrence(chunk):
    d = _rand(9, B=2, T=32, H=2, dk=8, dv=6)
    o, hT = orc.forward(**d)
    o2, hT2 = cw.forward(**d, chunk=chunk)
    np.testing.assert_allclose(o2, o, atol=2e-12)
    np.testing.assert_allclose(hT2, hT, atol=2e-12)


def test_chunkwise_form_strong_decay_no_overflow():
    d = _rand(10, B=1, T=128, H=1, dk=8, dv=8, alpha_lo=0.01)
    d["alpha"] = np.random.default_rng(0).uniform(0.01, 0.3, d["alpha"].shape)
    o, hT = orc.forward(**d)
    o2, hT2 = cw.forward(**d, chunk=64)
    assert np.all(np.isfinite(o2))
    np.testing.assert_allclose(o2, o, atol=1e-11)
    np.testing.assert_allclose(hT2, hT, atol=1e-11)


def test_segment_invariance_and_decode_wrapper():
    d = _rand(11, B=2, T=24, H=2)
    o, hT = orc.forward(**d)
    first = {kk: (vv[:, :10] if kk != "h0" else vv) for kk, vv in d.items()}
    o1, h1 = orc.forward(**first)
    second = {kk: (vv[:, 10:] if kk != "h0" else h1) for kk, vv in d.items()}
    o2, h2 = orc.forward(**second)
    np.testing.assert_allclose(np.concatenate([o1, o2], axis=1), o, atol=1e-14)
    np.testing.assert_allclose(h2, hT, atol=1e-14)
    mv = lambda a: np.moveaxis(a, 1, 0)
    od, hd = orc.decode(d["h0"], mv(d["q"]), mv(d["k"]), mv(d["v"]), mv(d["beta"]),
                        mv(d["alpha"]), mv(d["lam"]))
    np.testing.assert_allclose(np.moveaxis(od, 0, 1), o, atol=1e-14)
    np.testing.assert_allclose(hd, hT, atol=1e-14)


def test_heads_and_batches_are_independent():
    d = _rand(12, B=2, T=16, H=3)
    o, hT = orc.forward(**d)
    for b in range(2):
        for hh in range(3):
            sl = {kk: (vv[b:b + 1, :, hh:hh + 1] if kk != "h0" else vv[b:b + 1, hh:hh + 1])
                  for kk, vv in d.items()}
            o1, h1 = orc.forward(**sl)
            np.testing.assert_allclose(o1[0, :, 0], o[b, :, hh], atol=1e-15)
            np.testing.assert_allclose(h1[0, 0], hT[b, hh], atol=1e-15)


def test_golden_fixture_reproduced():
    """The stored results of a tiny seeded problem (tests/golden/qdelta_tiny.txt, written by make_golden.py
    from the oracle alone) are reproduced: guards against unintended changes of the oracle's arithmetic."""
    import importlib.util
    here = os.path.dirname(os.path.abspath(__file__))
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    got = mod.compute()
    lines = [l for l in open(os.path.join(here, "golden", "qdelta_tiny.txt")) if not l.startswith("#")]
    assert len(lines) == 2 * len(got)
    for head, vals in zip(lines[0::2], lines[1::2]):
        f = head.split()
        name, shape = f[0], tuple(int(x) for x in f[1:])
        want = np.array([float(x) for x in vals.split()]).reshape(shape)
        assert np.asarray(got[name]).shape == shape
        np.testing.assert_allclose(np.asarray(got[name], np.float64), want, rtol=1e-13, atol=1e-15)
