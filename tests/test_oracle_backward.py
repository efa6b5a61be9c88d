"""Pins of the reverse-pass oracle (CPU only)."""
import numpy as np
import pytest

from oracle import recurrence as orc
from oracle import chunkwise_form as cw
import independent_forms as ind


def _rand(seed, B=1, T=6, H=2, dk=4, dv=3):
    r = np.random.default_rng(seed)
    unit = lambda x: x / np.linalg.norm(x, axis=-1, keepdims=True)
    d = dict(q=unit(r.standard_normal((B, T, H, dk))), k=unit(r.standard_normal((B, T, H, dk))),
             v=r.standard_normal((B, T, H, dv)), beta=r.uniform(0.1, 0.9, (B, T, H)),
             alpha=r.uniform(0.4, 0.95, (B, T, H)), lam=r.uniform(0.1, 0.9, (B, T, H)),
             h0=0.3 * r.standard_normal((B, H, dk, dv)))
    up = dict(dO=r.standard_normal((B, T, H, dv)), dhT=r.standard_normal((B, H, dk, dv)))
    return d, up


def _loss(d, up):
    o, hT = orc.forward(**d)
    return float(np.sum(o * up["dO"]) + np.sum(hT * up["dhT"]))


GRAD_OF = dict(q="dq", k="dk", v="dv", beta="dbeta", alpha="dalpha", lam="dlam", h0="dh0")


def test_finite_differences_all_inputs():
    d, up = _rand(0)
    g = orc.backward(**d, **up, ckpt=4)
    eps = 1e-6
    rng = np.random.default_rng(1)
    for name, gname in GRAD_OF.items():
        flat = d[name].reshape(-1)
        idxs = range(flat.size) if flat.size <= 40 else rng.choice(flat.size, 40, replace=False)
        for i in idxs:
            old = flat[i]
            flat[i] = old + eps; lp = _loss(d, up)
            flat[i] = old - eps; lm = _loss(d, up)
            flat[i] = old
            fd = (lp - lm) / (2 * eps)
            an = g[gname].reshape(-1)[i]
            assert abs(fd - an) <= 2e-7 * max(1.0, abs(fd)), (name, i, fd, an)


def test_directional_derivative_medium():
    d, up = _rand(2, B=2, T=48, H=2, dk=16, dv=12)
    g = orc.backward(**d, **up, ckpt=16)
    rng = np.random.default_rng(3)
    dirs = {n: rng.standard_normal(d[n].shape) for n in GRAD_OF}
    an = sum(np.sum(g[GRAD_OF[n]] * dirs[n]) for n in GRAD_OF)
    eps = 1e-6
    plus = {n: d[n] + eps * dirs[n] for n in GRAD_OF}
    minus = {n: d[n] - eps * dirs[n] for n in GRAD_OF}
    fd = (_loss(plus, up) - _loss(minus, up)) / (2 * eps)
    assert abs(fd - an) <= 1e-6 * max(1.0, abs(an))


@pytest.mark.parametrize("ckpt", [1, 5, 64])
def test_checkpoint_spacing_does_not_matter(ckpt):
    d, up = _rand(4, T=23)
    a = orc.backward(**d, **up, ckpt=7)
    b = orc.backward(**d, **up, ckpt=ckpt)
    for n in a:
        np.testing.assert_allclose(a[n], b[n], rtol=0, atol=1e-13)


@pytest.mark.parametrize("chunk", [1, 4, 8, 32])
def test_chunkwise_backward_equals_reverse_pass(chunk):
    d, up = _rand(5, B=2, T=32, H=2, dk=8, dv=6)
    a = orc.backward(**d, **up)
    b = cw.backward(**d, **up, chunk=chunk)
    for n in a:
        np.testing.assert_allclose(b[n], a[n], rtol=0, atol=5e-12, err_msg=n)


def test_optional_arguments():
    d, up = _rand(6, T=10)
    d1 = dict(d); d1["alpha"] = np.ones_like(d["alpha"]); d1["lam"] = np.zeros_like(d["lam"])
    a = orc.backward(**d1, **up)
    b = orc.backward(d["q"], d["k"], d["v"], d["beta"], None, None, d["h0"], up["dO"], up["dhT"])
    for n in a:
        np.testing.assert_allclose(a[n], b[n], rtol=0, atol=1e-14)
    d2 = dict(d); d2["h0"] = np.zeros_like(d["h0"])
    a = orc.backward(**d2, dO=up["dO"], dhT=np.zeros_like(up["dhT"]))
    b = orc.backward(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], None, up["dO"], None)
    for n in a:
        np.testing.assert_allclose(a[n], b[n], rtol=0, atol=1e-14)


def _gdr_loss(q, k, v, beta, alpha, S0, dO, dST):
    o, S = ind.gated_delta_rule(q, k, v, beta, alpha, S0)
    return float(np.sum(o * dO) + np.sum(S * dST))


def test_lambda_zero_gradients_match_gated_delta_rule_fd():
    # gradients of the ordinary gated delta rule (Eq. 3), by finite differences of the
    # independently coded rule, equal the oracle's gradients at lambda = 0
    d, up = _rand(7, T=8, H=1)
    d["lam"][:] = 0.0
    g = orc.backward(**d, **up)
    q, k, v = d["q"][0, :, 0].copy(), d["k"][0, :, 0].copy(), d["v"][0, :, 0].copy()
    beta, alpha = d["beta"][0, :, 0].copy(), d["alpha"][0, :, 0].copy()
    S0 = d["h0"][0, 0].T.copy()
    dO, dST = up["dO"][0, :, 0], up["dhT"][0, 0].T
    eps = 1e-6
    for arr, gname in ((q, "dq"), (k, "dk"), (v, "dv"), (beta, "dbeta"), (alpha, "dalpha")):
        ga = g[gname][0, :, 0]
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = arr[i]
            arr[i] = old + eps; lp = _gdr_loss(q, k, v, beta, alpha, S0, dO, dST)
            arr[i] = old - eps; lm = _gdr_loss(q, k, v, beta, alpha, S0, dO, dST)
            arr[i] = old
            assert abs((lp - lm) / (2 * eps) - ga[i]) <= 2e-7 * max(1.0, abs(ga[i])), (gname, i)


def test_logit_gates_forward_is_sigmoid_composition_and_gradients_match_finite_differences():
    # forward_logits / backward_logits: the gates are sigmoid(z); pinned by the values of the sigmoid at known points
    # and by central finite differences of the whole composite with respect to every logit
    assert np.allclose(orc.gates_from_logits(np.array([0.0, np.log(3.0), -np.log(3.0), 800.0, -800.0]))[0],
                       [0.5, 0.75, 0.25, 1.0, 0.0], rtol=0, atol=1e-15)
    d, up = _rand(21)
    r = np.random.default_rng(22)
    z = dict(beta=r.normal(0, 1.5, d["beta"].shape), alpha=r.normal(1.0, 1.0, d["alpha"].shape), lam=r.normal(-0.8, 1.0, d["lam"].shape))
    sig = lambda x: 1.0 / (1.0 + np.exp(-x))
    o1, h1 = orc.forward_logits(d["q"], d["k"], d["v"], z["beta"], z["alpha"], z["lam"], d["h0"])
    o2, h2 = orc.forward(d["q"], d["k"], d["v"], sig(z["beta"]), sig(z["alpha"]), sig(z["lam"]), d["h0"])
    assert np.allclose(o1, o2, rtol=1e-13, atol=1e-13) and np.allclose(h1, h2, rtol=1e-13, atol=1e-13)

    def loss():
        o, hT = orc.forward_logits(d["q"], d["k"], d["v"], z["beta"], z["alpha"], z["lam"], d["h0"])
        return float(np.sum(o * up["dO"]) + np.sum(hT * up["dhT"]))
    g = orc.backward_logits(d["q"], d["k"], d["v"], z["beta"], z["alpha"], z["lam"], d["h0"], up["dO"], up["dhT"], ckpt=4)
    eps = 1e-6
    for name, gname in (("beta", "dbeta"), ("alpha", "dalpha"), ("lam", "dlam")):
        flat, gflat = z[name].reshape(-1), g[gname].reshape(-1)
        for i in range(flat.size):
            old = flat[i]
            flat[i] = old + eps; lp = loss()
            flat[i] = old - eps; lm = loss()
            flat[i] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - gflat[i]) <= 1e-6 * max(1.0, abs(fd)), (name, i, fd, gflat[i])
    # the other gradients are those of the plain call at the same gate values; absent logits stay absent
    g0 = orc.backward(d["q"], d["k"], d["v"], sig(z["beta"]), sig(z["alpha"]), sig(z["lam"]), d["h0"], up["dO"], up["dhT"], ckpt=4)
    for n in ("dq", "dk", "dv", "dh0"):
        assert np.allclose(g[n], g0[n], rtol=1e-12, atol=1e-12)
    gn = orc.backward_logits(d["q"], d["k"], d["v"], z["beta"], None, None, d["h0"], up["dO"], up["dhT"], ckpt=4)
    assert gn["dalpha"] is None and gn["dlam"] is None


def test_l2_normalisation_stage_pinned():
    # unit rows up to the constant under the root, closed form on a 3-4-0 row, gradient orthogonal to the row
    # direction (for eps -> 0), and central finite differences through the whole composite for q and k
    x = np.array([[3.0, 4.0, 0.0]])
    assert np.allclose(orc.l2_normalize(x), x / np.sqrt(25.0 + orc.NORM_EPS), rtol=0, atol=1e-15)
    d, up = _rand(31)
    r = np.random.default_rng(32)
    d["q"] = 2.0 * r.standard_normal(d["q"].shape)          # un-normalised rows
    d["k"] = 0.5 * r.standard_normal(d["k"].shape)
    assert np.allclose(np.linalg.norm(orc.l2_normalize(d["q"]), axis=-1), 1.0, atol=1e-6)
    gx = orc.l2_normalize_backward(d["q"], r.standard_normal(d["q"].shape))
    assert np.max(np.abs(np.sum(gx * d["q"], axis=-1))) < 1e-5

    def loss():
        o, hT = orc.forward_fused(**d, norm_qk=True)
        return float(np.sum(o * up["dO"]) + np.sum(hT * up["dhT"]))
    g = orc.backward_fused(**d, **up, ckpt=4, norm_qk=True)
    eps = 1e-6
    for name, gname in (("q", "dq"), ("k", "dk"), ("v", "dv"), ("beta", "dbeta")):
        flat, gflat = d[name].reshape(-1), g[gname].reshape(-1)
        for i in range(0, flat.size, 3):
            old = flat[i]
            flat[i] = old + eps; lp = loss()
            flat[i] = old - eps; lm = loss()
            flat[i] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - gflat[i]) <= 2e-6 * max(1.0, abs(fd)), (name, i, fd, gflat[i])
    # rows that are already unit vectors: the stage changes nothing but the 1e-6 under the root
    d2, up2 = _rand(33)
    o1, h1 = orc.forward_fused(**d2, norm_qk=True)
    o2, h2 = orc.forward(**d2)
    assert np.allclose(o1, o2, rtol=0, atol=1e-5) and np.allclose(h1, h2, rtol=0, atol=1e-5)
