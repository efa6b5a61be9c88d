"""Seeded synthetic inputs for the Q-Delta kernels and for their CPU checker.

This module holds NONE of the method's arithmetic: it only draws random
tensors with the shapes and value distributions of the five benchmark
configurations, rounds them once to the storage dtype, and hands the same bytes
to whoever asks.  It depends on numpy only and never touches the CUDA library.

Draw order (independent child streams of one seed): q, k, v, beta, alpha, lam,
h0, dO, dhT, key-pool, key-pool indices.  q and k are N(0,1) rows L2-normalised
per (b,t,h); v ~ N(0,1); beta, alpha, lam = sigmoid(N(0,1)) unless a regime
says otherwise; h0, dhT ~ N(0, std 0.02) in fp32; dO ~ N(0,1).
"""
from dataclasses import dataclass, replace

import numpy as np

__all__ = ["Config", "CONFIGS", "REGIMES", "round_bf16", "bf16_bits", "bits_to_f32",
           "make_chunk_inputs", "make_decode_state", "make_decode_tokens"]


@dataclass(frozen=True)
class Config:
    name: str
    B: int
    T: int
    H: int
    dk: int
    dv: int
    chunk: int
    dtype: str            # "f32" | "bf16" : storage dtype of q,k,v,coefficients,o,dO
    h0: bool              # random initial state (else zeros / absent)
    backward: bool        # also draw dO, dhT
    key_pool: int = 0     # >0: keys = pool vector + N(0, std 0.1) noise, renormalised
    regime: str = "config"
    seed: int = 0


CONFIGS = {
    # tiny fp32 forward
    "cfg0": Config("cfg0", 1, 256, 2, 64, 64, 64, "f32", False, False),
    # bf16 forward, LM-training shape
    "cfg1": Config("cfg1", 8, 2048, 16, 128, 128, 64, "bf16", True, False),
    # bf16 forward + backward at the same shape (headline)
    "cfg2": Config("cfg2", 8, 2048, 16, 128, 128, 64, "bf16", True, True),
    # long context, pooled keys
    "cfg3": Config("cfg3", 1, 32768, 32, 128, 128, 64, "bf16", True, True, key_pool=512),
    # decode: batch 256, 16 heads (T is the number of steps)
    "cfg4": Config("cfg4", 256, 1000, 16, 128, 128, 64, "bf16", True, False),
}

# coefficient regimes used for parity only (the default sigmoid(N(0,1)) forget
# gate erases the state within a few tokens, which could hide state-passing bugs)
REGIMES = ("config", "alpha_one", "alpha_slow", "lam_zero", "lam_one", "beta_spikes",
           "trained_like")


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 to the nearest bf16 (ties to even); returns fp32 holding bf16 values."""
    return bits_to_f32(bf16_bits(x))


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> uint16 bf16 bit patterns, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return round_bf16(x) if dtype == "bf16" else x


def _sigmoid(z):
    return 1.0 / (1.0 + np.exp(-z))


def _unit_rows(x):
    return x / np.sqrt(np.sum(x.astype(np.float64) ** 2, axis=-1, keepdims=True)).astype(np.float32)


def _coefficients(cfg, rng_b, rng_a, rng_l, shape):
    beta = _sigmoid(rng_b.standard_normal(shape, dtype=np.float32))
    alpha = _sigmoid(rng_a.standard_normal(shape, dtype=np.float32))
    lam = _sigmoid(rng_l.standard_normal(shape, dtype=np.float32))
    r = cfg.regime
    if r == "alpha_one":
        alpha = np.ones(shape, np.float32)
    elif r == "alpha_slow":
        alpha = (0.95 + 0.05 * rng_a.random(shape, dtype=np.float32)).astype(np.float32)
        alpha = np.minimum(alpha, np.float32(0.99999))
    elif r == "lam_zero":
        lam = np.zeros(shape, np.float32)
    elif r == "lam_one":
        lam = np.ones(shape, np.float32)
        alpha = (0.9 + 0.1 * rng_a.random(shape, dtype=np.float32)).astype(np.float32)
    elif r == "beta_spikes":
        u = rng_b.random(shape, dtype=np.float32)
        beta = np.where(u < 0.25, 0.0, np.where(u > 0.75, 1.0, beta)).astype(np.float32)
        alpha = (0.9 + 0.1 * rng_a.random(shape, dtype=np.float32)).astype(np.float32)
    elif r == "trained_like":
        beta = _sigmoid(-3.0 + 0.5 * rng_b.standard_normal(shape, dtype=np.float32))
        lam = _sigmoid(-0.8 + 0.5 * rng_l.standard_normal(shape, dtype=np.float32))
        alpha = _sigmoid(4.0 + rng_a.standard_normal(shape, dtype=np.float32))
    elif r != "config":
        raise ValueError("unknown regime %r" % r)
    return beta.astype(np.float32), alpha.astype(np.float32), lam.astype(np.float32)


def make_chunk_inputs(cfg: Config, **overrides) -> dict:
    """Inputs of one chunkwise forward (+backward) call.

    Returns fp32 numpy arrays whose values are exactly representable in
    ``cfg.dtype``: q,k [B,T,H,dk]; v [B,T,H,dv]; beta,alpha,lam [B,T,H];
    h0 [B,H,dk,dv] or None; and, if cfg.backward, dO [B,T,H,dv], dhT [B,H,dk,dv].
    """
    if overrides:
        cfg = replace(cfg, **overrides)
    ss = np.random.SeedSequence(cfg.seed).spawn(11)
    rq, rk, rv, rb, ra, rl, rh, rdo, rdh, rpool, ridx = (np.random.default_rng(s) for s in ss)
    B, T, H, dk, dv = cfg.B, cfg.T, cfg.H, cfg.dk, cfg.dv
    q = _unit_rows(rq.standard_normal((B, T, H, dk), dtype=np.float32))
    if cfg.key_pool > 0:
        pool = _unit_rows(rpool.standard_normal((B, H, cfg.key_pool, dk), dtype=np.float32))
        idx = ridx.integers(0, cfg.key_pool, size=(B, T, H))
        k = rk.standard_normal((B, T, H, dk), dtype=np.float32) * np.float32(0.1)
        bi = np.arange(B)[:, None, None]
        hi = np.arange(H)[None, None, :]
        k += pool[bi, hi, idx]
        k = _unit_rows(k)
    else:
        k = _unit_rows(rk.standard_normal((B, T, H, dk), dtype=np.float32))
    v = rv.standard_normal((B, T, H, dv), dtype=np.float32)
    beta, alpha, lam = _coefficients(cfg, rb, ra, rl, (B, T, H))
    out = dict(q=_store(q, cfg.dtype), k=_store(k, cfg.dtype), v=_store(v, cfg.dtype),
               beta=_store(beta, cfg.dtype), alpha=_store(alpha, cfg.dtype),
               lam=_store(lam, cfg.dtype), h0=None)
    # alpha must stay inside (0,1] after rounding
    out["alpha"] = np.clip(out["alpha"], np.float32(2.0 ** -20), np.float32(1.0))
    if cfg.h0:
        out["h0"] = (rh.standard_normal((B, H, dk, dv), dtype=np.float32) * np.float32(0.02))
    if cfg.backward:
        out["dO"] = _store(rdo.standard_normal((B, T, H, dv), dtype=np.float32), cfg.dtype)
        out["dhT"] = (rdh.standard_normal((B, H, dk, dv), dtype=np.float32) * np.float32(0.02))
    return out


def make_decode_state(cfg: Config) -> np.ndarray:
    """Initial fp32 decode states [batch,H,dk,dv] ~ N(0, std 0.02)."""
    rng = np.random.default_rng(np.random.SeedSequence([cfg.seed, 0xDEC0DE]))
    return rng.standard_normal((cfg.B, cfg.H, cfg.dk, cfg.dv), dtype=np.float32) * np.float32(0.02)


def make_decode_tokens(cfg: Config, step0: int, nsteps: int) -> dict:
    """Token inputs of decode steps [step0, step0+nsteps).

    Each step has its own counter-based stream, so any window of steps can be
    drawn without drawing the ones before it.  Returns q,k [n,batch,H,dk],
    v [n,batch,H,dv], beta,alpha,lam [n,batch,H] (fp32 values representable in
    cfg.dtype)."""
    Bn, H, dk, dv = cfg.B, cfg.H, cfg.dk, cfg.dv
    q = np.empty((nsteps, Bn, H, dk), np.float32); k = np.empty_like(q)
    v = np.empty((nsteps, Bn, H, dv), np.float32)
    beta = np.empty((nsteps, Bn, H), np.float32); alpha = np.empty_like(beta); lam = np.empty_like(beta)
    for i in range(nsteps):
        rng = np.random.default_rng(np.random.SeedSequence([cfg.seed, 0x70CE, step0 + i]))
        q[i] = _unit_rows(rng.standard_normal((Bn, H, dk), dtype=np.float32))
        k[i] = _unit_rows(rng.standard_normal((Bn, H, dk), dtype=np.float32))
        v[i] = rng.standard_normal((Bn, H, dv), dtype=np.float32)
        beta[i], alpha[i], lam[i] = _coefficients(cfg, rng, rng, rng, (Bn, H))
    out = dict(q=_store(q, cfg.dtype), k=_store(k, cfg.dtype), v=_store(v, cfg.dtype),
               beta=_store(beta, cfg.dtype), alpha=_store(alpha, cfg.dtype),
               lam=_store(lam, cfg.dtype))
    out["alpha"] = np.clip(out["alpha"], np.float32(2.0 ** -20), np.float32(1.0))
    return out
