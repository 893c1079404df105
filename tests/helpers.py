"""Shared test helpers: model construction for both sides, error metric."""
import numpy as np

import srm_inputs as I


def oracle_for(shape, W, dtype=np.float64):
    from oracle import srm_oracle as O
    return O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W,
                       n_heads=shape.n_heads, ln_eps=shape.ln_eps, dtype=dtype)


def rel_err_rows(got, want) -> float:
    """max over rows of max_i |got - want| / max_j |want_j| (rows = last axis)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    num = np.max(np.abs(got - want), axis=-1)
    den = np.maximum(np.max(np.abs(want), axis=-1), 1e-30)
    return float(np.max(num / den))


def top2_margin(logits) -> np.ndarray:
    part = np.partition(np.asarray(logits), -2, axis=-1)
    return part[..., -1] - part[..., -2]


def custom_shape(**kw):
    base = dict(n_layers=2, d_model=64, vocab=256, n_ctx=32, dtype="fp32", seed=0)
    base.update(kw)
    return I.SRMShape(**base)
