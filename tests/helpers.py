"""Shared test helpers: model construction for both sides, error metric."""
import functools

import numpy as np

import srm_inputs as I


@functools.lru_cache(maxsize=2)
def weights_for(name: str):
    """Seeded weights of a benchmark configuration (drawing the larger ones takes most of a minute: shared
    between the tests of one session; treat as read-only)."""
    return I.make_weights(I.CONFIGS[name])


def oracle_for(shape, W, dtype=np.float64):
    from oracle import srm_oracle as O
    return O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W,
                       n_heads=shape.n_heads, ln_eps=shape.ln_eps, dtype=dtype,
                       mixer=shape.mixer, kernel_size=shape.kernel_size)


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


def topp_is_strict(row, p, T, det, tol=2e-6):
    """True when neither decision of nucleus sampling is within rounding (fp32 exp, 2^-31 weight grid, against
    fp64) of flipping the drawn token. The nucleus closes where the descending cumulative mass reaches p Z: if
    that is within tol, a token at the edge may flip in or out, which moves u * mass by at most that token's
    weight. The draw compares u * mass with the CDF edges of the drawn token."""
    from oracle import srm_oracle as O
    order = O.topk_order(row.astype(np.float64), row.shape[0])
    w = np.exp((row[order].astype(np.float64) - row[order[0]]) / T)
    c = np.cumsum(w)
    m = len(det["ids"]) - 1
    g1 = (c[m] - p * c[-1]) / c[-1] if m < len(c) - 1 else np.inf        # (the whole vocabulary cannot grow)
    if m > 0 and p < 1.0:                            # (p = 1 keeps everything, whatever the last weights are)
        g1 = min(g1, (p * c[-1] - c[m - 1]) / c[-1])
    edge = 0.0 if g1 > tol else max(w[m], w[min(m + 1, len(w) - 1)]) / c[m]
    cdf, thr, k = det["cdf"], det["thr"], det["pick"]
    g2 = (cdf[k] - thr) / cdf[-1]
    if k > 0:
        g2 = min(g2, (thr - cdf[k - 1]) / cdf[-1])
    return g2 > tol + 2 * edge
