"""Seeded synthetic inputs for the Structured Recurrent Mixer (SRM) decode path.

This module only *draws numbers*: model shapes, random-init parameters, prompts.
It contains none of the method's arithmetic (no mixing, no norms, no sampling), so
both the CPU oracle's tests and the CUDA path's tests can be fed from it without
sharing any code of the method itself.

Shapes follow the paper's generation benchmarks (Tables 1, 2 and 11: d_model 512
or 1024, 8 or 16 layers, 8k..32k vocabulary, fixed-length generation at large
batch) and the GRPO rollout shape (a few prompts, each replicated many times).
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np


@dataclass(frozen=True)
class SRMShape:
    """Static description of one SRM model (notation: L layers, d model width,
    h heads of width d/h, F = ffn_mult*d, V vocabulary, n_ctx positions)."""
    n_layers: int
    d_model: int
    vocab: int
    n_ctx: int
    n_heads: int = 4
    ffn_mult: int = 4
    dtype: str = "bf16"        # "fp32" or "bf16" (weights + GEMM inputs; fp32 accumulate)
    seed: int = 0
    ln_eps: float = 1e-5
    head_proj: bool = False    # per-head input projections I_h (stacked: W_in[d,d]) and output projection W_out[d,d]
    mixer: str = "mixed"       # "mixed" (half row-repeat, half column-repeat heads), "combined" (every head holds both
                               # matrices, outputs linearly combined, twice the cache) or "kernel" (kernel_size filters)
    kernel_size: int = 1       # number of column-repeat filters of the "kernel" mixer (Eq. 11)

    @property
    def d_ffn(self) -> int:
        return self.ffn_mult * self.d_model

    @property
    def d_head(self) -> int:
        return self.d_model // self.n_heads

    def as_dict(self):
        return asdict(self)


# The five benchmark configurations (model part only; workloads below).
CONFIGS = {
    "tiny":  SRMShape(n_layers=2,  d_model=64,   vocab=256,   n_ctx=32,   dtype="fp32", seed=0),
    "small": SRMShape(n_layers=8,  d_model=512,  vocab=8000,  n_ctx=512,  dtype="bf16", seed=1),
    "mid":   SRMShape(n_layers=16, d_model=1024, vocab=32000, n_ctx=1024, dtype="bf16", seed=2),
    "rl":    SRMShape(n_layers=24, d_model=1536, vocab=32000, n_ctx=1024, dtype="bf16", seed=3),
}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result is fp32 holding
    bf16-representable values. Pure input quantisation, so that the oracle and the
    device both start from *identical* parameter values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of already bf16-representable fp32 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    assert not np.any(u & 0xFFFF), "values are not bf16-representable"
    return (u >> 16).astype(np.uint16)


def make_weights(shape: SRMShape, *, std: float = 0.02, alpha_std: float | None = None,
                 beta_std: float | None = None, lam_lo: float = 0.9) -> dict:
    """Random-init parameters, N(0, std^2) from `shape.seed`.

    Returns a dict of fp32 numpy arrays:
      E[V,d], lnf_g[d], lnf_b[d], W_lm[V,d], and a list "layers" of dicts with
      ln1_g, ln1_b, alpha[h,n_ctx], beta[n_ctx,d], lam[h], ln2_g, ln2_b,
      W1[F,d], b1[F], W2[d,F], b2[d], and with shape.head_proj also W_in[d,d] (rows g*d_h..(g+1)*d_h are
      head g's input projection I_g) and W_out[d,d] (the output projection P_out).
    Norm gains are 1 + N(0,std^2) and norm shifts N(0,std^2) so that the affine part of
    every norm is exercised. The decay constants lam are uniform on (lam_lo, 1) except
    head 0 of each layer, which is exactly 1 (the closed end of the allowed interval).
    In bf16 mode the matrices (E, W1, W2, W_lm, W_in, W_out) are rounded to bf16 once, here.
    """
    rng = np.random.Generator(np.random.Philox(key=shape.seed))
    d, F, V, n, h = shape.d_model, shape.d_ffn, shape.vocab, shape.n_ctx, shape.n_heads
    a_std = std if alpha_std is None else alpha_std
    b_std = std if beta_std is None else beta_std

    def nrm(*s, sd=std):
        return (rng.standard_normal(s, dtype=np.float32) * np.float32(sd)).astype(np.float32)

    def mat(*s):
        w = nrm(*s)
        return round_to_bf16(w) if shape.dtype == "bf16" else w

    W = {"E": mat(V, d), "layers": []}
    for _ in range(shape.n_layers):
        lam = rng.uniform(lam_lo, 1.0, size=h).astype(np.float32)
        lam[0] = 1.0
        W["layers"].append({
            "ln1_g": (1.0 + nrm(d)).astype(np.float32), "ln1_b": nrm(d),
            "alpha": nrm(h, n, sd=a_std), "beta": nrm(n, d, sd=b_std), "lam": lam,
            "ln2_g": (1.0 + nrm(d)).astype(np.float32), "ln2_b": nrm(d),
            "W1": mat(F, d), "b1": nrm(F), "W2": mat(d, F), "b2": nrm(d),
        })
        lw = W["layers"][-1]
        if shape.mixer == "combined":      # second set of repeated weights and decays, and the combination weights
            lam_c = rng.uniform(lam_lo, 1.0, size=h).astype(np.float32)
            lam_c[-1] = 1.0
            lw["alpha_col"] = nrm(h, n, sd=a_std)
            lw["lam_col"] = lam_c
            lw["w_comb"] = (0.5 + 0.5 * rng.random(size=(h, 2))).astype(np.float32)
        elif shape.mixer == "kernel":      # k filters instead of h heads
            k = shape.kernel_size
            lam_k = rng.uniform(lam_lo, 1.0, size=k).astype(np.float32)
            lam_k[0] = 1.0
            lw["alpha"] = nrm(k, n, sd=a_std)
            lw["lam"] = lam_k
        if shape.head_proj:        # drawn last, so the tensors above do not depend on the switch within a layer
            W["layers"][-1]["W_in"] = mat(d, d)
            W["layers"][-1]["W_out"] = mat(d, d)
    W["lnf_g"] = (1.0 + nrm(d)).astype(np.float32)
    W["lnf_b"] = nrm(d)
    W["W_lm"] = mat(V, d)
    return W


def uniform_prompts(batch: int, n: int, vocab: int, seed: int) -> np.ndarray:
    """int32 [batch, n] token ids uniform on [0, vocab)."""
    rng = np.random.Generator(np.random.Philox(key=seed + 1_000_003))
    return rng.integers(0, vocab, size=(batch, n), dtype=np.int64).astype(np.int32)


def zipf_prompts(batch: int, n: int, vocab: int, seed: int, s: float = 1.1) -> np.ndarray:
    """int32 [batch, n] token ids with P(id = r-1) proportional to r^-s, r = 1..vocab
    (inverse-CDF draw)."""
    rng = np.random.Generator(np.random.Philox(key=seed + 2_000_003))
    p = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(p)
    cdf /= cdf[-1]
    u = rng.random(size=(batch, n))
    ids = np.searchsorted(cdf, u, side="right")
    return np.minimum(ids, vocab - 1).astype(np.int32)


def replicated_prompts(n_prompts: int, replicas: int, n: int, vocab: int, seed: int,
                       s: float = 1.1) -> np.ndarray:
    """Rollout shape: `n_prompts` distinct Zipf prompts, each repeated `replicas` times;
    row index = prompt * replicas + replica."""
    base = zipf_prompts(n_prompts, n, vocab, seed, s)
    return np.repeat(base, replicas, axis=0)


# Workloads of the five benchmark configurations.
WORKLOADS = {
    "tiny":  dict(model="tiny",  batch=4,     prompt_len=8,   gen=24,  prompts="uniform", sampling="greedy"),
    "small": dict(model="small", batch=256,   prompt_len=128, gen=384, prompts="uniform", sampling="greedy"),
    "mid":   dict(model="mid",   batch=4096,  prompt_len=256, gen=768, prompts="zipf",    sampling="greedy"),
    "sweep": dict(model="mid",   batch=None,  prompt_len=128, gen=256, prompts="uniform", sampling="greedy"),
    "rl":    dict(model="rl",    batch=16384, prompt_len=200, gen=512, prompts="replicated",
                  n_prompts=16, replicas=1024, sampling="topk", top_k=50, temperature=0.8),
}


def make_prompts(workload: str, batch: int | None = None) -> np.ndarray:
    w = WORKLOADS[workload]
    shape = CONFIGS[w["model"]]
    B = w["batch"] if batch is None else batch
    if w["prompts"] == "uniform":
        return uniform_prompts(B, w["prompt_len"], shape.vocab, shape.seed)
    if w["prompts"] == "zipf":
        return zipf_prompts(B, w["prompt_len"], shape.vocab, shape.seed)
    reps = max(1, B // w["n_prompts"])
    return replicated_prompts(w["n_prompts"], reps, w["prompt_len"], shape.vocab, shape.seed)[:B]
