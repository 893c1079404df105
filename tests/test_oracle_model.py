"""Whole-model oracle checks: parallel == recurrent (1e-9 in fp64), causality, an
independent vectorised PyTorch restatement, generation bookkeeping, input generators."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from oracle import srm_oracle as O


def _tiny(alpha_std=None, **kw):
    shape = I.CONFIGS["tiny"]
    W = I.make_weights(shape, alpha_std=alpha_std, **kw)
    return shape, W, O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W,
                                 n_heads=shape.n_heads, ln_eps=shape.ln_eps)


@pytest.mark.parametrize("alpha_std", [None, 0.5])
def test_parallel_equals_recurrent_full_model(alpha_std):
    shape, W, orc = _tiny(alpha_std)
    toks = I.uniform_prompts(4, shape.n_ctx, shape.vocab, seed=11)
    lp, sp = orc.forward_parallel(toks)
    lr, sr = orc.prefill_recurrent(toks)
    assert np.max(np.abs(lp - lr)) < 1e-9
    assert np.max(np.abs(sp - sr)) < 1e-9


def test_tiny_config_generation_then_parallel_recheck():
    """Config 'tiny': 4 prompts of 8 tokens, greedy-decode 24 tokens with the recurrent form,
    then the parallel form over the full 32-token sequences gives the same logits."""
    shape, W, orc = _tiny()
    w = I.WORKLOADS["tiny"]
    prompts = I.make_prompts("tiny")
    assert prompts.shape == (4, 8)
    toks, logits, _ = orc.generate(prompts, w["gen"])
    full = np.concatenate([prompts, toks], axis=1)
    assert full.shape == (4, 32)
    lp, _ = orc.forward_parallel(full)
    for k in range(w["gen"]):
        assert np.max(np.abs(lp[:, 7 + k] - logits[k])) < 1e-9
        assert np.array_equal(np.argmax(lp[:, 7 + k], -1), toks[:, k])


def test_causality():
    shape, W, orc = _tiny(alpha_std=0.5)
    toks = I.uniform_prompts(2, 16, shape.vocab, seed=12)
    base, _ = orc.forward_parallel(toks)
    for t in [0, 5, 15]:
        alt = toks.copy()
        alt[:, t] = (alt[:, t] + 1) % shape.vocab
        out, _ = orc.forward_parallel(alt)
        assert np.array_equal(out[:, :t], base[:, :t])          # bit-identical before t
        assert np.max(np.abs(out[:, t] - base[:, t])) > 0       # and really different at t


def test_model_against_vectorised_torch_restatement():
    """Same reading of the block, written independently with torch.nn.functional and a
    broadcast (not looped) construction of the masked mixing matrices."""
    shape, W, orc = _tiny(alpha_std=0.3)
    toks = I.uniform_prompts(3, 20, shape.vocab, seed=13)
    got, got_state = orc.forward_parallel(toks)
    F = torch.nn.functional
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    n, d, h = 20, shape.d_model, shape.n_heads
    dh = d // h
    x = t(W["E"])[torch.from_numpy(toks).long()]
    ii = torch.arange(n)[:, None]; jj = torch.arange(n)[None, :]
    for lw in W["layers"]:
        z = F.layer_norm(x, (d,), t(lw["ln1_g"]), t(lw["ln1_b"]), shape.ln_eps)
        ys = []
        for g in range(h):
            lam = float(lw["lam"][g]); al = t(lw["alpha"][g][:n])
            decay = torch.where(jj >= ii, torch.tensor(lam, dtype=torch.float64) ** (jj - ii).clamp(min=0),
                                torch.zeros((), dtype=torch.float64))
            M = decay * (al[:, None] if g < h // 2 else al[None, :])
            zg = z[..., g * dh:(g + 1) * dh]                      # [B, n, dh]
            ys.append(torch.einsum("bic,ij->bjc", zg, M))
        x = x + torch.cat(ys, -1) + t(lw["beta"][:n])
        a = F.layer_norm(x, (d,), t(lw["ln2_g"]), t(lw["ln2_b"]), shape.ln_eps)
        x = x + F.linear(F.gelu(F.linear(a, t(lw["W1"]), t(lw["b1"]))), t(lw["W2"]), t(lw["b2"]))
    want = F.linear(F.layer_norm(x, (d,), t(W["lnf_g"]), t(W["lnf_b"]), shape.ln_eps), t(W["W_lm"])).numpy()
    assert np.max(np.abs(got - want)) < 1e-10


def test_fp32_oracle_close_to_fp64():
    shape, W, orc = _tiny()
    o32 = O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W, dtype=np.float32)
    toks = I.uniform_prompts(2, 12, shape.vocab, seed=14)
    l64, _ = orc.prefill_recurrent(toks)
    l32, _ = o32.prefill_recurrent(toks)
    assert l32.dtype == np.float32
    assert np.max(np.abs(l32 - l64)) / np.max(np.abs(l64)) < 1e-5


def test_input_generators():
    a = np.array([1.0, 1.00390625, 1.001953125, -3.1415926, 1e-3], dtype=np.float32)
    r = I.round_to_bf16(a)
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(r, want)
    assert I.bf16_bits(r).dtype == np.uint16
    z = I.zipf_prompts(64, 256, 32000, seed=2)
    assert z.min() >= 0 and z.max() < 32000
    assert (z == 0).mean() > 0.05 and (z < 10).mean() > 0.2      # heavy head of the Zipf law
    rp = I.make_prompts("rl", batch=64)
    assert rp.shape == (64, 200) and np.array_equal(rp[0], rp[3]) and not np.array_equal(rp[0], rp[4])
    W1 = I.make_weights(I.CONFIGS["tiny"]); W2 = I.make_weights(I.CONFIGS["tiny"])
    assert np.array_equal(W1["E"], W2["E"])
    for lw in W1["layers"]:
        assert lw["lam"][0] == 1.0 and np.all(lw["lam"] > 0.9) and np.all(lw["lam"] <= 1.0)
