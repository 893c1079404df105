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


# ---- the model built from the further mixer variants (linearly combined heads; kernels of size k, Eq. 11) ----

def _variant(mixer, k=1, alpha_std=0.4):
    import dataclasses
    shape = dataclasses.replace(I.CONFIGS["tiny"], mixer=mixer, kernel_size=k)
    W = I.make_weights(shape, alpha_std=alpha_std)
    return shape, W, O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W, n_heads=shape.n_heads,
                                 ln_eps=shape.ln_eps, mixer=mixer, kernel_size=k)


@pytest.mark.parametrize("mixer,k", [("combined", 1), ("kernel", 4), ("kernel", 8), ("kernel", 1)])
def test_variant_model_parallel_equals_recurrent_and_is_causal(mixer, k):
    """The model-level facts the mathematics fixes hold for the variant models too: the explicit n x n matrices
    (the definition) and the recurrence give the same logits and the same cache to 1e-9 in fp64; a later token
    cannot change an earlier output."""
    shape, W, orc = _variant(mixer, k)
    toks = I.uniform_prompts(3, 20, shape.vocab, seed=14)
    lp, sp = orc.forward_parallel(toks)
    lr, sr = orc.prefill_recurrent(toks)
    C = {"combined": 2, "kernel": k}[mixer]
    assert sp.shape == (shape.n_layers, C, 3, shape.d_model) and sr.shape == sp.shape
    assert np.max(np.abs(lp - lr)) < 1e-9 and np.max(np.abs(sp - sr)) < 1e-9
    alt = toks.copy()
    alt[:, 9] = (alt[:, 9] + 1) % shape.vocab
    out, _ = orc.forward_parallel(alt)
    assert np.array_equal(out[:, :9], lp[:, :9]) and np.max(np.abs(out[:, 9] - lp[:, 9])) > 0


def test_combined_model_with_one_matrix_switched_off_per_head_is_the_mixed_model():
    """Combination weights (1, 0) on the first half of the heads and (0, 1) on the second half leave exactly the
    mixed-head model (row-repeat heads first, column-repeat heads second) with the matching parameters."""
    shape, W, orc = _variant("combined")
    h = shape.n_heads
    Wm = {k: v for k, v in W.items() if k != "layers"}
    Wm["layers"] = []
    for lw in W["layers"]:
        lw["w_comb"] = np.array([[1.0, 0.0]] * (h // 2) + [[0.0, 1.0]] * (h // 2), dtype=np.float32)
        m = {k: v for k, v in lw.items() if k not in ("alpha_col", "lam_col", "w_comb")}
        m["alpha"] = np.concatenate([lw["alpha"][:h // 2], lw["alpha_col"][h // 2:]])
        m["lam"] = np.concatenate([lw["lam"][:h // 2], lw["lam_col"][h // 2:]])
        Wm["layers"].append(m)
    orc_c = O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W, mixer="combined")
    orc_m = O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, Wm)
    toks = I.uniform_prompts(2, 12, shape.vocab, seed=15)
    lc, sc = orc_c.forward_parallel(toks)
    lm, sm = orc_m.forward_parallel(toks)
    assert np.max(np.abs(lc - lm)) < 1e-12
    dh = shape.d_model // h
    half = (h // 2) * dh
    assert np.max(np.abs(sc[:, 0, :, :half] - sm[:, :, :half])) < 1e-12       # row-repeat sum terms of the first heads
    assert np.max(np.abs(sc[:, 1, :, half:] - sm[:, :, half:])) < 1e-12       # column-repeat sum terms of the others


def test_kernel_model_of_size_one_is_a_model_of_column_repeat_heads():
    """k = 1: Eq. 11 is a single column-repeat matrix over all channels, i.e. the mixed-head recurrence with every
    head column-repeat and the same alpha, lambda: checked through Eq. 3's closed form on the first layer."""
    shape, W, orc = _variant("kernel", 1)
    toks = I.uniform_prompts(2, 10, shape.vocab, seed=16)
    _, _, xs = orc.forward_parallel(toks, keep_x=True)
    lw = orc.layers[0]
    x0 = orc.E[toks]
    z = O.layer_norm(x0, lw["ln1_g"], lw["ln1_b"], shape.ln_eps)
    n = toks.shape[1]
    y = np.zeros_like(z)
    for j in range(n):                              # Eq. 3: y_j = alpha_j sum_{i <= j} lambda^(j - i) z_i + beta_j
        acc = sum(lw["lam"][0] ** (j - i) * z[:, i] for i in range(j + 1))
        y[:, j] = lw["alpha"][0][j] * acc + lw["beta"][j]
    x1 = x0 + y
    x1 = x1 + O.feed_forward(O.layer_norm(x1, lw["ln2_g"], lw["ln2_b"], shape.ln_eps), lw["W1"], lw["b1"], lw["W2"], lw["b2"])
    assert np.max(np.abs(xs[0] - x1)) < 1e-10
