"""Pins for the head-projection variant of the token mixer (Method/Architecture, Eq. 10):
Y = P_out (concat_g [(I_g X) M_g + beta_g]), X in R^{d x n} with one column per position."""
import dataclasses

import numpy as np

import srm_inputs as I
from oracle import srm_oracle as O


def _layer(rng, d, h, n, with_proj=True):
    lw = dict(alpha=rng.normal(size=(h, n)), beta=rng.normal(size=(n, d)), lam=rng.uniform(0.9, 1.0, size=h))
    if with_proj:
        lw["W_in"] = rng.normal(size=(d, d)) / np.sqrt(d)
        lw["W_out"] = rng.normal(size=(d, d)) / np.sqrt(d)
    return lw


def test_eq10_brute_force_in_the_papers_orientation():
    """Written the way the paper prints it: X is d x n, head g has its own I_g (d_h x d), its d_h x n block is
    multiplied from the right by the n x n matrix M_g, its bias block is added, the blocks are stacked and
    P_out (d x d) is applied from the left."""
    rng = np.random.default_rng(0)
    d, h, n = 8, 4, 6
    dh = d // h
    lw = _layer(rng, d, h, n)
    Z = rng.normal(size=(n, d))                       # oracle layout: one row per position
    X = Z.T                                           # paper layout: one column per position
    blocks = []
    for g, kind in enumerate(O.head_kinds(h)):
        I_g = lw["W_in"][g * dh:(g + 1) * dh, :]
        M_g = np.zeros((n, n))
        for i in range(n):
            for j in range(i, n):
                M_g[i, j] = lw["lam"][g] ** (j - i) * (lw["alpha"][g][i] if kind == "row" else lw["alpha"][g][j])
        B_g = lw["beta"][:, g * dh:(g + 1) * dh].T    # d_h x n
        blocks.append((I_g @ X) @ M_g + B_g)
    want = (lw["W_out"] @ np.concatenate(blocks, axis=0)).T
    got, _ = O.token_mixer_parallel(Z, lw, h)
    assert np.max(np.abs(got - want)) < 1e-12


def test_identity_projections_reduce_to_the_unprojected_mixer():
    rng = np.random.default_rng(1)
    d, h, n = 16, 4, 9
    lw = _layer(rng, d, h, n, with_proj=False)
    Z = rng.normal(size=(n, d))
    y0, s0 = O.token_mixer_parallel(Z, lw, h)
    lw_id = dict(lw, W_in=np.eye(d), W_out=np.eye(d))
    y1, s1 = O.token_mixer_parallel(Z, lw_id, h)
    assert np.array_equal(y0, y1) and np.array_equal(s0, s1)
    # and a transposed / swapped use of the projections would not pass: a permutation as W_in must permute channels
    perm = rng.permutation(d)
    Pm = np.eye(d)[perm]                               # (Pm z)[i] = z[perm[i]]
    y2, _ = O.token_mixer_parallel(Z, dict(lw, W_in=Pm, W_out=np.eye(d)), h)
    y2_want, _ = O.mixer_parallel(Z[:, perm], lw["alpha"], lw["beta"], lw["lam"], h)
    assert np.max(np.abs(y2 - y2_want)) < 1e-12


def test_parallel_equals_recurrent_with_projections_and_state_is_of_projected_values():
    rng = np.random.default_rng(2)
    d, h, n = 16, 4, 12
    lw = _layer(rng, d, h, n)
    Z = rng.normal(size=(n, d))
    yp, sp = O.token_mixer_parallel(Z, lw, h)
    S = np.zeros(d)
    for t in range(n):
        yt, S = O.token_mixer_recurrent(Z[t], S, t, lw, h)
        assert np.max(np.abs(yt - yp[t])) < 1e-9
    assert np.max(np.abs(S - sp)) < 1e-9
    # the cache is d numbers per layer and sample, as without projections, and it is the sum term of Q = Z W_in^T
    Q = Z @ lw["W_in"].T
    _, s_q = O.mixer_parallel(Q, lw["alpha"], lw["beta"], lw["lam"], h)
    assert sp.shape == (d,) and np.array_equal(sp, s_q)


def test_full_model_with_projections_parallel_equals_recurrent_and_is_causal():
    shape = dataclasses.replace(I.CONFIGS["tiny"], head_proj=True)
    W = I.make_weights(shape, alpha_std=0.5)
    assert W["layers"][0]["W_in"].shape == (64, 64) and W["layers"][1]["W_out"].shape == (64, 64)
    orc = O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W, n_heads=shape.n_heads)
    toks = I.uniform_prompts(3, 20, shape.vocab, seed=5)
    lp, sp = orc.forward_parallel(toks)
    lr, sr = orc.prefill_recurrent(toks)
    assert np.max(np.abs(lp - lr)) < 1e-9 and np.max(np.abs(sp - sr)) < 1e-9
    toks2 = toks.copy()
    toks2[:, 13] = (toks2[:, 13] + 1) % shape.vocab
    lp2, _ = orc.forward_parallel(toks2)
    assert np.array_equal(lp2[:, :13], lp[:, :13]) and not np.array_equal(lp2[:, 13:], lp[:, 13:])
    # the projections matter: dropping them changes the logits
    W0 = {**W, "layers": [{k: v for k, v in lw.items() if k not in ("W_in", "W_out")} for lw in W["layers"]]}
    orc0 = O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W0, n_heads=shape.n_heads)
    assert np.max(np.abs(orc0.forward_parallel(toks)[0] - lp)) > 1e-3


def test_weights_without_the_switch_are_unchanged_by_it():
    a = I.make_weights(I.CONFIGS["tiny"])
    b = I.make_weights(dataclasses.replace(I.CONFIGS["tiny"], head_proj=True))
    assert np.array_equal(a["E"], b["E"]) and np.array_equal(a["layers"][0]["W1"], b["layers"][0]["W1"])
    assert "W_in" not in a["layers"][0]
