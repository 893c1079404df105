"""Pins for the oracle's norm, activation, Philox generator and token selection."""
import ctypes
import math
import os

import numpy as np
import pytest
import torch

from oracle import srm_oracle as O


def test_layer_norm_moments_and_library():
    rng = np.random.default_rng(0)
    x = rng.normal(2.0, 3.0, size=(5, 64))
    y = O.layer_norm(x, np.ones(64), np.zeros(64), 0.0)
    np.testing.assert_allclose(y.mean(-1), 0, atol=1e-13)
    np.testing.assert_allclose(y.var(-1), 1, rtol=1e-12)      # biased variance
    g, b = rng.normal(size=64), rng.normal(size=64)
    want = torch.nn.functional.layer_norm(torch.from_numpy(x), (64,), torch.from_numpy(g),
                                          torch.from_numpy(b), 1e-5).numpy()
    np.testing.assert_allclose(O.layer_norm(x, g, b, 1e-5), want, rtol=1e-12, atol=1e-12)


def test_gelu_identities_and_library():
    x = np.linspace(-6, 6, 241)
    y = O.gelu_erf(x)
    assert O.gelu_erf(np.zeros(1))[0] == 0.0
    np.testing.assert_allclose(y - O.gelu_erf(-x), x, atol=1e-14)          # gelu(x) - gelu(-x) = x
    np.testing.assert_allclose(y, [0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in x], atol=1e-15)
    want = torch.nn.functional.gelu(torch.from_numpy(x), approximate="none").numpy()
    np.testing.assert_allclose(y, want, atol=1e-14)
    # the tanh approximation is a different function: must be distinguishable
    tanh = torch.nn.functional.gelu(torch.from_numpy(x), approximate="tanh").numpy()
    assert np.max(np.abs(y - tanh)) > 1e-4


def test_feed_forward_against_torch_linear():
    rng = np.random.default_rng(1)
    d, F = 8, 32
    a = rng.normal(size=(3, d)); W1 = rng.normal(size=(F, d)); b1 = rng.normal(size=F)
    W2 = rng.normal(size=(d, F)); b2 = rng.normal(size=d)
    t = torch.from_numpy
    want = torch.nn.functional.linear(
        torch.nn.functional.gelu(torch.nn.functional.linear(t(a), t(W1), t(b1))), t(W2), t(b2)).numpy()
    np.testing.assert_allclose(O.feed_forward(a, W1, b1, W2, b2), want, rtol=1e-12, atol=1e-12)


# ---- Philox4x32-10 ---------------------------------------------------------------------

def _curand_host_philox(seed, offset, count=4):
    """Raw 32-bit outputs of cuRAND's HOST Philox4_32_10 generator (runs on the CPU)."""
    for name in ("libcurand.so", "libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so"):
        try:
            lib = ctypes.CDLL(name)
            break
        except OSError:
            lib = None
    if lib is None:
        pytest.skip("libcurand not found")
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0   # CURAND_RNG_PSEUDO_PHILOX4_32_10
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset)) == 0
    out = (ctypes.c_uint32 * count)()
    assert lib.curandGenerate(gen, out, ctypes.c_size_t(count)) == 0
    lib.curandDestroyGenerator(gen)
    return [int(v) for v in out]


@pytest.mark.parametrize("seed", [0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF])
def test_philox_matches_curand_host_generator(seed):
    """cuRAND's host Philox4_32_10 generator maps the seed to the key (low word, high word)
    and emits, as its k-th group of four outputs, the Philox block of counter (0, 0, k, 0).
    Every round after the first sees four non-zero counter words, so a wrong multiplier,
    Weyl constant, word placement or round count anywhere changes these outputs."""
    n_blocks = 8192
    raw = _curand_host_philox(seed, 0, 4 * n_blocks)
    key = (seed & 0xFFFFFFFF, seed >> 32)
    for k in [0, 1, 2, 3, 100, 4095, 4096, 8191]:
        assert list(O.philox4x32_10((0, 0, k, 0), key)) == raw[4 * k: 4 * k + 4]


def test_philox_structure():
    key = (123, 456)
    seen = {O.philox4x32_10((c, s, 0, 0), key) for c in range(64) for s in range(64)}
    assert len(seen) == 64 * 64                                   # a bijection never collides
    assert O.philox4x32_10((1, 2, 0, 0), key) != O.philox4x32_10((2, 1, 0, 0), key)
    assert O.philox4x32_10((1, 2, 0, 0), (123, 457)) != O.philox4x32_10((1, 2, 0, 0), key)
    us = np.array([O.philox_uniform(9, b, s) for b in range(200) for s in range(50)])
    assert us.min() >= 0.0 and us.max() < 1.0
    assert abs(us.mean() - 0.5) < 0.01 and abs(us.var() - 1 / 12) < 0.005
    assert np.all(us == us.astype(np.float32))                   # 24-bit fractions are exact in fp32


# ---- token selection -------------------------------------------------------------------

def test_greedy_lowest_id_among_ties():
    lg = np.array([[0.0, 3.0, 3.0, 1.0], [5.0, 5.0, 5.0, 5.0], [-1.0, -2.0, -0.5, -0.5]])
    assert O.select_greedy(lg).tolist() == [1, 0, 2]


def test_topk_order_bruteforce():
    rng = np.random.default_rng(2)
    row = np.round(rng.normal(size=200), 1)            # many exact ties
    ids = O.topk_order(row, 50)
    want = sorted(range(200), key=lambda i: (-row[i], i))[:50]
    assert ids.tolist() == want


def test_topk_sampling_decision_bruteforce():
    rng = np.random.default_rng(3)
    V, k, T, seed = 300, 50, 0.8, 77
    lg = rng.normal(size=(6, V))
    toks, det = O.select_topk(lg, k, T, seed, np.arange(6), step=5, return_detail=True)
    for b in range(6):
        order = sorted(range(V), key=lambda i: (-lg[b, i], i))[:k]
        p = np.array([math.exp((lg[b, i] - lg[b, order[0]]) / T) for i in order])
        p /= p.sum()
        u = O.philox_uniform(seed, b, 5)
        acc, pick = 0.0, order[-1]
        for i, pi in zip(order, p):
            acc += pi
            if acc > u:
                pick = i
                break
        assert toks[b] == pick
        assert toks[b] in order


def test_topk_sampling_frequencies_match_softmax():
    V, k, T = 64, 8, 0.8
    rng = np.random.default_rng(4)
    row = rng.normal(size=V) * 2
    N = 20000
    lg = np.broadcast_to(row, (N, V))
    toks = O.select_topk(lg, k, T, seed=5, sample_idx=np.arange(N), step=0)
    order = O.topk_order(row, k)
    p = np.exp((row[order] - row[order[0]]) / T); p /= p.sum()
    freq = np.array([(toks == i).mean() for i in order])
    sigma = np.sqrt(p * (1 - p) / N)
    assert np.all(np.abs(freq - p) < 4.5 * sigma + 1e-4)
    assert set(np.unique(toks)) <= set(order.tolist())
    # distinct steps give a different stream for the same sample
    t2 = O.select_topk(lg[:200], k, T, seed=5, sample_idx=np.arange(200), step=1)
    assert np.any(t2 != toks[:200])


# ---- nucleus (top-p) sampling ------------------------------------------------------------------

def _probs(row, T):
    w = np.array([math.exp((v - max(row)) / T) for v in row])
    return w / w.sum()


def test_nucleus_is_the_smallest_set_of_most_probable_tokens_with_mass_p_bruteforce():
    """All 2^V subsets of a small vocabulary: among the sets whose mass reaches p the nucleus has the fewest
    tokens, and among those of that size the largest mass (it takes the most probable tokens)."""
    import itertools
    rng = np.random.default_rng(11)
    V, T = 10, 0.7
    for trial in range(6):
        row = rng.normal(size=V) * 1.5
        pr = _probs(row, T)
        for p in (0.3, 0.6, 0.9, 0.99):
            ids, w = O.nucleus(row, p, T)
            best = None
            for r in range(1, V + 1):
                sets = [s for s in itertools.combinations(range(V), r) if sum(pr[list(s)]) >= p - 1e-15]
                if sets:
                    best = max(sets, key=lambda s: sum(pr[list(s)]))
                    break
            assert sorted(ids.tolist()) == sorted(best)
            # the weights are the unnormalised probabilities of exactly those tokens, most probable first
            assert np.allclose(w / w.sum(), pr[ids] / pr[ids].sum(), rtol=1e-12)
            assert np.all(np.diff(row[ids]) <= 0)


def test_nucleus_ties_and_limits():
    row = np.array([1.0, 3.0, 3.0, 3.0, 0.0, 3.0])
    # four equal maxima of probability ~0.23 each: p = 0.5 needs three of them, the lowest ids
    ids, _ = O.nucleus(row, 0.5, 1.0)
    assert ids.tolist() == [1, 2, 3]
    assert O.nucleus(row, 1e-9, 1.0)[0].tolist() == [1]               # p -> 0: the argmax alone
    assert sorted(O.nucleus(row, 1.0, 1.0)[0].tolist()) == list(range(6))    # p = 1: everything
    # a mass reached exactly keeps the prefix that reaches it, no more (probabilities 1/2, 1/4, 1/8, 1/8)
    dyadic = np.log(np.array([0.5, 0.25, 0.125, 0.125]))
    assert O.nucleus(dyadic, 0.75, 1.0)[0].tolist() == [0, 1]


def test_topp_with_p_one_is_plain_inverse_cdf_sampling_and_with_small_p_greedy():
    rng = np.random.default_rng(12)
    B, V, T, seed = 40, 97, 0.7, 9
    lg = rng.normal(size=(B, V)) * 2
    toks = O.select_topp(lg, 1.0, T, seed, np.arange(B), step=3)
    for b in range(B):
        w = np.exp((lg[b] - lg[b].max()) / T)
        c = np.cumsum(w)
        u = O.philox_uniform(seed, b, 3)
        assert toks[b] == min(int(np.searchsorted(c, u * c[-1], side="right")), V - 1)
    assert np.array_equal(O.select_topp(lg, 1e-12, T, seed, np.arange(B), step=3), O.select_greedy(lg))


def test_topp_sampling_frequencies_match_the_renormalised_nucleus():
    V, p, T = 64, 0.9, 0.7
    rng = np.random.default_rng(13)
    row = rng.normal(size=V) * 2
    N = 20000
    lg = np.broadcast_to(row, (N, V))
    toks = O.select_topp(lg, p, T, seed=6, sample_idx=np.arange(N), step=0)
    ids, w = O.nucleus(row, p, T)
    pr = w / w.sum()
    assert 1 < len(ids) < V
    freq = np.array([(toks == i).mean() for i in ids])
    sigma = np.sqrt(pr * (1 - pr) / N)
    assert np.all(np.abs(freq - pr) < 4.5 * sigma + 1e-4)
    assert set(np.unique(toks)) <= set(ids.tolist())
    # the mass outside the nucleus is below 1 - p, and dropping the least probable member breaks the bound
    full = _probs(row, T)
    assert full[ids].sum() >= p > full[ids[:-1]].sum()
