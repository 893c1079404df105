"""Pins for the oracle's token mixer: printed matrices, closed forms, brute force,
textbook special cases, parallel == recurrent, causality, op count and cache size."""
import os

import numpy as np
import pytest

from oracle import srm_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_symbolic(path, env):
    rows = []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        rows.append([eval(tok, {}, env) for tok in line.split()])
    return np.array(rows, dtype=np.float64)


def test_row_repeat_matrix_matches_printed_eq1():
    rng = np.random.default_rng(0)
    a = rng.normal(size=3)
    lam = 0.93
    want = _read_symbolic(os.path.join(GOLD, "eq1_row_repeat_n3.txt"),
                          dict(a0=a[0], a1=a[1], a2=a[2], l=lam))
    got = O.mixing_matrix("row", a, lam, 3)
    np.testing.assert_allclose(got, want, rtol=1e-14, atol=0)
    # a transposed or column-repeat construction must NOT match
    assert not np.allclose(O.mixing_matrix("col", a, lam, 3), want)
    assert not np.allclose(got.T, want)


def test_col_repeat_matrix_matches_printed_eq3():
    rng = np.random.default_rng(1)
    a = rng.normal(size=4)
    lam = 0.97
    want = _read_symbolic(os.path.join(GOLD, "eq3_col_repeat_pattern.txt"),
                          dict(a0=a[0], a1=a[1], a2=a[2], a3=a[3], l=lam))
    got = O.mixing_matrix("col", a, lam, 4)
    np.testing.assert_allclose(got, want, rtol=1e-14, atol=0)
    assert not np.allclose(O.mixing_matrix("row", a, lam, 4), want)


def _rand_layer(rng, n, d, h, lam_one_head0=True):
    alpha = rng.normal(size=(h, n))
    beta = rng.normal(size=(n, d))
    lam = rng.uniform(0.9, 1.0, size=h)
    if lam_one_head0:
        lam[0] = 1.0
    return alpha, beta, lam


def test_parallel_form_equals_bruteforce_XM_plus_B():
    """Y = X M + B written with scalar loops over (channel, i, j) on tiny inputs."""
    rng = np.random.default_rng(2)
    n, d, h = 7, 8, 4
    dh = d // h
    alpha, beta, lam = _rand_layer(rng, n, d, h)
    Z = rng.normal(size=(n, d))
    Y, _ = O.mixer_parallel(Z, alpha, beta, lam, h)
    for c in range(d):
        g = c // dh
        for j in range(n):
            acc = 0.0
            for i in range(j + 1):
                coeff = alpha[g][i] if g < h // 2 else alpha[g][j]
                acc += Z[i, c] * (lam[g] ** (j - i)) * coeff
            assert abs(Y[j, c] - (acc + beta[j, c])) < 1e-12


def test_recurrent_outputs_equal_closed_forms_eq2_eq3():
    """Y_n = a_n X_n + b_n + sum_{m<n} l^(n-m) a_m X_m (row);
       Y_n = a_n X_n + b_n + a_n sum_{m<n} l^(n-m) X_m (column), as direct O(n^2) sums."""
    rng = np.random.default_rng(3)
    n, d, h = 9, 8, 4
    dh = d // h
    alpha, beta, lam = _rand_layer(rng, n, d, h)
    Z = rng.normal(size=(n, d))
    S = np.zeros(d)
    for t in range(n):
        y, S = O.mixer_recurrent_step(Z[t], S, t, alpha, beta, lam, h)
        for c in range(d):
            g = c // dh
            if g < h // 2:
                tail = sum(lam[g] ** (t - m) * alpha[g][m] * Z[m, c] for m in range(t))
                want = alpha[g][t] * Z[t, c] + beta[t, c] + tail
            else:
                tail = sum(lam[g] ** (t - m) * Z[m, c] for m in range(t))
                want = alpha[g][t] * Z[t, c] + beta[t, c] + alpha[g][t] * tail
            assert abs(y[c] - want) < 1e-12
    # the cache handed on after n tokens is the sum term position n would use
    _, S_par = O.mixer_parallel(Z, alpha, beta, lam, h)
    np.testing.assert_allclose(S, S_par, rtol=0, atol=1e-12)


def test_mixer_parallel_equals_recurrent_1e9():
    rng = np.random.default_rng(4)
    n, d, h = 32, 16, 4
    alpha, beta, lam = _rand_layer(rng, n, d, h)
    Z = rng.normal(size=(n, d))
    Y, S_n = O.mixer_parallel(Z, alpha, beta, lam, h)
    S = np.zeros(d)
    for t in range(n):
        y, S = O.mixer_recurrent_step(Z[t], S, t, alpha, beta, lam, h)
        assert np.max(np.abs(y - Y[t])) < 1e-9
    assert np.max(np.abs(S - S_n)) < 1e-9


def test_cumsum_special_cases():
    """lambda = 1, alpha = 1, beta = 0: both head kinds give the inclusive running sum;
    column head with lambda = 1: alpha_n * running sum; alpha = 0: y = beta."""
    rng = np.random.default_rng(5)
    n, d, h = 12, 8, 4
    Z = rng.normal(size=(n, d))
    one = np.ones((h, n)); zero_b = np.zeros((n, d)); lam1 = np.ones(h)
    Y, _ = O.mixer_parallel(Z, one, zero_b, lam1, h)
    np.testing.assert_allclose(Y, np.cumsum(Z, axis=0), atol=1e-12)
    S = np.zeros(d)
    for t in range(n):
        y, S = O.mixer_recurrent_step(Z[t], S, t, one, zero_b, lam1, h)
        np.testing.assert_allclose(y, np.cumsum(Z, axis=0)[t], atol=1e-12)
    alpha = rng.normal(size=(h, n))
    Y, _ = O.mixer_parallel(Z, alpha, zero_b, lam1, h)
    col = slice(d // 2, d)
    dh = d // h
    a_cols = np.repeat(alpha[h // 2:], dh, axis=0).T          # [n, d/2]
    np.testing.assert_allclose(Y[:, col], a_cols * np.cumsum(Z, axis=0)[:, col], atol=1e-12)
    beta = rng.normal(size=(n, d))
    Y, _ = O.mixer_parallel(Z, np.zeros((h, n)), beta, rng.uniform(0.9, 1, h), h)
    np.testing.assert_allclose(Y, beta, atol=0)
    # n = 1: y_0 = alpha_0 z_0 + beta_0 for both kinds
    Y, _ = O.mixer_parallel(Z[:1], alpha, beta, lam1, h)
    np.testing.assert_allclose(Y[0], np.repeat(alpha[:, 0], dh) * Z[0] + beta[0], atol=1e-14)


def test_geometric_decay_special_case():
    """Constant input, alpha = 1, beta = 0, decay l: the column/row output at position t is
    the geometric series (1 - l^(t+1)) / (1 - l)."""
    n, d, h = 20, 4, 4
    lam = np.array([0.9, 0.95, 0.91, 0.99])
    Z = np.ones((n, d))
    Y, S = O.mixer_parallel(Z, np.ones((h, n)), np.zeros((n, d)), lam, h)
    t = np.arange(n)[:, None]
    want = (1 - lam[None, :] ** (t + 1)) / (1 - lam[None, :])
    np.testing.assert_allclose(Y, want, rtol=1e-12)
    np.testing.assert_allclose(S, lam * (1 - lam ** n) / (1 - lam), rtol=1e-12)


class _CountingArray(np.ndarray):
    """ndarray that counts elementwise multiplies / adds done on d_head-sized vectors."""
    counts = {"mul": 0, "add": 0}

    def __array_ufunc__(self, ufunc, method, *inputs, **kw):
        args = [np.asarray(i) if isinstance(i, _CountingArray) else i for i in inputs]
        if "out" in kw:
            kw["out"] = tuple(np.asarray(o) if isinstance(o, _CountingArray) else o for o in kw["out"])
        res = getattr(ufunc, method)(*args, **kw)
        if ufunc is np.multiply:
            _CountingArray.counts["mul"] += 1
        elif ufunc is np.add:
            _CountingArray.counts["add"] += 1
        return res.view(_CountingArray) if isinstance(res, np.ndarray) else res


def test_op_count_and_cache_size():
    """Per head and step: at most two scalar-vector multiplies for the output/cache
    update plus vector additions; the cache is exactly one d-vector per layer."""
    n, d, h = 4, 8, 4
    rng = np.random.default_rng(6)
    alpha, beta, lam = _rand_layer(rng, n, d, h)
    z = rng.normal(size=d).view(_CountingArray)
    S = np.zeros(d).view(_CountingArray)
    _CountingArray.counts.update(mul=0, add=0)
    y, S2 = O.mixer_recurrent_step(z, S, 1, alpha, beta, lam, h)
    assert _CountingArray.counts["mul"] == 2 * h       # alpha_t * v and lambda * v, per head
    assert np.asarray(S2).shape == (d,)                # cache: d numbers per layer per sample
