"""Pins for the oracle's two further token-mixer variants: linearly combined heads (Architecture) and
non-unitary kernels (Eq. 11). Each pin is independent of the function it checks: scalar-loop
evaluations of the printed definitions, reductions to the plain mixer, closed forms."""
import numpy as np
import pytest

from oracle import srm_oracle as O


def _params(rng, h, n, d):
    return dict(alpha_r=rng.uniform(0.5, 1.5, (h, n)), alpha_c=rng.uniform(0.5, 1.5, (h, n)),
                lam_r=rng.uniform(0.6, 0.99, h), lam_c=rng.uniform(0.6, 0.99, h),
                w=rng.uniform(-1.0, 1.0, (h, 2)), beta=rng.standard_normal((n, d)))


def test_combined_heads_scalar_loop_definition():
    """Output position j of channel c is a weighted sum over input positions i <= j: row-repeat
    weight lam_r^(j-i) alpha_r[i], column-repeat weight lam_c^(j-i) alpha_c[j] (Eq. 1, Eq. 3)."""
    rng = np.random.default_rng(0)
    h, n, d = 2, 7, 8
    p = _params(rng, h, n, d)
    Z = rng.standard_normal((n, d))
    Y, _, _ = O.combined_parallel(Z, n_heads=h, **p)
    dh = d // h
    for j in range(n):
        for c in range(d):
            g = c // dh
            acc = p["beta"][j, c]
            for i in range(j + 1):
                acc += p["w"][g, 0] * p["lam_r"][g] ** (j - i) * p["alpha_r"][g, i] * Z[i, c]
                acc += p["w"][g, 1] * p["lam_c"][g] ** (j - i) * p["alpha_c"][g, j] * Z[i, c]
            assert abs(Y[j, c] - acc) < 1e-12


def test_combined_heads_with_unit_weights_reduce_to_mixed_heads():
    """Weights (1, 0) on the first half of the heads and (0, 1) on the second half give the mixed-head layer."""
    rng = np.random.default_rng(1)
    h, n, d = 4, 9, 16
    p = _params(rng, h, n, d)
    p["w"] = np.array([[1.0, 0.0], [1.0, 0.0], [0.0, 1.0], [0.0, 1.0]])
    Z = rng.standard_normal((n, d))
    Y, S_r, S_c = O.combined_parallel(Z, n_heads=h, **p)
    alpha = np.concatenate([p["alpha_r"][:2], p["alpha_c"][2:]])
    lam = np.concatenate([p["lam_r"][:2], p["lam_c"][2:]])
    Ym, Sm = O.mixer_parallel(Z, alpha, p["beta"], lam, h)
    assert np.allclose(Y, Ym, atol=1e-12)
    assert np.allclose(np.concatenate([S_r[:8], S_c[8:]]), Sm, atol=1e-12)


def test_combined_heads_closed_form_for_constant_input():
    """z = 1, alpha = a, lambda = l: the row part is a (1 - l^(j+1)) / (1 - l), so is the column part."""
    h, n, d = 1, 12, 2
    a_r, a_c, l_r, l_c = 0.7, 1.3, 0.9, 0.8
    Y, S_r, S_c = O.combined_parallel(np.ones((n, d)), np.full((h, n), a_r), np.full((h, n), a_c), np.zeros((n, d)),
                                      np.array([l_r]), np.array([l_c]), np.array([[2.0, -3.0]]), h)
    for j in range(n):
        want = 2.0 * a_r * (1 - l_r ** (j + 1)) / (1 - l_r) - 3.0 * a_c * (1 - l_c ** (j + 1)) / (1 - l_c)
        assert np.allclose(Y[j], want, atol=1e-12)
    assert np.allclose(S_r, a_r * l_r * (1 - l_r ** n) / (1 - l_r)) and np.allclose(S_c, l_c * (1 - l_c ** n) / (1 - l_c))


def test_combined_heads_recurrent_equals_parallel_with_twice_the_cache():
    rng = np.random.default_rng(2)
    h, n, d = 4, 20, 32
    p = _params(rng, h, n, d)
    Z = rng.standard_normal((3, n, d))
    S_r, S_c = np.zeros((3, d)), np.zeros((3, d))
    Yr = np.empty_like(Z)
    for t in range(n):
        Yr[:, t], S_r, S_c = O.combined_recurrent_step(Z[:, t], S_r, S_c, t, n_heads=h, **p)
    assert S_r.shape == (3, d) and S_c.shape == (3, d)          # 2 d values per sample and layer
    for b in range(3):
        Y, Pr, Pc = O.combined_parallel(Z[b], n_heads=h, **p)
        assert np.allclose(Yr[b], Y, atol=1e-10)
        assert np.allclose(S_r[b], Pr, atol=1e-10) and np.allclose(S_c[b], Pc, atol=1e-10)


# ---- Eq. 11 ---------------------------------------------------------------------------------

def _kparams(rng, k, n, d):
    return rng.uniform(0.5, 1.5, (k, n)), rng.standard_normal((n, d)), rng.uniform(0.6, 0.99, k)


def test_kernel_mixer_scalar_loop_on_the_padded_rows():
    """Eq. 11 entry by entry: Y[c, j] = sum_i sum_{m<=j} Xpad[c+i, m] W_i[m, j] + beta, W_i column-repeat."""
    rng = np.random.default_rng(3)
    k, n, d = 3, 6, 5
    alpha, beta, lam = _kparams(rng, k, n, d)
    Z = rng.standard_normal((n, d))
    Y, _ = O.kernel_parallel(Z, alpha, beta, lam, k)
    for j in range(n):
        for c in range(d):
            acc = beta[j, c]
            for i in range(k):
                for m in range(j + 1):
                    x = Z[m, c + i] if c + i < d else 0.0          # zero padding past the last channel
                    acc += x * lam[i] ** (j - m) * alpha[i, j]
            assert abs(Y[j, c] - acc) < 1e-12


def test_kernel_mixer_with_k_one_is_a_column_repeat_head():
    rng = np.random.default_rng(4)
    n, d = 10, 8
    alpha, beta, lam = _kparams(rng, 1, n, d)
    Z = rng.standard_normal((n, d))
    Y, P = O.kernel_parallel(Z, alpha, beta, lam, 1)
    M = O.mixing_matrix("col", alpha[0], lam[0], n)
    assert np.allclose(Y, (Z.T @ M).T + beta, atol=1e-12)
    # a two-head mixed layer's second (column-repeat) head computes the same thing on its channels
    Ym, Sm = O.mixer_parallel(Z, np.stack([alpha[0], alpha[0]]), beta, np.array([lam[0], lam[0]]), 2)
    assert np.allclose(Y[:, d // 2:], Ym[:, d // 2:], atol=1e-12) and np.allclose(P[0, d // 2:], Sm[d // 2:], atol=1e-12)


def test_kernel_mixer_shift_structure():
    """A one-hot input in channel c0 reaches output channels c0-k+1..c0 only, through filter i = c0 - c."""
    k, n, d, c0 = 4, 5, 10, 6
    alpha = np.arange(1, k + 1, dtype=np.float64)[:, None] * np.ones((k, n))
    lam = np.full(k, 0.5)
    Z = np.zeros((n, d))
    Z[0, c0] = 1.0
    Y, _ = O.kernel_parallel(Z, alpha, np.zeros((n, d)), lam, k)
    for j in range(n):
        for c in range(d):
            i = c0 - c
            want = (i + 1) * 0.5 ** j if 0 <= i < k else 0.0
            assert abs(Y[j, c] - want) < 1e-14


@pytest.mark.parametrize("k", [1, 4, 8])
def test_kernel_mixer_recurrent_equals_parallel_with_k_times_the_cache(k):
    rng = np.random.default_rng(5 + k)
    n, d = 16, 24
    alpha, beta, lam = _kparams(rng, k, n, d)
    Z = rng.standard_normal((2, n, d))
    P = np.zeros((k, 2, d))
    Yr = np.empty_like(Z)
    for t in range(n):
        Yr[:, t], P = O.kernel_recurrent_step(Z[:, t], P, t, alpha, beta, lam, k)
    assert P.shape == (k, 2, d)
    for b in range(2):
        Y, Pn = O.kernel_parallel(Z[b], alpha, beta, lam, k)
        assert np.allclose(Yr[b], Y, atol=1e-10) and np.allclose(P[:, b], Pn, atol=1e-10)
