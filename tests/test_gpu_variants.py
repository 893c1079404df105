"""Parity of the two further token-mixer variants (linearly combined heads; non-unitary kernels, Eq. 11),
called through the C ABI, against the CPU oracle: several recurrent steps from random caches, every output
and every cache element compared. fp32 kernel against the fp64 oracle on the same fp32 inputs: one rounding
per operation in sums of at most k + 2 terms of magnitude O(10), so 2e-5 absolute is ample."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 2e-5


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV)


def _f32(a):
    return np.asarray(a, np.float32).astype(np.float64)


@pytest.mark.parametrize("R,d,h", [(37, 64, 4), (300, 1024, 4), (5, 1536, 2), (1, 8, 2), (4099, 256, 1)])
def test_combined_heads_step_matches_oracle(R, d, h):
    import paper_2605_08696_b200 as P
    from oracle import srm_oracle as O
    rng = np.random.default_rng(R + d)
    n_ctx = 12
    ar, ac = _f32(rng.uniform(0.5, 1.5, (h, n_ctx))), _f32(rng.uniform(0.5, 1.5, (h, n_ctx)))
    lr, lc = _f32(rng.uniform(0.6, 0.99, h)), _f32(rng.uniform(0.6, 0.99, h))
    w, beta = _f32(rng.uniform(-1, 1, (h, 2))), _f32(rng.standard_normal((n_ctx, d)))
    S_r, S_c = _f32(rng.standard_normal((R, d))), _f32(rng.standard_normal((R, d)))
    dS_r, dS_c, dy = _t(S_r), _t(S_c), torch.empty(R, d, device=DEV)
    dev = [_t(a) for a in (ar, ac, beta, lr, lc, w)]
    for t in (3, 4, 11):
        z = _f32(rng.standard_normal((R, d)))
        y, S_r, S_c = O.combined_recurrent_step(z, S_r, S_c, t, ar, ac, beta, lr, lc, w, h)
        P.k_mixer_combined_step(t, _t(z), dS_r, dS_c, dev[0], dev[1], dev[2], dev[3], dev[4], dev[5], dy)
        torch.cuda.synchronize()
        assert np.abs(dy.cpu().numpy() - y).max() < TOL
        assert np.abs(dS_r.cpu().numpy() - S_r).max() < TOL and np.abs(dS_c.cpu().numpy() - S_c).max() < TOL


@pytest.mark.parametrize("R,d,k", [(37, 64, 4), (300, 1024, 8), (5, 1536, 4), (3, 8, 8), (2, 4, 1), (4099, 256, 16),
                                   (9, 2052, 3)])
def test_kernel_mixer_step_matches_oracle(R, d, k):
    import paper_2605_08696_b200 as P
    from oracle import srm_oracle as O
    rng = np.random.default_rng(R + d + k)
    n_ctx = 9
    alpha, lam = _f32(rng.uniform(0.5, 1.5, (k, n_ctx))), _f32(rng.uniform(0.6, 0.99, k))
    beta = _f32(rng.standard_normal((n_ctx, d)))
    Pc = _f32(rng.standard_normal((k, R, d)))
    dP, dy = _t(Pc), torch.empty(R, d, device=DEV)
    da, db, dl = _t(alpha), _t(beta), _t(lam)
    for t in (0, 5, 8):
        z = _f32(rng.standard_normal((R, d)))
        y, Pc = O.kernel_recurrent_step(z, Pc, t, alpha, beta, lam, k)
        P.k_mixer_kernel_step(t, _t(z), dP, da, db, dl, dy)
        torch.cuda.synchronize()
        assert np.abs(dy.cpu().numpy() - y).max() < TOL * k
        assert np.abs(dP.cpu().numpy() - Pc).max() < TOL


def test_variant_steps_from_zero_cache_reproduce_the_parallel_form():
    """A whole short sequence through the kernels, from empty caches, against the explicit n x n matrices."""
    import paper_2605_08696_b200 as P
    from oracle import srm_oracle as O
    rng = np.random.default_rng(0)
    n, d, h, k = 10, 128, 4, 4
    Z = _f32(rng.standard_normal((n, d)))
    beta = _f32(rng.standard_normal((n, d)))
    ar, ac = _f32(rng.uniform(0.5, 1.5, (h, n))), _f32(rng.uniform(0.5, 1.5, (h, n)))
    lr, lc, w = _f32(rng.uniform(0.6, 0.99, h)), _f32(rng.uniform(0.6, 0.99, h)), _f32(rng.uniform(-1, 1, (h, 2)))
    Y, S_r, S_c = O.combined_parallel(Z, ar, ac, beta, lr, lc, w, h)
    dS_r, dS_c, dy = torch.zeros(1, d, device=DEV), torch.zeros(1, d, device=DEV), torch.empty(1, d, device=DEV)
    dev = [_t(a) for a in (ar, ac, beta, lr, lc, w)]
    for t in range(n):
        P.k_mixer_combined_step(t, _t(Z[t:t + 1]), dS_r, dS_c, *dev, dy)
        assert np.abs(dy.cpu().numpy()[0] - Y[t]).max() < 1e-4
    assert np.abs(dS_r.cpu().numpy()[0] - S_r).max() < 1e-4 and np.abs(dS_c.cpu().numpy()[0] - S_c).max() < 1e-4

    alpha, lam = _f32(rng.uniform(0.5, 1.5, (k, n))), _f32(rng.uniform(0.6, 0.99, k))
    Yk, Pk = O.kernel_parallel(Z, alpha, beta, lam, k)
    dP = torch.zeros(k, 1, d, device=DEV)
    for t in range(n):
        P.k_mixer_kernel_step(t, _t(Z[t:t + 1]), dP, _t(alpha), _t(beta), _t(lam), dy)
        assert np.abs(dy.cpu().numpy()[0] - Yk[t]).max() < 2e-4
    assert np.abs(dP.cpu().numpy()[:, 0] - Pk).max() < 1e-4


def test_variant_steps_reject_bad_arguments():
    import paper_2605_08696_b200 as P
    z = torch.zeros(2, 8, device=DEV)
    S = torch.zeros(2, 8, device=DEV)
    a = torch.ones(2, 4, device=DEV)
    beta = torch.zeros(4, 8, device=DEV)
    lam = torch.ones(2, device=DEV)
    w = torch.ones(2, 2, device=DEV)
    with pytest.raises(P.SRMError) as e:
        P.k_mixer_combined_step(4, z, S, S.clone(), a, a, beta, lam, lam, w, z.clone())     # t == n_ctx
    assert e.value.code == -5                  # SRM_ERR_CTX_OVERFLOW
    a3 = torch.ones(3, 4, device=DEV)
    with pytest.raises(P.SRMError) as e:
        P.k_mixer_combined_step(0, z, S, S.clone(), a3, a3, beta, torch.ones(3, device=DEV), torch.ones(3, device=DEV),
                                torch.ones(3, 2, device=DEV), z.clone())                     # 8 channels, 3 heads
    assert e.value.code == -2                  # SRM_ERR_UNSUPPORTED
    with pytest.raises(P.SRMError) as e:
        P.k_mixer_kernel_step(0, z, torch.zeros(17, 2, 8, device=DEV), torch.ones(17, 4, device=DEV), beta,
                              torch.ones(17, device=DEV), z.clone())                          # k > 16
    assert e.value.code == -2
    # R = 0 is a no-op
    e0 = torch.zeros(0, 8, device=DEV)
    P.k_mixer_combined_step(0, e0, e0.clone(), e0.clone(), a, a, beta, lam, lam, w, e0.clone())
    P.k_mixer_kernel_step(0, e0, torch.zeros(2, 0, 8, device=DEV), a, beta, lam, e0.clone())


# ---- whole sequences (the prefill form) -----------------------------------------------------

@pytest.mark.parametrize("Bp,n,d,h", [(3, 10, 64, 4), (37, 33, 256, 2), (2, 5, 1536, 4), (300, 7, 128, 1)])
def test_combined_heads_scan_matches_the_explicit_matrices(Bp, n, d, h):
    import paper_2605_08696_b200 as P
    from oracle import srm_oracle as O
    rng = np.random.default_rng(Bp + n + d)
    ar, ac = _f32(rng.uniform(0.5, 1.5, (h, n))), _f32(rng.uniform(0.5, 1.5, (h, n)))
    lr, lc = _f32(rng.uniform(0.6, 0.99, h)), _f32(rng.uniform(0.6, 0.99, h))
    w, beta = _f32(rng.uniform(-1, 1, (h, 2))), _f32(rng.standard_normal((n, d)))
    Z = _f32(rng.standard_normal((Bp, n, d)))
    dS_r, dS_c = torch.zeros(Bp, d, device=DEV), torch.zeros(Bp, d, device=DEV)
    dY = torch.empty(Bp, n, d, device=DEV)
    P.k_mixer_combined_scan(0, _t(Z), dS_r, dS_c, _t(ar), _t(ac), _t(beta), _t(lr), _t(lc), _t(w), dY)
    Y, Sr, Sc = dY.cpu().numpy(), dS_r.cpu().numpy(), dS_c.cpu().numpy()
    for b in list(range(min(Bp, 4))) + [Bp - 1]:
        Yo, Sro, Sco = O.combined_parallel(Z[b], ar, ac, beta, lr, lc, w, h)
        assert np.abs(Y[b] - Yo).max() < 1e-4
        assert np.abs(Sr[b] - Sro).max() < 1e-4 and np.abs(Sc[b] - Sco).max() < 1e-4


@pytest.mark.parametrize("Bp,n,d,k", [(3, 10, 64, 4), (37, 33, 256, 8), (2, 5, 1536, 4), (150, 7, 128, 1), (2, 6, 2052, 3),
                                      (2, 9, 8, 8)])
def test_kernel_mixer_scan_matches_eq11_on_explicit_matrices(Bp, n, d, k):
    import paper_2605_08696_b200 as P
    from oracle import srm_oracle as O
    rng = np.random.default_rng(Bp + n + d + k)
    alpha, lam = _f32(rng.uniform(0.5, 1.5, (k, n))), _f32(rng.uniform(0.6, 0.99, k))
    beta = _f32(rng.standard_normal((n, d)))
    Z = _f32(rng.standard_normal((Bp, n, d)))
    dP, dY = torch.zeros(k, Bp, d, device=DEV), torch.empty(Bp, n, d, device=DEV)
    P.k_mixer_kernel_scan(0, _t(Z), dP, _t(alpha), _t(beta), _t(lam), dY)
    Y, Pc = dY.cpu().numpy(), dP.cpu().numpy()
    for b in list(range(min(Bp, 4))) + [Bp - 1]:
        Yo, Po = O.kernel_parallel(Z[b], alpha, beta, lam, k)
        assert np.abs(Y[b] - Yo).max() < 1e-4 * k
        assert np.abs(Pc[:, b] - Po).max() < 1e-4


def test_variant_scans_continue_from_a_cache_and_agree_with_the_steps():
    """A sequence in two pieces (positions 0..5, then 6..11 from the cache of the first piece) equals the sequence
    in one piece bit for bit, and the step kernels continue from the same caches."""
    import paper_2605_08696_b200 as P
    rng = np.random.default_rng(9)
    Bp, n, d, h, k = 5, 12, 128, 4, 4
    Z = _t(rng.standard_normal((Bp, n, d)))
    beta = _t(rng.standard_normal((n + 1, d)))
    ar, ac = _t(rng.uniform(0.5, 1.5, (h, n + 1))), _t(rng.uniform(0.5, 1.5, (h, n + 1)))
    lr, lc, w = _t(rng.uniform(0.6, 0.99, h)), _t(rng.uniform(0.6, 0.99, h)), _t(rng.uniform(-1, 1, (h, 2)))
    z0 = lambda *s: torch.zeros(*s, device=DEV)
    S1, C1, Y1 = z0(Bp, d), z0(Bp, d), z0(Bp, n, d)
    P.k_mixer_combined_scan(0, Z, S1, C1, ar, ac, beta, lr, lc, w, Y1)
    S2, C2, Ya, Yb = z0(Bp, d), z0(Bp, d), z0(Bp, 6, d), z0(Bp, 6, d)
    P.k_mixer_combined_scan(0, Z[:, :6].contiguous(), S2, C2, ar, ac, beta, lr, lc, w, Ya)
    P.k_mixer_combined_scan(6, Z[:, 6:].contiguous(), S2, C2, ar, ac, beta, lr, lc, w, Yb)
    assert torch.equal(torch.cat([Ya, Yb], 1), Y1) and torch.equal(S1, S2) and torch.equal(C1, C2)
    zt, y_scan, y_step = _t(rng.standard_normal((Bp, 1, d))), z0(Bp, 1, d), z0(Bp, d)
    S3, C3 = S1.clone(), C1.clone()
    P.k_mixer_combined_scan(n, zt, S1, C1, ar, ac, beta, lr, lc, w, y_scan)
    P.k_mixer_combined_step(n, zt[:, 0].contiguous(), S3, C3, ar, ac, beta, lr, lc, w, y_step)
    assert torch.equal(y_scan[:, 0], y_step) and torch.equal(S1, S3) and torch.equal(C1, C3)

    al, lk = _t(rng.uniform(0.5, 1.5, (k, n + 1))), _t(rng.uniform(0.6, 0.99, k))
    P1, P2 = z0(k, Bp, d), z0(k, Bp, d)
    P.k_mixer_kernel_scan(0, Z, P1, al, beta, lk, Y1)
    P.k_mixer_kernel_scan(0, Z[:, :6].contiguous(), P2, al, beta, lk, Ya)
    P.k_mixer_kernel_scan(6, Z[:, 6:].contiguous(), P2, al, beta, lk, Yb)
    assert torch.equal(torch.cat([Ya, Yb], 1), Y1) and torch.equal(P1, P2)
    P3 = P1.clone()
    P.k_mixer_kernel_scan(n, zt, P1, al, beta, lk, y_scan)
    P.k_mixer_kernel_step(n, zt[:, 0].contiguous(), P3, al, beta, lk, y_step)
    assert torch.equal(y_scan[:, 0], y_step) and torch.equal(P1, P3)
