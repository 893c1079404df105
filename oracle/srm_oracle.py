"""CPU oracle for the Structured Recurrent Mixer (SRM): TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct numpy implementation (fp64 by default) of what the
CUDA path computes: the sequence-parallel form (explicit token-mixing matrices), the
recurrent form (constant-size per-sample state), the channel-mixing feed-forward,
the LM head and the two token-selection rules. Only the tests, the smoke check and
the benchmark's CPU-baseline leg may import it. It shares no code with the CUDA path
and does not import it; inputs (weights, prompts) are passed in as numpy arrays.

Notation follows the paper's Method section: X, Y in R^{d x n} hold one column per
position, Y = X M + B with M in R^{n x n} upper-triangular (entry [i, j] weights
input position i in output position j, so i <= j), alpha the repeated weight vector,
lambda the decay constant, beta the per-position bias, and the "cache" is the sum
term of Eq. 2 / Eq. 3. Arrays here are stored position-major, Z[n, d] = X^T.

Parity status of each function (what pins it, see tests/test_oracle_*.py):
  mixing_matrix            pinned: printed 3x3 matrix of Eq. 1, printed pattern of Eq. 3
  mixer_parallel           pinned: brute-force loops, cumulative-sum special cases
  mixer_recurrent_step     pinned: closed forms of Eq. 2 / Eq. 3, equality with the
                           parallel form to 1e-9, op count, cache size d per layer
  layer_norm, gelu_erf     pinned: moments / identities / tabulated erf values
  philox4x32_10            pinned: cuRAND's host Philox4_32_10 generator, bijectivity
  select_greedy, select_topk  pinned: brute-force sort, frequency test
  select_topp              pinned: brute force over all subsets (smallest set of most probable tokens
                           with mass >= p), p = 1 == plain inverse-CDF sampling (numpy searchsorted),
                           p -> 0 == greedy, frequency test against the renormalised nucleus
  token_mixer_parallel / _recurrent with head projections (Eq. 10)
                           pinned: brute-force Eq. 10 in the paper's d x n orientation with explicit
                           per-head I_g, identity projections == no projections, parallel == recurrent
  combined_parallel / combined_recurrent_step (linearly combined heads, Architecture)
                           pinned: scalar-loop definition, weights (1, 0) / (0, 1) == the mixed-head
                           mixer, closed form for constant inputs, parallel == recurrent, cache size 2 d
  kernel_parallel / kernel_recurrent_step (non-unitary kernels, Eq. 11)
                           pinned: scalar-loop evaluation of Eq. 11 on the padded d+k rows, k = 1 == a
                           column-repeat head, shift structure (a one-hot channel spreads to the k
                           channels below it), parallel == recurrent, cache size k d
  SRMOracle (full model logits)  PARITY UNPINNED beyond self-consistency (parallel ==
                           recurrent, causality): the paper prints no activations and
                           its architecture figure is missing, so the block structure
                           (pre-norm residual blocks, LayerNorm, erf-GELU FFN with
                           biases, untied bias-free LM head) is a stated reading.
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf


# --------------------------------------------------------------------------------------
# Token mixing (Method / Architecture: Eq. 1, Eq. 2, Eq. 3)
# --------------------------------------------------------------------------------------

def mixing_matrix(kind: str, alpha, lam: float, n: int, dtype=np.float64) -> np.ndarray:
    """Explicit n x n token-mixing matrix M of one head.

    kind "row"   : row i repeats alpha[i], decayed by lam per diagonal (Eq. 1):
                   M[i, j] = lam^(j-i) * alpha[i]  for i <= j, else 0.
    kind "col"   : column j repeats alpha[j] (Eq. 3):
                   M[i, j] = lam^(j-i) * alpha[j]  for i <= j, else 0.
    Built with scalar loops on purpose (brute-force definition).
    """
    M = np.zeros((n, n), dtype=dtype)
    for i in range(n):
        for j in range(i, n):
            a = alpha[i] if kind == "row" else alpha[j]
            M[i, j] = dtype(lam) ** (j - i) * dtype(a)
    return M


def head_kinds(n_heads: int):
    """'Mixed' heads: the first half of the heads are row-repeat, the second half
    column-repeat; outputs are concatenated (Architecture, mixed heads)."""
    return ["row" if g < n_heads // 2 else "col" for g in range(n_heads)]


def mixer_parallel(Z: np.ndarray, alpha: np.ndarray, beta: np.ndarray, lam: np.ndarray,
                   n_heads: int, matrices=None):
    """Sequence-parallel token mixing of one layer for one sample.

    Z[n, d] are the (normed) inputs, one row per position. For head g with channel
    slice c, Y[:, c]^T = Z[:, c]^T M_g + beta[:n, c]^T   (Y = X M + B).
    Also returns the hand-off cache S_n[d], i.e. the sum term of Eq. 2 / Eq. 3 that
    position n would use:  row heads  S_n = sum_{m<n} lam^(n-m) alpha[m] z_m,
                           col heads  S_n = sum_{m<n} lam^(n-m) z_m.
    `matrices` may hold the per-head M already built by mixing_matrix for this n (they do
    not depend on the sample).
    """
    n, d = Z.shape
    dh = d // n_heads
    dt = Z.dtype.type
    Y = np.empty_like(Z)
    S = np.zeros(d, dtype=Z.dtype)
    for g, kind in enumerate(head_kinds(n_heads)):
        c = slice(g * dh, (g + 1) * dh)
        M = matrices[g] if matrices is not None else mixing_matrix(kind, alpha[g], lam[g], n, dtype=dt)
        X = Z[:, c].T                               # d_h x n, columns = positions
        Y[:, c] = (X @ M).T + beta[:n, c]
        for m in range(n):
            w = dt(lam[g]) ** (n - m)
            if kind == "row":
                w = w * dt(alpha[g][m])
            S[c] += w * Z[m, c]
    return Y, S


def mixer_recurrent_step(z: np.ndarray, S: np.ndarray, t: int, alpha: np.ndarray,
                         beta: np.ndarray, lam: np.ndarray, n_heads: int):
    """One recurrent token-mixing step at absolute position t (batched over rows).

    z[..., d] normed input of position t, S[..., d] the cache (sum term) for position t.
    row heads (Eq. 2):  y = alpha_t z + beta_t + S ;      S' = lam (S + alpha_t z)
    col heads (Eq. 3):  y = alpha_t (z + S) + beta_t ;    S' = lam (S + z)
    so that S'(t+1) = sum_{m<=t} lam^(t+1-m) [alpha_m] z_m is the sum term of t+1.
    """
    d = z.shape[-1]
    dh = d // n_heads
    dt = z.dtype.type
    y = np.empty_like(z)
    S_new = np.empty_like(S)
    for g, kind in enumerate(head_kinds(n_heads)):
        c = slice(g * dh, (g + 1) * dh)
        a, l = dt(alpha[g][t]), dt(lam[g])
        if kind == "row":
            u = a * z[..., c]
            y[..., c] = u + beta[t, c] + S[..., c]
            S_new[..., c] = l * (S[..., c] + u)
        else:
            v = z[..., c] + S[..., c]
            y[..., c] = a * v + beta[t, c]
            S_new[..., c] = l * v
    return y, S_new


# --------------------------------------------------------------------------------------
# Channel mixing and norms (stated reading: pre-norm residual block, LayerNorm with
# affine parameters and biased variance, Linear -> exact erf GELU -> Linear, with biases)
# --------------------------------------------------------------------------------------

def layer_norm(x: np.ndarray, g: np.ndarray, b: np.ndarray, eps: float) -> np.ndarray:
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + x.dtype.type(eps)) * g + b


def gelu_erf(x: np.ndarray) -> np.ndarray:
    return (0.5 * x * (1.0 + _erf(x / np.sqrt(2.0)))).astype(x.dtype)


def feed_forward(a: np.ndarray, W1, b1, W2, b2) -> np.ndarray:
    """FFN(a) = W2 gelu(W1 a + b1) + b2, weights stored [out, in]."""
    return gelu_erf(a @ W1.T + b1) @ W2.T + b2


# --------------------------------------------------------------------------------------
# Token selection
# --------------------------------------------------------------------------------------

_M0, _M1 = 0xD2511F53, 0xCD9E8D57
_W0, _W1 = 0x9E3779B9, 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """Philox4x32 with 10 rounds (Salmon et al., 'Parallel random numbers: as easy as
    1, 2, 3', SC'11). counter = 4 uint32 words, key = 2 uint32 words -> 4 uint32 words."""
    c0, c1, c2, c3 = (int(v) & _MASK for v in counter)
    k0, k1 = (int(v) & _MASK for v in key)
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        c0, c1, c2, c3 = ((p1 >> 32) ^ c1 ^ k0) & _MASK, p1 & _MASK, \
                         ((p0 >> 32) ^ c3 ^ k1) & _MASK, p0 & _MASK
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def philox_uniform(seed: int, sample_idx: int, step: int) -> float:
    """u in [0,1) for (seed, sample, step): the first output word of Philox4x32-10 with
    key (seed low word, seed high word) and counter (sample_idx, step, 0, 0), keeping
    its top 24 bits: u = (r >> 8) * 2^-24 (exactly representable in fp32)."""
    r = philox4x32_10((sample_idx, step, 0, 0), (seed & _MASK, (seed >> 32) & _MASK))[0]
    return (r >> 8) * (1.0 / 16777216.0)


def select_greedy(logits: np.ndarray) -> np.ndarray:
    """argmax over the vocabulary; among equal maxima the smallest id wins."""
    return np.argmax(logits, axis=-1).astype(np.int32)   # numpy returns the first maximum


def topk_order(row: np.ndarray, k: int) -> np.ndarray:
    """ids of the k largest logits ordered by (logit descending, id ascending)."""
    ids = np.lexsort((np.arange(row.shape[0]), -row))     # primary -row, secondary id
    return ids[:k]


def select_topk(logits: np.ndarray, k: int, temperature: float, seed: int,
                sample_idx: np.ndarray, step: int, return_detail: bool = False):
    """Temperature + top-k sampling by inverse CDF.

    For each row: keep the k largest logits in (logit desc, id asc) order,
    w_i = exp((l_i - l_0) / T), c_i = w_0 + ... + w_i, u = philox_uniform(...);
    the token is the first i with c_i > u * c_{k-1} (the last one if none).
    """
    B = logits.shape[0]
    out = np.empty(B, dtype=np.int32)
    detail = []
    for b in range(B):
        row = logits[b].astype(np.float64)
        ids = topk_order(row, k)
        w = np.exp((row[ids] - row[ids[0]]) / temperature)
        c = np.cumsum(w)
        u = philox_uniform(seed, int(sample_idx[b]), step)
        thr = u * c[-1]
        pick = len(ids) - 1
        for i in range(len(ids)):
            if c[i] > thr:
                pick = i
                break
        out[b] = ids[pick]
        if return_detail:
            detail.append(dict(ids=ids, cdf=c, thr=thr, pick=pick, u=u))
    return (out, detail) if return_detail else out


def nucleus(row: np.ndarray, p: float, temperature: float):
    """(ids of the nucleus in (logit desc, id asc) order, their weights): with probabilities
    softmax(row / T), the shortest prefix of that order whose probability mass reaches p
    (Holtzman et al., 'The curious case of neural text degeneration', ICLR 2020: the smallest
    set of most probable tokens with total probability >= p). Weights are exp((l - max) / T)."""
    row = row.astype(np.float64)
    order = topk_order(row, row.shape[0])
    w = np.exp((row[order] - row[order[0]]) / temperature)
    c = np.cumsum(w)
    m = int(np.searchsorted(c, p * c[-1], side="left"))     # first prefix with mass >= p
    m = min(m, len(order) - 1)
    return order[: m + 1], w[: m + 1]


def select_topp(logits: np.ndarray, p: float, temperature: float, seed: int,
                sample_idx: np.ndarray, step: int, return_detail: bool = False):
    """Temperature + nucleus (top-p) sampling, the sampler of the paper's GRPO rollouts
    (Training details: top-p 0.9, temperature 0.7). Tokens outside the nucleus get probability
    zero; the token is drawn from what is left by inverse CDF over the vocabulary in id order:
    c_v = sum of the nucleus weights with id <= v, u = philox_uniform(...), the token is the
    first nucleus id v with c_v > u * c_last (the last nucleus id if none)."""
    B = logits.shape[0]
    out = np.empty(B, dtype=np.int32)
    detail = []
    for b in range(B):
        ids, w = nucleus(logits[b], p, temperature)
        by_id = np.argsort(ids, kind="stable")
        ids, w = ids[by_id], w[by_id]
        c = np.cumsum(w)
        u = philox_uniform(seed, int(sample_idx[b]), step)
        thr = u * c[-1]
        pick = len(ids) - 1
        for i in range(len(ids)):
            if c[i] > thr:
                pick = i
                break
        out[b] = ids[pick]
        if return_detail:
            detail.append(dict(ids=ids, cdf=c, thr=thr, pick=pick, u=u))
    return (out, detail) if return_detail else out


# --------------------------------------------------------------------------------------
# Head projections (Method / Architecture, Eq. 10): Y = P_out (concat_g [(I_g X) M_g + beta_g])
# --------------------------------------------------------------------------------------

def token_mixer_parallel(Z: np.ndarray, lw: dict, n_heads: int, matrices=None):
    """Sequence-parallel token-mixing block of one layer for one sample, Z[n, d] (normed inputs).
    Without projections this is mixer_parallel. With lw["W_in"] (rows g*d_h..(g+1)*d_h = I_g) and
    lw["W_out"] (= P_out): every position is projected, Q = Z W_in^T, the heads of Q are mixed along
    the sequence, and the concatenated result is projected back, Y = (.) W_out^T. The cache is the
    sum term of the PROJECTED values."""
    if "W_in" not in lw:
        return mixer_parallel(Z, lw["alpha"], lw["beta"], lw["lam"], n_heads, matrices)
    Q = Z @ lw["W_in"].T
    Yh, S = mixer_parallel(Q, lw["alpha"], lw["beta"], lw["lam"], n_heads, matrices)
    return Yh @ lw["W_out"].T, S


def token_mixer_recurrent(z: np.ndarray, S: np.ndarray, t: int, lw: dict, n_heads: int):
    """Recurrent counterpart of token_mixer_parallel for position t (batched over rows)."""
    if "W_in" not in lw:
        return mixer_recurrent_step(z, S, t, lw["alpha"], lw["beta"], lw["lam"], n_heads)
    q = z @ lw["W_in"].T
    yh, S_new = mixer_recurrent_step(q, S, t, lw["alpha"], lw["beta"], lw["lam"], n_heads)
    return yh @ lw["W_out"].T, S_new


# --------------------------------------------------------------------------------------
# Linearly combined heads (Architecture: every head holds one row-repeat and one column-repeat
# matrix and its output is a linear combination of the two products; twice the cache).
# Reading: the combination weights are two scalars per head, w[g] = (w_row, w_col); the per-position
# bias beta is added once.
# --------------------------------------------------------------------------------------

def combined_parallel(Z, alpha_r, alpha_c, beta, lam_r, lam_c, w, n_heads: int):
    """Z[n, d] -> Y[n, d] and the two hand-off caches S_r[d], S_c[d] for position n.
    Head g, channel slice c:  Y_c^T = w[g,0] Z_c^T M_row(alpha_r[g], lam_r[g])
                                    + w[g,1] Z_c^T M_col(alpha_c[g], lam_c[g]) + beta_c^T."""
    n, d = Z.shape
    dh = d // n_heads
    dt = Z.dtype.type
    Y = np.empty_like(Z)
    S_r = np.zeros(d, dtype=Z.dtype)
    S_c = np.zeros(d, dtype=Z.dtype)
    for g in range(n_heads):
        c = slice(g * dh, (g + 1) * dh)
        Mr = mixing_matrix("row", alpha_r[g], lam_r[g], n, dtype=dt)
        Mc = mixing_matrix("col", alpha_c[g], lam_c[g], n, dtype=dt)
        X = Z[:, c].T
        Y[:, c] = (dt(w[g][0]) * (X @ Mr) + dt(w[g][1]) * (X @ Mc)).T + beta[:n, c]
        for m in range(n):
            S_r[c] += dt(lam_r[g]) ** (n - m) * dt(alpha_r[g][m]) * Z[m, c]
            S_c[c] += dt(lam_c[g]) ** (n - m) * Z[m, c]
    return Y, S_r, S_c


def combined_recurrent_step(z, S_r, S_c, t: int, alpha_r, alpha_c, beta, lam_r, lam_c, w, n_heads: int):
    """Recurrent form of combined_parallel at position t (batched over leading dimensions):
      y    = w_row (alpha_r[t] z + S_r) + w_col alpha_c[t] (z + S_c) + beta_t      (Eq. 2 and Eq. 3, combined)
      S_r' = lam_r (S_r + alpha_r[t] z) ;  S_c' = lam_c (S_c + z)."""
    d = z.shape[-1]
    dh = d // n_heads
    dt = z.dtype.type
    y = np.empty_like(z)
    Sr_new, Sc_new = np.empty_like(S_r), np.empty_like(S_c)
    for g in range(n_heads):
        c = slice(g * dh, (g + 1) * dh)
        ar, ac = dt(alpha_r[g][t]), dt(alpha_c[g][t])
        u = ar * z[..., c]
        v = z[..., c] + S_c[..., c]
        y[..., c] = dt(w[g][0]) * (u + S_r[..., c]) + dt(w[g][1]) * (ac * v) + beta[t, c]
        Sr_new[..., c] = dt(lam_r[g]) * (S_r[..., c] + u)
        Sc_new[..., c] = dt(lam_c[g]) * v
    return y, Sr_new, Sc_new


# --------------------------------------------------------------------------------------
# Non-unitary kernels (Architecture, Eq. 11): Y = sum_{i<k} X_(i:d+i, :) W_i + beta with k column-repeat
# matrices W_i and X zero-padded to d + k rows, stride 1.
# Readings: the sum runs over the k filters i = 0..k-1 (the printed upper limit k would index a filter
# that W in R^{k x n x n} does not have); the zero rows follow the d hidden channels, so that output
# channel c mixes hidden channels c..c+k-1 and channels past d-1 contribute nothing; one set of k filters
# serves the whole hidden dimension (the equation has no head index).
# --------------------------------------------------------------------------------------

def kernel_parallel(Z, alpha, beta, lam, k: int):
    """Z[n, d] -> Y[n, d] by Eq. 11 as written, and the hand-off cache P[k, d] for position n:
    P[i] = sum_{m<n} lam[i]^(n-m) z_m (the sum term of Eq. 3 for filter i over the unpadded channels).
    alpha[k, >=n], lam[k], beta[>=n, d]."""
    n, d = Z.shape
    dt = Z.dtype.type
    Xpad = np.zeros((d + k, n), dtype=Z.dtype)
    Xpad[:d] = Z.T
    Yt = np.zeros((d, n), dtype=Z.dtype)
    for i in range(k):
        Yt += Xpad[i:d + i, :] @ mixing_matrix("col", alpha[i], lam[i], n, dtype=dt)
    P = np.zeros((k, d), dtype=Z.dtype)
    for i in range(k):
        for m in range(n):
            P[i] += dt(lam[i]) ** (n - m) * Z[m]
    return Yt.T + beta[:n], P


def kernel_recurrent_step(z, P, t: int, alpha, beta, lam, k: int):
    """Recurrent form of kernel_parallel at position t. z[..., d], P[k, ..., d].
      v_i = z + P_i ;  y[c] = sum_i alpha[i][t] v_i[c + i] (terms with c + i >= d are the zero padding) + beta_t[c]
      P_i' = lam[i] v_i."""
    d = z.shape[-1]
    dt = z.dtype.type
    y = np.zeros_like(z)
    P_new = np.empty_like(P)
    for i in range(k):
        v = z + P[i]
        y[..., :d - i] += dt(alpha[i][t]) * v[..., i:]
        P_new[i] = dt(lam[i]) * v
    return y + beta[t], P_new


# --------------------------------------------------------------------------------------
# The model
# --------------------------------------------------------------------------------------

class SRMOracle:
    """Whole-model oracle. `W` is the parameter dict of srm_inputs.make_weights (any dict
    of numpy arrays with those names works); all arithmetic runs in `dtype`."""

    def __init__(self, n_layers, d_model, vocab, n_ctx, W, n_heads=4, ln_eps=1e-5,
                 dtype=np.float64, mixer="mixed", kernel_size=1):
        """mixer: "mixed" (Eq. 2 / Eq. 3 heads side by side; cache [L, B, d]), "combined" (every head holds a
        row-repeat and a column-repeat matrix, outputs linearly combined; cache [L, 2, B, d]) or "kernel"
        (Eq. 11 with kernel_size filters; cache [L, k, B, d]). Head projections go with "mixed" only."""
        self.L, self.d, self.V, self.n_ctx, self.h = n_layers, d_model, vocab, n_ctx, n_heads
        self.eps, self.dt = ln_eps, dtype
        assert mixer in ("mixed", "combined", "kernel")
        self.mixer, self.k = mixer, kernel_size
        self.C = {"mixed": 1, "combined": 2, "kernel": kernel_size}[mixer]     # d-vectors of cache per layer and sample
        cv = lambda a: np.asarray(a, dtype=dtype)
        self.E, self.W_lm = cv(W["E"]), cv(W["W_lm"])
        self.lnf_g, self.lnf_b = cv(W["lnf_g"]), cv(W["lnf_b"])
        self.layers = [{k: cv(v) for k, v in lw.items()} for lw in W["layers"]]
        assert len(self.layers) == n_layers

    # -- sequence-parallel form --------------------------------------------------------
    def forward_parallel(self, tokens: np.ndarray, keep_x: bool = False):
        """tokens int[B, n] -> logits[B, n, V] for every position, hand-off cache
        state[L, B, d] (what position n would read). Token mixing uses the explicit
        matrices of Eq. 1 / Eq. 3 per head."""
        B, n = tokens.shape
        assert n <= self.n_ctx
        x = self.E[tokens]                                   # [B, n, d]; no positional embedding
        state = self.init_state(B)
        xs = []
        for l, lw in enumerate(self.layers):
            z = layer_norm(x, lw["ln1_g"], lw["ln1_b"], self.eps)
            y = np.empty_like(z)
            if self.mixer == "combined":
                for b in range(B):
                    y[b], state[l, 0, b], state[l, 1, b] = combined_parallel(
                        z[b], lw["alpha"], lw["alpha_col"], lw["beta"], lw["lam"], lw["lam_col"], lw["w_comb"], self.h)
            elif self.mixer == "kernel":
                for b in range(B):
                    y[b], state[l, :, b] = kernel_parallel(z[b], lw["alpha"], lw["beta"], lw["lam"], self.k)
            else:
                Ms = [mixing_matrix(kind, lw["alpha"][g], lw["lam"][g], n, dtype=self.dt)
                      for g, kind in enumerate(head_kinds(self.h))]
                for b in range(B):
                    y[b], state[l, b] = token_mixer_parallel(z[b], lw, self.h, Ms)
            x = x + y
            a = layer_norm(x, lw["ln2_g"], lw["ln2_b"], self.eps)
            x = x + feed_forward(a, lw["W1"], lw["b1"], lw["W2"], lw["b2"])
            if keep_x:
                xs.append(x.copy())
        logits = layer_norm(x, self.lnf_g, self.lnf_b, self.eps) @ self.W_lm.T
        return (logits, state, xs) if keep_x else (logits, state)

    # -- recurrent form ----------------------------------------------------------------
    def init_state(self, B: int) -> np.ndarray:
        if self.mixer == "mixed":
            return np.zeros((self.L, B, self.d), dtype=self.dt)
        return np.zeros((self.L, self.C, B, self.d), dtype=self.dt)

    def decode_step(self, state: np.ndarray, tok: np.ndarray, pos: int, keep_x: bool = False):
        """Consume tok[B] at absolute position `pos`: returns logits[B, V] (predicting
        position pos+1) and the updated cache state'[L, B, d]."""
        assert 0 <= pos < self.n_ctx
        x = self.E[tok]                                      # [B, d]
        new_state = np.empty_like(state)
        xs = []
        for l, lw in enumerate(self.layers):
            z = layer_norm(x, lw["ln1_g"], lw["ln1_b"], self.eps)
            if self.mixer == "combined":
                y, new_state[l, 0], new_state[l, 1] = combined_recurrent_step(
                    z, state[l, 0], state[l, 1], pos, lw["alpha"], lw["alpha_col"], lw["beta"], lw["lam"], lw["lam_col"],
                    lw["w_comb"], self.h)
            elif self.mixer == "kernel":
                y, new_state[l] = kernel_recurrent_step(z, state[l], pos, lw["alpha"], lw["beta"], lw["lam"], self.k)
            else:
                y, new_state[l] = token_mixer_recurrent(z, state[l], pos, lw, self.h)
            x = x + y
            a = layer_norm(x, lw["ln2_g"], lw["ln2_b"], self.eps)
            x = x + feed_forward(a, lw["W1"], lw["b1"], lw["W2"], lw["b2"])
            if keep_x:
                xs.append(x.copy())
        logits = layer_norm(x, self.lnf_g, self.lnf_b, self.eps) @ self.W_lm.T
        return (logits, new_state, xs) if keep_x else (logits, new_state)

    def prefill_recurrent(self, tokens: np.ndarray):
        """The recurrent form applied position by position to a prompt:
        logits[B, n, V] and the cache after n tokens."""
        B, n = tokens.shape
        state = self.init_state(B)
        out = np.empty((B, n, self.V), dtype=self.dt)
        for t in range(n):
            out[:, t], state = self.decode_step(state, tokens[:, t], t)
        return out, state

    # -- generation --------------------------------------------------------------------
    def generate(self, prompts: np.ndarray, gen: int, sampling: dict | None = None,
                 sample_idx: np.ndarray | None = None, parallel_prefill: bool = True):
        """Prefill the prompts, then produce `gen` tokens per sample. Generated token k
        is selected from the logits of position n-1+k and uses Philox step k.
        Returns tokens[B, gen], the per-step logits[gen, B, V] and the final state."""
        B, n = prompts.shape
        sampling = sampling or {"mode": "greedy"}
        sidx = np.arange(B) if sample_idx is None else sample_idx
        if parallel_prefill:
            lg, state = self.forward_parallel(prompts)
        else:
            lg, state = self.prefill_recurrent(prompts)
        logits = lg[:, -1]
        toks = np.empty((B, gen), dtype=np.int32)
        all_logits = np.empty((gen, B, self.V), dtype=self.dt)
        for k in range(gen):
            all_logits[k] = logits
            toks[:, k] = self.select(logits, sampling, sidx, k)
            if k + 1 < gen:
                logits, state = self.decode_step(state, toks[:, k], n + k)
        return toks, all_logits, state

    @staticmethod
    def select(logits, sampling, sample_idx, step):
        if sampling.get("mode", "greedy") == "greedy":
            return select_greedy(logits)
        if sampling["mode"] == "topp":
            return select_topp(logits, sampling["top_p"], sampling["temperature"],
                               sampling["seed"], sample_idx, step)
        return select_topk(logits, sampling["top_k"], sampling["temperature"],
                           sampling["seed"], sample_idx, step)
