"""fp64 CPU oracle for the GRASS per-layer structured-sparse gradient step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain restatement of the
method that the CUDA library is checked against.  It is imported by the test
suite, by the smoke check and by the benchmark's CPU-baseline leg, and by
nothing else; it shares no code with the CUDA path and must never serve as a
fallback for it.

Every function follows one passage of the GRASS paper (arXiv 2406.17660) and
says which.  All floating point is numpy float64; inputs of lower precision
(bf16 / fp32 values held in float32 arrays) are widened exactly.

Notation (Section 3 and Algorithm 1 of the paper):
    W   m x n weight matrix            dY  T x m gradient w.r.t. layer outputs
    X   T x n layer inputs             G   = dY^T X, the m x n weight gradient
    sigma_j  row picked by the j-th column of P (0-based here)
    rho_j    j-th diagonal entry of the scaling matrix rho;  P^T = rho B
    G_C = P^T G   (r x n),   Delta = U from Adam,   W <- W + alpha P Delta

Conventions the paper leaves open (each is a stated reading, not a fact of
the paper): rows are 0-based; ties in top-r go to the lowest row index; the
selected rows are reported in ascending row order; random draws come from
Philox4x32-10 words turned into u = word * 2^-32 and inverted through the
running sum of the row norms.

Pins (tests/test_oracle_pins.py): the dense triple loop for the projection,
brute-force subset search for top-r, Monte-Carlo unbiasedness and the
closed-form variance for the sampler, torch.optim.Adam for the dense special
case, the Algorithm-4 form of the loop, the index-coverage value printed in
the paper's appendix and published Philox known-answer vectors.
Parity unpinned: the Philox counter layout, the ascending output order and the
exponential-race realisation of the without-replacement variants are
conventions of this build; nothing in the paper can confirm or refute them
(the distribution the race produces is pinned against the sequential
definition).
"""
from __future__ import annotations

import numpy as np

TOPR = 0
MULTINOMIAL_NORM = 1       # q ~ lambda,   with replacement, rho = 1/sqrt(r q)
MULTINOMIAL_NORM2 = 2      # q ~ lambda^2, with replacement, rho = 1/sqrt(r q)
UNIFORM = 3                # q = 1/m,      with replacement, rho = sqrt(m/r)
MULTINOMIAL_NORM_NR = 4    # the three distributions without replacement, rho = 1
MULTINOMIAL_NORM2_NR = 5
UNIFORM_NR = 6

# Tag placed in the fourth counter word of every Philox call made by select.
PHILOX_STREAM_TAG = 0x47524153


# --------------------------------------------------------------------------
# Row norms of the weight gradient (Section 3.2: lambda_k = ||G_k||_2)
# --------------------------------------------------------------------------
def dense_grad(dY, X):
    """G_W = (nabla_y L)^T X, the chain-rule form of Section 3.1 (a plain sum
    over tokens, no division by T)."""
    dY = np.asarray(dY, dtype=np.float64)
    X = np.asarray(X, dtype=np.float64)
    return dY.T @ X


def row_norms(G):
    """lambda_k = sqrt(sum_c G[k,c]^2) for every row k (Section 3.2, the row
    norms that Top-r and Multinomial-Norm are built from)."""
    G = np.asarray(G, dtype=np.float64)
    return np.sqrt(np.sum(G * G, axis=1))


def grad_row_norms(dY, X):
    """Row norms of G_W = dY^T X: what a refresh iteration feeds to compute_P."""
    return row_norms(dense_grad(dY, X))


# --------------------------------------------------------------------------
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
# easy as 1, 2, 3", SC'11).  Written out with Python integers.
# --------------------------------------------------------------------------
_PHILOX_M0 = 0xD2511F53
_PHILOX_M1 = 0xCD9E8D57
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """Ten rounds of Philox-4x32.  counter: 4 words, key: 2 words -> 4 words."""
    c0, c1, c2, c3 = (int(c) & _MASK32 for c in counter)
    k0, k1 = (int(k) & _MASK32 for k in key)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK32
        hi1, lo1 = p1 >> 32, p1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK32, lo1, (hi0 ^ c3 ^ k1) & _MASK32, lo0
        k0 = (k0 + _PHILOX_W0) & _MASK32
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return (c0, c1, c2, c3)


def draw_words(r, seed, layer_id, epoch):
    """The r 32-bit words consumed by one selection refresh.

    Draw j takes output word (j mod 4) of the Philox block whose key is the
    64-bit seed split into (low, high) words and whose counter is
    (j div 4, layer_id, epoch, PHILOX_STREAM_TAG).  Being counter-based, the
    stream is a pure function of (seed, layer_id, epoch, j).
    """
    key = (seed & _MASK32, (seed >> 32) & _MASK32)
    words = np.empty(r, dtype=np.uint64)
    block = None
    for j in range(r):
        if j % 4 == 0:
            block = philox4x32_10((j // 4, layer_id, epoch, PHILOX_STREAM_TAG), key)
        words[j] = block[j % 4]
    return words


# --------------------------------------------------------------------------
# compute_P (Section 3.2)
# --------------------------------------------------------------------------
class DegenerateNorms(ValueError):
    """Raised when the norms cannot define a selection (negative, non-finite,
    or all zero where a distribution is needed)."""


def _check_norms(norms):
    lam = np.asarray(norms, dtype=np.float64)
    if lam.ndim != 1 or not np.all(np.isfinite(lam)) or np.any(lam < 0):
        raise DegenerateNorms("row norms must be finite and non-negative")
    return lam


def select_topr(norms, r):
    """Top-r (Section 3.2 B): rho = 1 and sigma = the rows with the r largest
    norms.  Ties go to the lower row index; output ascending by row."""
    lam = _check_norms(norms)
    m = lam.shape[0]
    if not 1 <= r <= m:
        raise ValueError("need 1 <= r <= m")
    order = sorted(range(m), key=lambda k: (-lam[k], k))
    sigma = np.array(sorted(order[:r]), dtype=np.int64)
    rho = np.ones(r, dtype=np.float64)
    return sigma, rho


def sampling_weights(lam, method):
    """Unnormalised q of the three sampling distributions of Section 3.2 A."""
    if method in (MULTINOMIAL_NORM, MULTINOMIAL_NORM_NR):
        return lam.copy()                       # Multinomial-Norm (Theorem 1)
    if method in (MULTINOMIAL_NORM2, MULTINOMIAL_NORM2_NR):
        return lam * lam                        # Multinomial-Norm^2 (subspace preservation)
    if method in (UNIFORM, UNIFORM_NR):
        return np.ones_like(lam)                # Uniform
    raise ValueError("not a sampling method")


def select_with_replacement(norms, r, method, seed, layer_id, epoch):
    """Sampling with replacement (Section 3.2 A): sigma_j i.i.d. ~ Multinomial(1, q) with
    q = w / sum(w), w from sampling_weights; rho_j = 1 / sqrt(r * q_{sigma_j}).

    Draw j inverts the running sum c_k = sum_{i<=k} w_i at u_j * S with
    u_j = word_j * 2^-32: sigma_j = min{k : c_k > u_j S}, so a zero-weight row
    is never drawn.  The r pairs are reported ascending by row (repeats kept).
    """
    lam = _check_norms(norms)
    m = lam.shape[0]
    if not 1 <= r <= m:
        raise ValueError("need 1 <= r <= m")
    w = sampling_weights(lam, method)
    c = np.cumsum(w)
    S = c[-1]
    if not S > 0:
        raise DegenerateNorms("all sampling weights are zero")
    words = draw_words(r, seed, layer_id, epoch)
    sigma = np.empty(r, dtype=np.int64)
    for j in range(r):
        u = float(words[j]) * 2.0 ** -32
        k = int(np.searchsorted(c, u * S, side="right"))
        sigma[j] = min(k, m - 1)
    sigma.sort()
    q = w[sigma] / S
    rho = 1.0 / np.sqrt(r * q)
    return sigma, rho


def select_multinomial_norm(norms, r, seed, layer_id, epoch):
    """Multinomial-Norm with replacement (Section 3.2 A, Theorem 1): q_k = lambda_k / sum(lambda)."""
    return select_with_replacement(norms, r, MULTINOMIAL_NORM, seed, layer_id, epoch)


def nr_scores(norms, method, seed, layer_id, epoch):
    """Scores whose r largest entries are a sample without replacement.

    The paper's "-NR" variants (Section 3.2 A) draw r distinct rows, each draw
    from q restricted to the rows not yet drawn, and set rho = 1; it does not
    say how the draws are made.  This build uses the exponential-race form of
    that sequential scheme (Efraimidis & Spirakis 2006): row k gets
    t_k = -log(u_k) / w_k with u_k uniform on (0, 1); the rows with the r
    smallest t -- equivalently the r largest scores w_k / (-log u_k) -- are
    distributed exactly as r successive draws without replacement.
    u_k = (word_k + 1/2) * 2^-32, word_k = Philox word (k mod 4) of block
    (k div 4, layer_id, epoch, tag).  Scores are fp64 and ranked as such (ties to
    the lower row); an implementation that ranks rounded scores may differ only
    where two scores at the selection threshold agree to its rounding.
    """
    lam = _check_norms(norms)
    m = lam.shape[0]
    w = sampling_weights(lam, method)
    words = draw_words(m, seed, layer_id, epoch).astype(np.float64)
    u = (words + 0.5) * 2.0 ** -32
    return w / -np.log(u)


def select_without_replacement(norms, r, method, seed, layer_id, epoch):
    """The -NR variants: r distinct rows, rho = 1, ascending by row."""
    lam = _check_norms(norms)
    m = lam.shape[0]
    if not 1 <= r <= m:
        raise ValueError("need 1 <= r <= m")
    if np.count_nonzero(sampling_weights(lam, method) > 0) < r:
        raise DegenerateNorms("fewer than r rows have positive weight")
    return select_topr(nr_scores(norms, method, seed, layer_id, epoch), r)


def select(norms, r, method, seed=0, layer_id=0, epoch=0):
    if method == TOPR:
        return select_topr(norms, r)
    if method in (MULTINOMIAL_NORM, MULTINOMIAL_NORM2, UNIFORM):
        return select_with_replacement(norms, r, method, seed, layer_id, epoch)
    if method in (MULTINOMIAL_NORM_NR, MULTINOMIAL_NORM2_NR, UNIFORM_NR):
        return select_without_replacement(norms, r, method, seed, layer_id, epoch)
    raise ValueError("unknown selection method")


# --------------------------------------------------------------------------
# Projected gradient (Section 3.1, "Efficient Gradient Projection")
# --------------------------------------------------------------------------
def project_grad(dY, X, sigma, rho=None):
    """G_C = rho ((B dY^T) X):  G_C[j, :] = rho_j * sum_t dY[t, sigma_j] X[t, :].
    Repeated rows in sigma give repeated rows of G_C."""
    dY = np.asarray(dY, dtype=np.float64)
    X = np.asarray(X, dtype=np.float64)
    sigma = np.asarray(sigma, dtype=np.int64)
    picked = dY[:, sigma]                      # B dY^T, transposed: T x r
    Gc = picked.T @ X                          # r x n
    if rho is not None:
        Gc = np.asarray(rho, dtype=np.float64)[:, None] * Gc
    return Gc


# --------------------------------------------------------------------------
# Adam on the subspace state (Appendix A, adam.init / adam.update)
# --------------------------------------------------------------------------
def adam_init(r, n):
    return np.zeros((r, n)), np.zeros((r, n))


def adam_update(M, V, g, lr, beta1, beta2, eps, step):
    """One adam.update: returns (M_new, V_new, U).  `step` is t >= 1, the
    number of updates since the state was last zeroed."""
    if step < 1:
        raise ValueError("step counts from 1")
    g = np.asarray(g, dtype=np.float64)
    M_new = beta1 * np.asarray(M, dtype=np.float64) + (1.0 - beta1) * g
    V_new = beta2 * np.asarray(V, dtype=np.float64) + (1.0 - beta2) * g * g
    M_star = M_new / (1.0 - beta1 ** step)
    V_star = V_new / (1.0 - beta2 ** step)
    U = -lr * M_star / (np.sqrt(V_star) + eps)
    return M_new, V_new, U


# --------------------------------------------------------------------------
# Sparse weight update (Algorithm 1, "Apply update"; Section 3.1)
# --------------------------------------------------------------------------
def round_to_bf16(x):
    """Round float64 values to the nearest bfloat16 (ties to even), returned
    as float64.  bfloat16 = sign, 8 exponent bits, 7 stored fraction bits."""
    x = np.asarray(x, dtype=np.float64)
    out = np.array(x, copy=True)
    finite = np.isfinite(x) & (x != 0)
    mant, expo = np.frexp(x[finite])             # x = mant * 2^expo, 0.5 <= |mant| < 1
    expo = np.maximum(expo, -125)                # below 2^-126 the spacing stays 2^-133
    scale = np.ldexp(1.0, expo - 8)              # spacing of bf16 values in that binade
    out[finite] = np.rint(x[finite] / scale) * scale   # rint = ties to even
    out[np.abs(out) >= 2.0 ** 128] *= np.inf     # past the largest bf16: overflow
    return out


def scatter_update(W, U, sigma, rho, alpha, w_is_bf16=False):
    """W <- W + alpha P Delta with P = (rho B)^T: only rows sigma_j change,
    row sigma_j gains alpha * rho_j * U[j, :], repeated rows add up.  With
    w_is_bf16 the sum is rounded once to bfloat16 at the end."""
    W = np.array(W, dtype=np.float64, copy=True)
    U = np.asarray(U, dtype=np.float64)
    sigma = np.asarray(sigma, dtype=np.int64)
    r = sigma.shape[0]
    rho = np.ones(r) if rho is None else np.asarray(rho, dtype=np.float64)
    for j in range(r):
        W[sigma[j], :] += alpha * rho[j] * U[j, :]
    if w_is_bf16:
        touched = np.unique(sigma)
        W[touched, :] = round_to_bf16(W[touched, :])
    return W


# --------------------------------------------------------------------------
# The loop (Algorithm 1, GRASS instantiation)
# --------------------------------------------------------------------------
def layer_steps(W, batches, r, method, K, alpha, lr, beta1, beta2, eps,
                reset_state=True, seed=0, layer_id=0, w_is_bf16=False,
                trace=None):
    """Run Algorithm 1 for len(batches) iterations t = 0, 1, ...

    batches[t] = (dY_t, X_t).  Every K iterations P is recomputed from this
    iteration's own gradient and (optionally) the Adam state is zeroed; then
    G_C = P^T G, Adam, and the row-sparse apply.  Returns the final
    (W, M, V, sigma, rho).  If `trace` is a list, one dict per iteration with
    every intermediate is appended to it.
    """
    W = np.array(W, dtype=np.float64, copy=True)
    n = W.shape[1]
    M, V = adam_init(r, n)
    sigma = rho = None
    adam_step = 0
    for t, (dY, X) in enumerate(batches):
        norms = None
        if t % K == 0:
            norms = row_norms(dense_grad(dY, X))
            sigma, rho = select(norms, r, method, seed, layer_id, t // K)
            if reset_state:
                M, V = adam_init(r, n)
                adam_step = 0
        adam_step += 1
        Gc = project_grad(dY, X, sigma, rho)
        M, V, U = adam_update(M, V, Gc, lr, beta1, beta2, eps, adam_step)
        W = scatter_update(W, U, sigma, rho, alpha, w_is_bf16)
        if trace is not None:
            trace.append(dict(t=t, norms=norms, sigma=sigma.copy(), rho=rho.copy(),
                              Gc=Gc, M=M.copy(), V=V.copy(), U=U, W=W.copy(),
                              adam_step=adam_step))
    return W, M, V, sigma, rho


# --------------------------------------------------------------------------
# Projecting the smaller dimension (Section 4.1: "P is applied to project the
# smaller dimension of G_W")
# --------------------------------------------------------------------------
def scatter_update_cols(W, U, sigma, rho, alpha, w_is_bf16=False):
    """Column form of the apply step: W <- W + alpha * Delta P^T with P in R^{n x r}
    selecting columns: W[:, sigma_j] += alpha * rho_j * U[j, :], U being r x m."""
    W = np.array(W, dtype=np.float64, copy=True)
    U = np.asarray(U, dtype=np.float64)
    sigma = np.asarray(sigma, dtype=np.int64)
    r = sigma.shape[0]
    rho = np.ones(r) if rho is None else np.asarray(rho, dtype=np.float64)
    for j in range(r):
        W[:, sigma[j]] += alpha * rho[j] * U[j, :]
    if w_is_bf16:
        touched = np.unique(sigma)
        W[:, touched] = round_to_bf16(W[:, touched])
    return W


def layer_steps_cols(W, batches, r, method, K, alpha, lr, beta1, beta2, eps, **kw):
    """Algorithm 1 with the projection on the input dimension n (used when m > n):
    G_C = G_W P is m x r, kept here as its transpose (r x m).  Selecting columns of
    G_W = dY^T X is selecting rows of G_W^T = X^T dY, so this is Algorithm 1 on W^T
    with the roles of dY and X exchanged."""
    swapped = [(X, dY) for dY, X in batches]
    trace = kw.get("trace")
    Wt, M, V, sigma, rho = layer_steps(np.asarray(W, dtype=np.float64).T, swapped, r, method, K,
                                       alpha, lr, beta1, beta2, eps, **kw)
    if trace is not None:
        for rec in trace:
            rec["W"] = rec["W"].T
    return Wt.T, M, V, sigma, rho
