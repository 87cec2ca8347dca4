"""Pins of the fp64 oracle against what the paper and the mathematics fix.

Nothing here touches the CUDA path.  Each test is chosen so that a plausible
slip in the oracle (a dropped rho, a transposed operand, a wrong tie-break, a
wrong bias correction, an off-by-one in the inverse CDF) makes it fail.
"""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import accounting
from oracle import grass_oracle as oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def _small_problem(rng, T=6, m=16, n=8, skew=1.0):
    dY = rng.standard_normal((T, m)) * np.exp(skew * rng.standard_normal(m))[None, :]
    X = rng.standard_normal((T, n))
    return dY, X


# ---- projection: G_C = rho ((B dY^T) X) is rows of the dense gradient (Section 3.1) ----
def test_projection_equals_scaled_rows_of_dense_triple_loop():
    rng = np.random.default_rng(1)
    T, m, n = 5, 7, 4
    dY, X = _small_problem(rng, T, m, n)
    G = np.zeros((m, n))
    for k in range(m):
        for c in range(n):
            for t in range(T):
                G[k, c] += dY[t, k] * X[t, c]
    sigma = np.array([0, 2, 2, 6])
    rho = np.array([0.5, 2.0, 3.0, 1.25])
    Gc = oracle.project_grad(dY, X, sigma, rho)
    assert Gc.shape == (4, n)
    for j in range(4):
        np.testing.assert_allclose(Gc[j], rho[j] * G[sigma[j]], rtol=1e-12, atol=1e-14)
    # r = m, identity sigma, rho = 1 is the textbook product dY^T X
    np.testing.assert_allclose(oracle.project_grad(dY, X, np.arange(m)), G, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(oracle.dense_grad(dY, X), G, rtol=1e-12, atol=1e-14)
    # row norms against the definition, element by element
    lam = oracle.row_norms(G)
    for k in range(m):
        assert abs(lam[k] - sum(v * v for v in G[k]) ** 0.5) <= 1e-13 * lam[k]


# ---- top-r minimises ||P P^T G - G||_F^2 (Section 3.2 B), brute force over all subsets ----
@pytest.mark.parametrize("m,r", [(6, 2), (9, 4), (10, 3)])
def test_topr_is_the_minimiser_by_brute_force(m, r):
    rng = np.random.default_rng(m * 10 + r)
    G = rng.standard_normal((m, 5)) * np.exp(rng.standard_normal(m))[:, None]
    lam = oracle.row_norms(G)
    sigma, rho = oracle.select_topr(lam, r)
    assert np.all(rho == 1.0) and list(sigma) == sorted(sigma) and len(set(sigma)) == r

    def err(rows):
        R = G.copy()
        R[list(rows)] = 0.0          # P P^T G keeps the chosen rows, zeroes the rest
        return np.sum(R * R)

    best = min(itertools.combinations(range(m), r), key=err)
    assert tuple(sigma) == best
    unselected = np.setdiff1d(np.arange(m), sigma)
    assert abs(err(sigma) - np.sum(lam[unselected] ** 2)) < 1e-12


def test_topr_ties_go_to_lowest_index():
    lam = np.array([1.0, 3.0, 3.0, 0.5, 3.0, 3.0, 0.0, 0.0])
    assert list(oracle.select_topr(lam, 3)[0]) == [1, 2, 4]
    assert list(oracle.select_topr(lam, 5)[0]) == [0, 1, 2, 4, 5]
    assert list(oracle.select_topr(lam, 7)[0]) == [0, 1, 2, 3, 4, 5, 6]
    assert list(oracle.select_topr(np.zeros(5), 2)[0]) == [0, 1]
    with pytest.raises(oracle.DegenerateNorms):
        oracle.select_topr(np.array([1.0, np.nan]), 1)


# ---- Philox4x32-10 known answers ----
def test_philox_known_answers():
    rows = _rows("philox4x32_10_kat.txt")
    assert len(rows) == 3
    for row in rows:
        w = [int(x, 16) for x in row]
        assert list(oracle.philox4x32_10(w[0:4], w[4:6])) == w[6:10]


def test_draw_words_layout():
    seed = 0x0123456789ABCDEF
    words = oracle.draw_words(7, seed, layer_id=3, epoch=9)
    key = (0x89ABCDEF, 0x01234567)
    b0 = oracle.philox4x32_10((0, 3, 9, oracle.PHILOX_STREAM_TAG), key)
    b1 = oracle.philox4x32_10((1, 3, 9, oracle.PHILOX_STREAM_TAG), key)
    assert [int(w) for w in words] == list(b0) + list(b1[:3])


# ---- the sampler: frequencies, rho, unbiasedness, variance (Section 3.2 A, Appendices C, D) ----
def test_multinomial_inverse_cdf_by_hand():
    lam = np.array([0.0, 2.0, 0.0, 1.0, 1.0])          # S = 4, c = [0,2,2,3,4]
    r = 4
    words = oracle.draw_words(r, 11, 0, 0)
    expect = []
    for w in words:
        x = float(w) / 2 ** 32 * 4.0
        expect.append(1 if x < 2 else (3 if x < 3 else 4))
    sigma, rho = oracle.select_multinomial_norm(lam, r, 11, 0, 0)
    assert list(sigma) == sorted(expect)
    q = lam / 4.0
    np.testing.assert_allclose(rho, 1 / np.sqrt(r * q[sigma]), rtol=1e-15)
    with pytest.raises(oracle.DegenerateNorms):
        oracle.select_multinomial_norm(np.zeros(5), 2, 0, 0, 0)


def test_multinomial_frequencies_chi_square():
    lam = np.array([5.0, 0.1, 1.0, 0.0, 2.5, 0.4, 8.0, 1.0])
    q = lam / lam.sum()
    r, epochs = 8, 3000
    counts = np.zeros(8)
    for e in range(epochs):
        sigma, _ = oracle.select_multinomial_norm(lam, r, seed=77, layer_id=2, epoch=e)
        counts += np.bincount(sigma, minlength=8)
    assert counts[3] == 0                                # zero-norm row is never drawn
    nz = q > 0
    expected = q[nz] * r * epochs
    chi2 = np.sum((counts[nz] - expected) ** 2 / expected)
    assert chi2 < 24.3                                   # 99.9 % point of chi^2 with 6 dof is 22.5


def test_reconstruction_is_unbiased_with_closed_form_variance():
    """E[P P^T G] = G (Appendix C) and the total variance equals
    (1/r)(sum_k lambda_k^2 / q_k - ||G||_F^2), which follows from
    E[P P^T P P^T] = (1/r) diag(1/q) + ((r-1)/r) I (Appendix D).  rho enters
    twice: once in P^T G and once in P Delta."""
    rng = np.random.default_rng(5)
    T, m, n, r = 6, 16, 8, 4
    dY, X = _small_problem(rng, T, m, n, skew=0.7)
    G = oracle.dense_grad(dY, X)
    lam = oracle.row_norms(G)
    q = lam / lam.sum()
    epochs = 40000
    s1 = np.zeros((m, n))
    s2 = np.zeros((m, n))
    for e in range(epochs):
        sigma, rho = oracle.select_multinomial_norm(lam, r, seed=123, layer_id=1, epoch=e)
        Gc = oracle.project_grad(dY, X, sigma, rho)
        R = oracle.scatter_update(np.zeros((m, n)), Gc, sigma, rho, alpha=1.0)
        s1 += R
        s2 += R * R
    mean = s1 / epochs
    var_elem = (1 - q)[:, None] / (r * q)[:, None] * G * G          # per-element closed form
    se = np.sqrt(var_elem / epochs)
    assert np.all(np.abs(mean - G) <= 5 * se + 1e-12)
    emp_total_var = np.sum(s2 / epochs - mean * mean)
    closed = (np.sum(lam ** 2 / q) - np.sum(G * G)) / r
    assert abs(closed - (lam.sum() ** 2 - np.sum(lam ** 2)) / r) < 1e-9 * closed
    assert abs(emp_total_var - closed) < 0.05 * closed
    # Theorem 1: q ~ lambda gives less total variance than uniform or q ~ lambda^2
    for other in (np.full(m, 1 / m), lam ** 2 / np.sum(lam ** 2)):
        assert closed <= (np.sum(lam ** 2 / other) - np.sum(G * G)) / r + 1e-12
    assert emp_total_var < (np.sum(lam ** 2 * m) - np.sum(G * G)) / r


def test_dropping_rho_from_the_apply_step_would_be_biased():
    """Guards the pin above: without rho in P Delta the mean is visibly off."""
    rng = np.random.default_rng(5)
    dY, X = _small_problem(rng, 6, 16, 8, skew=0.7)
    G = oracle.dense_grad(dY, X)
    lam = oracle.row_norms(G)
    s1 = np.zeros_like(G)
    for e in range(4000):
        sigma, rho = oracle.select_multinomial_norm(lam, 4, 123, 1, e)
        s1 += oracle.scatter_update(np.zeros_like(G), oracle.project_grad(dY, X, sigma, rho),
                                    sigma, None, 1.0)
    assert np.linalg.norm(s1 / 4000 - G) > 0.2 * np.linalg.norm(G)


def test_index_coverage_matches_the_papers_printed_value():
    (m, r, updates, pct), = _rows("index_coverage.txt")
    m, r, updates, pct = int(m), int(r), int(updates), float(pct)
    formula = 1 - ((1 - 1 / m) ** r) ** updates
    assert round(100 * formula, 2) == pct
    lam = np.ones(m)                                      # equal norms: the sampler is uniform
    cover = []
    for trial in range(120):
        seen = np.zeros(m, dtype=bool)
        for e in range(updates):
            sigma, rho = oracle.select_multinomial_norm(lam, r, seed=1000 + trial, layer_id=0, epoch=e)
            seen[sigma] = True
        cover.append(seen.mean())
    np.testing.assert_allclose(rho, np.sqrt(m / r), rtol=1e-14)
    assert abs(np.mean(cover) - formula) < 0.0025         # 4 standard errors of the mean


# ---- Adam and the apply step ----
def test_adam_first_step_closed_form_and_bias_correction():
    rng = np.random.default_rng(2)
    g = rng.standard_normal((3, 5))
    M, V = oracle.adam_init(3, 5)
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    M1, V1, U1 = oracle.adam_update(M, V, g, lr, b1, b2, eps, 1)
    np.testing.assert_allclose(U1, -lr * g / (np.abs(g) + eps), rtol=1e-12)
    np.testing.assert_allclose(M1, 0.1 * g, rtol=1e-12)
    np.testing.assert_allclose(V1, 0.001 * g * g, rtol=1e-12)
    with pytest.raises(ValueError):
        oracle.adam_update(M, V, g, lr, b1, b2, eps, 0)


def test_full_rank_identity_projection_is_dense_adam():
    """r = m, rho = 1, alpha = 1: the loop is Adam on W with gradient dY^T X."""
    rng = np.random.default_rng(3)
    T, m, n = 9, 6, 5
    W0 = rng.standard_normal((m, n)) * 0.02
    batches = [_small_problem(rng, T, m, n) for _ in range(3)]
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    W, M, V, sigma, rho = oracle.layer_steps(W0, batches, r=m, method=oracle.TOPR, K=1, alpha=1.0,
                                             lr=lr, beta1=b1, beta2=b2, eps=eps, reset_state=False)
    assert list(sigma) == list(range(m)) and np.all(rho == 1)
    p = torch.nn.Parameter(torch.tensor(W0, dtype=torch.float64))
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=0, amsgrad=False)
    for dY, X in batches:
        p.grad = torch.tensor(dY).T @ torch.tensor(X)
        opt.step()
    np.testing.assert_allclose(W, p.detach().numpy(), rtol=1e-9, atol=1e-12)
    st = opt.state[p]
    np.testing.assert_allclose(M, st["exp_avg"].numpy(), rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(V, st["exp_avg_sq"].numpy(), rtol=1e-10, atol=1e-16)


def test_apply_touches_only_selected_rows_and_sums_repeats():
    rng = np.random.default_rng(4)
    W = rng.standard_normal((8, 3))
    U = rng.standard_normal((4, 3))
    sigma = np.array([1, 5, 5, 6])
    rho = np.array([2.0, 0.5, 4.0, 1.0])
    out = oracle.scatter_update(W, U, sigma, rho, alpha=0.25)
    for k in (0, 2, 3, 4, 7):
        assert np.array_equal(out[k], W[k])               # bit-identical
    np.testing.assert_allclose(out[1], W[1] + 0.25 * 2.0 * U[0], rtol=1e-15)
    np.testing.assert_allclose(out[5], W[5] + 0.25 * (0.5 * U[1] + 4.0 * U[2]), rtol=1e-15)
    np.testing.assert_allclose(out[6], W[6] + 0.25 * U[3], rtol=1e-15)


def test_loop_equals_the_explicit_A_matrix_form():
    """Algorithm 1 against Algorithm 4 (Appendix B): keep A = sum of alpha*Delta
    explicitly, fold W0 <- W0 + P A at every refresh, and compare W0 + P A."""
    rng = np.random.default_rng(6)
    T, m, n, r, K, steps = 7, 12, 5, 4, 3, 8
    W_init = rng.standard_normal((m, n))
    batches = [_small_problem(rng, T, m, n) for _ in range(steps)]
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8)
    for method, reset in ((oracle.MULTINOMIAL_NORM, True), (oracle.TOPR, False)):
        trace = []
        oracle.layer_steps(W_init, batches, r, method, K, alpha=0.25, reset_state=reset,
                           seed=9, layer_id=4, trace=trace, **hp)
        W0 = W_init.copy()
        A = np.zeros((r, n))
        P = np.zeros((m, r))
        M, V = oracle.adam_init(r, n)
        s = 0
        for t, (dY, X) in enumerate(batches):
            G = np.asarray(dY).T @ np.asarray(X)
            if t % K == 0:
                W0 = W0 + P @ A
                A = np.zeros((r, n))
                sigma, rho = oracle.select(oracle.row_norms(G), r, method, 9, 4, t // K)
                P = np.zeros((m, r))
                P[sigma, np.arange(r)] = rho               # P = (rho B)^T, dense
                if reset:
                    M, V = oracle.adam_init(r, n)
                    s = 0
            s += 1
            M, V, U = oracle.adam_update(M, V, P.T @ G, hp["lr"], hp["beta1"], hp["beta2"],
                                         hp["eps"], s)
            A = A + 0.25 * U
            np.testing.assert_allclose(trace[t]["W"], W0 + P @ A, rtol=1e-11, atol=1e-13)
            untouched = np.setdiff1d(np.arange(m), sigma)
            prev = W_init if t == 0 else trace[t - 1]["W"]
            assert np.array_equal(trace[t]["W"][untouched], prev[untouched])


# ---- bf16 rounding helper ----
def test_bf16_rounding_matches_torch_conversion():
    rng = np.random.default_rng(8)
    x = np.concatenate([
        rng.standard_normal(4000) * np.exp(6 * rng.standard_normal(4000)),
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, -1.00390625, 3.3895314e38, 1e-40,
                  9.1835e-41, 4.5e-41, 2 ** -133, 2 ** -134, 1.5 * 2 ** -133, 65280.0, 65408.0]),
    ])
    x32 = x.astype(np.float32).astype(np.float64)          # exact fp32 values, as the GPU holds
    want = torch.tensor(x32, dtype=torch.float64).to(torch.float32).to(torch.bfloat16) \
        .to(torch.float64).numpy()
    got = oracle.round_to_bf16(x32)
    assert np.array_equal(got, want)
    W = np.array([[1.0, 2.0]])
    out = oracle.scatter_update(W, np.array([[2 ** -8, 2 ** -7]]), [0], None, 1.0, w_is_bf16=True)
    assert np.array_equal(out, np.array([[1.0, 2.0]]))     # both are ties: round to even


# ---- state-size accounting against the paper's 13B worked example ----
def test_memory_accounting_reproduces_13b_example():
    got = accounting.grass_memory_mib(hidden=5120, ffn=13824, layers=40, heads=40, vocab=32000,
                                      seq=256, batch=1, r=128)
    for name, val in _rows("memory_13b.txt"):
        assert round(got[name], 2) == float(val), name


# ---- the other sampling distributions of Section 3.2 A ----
def test_norm2_and_uniform_with_replacement_frequencies_and_rho():
    lam = np.array([3.0, 0.5, 1.0, 0.0, 2.0, 0.25])
    r, epochs = 6, 3000
    for method, w in ((oracle.MULTINOMIAL_NORM2, lam ** 2), (oracle.UNIFORM, np.ones(6))):
        q = w / w.sum()
        counts = np.zeros(6)
        for e in range(epochs):
            sigma, rho = oracle.select(lam, r, method, seed=5, layer_id=1, epoch=e)
            counts += np.bincount(sigma, minlength=6)
            np.testing.assert_allclose(rho, 1 / np.sqrt(r * q[sigma]), rtol=1e-14)
        nz = q > 0
        expected = q[nz] * r * epochs
        chi2 = np.sum((counts[nz] - expected) ** 2 / expected)
        assert chi2 < 20.5 if nz.sum() == 6 else chi2 < 18.5      # 99.9 % points, 5 and 4 dof
        assert np.all(counts[~nz] == 0)
    sigma, rho = oracle.select(lam, 3, oracle.UNIFORM, seed=1)
    np.testing.assert_allclose(rho, np.sqrt(6 / 3), rtol=1e-14)


def test_without_replacement_matches_sequential_sampling_exactly_in_distribution():
    """The exponential race must give each unordered pair the probability that two successive
    draws without replacement give it: w_a/S * w_b/(S - w_a) + w_b/S * w_a/(S - w_b)."""
    lam = np.array([1.0, 2.0, 3.0, 4.0])
    for method, w in ((oracle.MULTINOMIAL_NORM_NR, lam), (oracle.MULTINOMIAL_NORM2_NR, lam ** 2),
                      (oracle.UNIFORM_NR, np.ones(4))):
        S = w.sum()
        pairs = list(itertools.combinations(range(4), 2))
        p = np.array([w[a] / S * w[b] / (S - w[a]) + w[b] / S * w[a] / (S - w[b]) for a, b in pairs])
        assert abs(p.sum() - 1) < 1e-12
        epochs = 12000
        counts = np.zeros(len(pairs))
        for e in range(epochs):
            sigma, rho = oracle.select(lam, 2, method, seed=99, layer_id=0, epoch=e)
            assert len(set(sigma)) == 2 and np.all(rho == 1.0) and sigma[0] < sigma[1]
            counts[pairs.index(tuple(sigma))] += 1
        chi2 = np.sum((counts - p * epochs) ** 2 / (p * epochs))
        assert chi2 < 20.5                                         # 99.9 % point, 5 dof
    # r = m takes every row; too few positive weights is an error
    assert list(oracle.select(lam, 4, oracle.MULTINOMIAL_NORM_NR, seed=3)[0]) == [0, 1, 2, 3]
    with pytest.raises(oracle.DegenerateNorms):
        oracle.select(np.array([1.0, 0.0, 0.0]), 2, oracle.MULTINOMIAL_NORM_NR, seed=3)
    assert len(oracle.select(np.array([1.0, 0.0, 0.0]), 2, oracle.UNIFORM_NR, seed=3)[0]) == 2


# ---- projecting the input dimension (Section 4.1, smaller-dimension rule) ----
def test_column_projection_equals_dense_right_multiplication():
    """G_C = G_W P, Adam on it, W += alpha * Delta P^T, written with dense matrices."""
    rng = np.random.default_rng(12)
    T, m, n, r = 7, 9, 5, 3
    W0 = rng.standard_normal((m, n))
    batches = [_small_problem(rng, T, m, n) for _ in range(4)]
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8)
    trace = []
    oracle.layer_steps_cols(W0, batches, r, oracle.MULTINOMIAL_NORM, K=2, alpha=0.5,
                            reset_state=True, seed=8, layer_id=1, trace=trace, **hp)
    W = W0.copy()
    for t, (dY, X) in enumerate(batches):
        G = dY.T @ X                                              # m x n
        if t % 2 == 0:
            col_norms = np.sqrt(np.sum(G * G, axis=0))
            sigma, rho = oracle.select(col_norms, r, oracle.MULTINOMIAL_NORM, 8, 1, t // 2)
            P = np.zeros((n, r))
            P[sigma, np.arange(r)] = rho
            M, V = np.zeros((m, r)), np.zeros((m, r))
            s = 0
        s += 1
        Mt, Vt, Ut = oracle.adam_update(M.T, V.T, (G @ P).T, hp["lr"], hp["beta1"], hp["beta2"],
                                        hp["eps"], s)
        M, V = Mt.T, Vt.T
        W = W + 0.5 * Ut.T @ P.T
        np.testing.assert_allclose(trace[t]["W"], W, rtol=1e-11, atol=1e-13)
    U = rng.standard_normal((r, m))
    sig = np.array([0, 3, 3])
    rho3 = np.array([2.0, 0.5, 1.5])
    out = oracle.scatter_update_cols(W0, U, sig, rho3, 0.25)
    assert np.array_equal(out[:, [1, 2, 4]], W0[:, [1, 2, 4]])
    np.testing.assert_allclose(out[:, 3], W0[:, 3] + 0.25 * (0.5 * U[1] + 1.5 * U[2]), rtol=1e-15)
