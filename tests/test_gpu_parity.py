"""Parity of the CUDA library (through the C ABI) with the fp64 oracle, element by element.

Tolerances (stated by the build's acceptance criteria, and where tighter,
derived from the arithmetic):
  indices            bit-exact, except where the deciding fp64 quantity is within 1e-6 relative
  projected gradient relative Frobenius error <= 1e-2 for bf16 inputs (acceptance); the kernel
                     multiplies bf16 exactly and accumulates in fp32, so <= 1e-4 is also required
                     (catches a dropped token block that 1e-2 would let through); fp32 path 1e-5
  Adam M, V, U       1e-5 relative
  updated rows       fp32 W: 1e-5 relative; bf16 W: at most 1 bf16 ulp from the oracle's rounding
  unselected rows    bit-identical
"""
import numpy as np
import pytest
import torch

import paper_2406_17660_b200 as grass
from paper_2406_17660_b200 import synthetic as syn
from oracle import grass_oracle as oracle

pytestmark = pytest.mark.gpu
DEV = "cuda"


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def f64(t):
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def ws_bytes(nbytes):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=DEV)


# --------------------------------------------------------------------------- row norms
@pytest.mark.parametrize("m,n,ld,dtype", [
    (256, 256, 256, torch.float32),
    (37, 1001, 1001, torch.float32),       # no 128-bit path, ragged
    (64, 5461, 5464, torch.float32),       # padded pitch, tail columns
    (24, 11008, 11008, torch.float32),     # CTA-per-row path
    (9, 4099, 4104, torch.bfloat16),
    (300, 520, 520, torch.bfloat16),
    (1, 1, 1, torch.float32),
])
def test_row_norms(m, n, ld, dtype):
    g = torch.Generator().manual_seed(m * 7 + n)
    G = (torch.randn((m, n), generator=g) * torch.exp(torch.randn((m, 1), generator=g))).to(dtype)
    Gd = syn._padded(G.to(DEV), ld)
    norms = torch.full((m,), -1.0, dtype=torch.float32, device=DEV)
    grass.grass_row_norms(Gd, norms)
    grass.grass_device_status()
    want = oracle.row_norms(f64(G))
    np.testing.assert_allclose(f64(norms), want, rtol=1e-5, atol=0)


@pytest.mark.parametrize("T,m,n,dtype,ld", [
    (512, 256, 256, torch.float32, None),
    (100, 50, 70, torch.float32, None),
    (1024, 512, 512, torch.bfloat16, None),
    (777, 1376, 520, torch.bfloat16, None),              # 3 row blocks, ragged T
    (640, 300, 328, torch.bfloat16, None),               # ragged m and n
    (512, 2048, 5461, torch.bfloat16, 5464),             # padded pitch, n not a tile multiple
    (256, 13824, 640, torch.bfloat16, None),             # 27 row blocks
])
def test_grad_row_norms_without_forming_the_gradient(T, m, n, dtype, ld):
    X = syn.make_X(T, n, dtype, seed0=T + m)
    dY = syn.make_dY(T, m, dtype, seed0=T + m)
    Xd = syn._padded(X.to(DEV), ld or n)
    norms = torch.full((m,), -1.0, dtype=torch.float32, device=DEV)
    dt = grass.BF16 if dtype == torch.bfloat16 else grass.F32
    ws = ws_bytes(grass.grass_grad_row_norms_workspace_bytes(T, m, n, dt))
    dYd = syn._padded(dY.to(DEV), syn.pad_to(m, 8))      # the TMA path reads dY rows directly
    grass.grass_grad_row_norms(dYd, Xd, norms, ws)
    grass.grass_device_status()
    want = oracle.grad_row_norms(f64(dY), f64(X))
    np.testing.assert_allclose(f64(norms), want, rtol=1e-5)
    again = torch.empty_like(norms)
    grass.grass_grad_row_norms(dYd, Xd, again, ws)
    assert torch.equal(again, norms)                      # fixed summation order


# --------------------------------------------------------------------------- selection
def _gpu_select(norms_np, r, method, seed=0, layer_id=0, epoch=0):
    norms = torch.tensor(norms_np, dtype=torch.float32, device=DEV)
    m = norms.numel()
    idx = torch.full((r,), -7, dtype=torch.int32, device=DEV)
    rho = torch.full((r,), -7.0, dtype=torch.float32, device=DEV)
    ws = ws_bytes(grass.grass_select_workspace_bytes(m, r, method))
    grass.grass_select(norms, r, method, seed, layer_id, epoch, idx, rho, ws)
    status, detail = grass.grass_device_status(raise_on_error=False)
    return status, idx.cpu().numpy(), rho.cpu().numpy()


def _lognormal_norms(m, seed, zeros=0):
    rng = np.random.default_rng(seed)
    lam = np.exp(rng.standard_normal(m)).astype(np.float32)
    if zeros:
        lam[rng.choice(m, zeros, replace=False)] = 0.0
    return lam


@pytest.mark.parametrize("m,r", [(256, 32), (512, 128), (1000, 1), (1000, 1000), (13824, 1024),
                                 (5000, 4097)])
def test_select_topr_bit_exact(m, r):
    lam = _lognormal_norms(m, m + r, zeros=m // 10)
    status, idx, rho = _gpu_select(lam, r, grass.SEL_TOPR)
    assert status == 0
    sigma, _ = oracle.select_topr(lam, r)
    assert np.array_equal(idx, sigma)
    assert np.all(rho == 1.0)


def test_select_topr_ties_lowest_index():
    lam = np.zeros(3000, dtype=np.float32)
    lam[5::7] = 2.0          # many equal norms straddling the threshold
    lam[100] = 3.0
    lam[2999] = 3.0
    lam[0] = -0.0
    for r in (1, 2, 3, 50, 400, 431, 2000):
        status, idx, _ = _gpu_select(lam, r, grass.SEL_TOPR)
        assert status == 0
        assert np.array_equal(idx, oracle.select_topr(lam, r)[0]), r


def _check_multinomial(lam, r, seed, layer_id, epoch):
    status, idx, rho = _gpu_select(lam, r, grass.SEL_MULTINOMIAL_NORM, seed, layer_id, epoch)
    assert status == 0
    sigma, rho_ref = oracle.select_multinomial_norm(lam, r, seed, layer_id, epoch)
    if not np.array_equal(idx, sigma):
        # allowed only where a draw falls within 1e-6 (relative to the total) of a CDF step
        c = np.cumsum(lam.astype(np.float64))
        u = oracle.draw_words(r, seed, layer_id, epoch).astype(np.float64) * 2.0 ** -32 * c[-1]
        gap = np.min(np.abs(c[None, :] - u[:, None]), axis=1) / c[-1]
        assert np.sum(idx != sigma) <= np.sum(gap < 1e-6), "index mismatch beyond the near-tie allowance"
    else:
        np.testing.assert_allclose(rho, rho_ref, rtol=1e-6)
    assert np.all(np.diff(idx) >= 0)


@pytest.mark.parametrize("m,r,seed,layer_id,epoch", [
    (512, 128, 0, 0, 0), (512, 128, 0, 3, 17), (1376, 128, 12345678901234567, 55, 2),
    (13824, 1024, 7, 1, 1), (300, 300, 99, 0, 0), (2048, 512, 2 ** 63 + 5, 167, 4000000000),
    (64, 1, 1, 1, 1),
])
def test_select_multinomial_matches_oracle(m, r, seed, layer_id, epoch):
    _check_multinomial(_lognormal_norms(m, m * 3 + r, zeros=m // 8), r, seed, layer_id, epoch)


@pytest.mark.parametrize("method", [grass.SEL_MULTINOMIAL_NORM2, grass.SEL_UNIFORM])
@pytest.mark.parametrize("m,r", [(512, 128), (5461, 512), (13824, 1024)])
def test_select_other_distributions_with_replacement(method, m, r):
    lam = _lognormal_norms(m, m + r + method, zeros=m // 8)
    status, idx, rho = _gpu_select(lam, r, method, seed=21, layer_id=6, epoch=3)
    assert status == 0
    sigma, rho_ref = oracle.select(lam, r, method, seed=21, layer_id=6, epoch=3)
    if not np.array_equal(idx, sigma):
        w = oracle.sampling_weights(lam.astype(np.float64), method)
        c = np.cumsum(w)
        u = oracle.draw_words(r, 21, 6, 3).astype(np.float64) * 2.0 ** -32 * c[-1]
        gap = np.min(np.abs(c[None, :] - u[:, None]), axis=1) / c[-1]
        assert np.sum(idx != sigma) <= np.sum(gap < 1e-6)
    else:
        np.testing.assert_allclose(rho, rho_ref, rtol=1e-6)


@pytest.mark.parametrize("method", [grass.SEL_MULTINOMIAL_NORM_NR, grass.SEL_MULTINOMIAL_NORM2_NR,
                                    grass.SEL_UNIFORM_NR])
@pytest.mark.parametrize("m,r", [(512, 128), (2048, 512), (13824, 1024), (300, 260)])
def test_select_without_replacement(method, m, r):
    lam = _lognormal_norms(m, m + 5 * r + method, zeros=m // 10)
    status, idx, rho = _gpu_select(lam, r, method, seed=4242, layer_id=9, epoch=1)
    assert status == 0
    sigma, _ = oracle.select(lam, r, method, seed=4242, layer_id=9, epoch=1)
    assert np.all(rho == 1.0) and len(set(idx.tolist())) == r and np.all(np.diff(idx) > 0)
    if not np.array_equal(idx, sigma):
        # allowed only where the fp64 scores at the selection threshold are within 1e-6 relative
        sc = oracle.nr_scores(lam, method, 4242, 9, 1).astype(np.float64)
        thr = np.sort(sc)[-r]
        swapped = np.setxor1d(idx, sigma)
        assert np.all(np.abs(sc[swapped] - thr) <= 1e-6 * thr), "mismatch beyond the near-tie allowance"


@pytest.mark.parametrize("method", [grass.SEL_MULTINOMIAL_NORM, grass.SEL_MULTINOMIAL_NORM2])
def test_sampling_never_lands_on_a_zero_weight_row(method):
    """Many rows of zero weight between rows of very different weight: the fp64 running sum of a
    warp scan is not exactly monotone there, and a draw that landed on a zero-weight row would
    make rho infinite.  The kernel's running sum repeats the predecessor's entry on such rows."""
    rng = np.random.default_rng(77)
    for trial in range(4):
        m, r = 13824, 1024
        lam = np.exp(3.0 * rng.standard_normal(m)).astype(np.float32)
        lam[rng.random(m) < 0.6] = 0.0
        status, idx, rho = _gpu_select(lam, r, method, seed=trial, layer_id=trial, epoch=trial)
        assert status == 0
        assert np.all(lam[idx] > 0) and np.all(np.isfinite(rho)) and np.all(rho > 0)
        sigma, rho_ref = oracle.select(lam, r, method, seed=trial, layer_id=trial, epoch=trial)
        if np.array_equal(idx, sigma):
            np.testing.assert_allclose(rho, rho_ref, rtol=1e-6)
        else:
            c = np.cumsum(oracle.sampling_weights(lam.astype(np.float64), method))
            u = oracle.draw_words(r, trial, trial, trial).astype(np.float64) * 2.0 ** -32 * c[-1]
            gap = np.min(np.abs(c[None, :] - u[:, None]), axis=1) / c[-1]
            assert np.sum(idx != sigma) <= np.sum(gap < 1e-6)


def test_select_without_replacement_needs_enough_positive_rows():
    lam = np.zeros(64, dtype=np.float32)
    lam[:5] = 1.0
    status, idx, _ = _gpu_select(lam, 6, grass.SEL_MULTINOMIAL_NORM_NR)
    assert status == 4 and np.all(idx == -7)
    status, idx, _ = _gpu_select(lam, 5, grass.SEL_MULTINOMIAL_NORM_NR)
    assert status == 0 and np.array_equal(idx, np.arange(5))
    status, idx, _ = _gpu_select(lam, 6, grass.SEL_UNIFORM_NR)
    assert status == 0


def test_select_degenerate_inputs_leave_outputs_untouched():
    lam = _lognormal_norms(100, 1)
    for bad, method in ((np.nan, grass.SEL_TOPR), (np.inf, grass.SEL_TOPR), (-1.0, grass.SEL_TOPR),
                        (np.nan, grass.SEL_MULTINOMIAL_NORM)):
        x = lam.copy()
        x[41] = bad
        status, idx, rho = _gpu_select(x, 10, method)
        assert status == 4                       # GRASS_ERR_DEGENERATE
        assert np.all(idx == -7) and np.all(rho == -7.0)
    status, idx, rho = _gpu_select(np.zeros(100, dtype=np.float32), 10, grass.SEL_MULTINOMIAL_NORM)
    assert status == 4 and np.all(idx == -7)
    status, idx, _ = _gpu_select(np.zeros(100, dtype=np.float32), 10, grass.SEL_TOPR)
    assert status == 0 and np.array_equal(idx, np.arange(10))


# --------------------------------------------------------------------------- projection
def _project_case(T, m, n, r, dtype, seed, ldx=None, lddy=None, identity=False, dup=False,
                  with_rho=True, opts=None):
    X = syn.make_X(T, n, dtype, seed0=seed, ld=ldx)
    dY = syn.make_dY(T, m, dtype, seed0=seed, ld=lddy)
    rng = np.random.default_rng(seed)
    if identity:
        sigma, idx_t = np.arange(m), None
        r = m
    else:
        sigma = np.sort(rng.choice(m, r, replace=dup))
        idx_t = torch.tensor(sigma, dtype=torch.int32, device=DEV)
    rho_np = (0.5 + rng.random(r)).astype(np.float32) if with_rho else None
    rho_t = None if rho_np is None else torch.tensor(rho_np, device=DEV)
    Xd = syn._padded(X.to(DEV), ldx or n)
    dYd = syn._padded(dY.to(DEV), lddy or m)
    Gc = torch.full((r, n), float("nan"), dtype=torch.float32, device=DEV)
    dt = grass.BF16 if dtype == torch.bfloat16 else grass.F32
    if opts is None:
        ws = ws_bytes(grass.grass_project_workspace_bytes(T, m, n, r, dt))
        grass.grass_project_grad(dYd, Xd, idx_t, rho_t, r, Gc, ws)
    else:
        plan = grass.grass_project_plan(1, T, m, n, r, opts)
        ws = ws_bytes(plan["workspace_bytes"])
        ws.fill_(0xA5)                       # the library must not rely on a clean workspace
        grass.grass_project_grad_ex([dYd], [Xd], [idx_t], None if rho_t is None else [rho_t], r,
                                    [Gc], ws, opts)
    grass.grass_device_status()
    want = oracle.project_grad(f64(dY), f64(X), sigma, rho_np)
    return f64(Gc), want


def _assert_close_gc(got, want, tol=1e-4):
    """Frobenius bound (the acceptance metric) plus an element-wise bound that localises a bad
    tile: no element off by more than tol of the largest expected magnitude."""
    assert np.all(np.isfinite(got))
    err = rel_fro(got, want)
    assert err <= tol, err
    worst = np.max(np.abs(got - want))
    assert worst <= tol * np.max(np.abs(want)), worst


@pytest.mark.parametrize("T,m,n,r", [(512, 256, 256, 32), (100, 50, 70, 7), (33, 65, 129, 65)])
def test_project_fp32(T, m, n, r):
    got, want = _project_case(T, m, n, r, torch.float32, seed=T + r, dup=(r == 7))
    _assert_close_gc(got, want, 1e-5)
    got, want = _project_case(T, m, n, r, torch.float32, seed=T, identity=True, with_rho=False)
    _assert_close_gc(got, want, 1e-5)


@pytest.mark.parametrize("T,m,n,r,ldx,kw", [
    (256, 256, 256, 64, None, {}),                       # one tile, 8 token blocks
    (1000, 300, 328, 100, None, {}),                     # ragged T, n, r
    (4096, 512, 512, 128, None, {"dup": True}),          # 60M-shaped, repeated rows
    (2048, 1376, 512, 128, None, {}),
    (3000, 1024, 2736, 256, None, {}),                   # 350M down-shaped, n not a tile multiple
    (2048, 2048, 5461, 512, 5464, {}),                   # 1B down-shaped, padded pitch
    (1536, 4096, 1024, 1024, None, {}),                  # two row blocks of 512
    (1024, 700, 640, 600, None, {}),                     # two row blocks of 320
    (777, 320, 200, 320, None, {"identity": True}),      # dense gradient, idx = NULL
    (64, 128, 128, 1, None, {}),                         # r = 1
    (31, 64, 64, 64, None, {"with_rho": False}),         # fewer tokens than one block
    (200, 50, 70, 20, 72, {}),                           # n not a multiple of 8 (padded pitch), odd m
    (64, 13824, 256, 13824, None, {"identity": True}),   # largest LLaMA row count, dense: 27 row blocks
    (96, 640, 128, 384, None, {}),                       # 384 rows: MMA chunks of 256 + 128, single CTA
    (96, 640, 512, 384, None, {}),                       # same through a CTA pair
    (3000, 512, 1024, 128, None, {"dup": True}),         # dense pick, wide n: in-kernel gather
    (700, 600, 1000, 64, None, {}),                      # in-kernel gather, single CTA, ragged T and n
    (2100, 256, 2048, 32, None, {}),                     # 32 rows padded to a 64-row tile
])
def test_project_bf16_tensor_core(T, m, n, r, ldx, kw):
    got, want = _project_case(T, m, n, r, torch.bfloat16, seed=T + n + r, ldx=ldx, **kw)
    assert rel_fro(got, want) <= 1e-2                     # acceptance tolerance
    _assert_close_gc(got, want, 1e-4)                     # what fp32 accumulation must deliver


def test_project_bf16_is_bit_reproducible_and_flags_bad_rows():
    T, m, n, r = 2048, 512, 512, 128
    X = syn.make_X(T, n, torch.bfloat16).to(DEV)
    dY = syn.make_dY(T, m, torch.bfloat16).to(DEV)
    idx = torch.arange(0, 4 * r, 4, dtype=torch.int32, device=DEV)
    ws = ws_bytes(grass.grass_project_workspace_bytes(T, m, n, r, grass.BF16))
    outs = []
    for _ in range(2):
        Gc = torch.empty((r, n), dtype=torch.float32, device=DEV)
        grass.grass_project_grad(dY, X, idx, None, r, Gc, ws)
        grass.grass_device_status()
        outs.append(Gc.clone())
    assert torch.equal(outs[0], outs[1])
    bad = idx.clone()
    bad[5] = m + 3
    Gc = torch.empty((r, n), dtype=torch.float32, device=DEV)
    grass.grass_project_grad(dY, X, bad, None, r, Gc, ws)
    status, detail = grass.grass_device_status(raise_on_error=False)
    assert status == 1 and detail == m + 3
    assert torch.all(Gc[5] == 0) and torch.equal(Gc[6], outs[0][6])


# --------------------------------------------------------------------------- Adam
@pytest.mark.parametrize("r,n,ld,step", [(32, 256, 256, 1), (128, 1376, 1376, 7), (5, 33, 40, 3),
                                         (3, 8, 9, 1000)])
def test_subspace_adam(r, n, ld, step):
    g = torch.Generator().manual_seed(r + n)
    Gc = torch.randn((r, n), generator=g) * torch.exp(2 * torch.randn((r, 1), generator=g))
    M = torch.randn((r, n), generator=g) * 0.1 if step > 1 else torch.zeros((r, n))
    V = torch.rand((r, n), generator=g) * 0.01 if step > 1 else torch.zeros((r, n))
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    Md, Vd = syn._padded(M.to(DEV), ld), syn._padded(V.to(DEV), ld)
    Ud = syn._padded(torch.zeros((r, n), device=DEV), ld)
    grass.grass_subspace_adam(Gc.to(DEV), Md, Vd, Ud, lr, b1, b2, eps, step)
    grass.grass_device_status()
    M1, V1, U1 = oracle.adam_update(f64(M), f64(V), f64(Gc), lr, b1, b2, eps, step)
    # 1e-5 relative to the size of the terms that were added: M mixes two signed terms, so an
    # element-wise bound relative to the (possibly cancelled) result would be ill-conditioned.
    scale_M = b1 * np.abs(f64(M)) + (1 - b1) * np.abs(f64(Gc))
    assert np.all(np.abs(f64(Md) - M1) <= 1e-5 * scale_M + 1e-30)
    np.testing.assert_allclose(f64(Vd), V1, rtol=1e-5, atol=1e-30)
    scale_U = lr * (scale_M / (1 - b1 ** step)) / (np.sqrt(V1 / (1 - b2 ** step)) + eps)
    assert np.all(np.abs(f64(Ud) - U1) <= 1e-5 * scale_U + 1e-30)
    assert rel_fro(f64(Md), M1) <= 1e-6 and rel_fro(f64(Ud), U1) <= 1e-6


# --------------------------------------------------------------------------- scatter
@pytest.mark.parametrize("m,n,ld,r,dtype", [
    (256, 256, 256, 32, torch.float32), (512, 1376, 1376, 128, torch.bfloat16),
    (100, 37, 40, 9, torch.bfloat16), (64, 5461, 5464, 16, torch.bfloat16),
    (50, 30, 30, 50, torch.float32),
])
def test_scatter_update(m, n, ld, r, dtype):
    rng = np.random.default_rng(m + n + r)
    W = syn.make_W(m, n, dtype, seed0=r)
    U = torch.tensor(rng.standard_normal((r, n)) * 1e-3, dtype=torch.float32)
    sigma = np.sort(rng.choice(m, r, replace=True))
    rho = (0.5 + 3 * rng.random(r)).astype(np.float32)
    Wd = syn._padded(W.to(DEV), ld)
    before = Wd.clone()
    grass.grass_scatter_update(Wd, U.to(DEV), torch.tensor(sigma, dtype=torch.int32, device=DEV),
                               torch.tensor(rho, device=DEV), 0.25)
    grass.grass_device_status()
    is_bf16 = dtype == torch.bfloat16
    want = oracle.scatter_update(f64(W), f64(U), sigma, rho, 0.25, w_is_bf16=is_bf16)
    got = f64(Wd)
    untouched = np.setdiff1d(np.arange(m), sigma)
    assert torch.equal(Wd[untouched], before[untouched])             # bit-identical
    touched = np.unique(sigma)
    if is_bf16:
        exact = oracle.scatter_update(f64(W), f64(U), sigma, rho, 0.25)[touched]
        ulp = np.ldexp(1.0, np.floor(np.log2(np.maximum(np.abs(exact), 2.0 ** -126))).astype(int) - 7)
        diff = np.abs(got[touched] - want[touched])
        assert np.all(diff <= ulp * 1.0001)
        assert np.mean(diff > 0) < 0.01                              # rounding-boundary cases only
    else:
        np.testing.assert_allclose(got[touched], want[touched], rtol=1e-5, atol=1e-9)


# --------------------------------------------------------------------------- whole step
def _run_layer(m, n, T, r, dtype, method, K, steps, alpha, reset, seed, layer_id=0):
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    W = syn.make_W(m, n, dtype, seed0=seed)
    batches = [(syn.make_dY(T, m, dtype, seed0=seed, step=t), syn.make_X(T, n, dtype, seed0=seed, step=t))
               for t in range(steps)]
    ws = grass.step.GrassWorkspace([(m, n)], T, r, dtype, method)
    Wd = W.to(DEV).clone()
    layer = grass.GrassLayer(Wd, r, method, K, alpha, lr, b1, b2, eps, reset_state=reset, seed=seed,
                             layer_id=layer_id, workspace=ws)
    trace = []
    oracle.layer_steps(f64(W), [(f64(a), f64(b)) for a, b in batches], r, method, K, alpha, lr, b1,
                       b2, eps, reset_state=reset, seed=seed, layer_id=layer_id,
                       w_is_bf16=(dtype == torch.bfloat16), trace=trace)
    for t, (dY, X) in enumerate(batches):
        before = layer.W.clone()
        M_prev, V_prev = f64(layer.M), f64(layer.V)
        layer.step(dY.to(DEV), X.to(DEV))
        grass.grass_device_status()
        ref = trace[t]
        assert np.array_equal(layer.idx.cpu().numpy(), ref["sigma"]), f"step {t}: rows differ"
        np.testing.assert_allclose(layer.rho.cpu().numpy(), ref["rho"], rtol=2e-5)
        tol = 1e-5 if dtype == torch.float32 else 1e-4
        _assert_close_gc(f64(layer.Gc), ref["Gc"], tol)
        # Adam and the apply step from the GPU's own G_C and previous state: this isolates the
        # update kernels from the GEMM's summation order, so the stated 1e-5 applies element-wise
        if reset and t % K == 0:
            M_prev[:] = 0.0
            V_prev[:] = 0.0
        g_gpu = f64(layer.Gc)
        M1, V1, U1 = oracle.adam_update(M_prev, V_prev, g_gpu, lr, b1, b2, eps, layer.adam_step)
        scale_M = b1 * np.abs(M_prev) + (1 - b1) * np.abs(g_gpu)
        assert np.all(np.abs(f64(layer.M) - M1) <= 1e-5 * scale_M + 1e-30), f"step {t}: M"
        np.testing.assert_allclose(f64(layer.V), V1, rtol=1e-5, atol=1e-30)
        s = layer.adam_step
        scale_U = lr * (scale_M / (1 - b1 ** s)) / (np.sqrt(V1 / (1 - b2 ** s)) + eps)
        assert np.all(np.abs(f64(layer.U) - U1) <= 1e-5 * scale_U + 1e-30), f"step {t}: U"
        sigma, rho_gpu = ref["sigma"], layer.rho.cpu().numpy()
        touched = np.unique(sigma)
        untouched = np.setdiff1d(np.arange(m), sigma)
        got = f64(layer.W)
        assert torch.equal(layer.W[untouched], before[untouched])      # bit-identical
        exact = oracle.scatter_update(f64(before), f64(layer.U), sigma, rho_gpu, alpha)[touched]
        if dtype == torch.float32:
            np.testing.assert_allclose(got[touched], exact, rtol=1e-5, atol=1e-9)
        else:
            want = oracle.round_to_bf16(exact)
            ulp = np.ldexp(1.0, np.floor(np.log2(np.maximum(np.abs(exact), 2.0 ** -126))).astype(int) - 7)
            diff = np.abs(got[touched] - want)
            assert np.all(diff <= ulp * 1.0001), f"step {t}: W off by more than one bf16 ulp"
            assert np.mean(diff > 0) < 0.01                             # rounding-boundary cases only
        # end to end against the oracle's own trajectory (secondary: the bf16 GEMM's fp32
        # summation order feeds into these)
        assert rel_fro(f64(layer.M), ref["M"]) <= tol
        assert rel_fro(f64(layer.V), ref["V"]) <= 2 * tol
        assert rel_fro(f64(layer.U), ref["U"]) <= 10 * tol
        if dtype == torch.float32:
            np.testing.assert_allclose(got, ref["W"], rtol=1e-5, atol=1e-8)
        else:
            assert np.max(np.abs(got - ref["W"])) <= 2.0 ** -7 * np.max(np.abs(ref["W"]))
            assert np.mean(got != ref["W"]) < 0.02
    return layer


def test_layer_steps_config1_fp32_topr():
    """m = n = 256, T = 512, r = 32, top-r, K = 1, 3 steps, fp32 everywhere, seed 0."""
    _run_layer(256, 256, 512, 32, torch.float32, grass.SEL_TOPR, K=1, steps=3, alpha=1.0,
               reset=True, seed=0)


def test_layer_steps_bf16_multinomial_with_refresh():
    """60M-shaped q projection at reduced T: multinomial-norm, rho, refresh at t = 0 and 2."""
    _run_layer(512, 512, 2048, 128, torch.bfloat16, grass.SEL_MULTINOMIAL_NORM, K=2, steps=4,
               alpha=0.25, reset=False, seed=3, layer_id=5)


@pytest.mark.parametrize("m,n", [(1024, 1024), (1024, 2736)], ids=["350m_q", "350m_down"])
def test_layer_steps_350m_topr_ten_steps_across_a_refresh(m, n):
    """LLaMA-350M q and down shapes, top-r, r = 256, K = 5, ten steps (refresh at t = 0 and 5,
    state reset on), at a token count the oracle affords; every step is checked element-wise."""
    _run_layer(m, n, 4096, 256, torch.bfloat16, grass.SEL_TOPR, K=5, steps=10, alpha=0.25,
               reset=True, seed=6, layer_id=1)


def test_layer_steps_bf16_topr_reset():
    _run_layer(1376, 512, 1024, 128, torch.bfloat16, grass.SEL_TOPR, K=2, steps=3, alpha=0.25,
               reset=True, seed=4)


# --------------------------------------------------------------------------- column projection
@pytest.mark.parametrize("m,n,ld,r,dtype", [
    (300, 256, 256, 64, torch.float32), (1376, 512, 512, 128, torch.bfloat16),
    (100, 77, 80, 40, torch.bfloat16), (64, 40, 40, 40, torch.float32),
])
def test_scatter_update_cols(m, n, ld, r, dtype):
    rng = np.random.default_rng(m + n + r)
    W = syn.make_W(m, n, dtype, seed0=r)
    U = torch.tensor(rng.standard_normal((r, m)) * 1e-3, dtype=torch.float32)
    sigma = np.sort(rng.choice(n, r, replace=True))          # repeats, some runs longer than a tile
    sigma[: min(r, 36)] = sigma[0]
    sigma = np.sort(sigma)
    rho = (0.5 + 3 * rng.random(r)).astype(np.float32)
    Wd = syn._padded(W.to(DEV), ld)
    before = Wd.clone()
    grass.grass_scatter_update_cols(Wd, U.to(DEV), torch.tensor(sigma, dtype=torch.int32, device=DEV),
                                    torch.tensor(rho, device=DEV), 0.25)
    grass.grass_device_status()
    is_bf16 = dtype == torch.bfloat16
    want = oracle.scatter_update_cols(f64(W), f64(U), sigma, rho, 0.25, w_is_bf16=is_bf16)
    got = f64(Wd)
    untouched = np.setdiff1d(np.arange(n), sigma)
    assert torch.equal(Wd[:, untouched], before[:, untouched])
    touched = np.unique(sigma)
    if is_bf16:
        exact = oracle.scatter_update_cols(f64(W), f64(U), sigma, rho, 0.25)[:, touched]
        ulp = np.ldexp(1.0, np.floor(np.log2(np.maximum(np.abs(exact), 2.0 ** -126))).astype(int) - 7)
        diff = np.abs(got[:, touched] - want[:, touched])
        assert np.all(diff <= ulp * 1.0001) and np.mean(diff > 0) < 0.01
    else:
        np.testing.assert_allclose(got[:, touched], want[:, touched], rtol=1e-5, atol=1e-9)


def test_layer_steps_projecting_the_input_dimension():
    """gate/up-shaped layer (m > n): the selection picks input features (columns of W)."""
    m, n, T, r = 1376, 512, 1024, 128
    dtype, method = torch.bfloat16, grass.SEL_MULTINOMIAL_NORM
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    W = syn.make_W(m, n, dtype, seed0=8)
    batches = [(syn.make_dY(T, m, dtype, seed0=8, step=t), syn.make_X(T, n, dtype, seed0=8, step=t))
               for t in range(3)]
    ws = grass.step.GrassWorkspace([(n, m)], T, r, dtype, method)
    layer = grass.GrassLayer(W.to(DEV).clone(), r, method, 2, 0.25, lr, b1, b2, eps, reset_state=True,
                             seed=8, layer_id=1, workspace=ws, side="cols")
    trace = []
    oracle.layer_steps_cols(f64(W), [(f64(a), f64(b)) for a, b in batches], r, method, 2, 0.25, lr,
                            b1, b2, eps, reset_state=True, seed=8, layer_id=1, w_is_bf16=True,
                            trace=trace)
    for t, (dY, X) in enumerate(batches):
        before = layer.W.clone()
        layer.step(dY.to(DEV), X.to(DEV))
        grass.grass_device_status()
        ref = trace[t]
        assert np.array_equal(layer.idx.cpu().numpy(), ref["sigma"])
        assert layer.Gc.shape == (r, m) and rel_fro(f64(layer.Gc), ref["Gc"]) <= 1e-4
        assert rel_fro(f64(layer.M), ref["M"]) <= 1e-4
        untouched = np.setdiff1d(np.arange(n), ref["sigma"])
        assert torch.equal(layer.W[:, untouched], before[:, untouched])
        got = f64(layer.W)
        assert np.max(np.abs(got - ref["W"])) <= 2.0 ** -7 * np.max(np.abs(ref["W"]))
        assert np.mean(got != ref["W"]) < 0.02


# --------------------------------------------------------------------------- fused Adam + apply
@pytest.mark.parametrize("m,n,ld,r,dtype,step", [
    (256, 256, 256, 32, torch.float32, 1), (512, 1376, 1376, 128, torch.bfloat16, 5),
    (100, 37, 40, 9, torch.bfloat16, 2), (4096, 4096, 4096, 1024, torch.bfloat16, 3),
])
def test_fused_adam_scatter_is_bit_identical_to_the_two_calls(m, n, ld, r, dtype, step):
    rng = np.random.default_rng(m + n + r)
    g = torch.Generator().manual_seed(r + n)
    Gc = (torch.randn((r, n), generator=g) * torch.exp(torch.randn((r, 1), generator=g))).to(DEV)
    M0 = (torch.randn((r, n), generator=g) * 0.1).to(DEV)
    V0 = (torch.rand((r, n), generator=g) * 0.01).to(DEV)
    sigma = np.sort(rng.choice(m, r, replace=True))
    idx = torch.tensor(sigma, dtype=torch.int32, device=DEV)
    rho = torch.tensor((0.5 + rng.random(r)).astype(np.float32), device=DEV)
    W0 = syn._padded(syn.make_W(m, n, dtype, seed0=r).to(DEV), ld)
    hp = (1e-3, 0.9, 0.999, 1e-8)
    M1, V1, U1, W1 = M0.clone(), V0.clone(), torch.empty_like(M0), W0.clone()
    grass.grass_subspace_adam(Gc, M1, V1, U1, *hp, step)
    grass.grass_scatter_update(W1, U1, idx, rho, 0.25)
    for keep in (True, False):
        M2, V2, W2 = M0.clone(), V0.clone(), W0.clone()
        U2 = torch.full_like(M0, float("nan")) if keep else None
        grass.grass_adam_scatter(Gc, M2, V2, U2, W2, idx, rho, *hp, step, 0.25)
        grass.grass_device_status()
        assert torch.equal(M2, M1) and torch.equal(V2, V1) and torch.equal(W2, W1)
        if keep:
            assert torch.equal(U2, U1)
    # and against the oracle, through the two-call path already checked element by element above
    Mo, Vo, Uo = oracle.adam_update(f64(M0), f64(V0), f64(Gc), *hp, step)
    assert rel_fro(f64(M1), Mo) <= 1e-6 and rel_fro(f64(U1), Uo) <= 1e-5


# --------------------------------------------------------------------------- bounded waits
def test_a_wait_that_nothing_completes_times_out_and_leaves_the_context_usable():
    grass.grass_device_status(raise_on_error=False)              # start from a clean status word
    grass.grass_selftest_bounded_wait(1_000_000)                 # ~0.5 ms at 1.9 GHz
    status, detail = grass.grass_device_status(raise_on_error=False)
    assert status == 7 and detail == 900                         # GRASS_ERR_TIMEOUT
    assert grass.grass_device_status(raise_on_error=False)[0] == 0   # reading clears it
    G = torch.ones((4, 16), device=DEV)
    norms = torch.empty(4, device=DEV)
    grass.grass_row_norms(G, norms)                              # the GPU still does work
    grass.grass_device_status()
    assert torch.allclose(norms, torch.full((4,), 4.0, device=DEV))


# --------------------------------------------------------------------------- batched layers
@pytest.mark.parametrize("count,T,m,n,r", [(4, 2048, 512, 512, 128), (2, 1500, 1376, 520, 100),
                                           (8, 512, 256, 256, 64), (3, 1024, 2048, 1024, 1024)])
def test_batched_projection_and_update_match_the_oracle_layer_by_layer(count, T, m, n, r):
    dt = torch.bfloat16
    rng = np.random.default_rng(count + T + r)
    dYs = [syn.make_dY(T, m, dt, seed0=5, proj=g) for g in range(count)]
    Xs = [syn.make_X(T, n, dt, seed0=5, proj=g) for g in range(count)]
    Ws = [syn.make_W(m, n, dt, seed0=5, proj=g) for g in range(count)]
    sig = [np.sort(rng.choice(m, r, replace=(g % 2 == 1))) for g in range(count)]
    rho = [(0.5 + rng.random(r)).astype(np.float32) for g in range(count)]
    dYd = [syn._padded(t.to(DEV), syn.pad_to(m, 8)) for t in dYs]
    Xd = [syn._padded(t.to(DEV), syn.pad_to(n, 8)) for t in Xs]
    Wd = [t.to(DEV).clone() for t in Ws]
    idx = [torch.tensor(s, dtype=torch.int32, device=DEV) for s in sig]
    rhod = [torch.tensor(x, device=DEV) for x in rho]
    Gc = [torch.full((r, n), float("nan"), dtype=torch.float32, device=DEV) for _ in range(count)]
    M = [torch.zeros((r, n), dtype=torch.float32, device=DEV) for _ in range(count)]
    V = [torch.zeros((r, n), dtype=torch.float32, device=DEV) for _ in range(count)]
    ws = ws_bytes(grass.grass_project_batched_workspace_bytes(count, T, m, n, r))
    grass.grass_project_grad_batched(dYd, Xd, idx, rhod, r, Gc, ws)
    grass.grass_adam_scatter_batched(Gc, M, V, None, Wd, idx, rhod, 1e-3, 0.9, 0.999, 1e-8, 1, 0.25)
    grass.grass_device_status()
    for g in range(count):
        want = oracle.project_grad(f64(dYs[g]), f64(Xs[g]), sig[g], rho[g])
        _assert_close_gc(f64(Gc[g]), want, 1e-4)
        # the update against the single-layer call on the same projected gradient: bit-identical
        M1 = torch.zeros_like(M[g]); V1 = torch.zeros_like(V[g]); W1 = Ws[g].to(DEV).clone()
        grass.grass_adam_scatter(Gc[g], M1, V1, None, W1, idx[g], rhod[g], 1e-3, 0.9, 0.999, 1e-8, 1, 0.25)
        assert torch.equal(M1, M[g]) and torch.equal(V1, V[g]) and torch.equal(W1, Wd[g])
        Mo, Vo, Uo = oracle.adam_update(np.zeros((r, n)), np.zeros((r, n)), want, 1e-3, 0.9, 0.999, 1e-8, 1)
        assert rel_fro(f64(M[g]), Mo) <= 1e-4


# --------------------------------------------------------------------------- resume
def test_resume_from_copied_state_is_bit_identical():
    """All state is caller-owned buffers plus (t, adam_step); selection is a pure function of
    (norms, seed, layer_id, epoch).  Six steps in one go equal three steps, a copy of the state
    into a fresh layer, and three more."""
    m, n, T, r, K = 512, 512, 1024, 128, 2
    dt, method = torch.bfloat16, grass.SEL_MULTINOMIAL_NORM
    W0 = syn.make_W(m, n, dt, seed0=31).to(DEV)
    batches = [(syn.make_dY(T, m, dt, seed0=31, step=t).to(DEV), syn.make_X(T, n, dt, seed0=31, step=t).to(DEV))
               for t in range(6)]

    def fresh(W):
        ws = grass.step.GrassWorkspace([(m, n)], T, r, dt, method)
        return grass.GrassLayer(W, r, method, K, 0.25, 1e-3, reset_state=False, seed=77, layer_id=3,
                                workspace=ws)

    a = fresh(W0.clone())
    for dY, X in batches:
        a.step(dY, X)
    b = fresh(W0.clone())
    for dY, X in batches[:3]:
        b.step(dY, X)
    c = fresh(b.W.clone())
    for name in ("M", "V", "idx", "rho"):
        getattr(c, name).copy_(getattr(b, name))
    c.t, c.adam_step = b.t, b.adam_step
    for dY, X in batches[3:]:
        c.step(dY, X)
    grass.grass_device_status()
    assert torch.equal(a.W, c.W) and torch.equal(a.M, c.M) and torch.equal(a.V, c.V)
    assert torch.equal(a.idx, c.idx)


# --------------------------------------------------------------------------- kernel variants
@pytest.mark.parametrize("mb", [1, 2, 4])
@pytest.mark.parametrize("pair", [grass.PAIR_NEVER, grass.PAIR_ALWAYS])
@pytest.mark.parametrize("gather", [grass.GATHER_PREPASS, grass.GATHER_IN_CTA, grass.GATHER_COOPERATIVE])
def test_every_tile_variant_of_the_projection_kernel(mb, pair, gather):
    """The host picks the tile shape from a cost model, so a given problem exercises one template
    instantiation.  Explicit options pin the n-blocks per CTA, single CTAs or CTA pairs, and the
    way the selected columns reach the GEMM (pre-pass, in-CTA gather, cooperative gather), so
    that every instantiation that can serve these shapes is run and checked against the oracle."""
    opts = dict(gather=gather, n_blocks_per_cta=mb, cta_pair=pair)
    seen = set()
    for T, m, n, r in [(1500, 512, 1024, 128), (900, 256, 520, 64), (1100, 640, 1024, 256),
                       (800, 1200, 1024, 448)]:
        plan = grass.grass_project_plan(1, T, m, n, r, opts)
        seen.add((plan["gather"], plan["n_blocks_per_cta"], plan["cta_pair"], plan["rows_per_tile"]))
        got, want = _project_case(T, m, n, r, torch.bfloat16, seed=T + r, dup=True, opts=opts)
        _assert_close_gc(got, want)
    assert len(seen) >= 3


@pytest.mark.parametrize("slices", [1, 2, 3, 7])
@pytest.mark.parametrize("T,m,n,r", [(2000, 512, 768, 192), (4100, 2048, 1024, 1024), (129, 300, 256, 40)])
def test_cooperative_gather_over_token_slices(T, m, n, r, slices):
    """Cooperative gather with the token sum cut into 1..7 slices (slices start on 128-token
    chunk borders; ragged last chunk; r not a multiple of the column group)."""
    opts = dict(gather=grass.GATHER_COOPERATIVE, token_slices=slices)
    got, want = _project_case(T, m, n, r, torch.bfloat16, seed=T + r + slices, opts=opts)
    _assert_close_gc(got, want)
    # fewer gather warps per CTA: same items, same bits
    opts["gather_warps"] = 1 + slices % 4
    again, _ = _project_case(T, m, n, r, torch.bfloat16, seed=T + r + slices, opts=opts)
    assert np.array_equal(again, got)


@pytest.mark.parametrize("seed", range(6))
def test_projection_on_random_small_shapes_all_gather_modes(seed):
    """Seeded random shapes (ragged T, m, n, r; repeated rows; with and without rho; 1..3 layers)
    through every gather mode and the plain call; every result against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    for _ in range(6):
        T = int(rng.integers(1, 700))
        m = int(rng.integers(1, 900))
        n = int(rng.integers(1, 600))
        r = int(rng.integers(1, m + 1))
        count = int(rng.integers(1, 4))
        ldx, lddy = syn.pad_to(n, 8), syn.pad_to(m, 8)
        Xs = [syn.make_X(T, n, torch.bfloat16, seed0=seed, proj=g) for g in range(count)]
        dYs = [syn.make_dY(T, m, torch.bfloat16, seed0=seed, proj=g) for g in range(count)]
        Xd = [syn._padded(t.to(DEV), ldx) for t in Xs]
        dYd = [syn._padded(t.to(DEV), lddy) for t in dYs]
        sig = [np.sort(rng.choice(m, r, replace=bool(rng.integers(0, 2)))) for _ in range(count)]
        rho = [(0.5 + rng.random(r)).astype(np.float32) for _ in range(count)]
        idx = [torch.tensor(x, dtype=torch.int32, device=DEV) for x in sig]
        rhod = [torch.tensor(x, device=DEV) for x in rho]
        want = [oracle.project_grad(f64(dYs[g]), f64(Xs[g]), sig[g], rho[g]) for g in range(count)]
        for gather in (grass.GATHER_AUTO, grass.GATHER_PREPASS, grass.GATHER_IN_CTA, grass.GATHER_COOPERATIVE):
            opts = dict(gather=gather, token_slices=int(rng.integers(0, 4)))
            ws = ws_bytes(grass.grass_project_plan(count, T, m, n, r, opts)["workspace_bytes"])
            ws.fill_(0x3C)
            Gc = [torch.full((r, n), float("nan"), dtype=torch.float32, device=DEV) for _ in range(count)]
            grass.grass_project_grad_ex(dYd, Xd, idx, rhod, r, Gc, ws, opts)
            grass.grass_device_status()
            for g in range(count):
                _assert_close_gc(f64(Gc[g]), want[g])


def test_cooperative_gather_is_bit_reproducible_and_matches_the_prepass():
    """Same tiling, same token slices: the cooperative gather and the pre-pass feed the GEMM the
    same operand bits, so the results are identical, run after run."""
    T, m, n, r = 3072, 2048, 1024, 512        # 24 chunks of 128 tokens: both cut it 16/16/16 blocks
    X = syn.make_X(T, n, torch.bfloat16, seed0=9).to(DEV)
    dY = syn.make_dY(T, m, torch.bfloat16, seed0=9).to(DEV)
    idx = torch.tensor(np.sort(np.random.default_rng(1).choice(m, r, replace=False)),
                       dtype=torch.int32, device=DEV)
    outs = []
    for gather in (grass.GATHER_COOPERATIVE, grass.GATHER_COOPERATIVE, grass.GATHER_PREPASS):
        opts = dict(gather=gather, token_slices=3)
        ws = ws_bytes(grass.grass_project_plan(1, T, m, n, r, opts)["workspace_bytes"])
        Gc = torch.empty((r, n), dtype=torch.float32, device=DEV)
        grass.grass_project_grad_ex([dY], [X], [idx], None, r, [Gc], ws, opts)
        grass.grass_device_status()
        outs.append(Gc)
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


def test_cooperative_gather_kernels_on_two_streams_at_once():
    """Two projections with the cooperative gather in flight on two streams: each kernel's gather
    warps serve only its own queue and never wait, so neither can starve the other, whichever
    CTAs happen to be resident.  Results equal the one-at-a-time results, bit for bit."""
    T, m, n, r = 8192, 2048, 2048, 512
    opts = dict(gather=grass.GATHER_COOPERATIVE)
    nbytes = grass.grass_project_plan(1, T, m, n, r, opts)["workspace_bytes"]
    jobs = []
    for k in range(2):
        X = syn.make_X(T, n, torch.bfloat16, seed0=40 + k).to(DEV)
        dY = syn.make_dY(T, m, torch.bfloat16, seed0=40 + k).to(DEV)
        idx = torch.tensor(np.sort(np.random.default_rng(k).choice(m, r, replace=False)),
                           dtype=torch.int32, device=DEV)
        jobs.append(dict(X=X, dY=dY, idx=idx, ws=ws_bytes(nbytes), stream=torch.cuda.Stream(),
                         Gc=torch.empty((r, n), dtype=torch.float32, device=DEV)))
    want = []
    for j in jobs:
        ref = torch.empty_like(j["Gc"])
        grass.grass_project_grad_ex([j["dY"]], [j["X"]], [j["idx"]], None, r, [ref], j["ws"], opts)
        want.append(ref)
    torch.cuda.synchronize()
    for _ in range(5):
        for j in jobs:
            j["stream"].wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(j["stream"]):
                grass.grass_project_grad_ex([j["dY"]], [j["X"]], [j["idx"]], None, r, [j["Gc"]], j["ws"], opts)
        torch.cuda.synchronize()
        grass.grass_device_status()
        for j, ref in zip(jobs, want):
            assert torch.equal(j["Gc"], ref)


def test_updates_with_repeated_rows_are_bit_reproducible():
    """Repeated rows are summed by one owner in a fixed order: two runs give the same bits."""
    m, n, r = 512, 1376, 256
    rng = np.random.default_rng(3)
    sigma = np.sort(rng.choice(40, r, replace=True))          # heavy repetition
    idx = torch.tensor(sigma, dtype=torch.int32, device=DEV)
    rho = torch.tensor((0.5 + rng.random(r)).astype(np.float32), device=DEV)
    g = torch.Generator().manual_seed(1)
    Gc = torch.randn((r, n), generator=g).to(DEV)
    W0 = syn.make_W(m, n, torch.bfloat16, seed0=2).to(DEV)
    outs = []
    for _ in range(2):
        W, M, V = W0.clone(), torch.zeros_like(Gc), torch.zeros_like(Gc)
        grass.grass_adam_scatter(Gc, M, V, None, W, idx, rho, 1e-3, 0.9, 0.999, 1e-8, 1, 0.25)
        W2 = W0.clone()
        U = torch.empty_like(Gc)
        grass.grass_subspace_adam(Gc, torch.zeros_like(Gc), torch.zeros_like(Gc), U, 1e-3, 0.9, 0.999, 1e-8, 1)
        grass.grass_scatter_update(W2, U, idx, rho, 0.25)
        grass.grass_device_status()
        outs.append((W, W2))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert torch.equal(outs[0][0], outs[0][1])
    want = oracle.scatter_update(f64(W0), oracle.adam_update(np.zeros((r, n)), np.zeros((r, n)), f64(Gc),
                                                            1e-3, 0.9, 0.999, 1e-8, 1)[2],
                                 sigma, rho.cpu().numpy(), 0.25, w_is_bf16=True)
    got = f64(outs[0][0])
    assert np.max(np.abs(got - want)) <= 2.0 ** -7 * np.max(np.abs(want))
    assert np.mean(got != want) < 0.01
