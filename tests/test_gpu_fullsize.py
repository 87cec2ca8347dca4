"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The fp64 oracle cannot form the whole r x n result at T = 32768..65536 in seconds, so whole output
rows are sampled: for a selected row j the oracle's G_C[j, :] = rho_j * X^T dY[:, sigma_j] is one
matrix-vector product, Adam and the apply step are row-local, and the row's new W follows.  The
tensor-core kernel's tiles, CTA pairs and split-K slices all contribute to every sampled row.
"""
import numpy as np
import pytest
import torch

import paper_2406_17660_b200 as grass
from paper_2406_17660_b200 import synthetic as syn
from oracle import grass_oracle as oracle

pytestmark = pytest.mark.gpu
DEV = "cuda"


def f64(t):
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


CASES = [
    # name, T, m, n, r, method (BASELINE config it belongs to)
    ("7b_q", 32768, 4096, 4096, 1024, grass.SEL_TOPR),                    # config 5
    ("7b_down", 32768, 4096, 11008, 1024, grass.SEL_TOPR),
    ("7b_q", 32768, 4096, 4096, 256, grass.SEL_TOPR),                     # config 5, r = 256
    ("13b_gate", 32768, 13824, 5120, 1024, grass.SEL_TOPR),               # largest row count, sparse pick
    ("13b_gate", 32768, 13824, 5120, 256, grass.SEL_TOPR),
    ("60m_gate", 65536, 1376, 512, 128, grass.SEL_MULTINOMIAL_NORM),      # config 2
    ("350m_down", 65536, 1024, 2736, 256, grass.SEL_TOPR),                # config 3 at full T
    ("1b_q", 65536, 2048, 2048, 512, grass.SEL_MULTINOMIAL_NORM),         # config 4: sampling with rho
    ("1b_down", 65536, 2048, 5461, 512, grass.SEL_MULTINOMIAL_NORM),      # padded pitch
    ("1b_q", 65536, 2048, 2048, 256, grass.SEL_MULTINOMIAL_NORM),         # config 4's r sweep
    ("1b_q", 65536, 2048, 2048, 128, grass.SEL_MULTINOMIAL_NORM),
    ("1b_q", 65536, 2048, 2048, 64, grass.SEL_MULTINOMIAL_NORM),
    ("1b_down", 65536, 2048, 5461, 512, grass.SEL_MULTINOMIAL_NORM_NR),   # the paper's 1B setting (-NR)
]


def _case_id(case):
    """Shape, r and the kernel variant the host plan picks for it (tile rows, n-blocks per CTA,
    pair or single CTA, token slices, how the selected columns are gathered)."""
    name, T, m, n, r, method = case
    try:
        p = grass.grass_project_plan(1, T, m, n, r)
        variant = (f"{['dense', 'prepass', 'incta', 'coop'][p['gather']]}-rows{p['rows_per_tile']}"
                   f"-mb{p['n_blocks_per_cta']}-{'pair' if p['cta_pair'] else 'single'}"
                   f"-s{p['token_slices']}")
    except Exception:
        variant = "unbuilt"
    return f"{name}-r{r}-sel{method}-{variant}"


@pytest.mark.parametrize("case", CASES, ids=[_case_id(c) for c in CASES])
def test_layer_step_on_sampled_rows(case):
    _, T, m, n, r, method = case
    dt = torch.bfloat16
    X = syn.make_X(T, n, dt, seed0=11)
    dY = syn.make_dY(T, m, dt, seed0=11)
    W = syn.make_W(m, n, dt, seed0=11)
    Xd = syn._padded(X.to(DEV), syn.pad_to(n, 8))            # 16-byte row pitch for the TMA path
    dYd = syn._padded(dY.to(DEV), syn.pad_to(m, 8))
    ws = grass.step.GrassWorkspace([(m, n)], T, r, dt, method)
    layer = grass.GrassLayer(W.to(DEV).clone(), r, method, K=200, alpha=0.25, lr=1e-3,
                             reset_state=True, seed=5, layer_id=2, workspace=ws)
    layer.step(dYd, Xd)
    grass.grass_device_status()

    idx = layer.idx.cpu().numpy()
    rho = layer.rho.cpu().numpy().astype(np.float64)
    norms = f64(ws.norms[:m])
    # the selection, from the GPU's own fp32 norms (same bits on both sides)
    sigma, rho_ref = oracle.select(norms.astype(np.float32), r, method, seed=5, layer_id=2, epoch=0)
    if method in (grass.SEL_MULTINOMIAL_NORM_NR, grass.SEL_MULTINOMIAL_NORM2_NR, grass.SEL_UNIFORM_NR) \
            and not np.array_equal(idx, sigma):
        # the kernel ranks fp32 scores: rows may differ only where fp64 scores at the threshold
        # agree to 1e-6 relative
        sc = oracle.nr_scores(norms.astype(np.float32), method, 5, 2, 0)
        thr = np.sort(sc)[-r]
        swapped = np.setxor1d(idx, sigma)
        assert np.all(np.abs(sc[swapped] - thr) <= 1e-6 * thr)
        assert np.all(rho == 1.0)                    # the rows below are checked for the GPU's pick
    else:
        assert np.array_equal(idx, sigma)
        np.testing.assert_allclose(rho, rho_ref, rtol=1e-6)
    # the norms themselves, on sampled rows of the dense gradient
    X64 = f64(X)
    rng = np.random.default_rng(T + n)
    for k in rng.choice(m, 4, replace=False):
        g_row = X64.T @ f64(dY[:, k])
        assert abs(norms[k] - np.linalg.norm(g_row)) <= 1e-4 * np.linalg.norm(g_row)
    # projected gradient, Adam and the apply step on sampled selected rows
    W64 = f64(W)
    Gc, M, V, U, Wn = (f64(t) for t in (layer.Gc, layer.M, layer.V, layer.U, layer.W))
    picks = rng.choice(r, 6, replace=False)
    for j in picks:
        g = rho[j] * (X64.T @ f64(dY[:, idx[j]]))
        err = np.linalg.norm(Gc[j] - g) / np.linalg.norm(g)
        assert err <= 1e-2 and err <= 1e-4, err
        assert np.max(np.abs(Gc[j] - g)) <= 1e-4 * np.max(np.abs(g))       # no bad tile in the row
        # Adam from the GPU's own G_C row (isolates the update kernel): 1e-5 element-wise
        M1, V1, U1 = oracle.adam_update(np.zeros(n), np.zeros(n), Gc[j], 1e-3, 0.9, 0.999, 1e-8, 1)
        np.testing.assert_allclose(M[j], M1, rtol=1e-5, atol=1e-30)
        np.testing.assert_allclose(V[j], V1, rtol=1e-5, atol=1e-30)
        np.testing.assert_allclose(U[j], U1, rtol=1e-5, atol=1e-12)
        # and end to end from the oracle's own row (secondary: carries the GEMM's rounding)
        M1, V1, U1 = oracle.adam_update(np.zeros(n), np.zeros(n), g, 1e-3, 0.9, 0.999, 1e-8, 1)
        assert np.linalg.norm(M[j] - M1) <= 1e-4 * np.linalg.norm(M1)
        assert np.linalg.norm(V[j] - V1) <= 2e-4 * np.linalg.norm(V1)
        assert np.linalg.norm(U[j] - U1) <= 1e-3 * np.linalg.norm(U1)
    for k in np.unique(idx[picks]):
        js = np.nonzero(idx == k)[0]                     # every repeat of this row
        upd = sum(0.25 * rho[j] * U[j] for j in js)      # the GPU's own U: isolates the apply step
        want = oracle.round_to_bf16(W64[k] + upd)
        ulp = np.ldexp(1.0, np.floor(np.log2(np.maximum(np.abs(want), 2.0 ** -126))).astype(int) - 7)
        assert np.all(np.abs(Wn[k] - want) <= ulp * 1.0001)
        assert np.mean(Wn[k] != want) < 0.01
    untouched = np.setdiff1d(np.arange(m), idx)
    assert torch.equal(layer.W[untouched].cpu(), W[untouched])


@pytest.mark.parametrize("T,m,n,r,count", [
    (32768, 4096, 4096, 1024, 4),      # 7B q,k,v,o
    (32768, 4096, 4096, 256, 4),
    (32768, 11008, 4096, 1024, 2),     # 7B gate, up
    (65536, 2048, 2048, 512, 4),       # 1B q,k,v,o
    (65536, 1024, 1024, 256, 4),       # 350M q,k,v,o
    (32768, 5120, 5120, 1024, 4),      # 13B q,k,v,o: three waves of tiles, long + short token slices
], ids=["7b_qkvo_r1024", "7b_qkvo_r256", "7b_gateup_r1024", "1b_qkvo_r512", "350m_qkvo_r256",
        "13b_qkvo_r1024"])
def test_batched_projection_on_sampled_rows(T, m, n, r, count):
    """Same-shaped projections of a block stepped as one group, as bench.py does: one set of
    launches over `count` layers (a different tiling plan from the single-layer call)."""
    dt = torch.bfloat16
    rng = np.random.default_rng(99)
    X = [syn.make_X(T, n, dt, seed0=21, proj=g) for g in range(count)]
    dY = [syn.make_dY(T, m, dt, seed0=21, proj=g) for g in range(count)]
    sig = [np.sort(rng.choice(m, r, replace=False)) for _ in range(count)]
    rho = [(0.5 + rng.random(r)).astype(np.float32) for _ in range(count)]
    Xd, dYd = [t.to(DEV) for t in X], [t.to(DEV) for t in dY]
    idx = [torch.tensor(s, dtype=torch.int32, device=DEV) for s in sig]
    rhod = [torch.tensor(x, device=DEV) for x in rho]
    Gc = [torch.full((r, n), float("nan"), dtype=torch.float32, device=DEV) for _ in range(count)]
    ws = torch.empty(grass.grass_project_batched_workspace_bytes(count, T, m, n, r),
                     dtype=torch.uint8, device=DEV)
    grass.grass_project_grad_batched(dYd, Xd, idx, rhod, r, Gc, ws)
    grass.grass_device_status()
    for g in range(count):
        X64 = f64(X[g])
        got = f64(Gc[g])
        assert np.all(np.isfinite(got))
        for j in rng.choice(r, 3, replace=False):
            want = rho[g][j] * (X64.T @ f64(dY[g][:, sig[g][j]]))
            err = np.linalg.norm(got[j] - want) / np.linalg.norm(want)
            assert err <= 1e-2 and err <= 1e-4, (g, j, err)
            assert np.max(np.abs(got[j] - want)) <= 1e-4 * np.max(np.abs(want))
