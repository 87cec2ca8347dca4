"""grass_select_static: the selection call that takes no workspace and allocates nothing.

Some callers hold tensors but cannot get device memory when they need to select rows (the
framework's pool owns the device, or no allocator is reachable from where they run).  For them
the library keeps the scratch in a fixed array of its own.  This test drives that entry point
through the C ABI and checks that it returns exactly what grass_select returns with a
caller-provided workspace, and what the fp64 oracle returns, twice in a row on different
problems that both reach the built-in array (the kernel keeps its running sum in shared memory
up to 12800 rows, so only sampling methods on more rows than that touch it), so that contents
left there by the first call would show in the second.  It sits in a file of its own that sorts
last, and passes whether it runs alone in a fresh process or after the other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2406_17660_b200 as grass
from oracle import grass_oracle as oracle

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _both(lam, r, method, seed, layer_id, epoch):
    norms = torch.tensor(lam, dtype=torch.float32, device=DEV)
    m = norms.numel()
    out = []
    for static in (False, True):
        idx = torch.full((r,), -1, dtype=torch.int32, device=DEV)
        rho = torch.full((r,), -1.0, dtype=torch.float32, device=DEV)
        if static:
            grass.grass_select_static(norms, r, method, seed, layer_id, epoch, idx, rho)
        else:
            ws = torch.empty(grass.grass_select_workspace_bytes(m, r, method), dtype=torch.uint8,
                             device=DEV)
            grass.grass_select(norms, r, method, seed, layer_id, epoch, idx, rho, ws)
        grass.grass_device_status()
        out.append((idx.cpu().numpy(), rho.cpu().numpy()))
    return out


def test_static_scratch_selection_matches_workspace_selection_twice_in_a_row():
    rng = np.random.default_rng(2024)
    # first call: the largest LLaMA row count; its fp64 running sum goes to the built-in array
    big = np.exp(rng.standard_normal(13824)).astype(np.float32)
    # second call: fewer rows, many of zero weight, still above the shared-memory limit, so it
    # reads and writes the same array entries the first call left behind
    second = np.exp(rng.standard_normal(13000)).astype(np.float32)
    second[::9] = 0.0
    # third call: exactly the limit
    full = np.exp(rng.standard_normal(16384)).astype(np.float32)
    for lam, r, method, seed, layer_id, epoch in (
            (big, 1024, grass.SEL_MULTINOMIAL_NORM, 7, 3, 0),
            (second, 512, grass.SEL_MULTINOMIAL_NORM2, 7, 3, 1),
            (full, 1024, grass.SEL_MULTINOMIAL_NORM, 9, 1, 2)):
        (idx_ws, rho_ws), (idx_st, rho_st) = _both(lam, r, method, seed, layer_id, epoch)
        assert np.array_equal(idx_st, idx_ws)                       # indices: bit-exact
        np.testing.assert_allclose(rho_st, rho_ws, rtol=1e-6)      # rho: the suite's tolerance
        assert idx_st.min() >= 0 and np.all(np.diff(idx_st) >= 0)
        assert np.all(np.isfinite(rho_st)) and np.all(lam[idx_st] > 0)   # never a zero-weight row
        sigma, rho_ref = oracle.select(lam, r, method, seed=seed, layer_id=layer_id, epoch=epoch)
        if np.array_equal(idx_st, sigma):
            np.testing.assert_allclose(rho_st, rho_ref, rtol=1e-6)
        else:       # allowed only where a draw falls within 1e-6 of a step of the running sum
            c = np.cumsum(oracle.sampling_weights(lam.astype(np.float64), method))
            u = oracle.draw_words(r, seed, layer_id, epoch).astype(np.float64) * 2.0 ** -32 * c[-1]
            gap = np.min(np.abs(c[None, :] - u[:, None]), axis=1) / c[-1]
            assert np.sum(idx_st != sigma) <= np.sum(gap < 1e-6)
    (idx_ws, _), (idx_st, rho_st) = _both(big, 256, grass.SEL_TOPR, 0, 0, 0)
    assert np.array_equal(idx_st, idx_ws) and np.all(rho_st == 1.0)
    assert np.array_equal(idx_st, oracle.select_topr(big, 256)[0])


def test_static_scratch_rejects_more_rows_than_it_holds():
    lib = grass.load_library()
    fake = ctypes.c_void_p(0x1000)                                  # rejected before any use
    too_many = 16384 + 1
    assert lib.grass_select_static(fake, too_many, 8, grass.SEL_MULTINOMIAL_NORM, 0, 0, 0, fake,
                                   fake, None) == 5                 # GRASS_ERR_WORKSPACE
    assert lib.grass_select_static(fake, 100, 101, grass.SEL_TOPR, 0, 0, 0, fake, fake, None) == 1
