"""grass_select_static: the selection call that takes no workspace and allocates nothing.

Some callers hold tensors but cannot get device memory when they need to select rows (the
framework's pool owns the device, or no allocator is reachable from where they run).  For them
the library keeps the scratch in a fixed array of its own.  This test drives that entry point
through the C ABI and checks that it returns exactly what grass_select returns with a
caller-provided workspace, twice in a row on different problems, so that contents left in the
shared array by the first call cannot leak into the second.  It sits in a file of its own that
sorts last, and passes whether it runs alone in a fresh process or after the other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2406_17660_b200 as grass

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
    # first call: the largest LLaMA row count, fills most of the built-in array
    big = np.exp(rng.standard_normal(13824)).astype(np.float32)
    # second call: a smaller problem whose rows overlap what the first call left behind
    small = np.exp(rng.standard_normal(512)).astype(np.float32)
    small[::9] = 0.0
    for lam, r, seed, layer_id, epoch in ((big, 1024, 7, 3, 0), (small, 128, 7, 3, 1)):
        (idx_ws, rho_ws), (idx_st, rho_st) = _both(lam, r, grass.SEL_MULTINOMIAL_NORM, seed,
                                                   layer_id, epoch)
        assert np.array_equal(idx_st, idx_ws)                       # indices: bit-exact
        np.testing.assert_allclose(rho_st, rho_ws, rtol=1e-6)      # rho: the suite's tolerance
        assert idx_st.min() >= 0 and np.all(np.diff(idx_st) >= 0)
    (idx_ws, _), (idx_st, rho_st) = _both(big, 256, grass.SEL_TOPR, 0, 0, 0)
    assert np.array_equal(idx_st, idx_ws) and np.all(rho_st == 1.0)


def test_static_scratch_rejects_more_rows_than_it_holds():
    lib = grass.load_library()
    fake = ctypes.c_void_p(0x1000)                                  # rejected before any use
    too_many = 16384 + 1
    assert lib.grass_select_static(fake, too_many, 8, grass.SEL_MULTINOMIAL_NORM, 0, 0, 0, fake,
                                   fake, None) == 5                 # GRASS_ERR_WORKSPACE
    assert lib.grass_select_static(fake, 100, 101, grass.SEL_TOPR, 0, 0, 0, fake, fake, None) == 1
