"""Host-only checks of the C ABI: the library builds, loads without a GPU, exports every
symbol include/grass.h declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2406_17660_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "grass.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(grass_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = _declared()
    assert "grass_project_grad" in names and len(names) >= 9
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(binding.exported_symbols())


def test_status_strings(lib):
    assert binding.grass_status_string(0) == "ok"
    seen = {binding.grass_status_string(i) for i in range(8)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert binding.grass_status_string(99) == "unknown status"


def test_argument_errors_are_returned_without_a_device(lib):
    null = ctypes.c_void_p(None)
    fake = ctypes.c_void_p(0x1000)          # never dereferenced: checks fail first
    assert lib.grass_row_norms(null, 0, 4, 4, 4, fake, null) == 1
    assert lib.grass_row_norms(fake, 0, 4, 4, 3, fake, null) == 1            # ld < n
    assert lib.grass_row_norms(fake, 7, 4, 4, 4, fake, null) == 3            # dtype
    assert lib.grass_select(fake, 10, 11, 0, 0, 0, 0, fake, fake, null, 0, null) == 1   # r > m
    assert lib.grass_select(fake, 10, 0, 0, 0, 0, 0, fake, fake, null, 0, null) == 1
    assert lib.grass_select(fake, 10, 5, 9, 0, 0, 0, fake, fake, null, 0, null) == 3    # method
    assert lib.grass_select(fake, 10, 5, 1, 0, 0, 0, fake, fake, null, 0, null) == 5    # no workspace
    assert lib.grass_project_grad(fake, 8, fake, 8, 1, 16, 8, 8, null, null, 4, fake, 8, null, 0,
                                  null) == 1                                 # idx NULL but r != m
    assert lib.grass_project_grad(fake, 8, fake, 8, 1, 16, 8, 8, fake, null, 9, fake, 8, null, 0,
                                  null) == 1                                 # r > m
    assert lib.grass_project_grad(fake, 8, fake, 4, 1, 16, 8, 8, fake, null, 4, fake, 8, null, 0,
                                  null) == 1                                 # ldx < n
    assert lib.grass_project_grad(fake, 8, fake, 12, 1, 16, 8, 8, fake, null, 4, fake, 8, null, 0,
                                  null) == 2                                 # bf16 pitch not 16-byte
    assert lib.grass_project_grad(fake, 1000, fake, 8, 1, 16, 1000, 8, fake, null, 4, fake, 8, null,
                                  0, null) == 5      # sparse pick: the gather pre-pass needs workspace
    assert lib.grass_subspace_adam(fake, 8, fake, fake, fake, 8, 4, 8, 1e-3, 0.9, 0.999, 1e-8, 0,
                                   null) == 1                                # step < 1
    assert lib.grass_subspace_adam(fake, 8, fake, fake, fake, 8, 4, 8, 1e-3, 1.0, 0.999, 1e-8, 1,
                                   null) == 1                                # beta1 = 1
    # empty problems are argument errors, not launches
    assert lib.grass_row_norms(fake, 0, 0, 4, 4, fake, null) == 1
    assert lib.grass_project_grad(fake, 8, fake, 8, 1, 0, 8, 8, fake, null, 4, fake, 8, null, 0,
                                  null) == 1                                 # T = 0
    assert lib.grass_project_grad(fake, 8, fake, 8, 1, 16, 8, 8, fake, null, 0, fake, 8, null, 0,
                                  null) == 1                                 # r = 0
    assert lib.grass_subspace_adam(fake, 8, fake, fake, fake, 8, 0, 8, 1e-3, 0.9, 0.999, 1e-8, 1,
                                   null) == 1                                # r = 0
    assert lib.grass_grad_row_norms(fake, 8, fake, 8, 1, 0, 8, 8, fake, null, 0, null) == 1
    assert lib.grass_selftest_bounded_wait(0, null) == 1
    assert lib.grass_scatter_update(fake, 1, 8, 8, 8, fake, 8, null, null, 4, 0.25, null) == 1
    assert lib.grass_scatter_update(fake, 5, 8, 8, 8, fake, 8, fake, null, 4, 0.25, null) == 3


def test_projection_options_and_limits_are_checked_on_the_host(lib):
    null = ctypes.c_void_p(None)
    fake = ctypes.c_void_p(0x1000)
    # more tokens than the 16-bit slice table can describe: rejected before anything is launched
    assert lib.grass_project_grad(fake, 1000, fake, 8, 1, 2 ** 31 - 1, 1000, 8, fake, null, 4, fake, 8,
                                  fake, 1 << 40, null) == 3
    # options out of range
    plan = binding.ProjectPlan()
    for bad in (dict(gather=4), dict(n_blocks_per_cta=3), dict(cta_pair=3), dict(token_slices=-1),
                dict(gather_warps=9)):
        opts = binding.ProjectOpts(**bad)
        assert lib.grass_project_plan(1, 1024, 512, 512, 128, ctypes.byref(opts), ctypes.byref(plan)) == 1
    # the plan query is host-only and honours explicit options
    p = binding.grass_project_plan(1, 4096, 2048, 1024, 512, dict(gather=binding.GATHER_PREPASS, token_slices=3))
    assert p["gather"] == binding.GATHER_PREPASS and p["token_slices"] == 3 and p["short_slices"] == 0
    assert p["rows_per_tile"] == 512 and p["workspace_bytes"] >= 4096 * 512 * 2 + 3 * 512 * 1024 * 4
    p = binding.grass_project_plan(1, 4096, 2048, 1024, 512, dict(gather=binding.GATHER_COOPERATIVE))
    assert p["gather"] == binding.GATHER_COOPERATIVE
    assert binding.grass_project_plan(1, 4096, 2048, 1024, 512)["gather"] == binding.GATHER_COOPERATIVE
    assert binding.grass_project_plan(4, 65536, 512, 512, 128)["gather"] == binding.GATHER_IN_CTA
    # in-CTA gather is only for tiles of at most 128 rows: the request falls back to the default
    assert binding.grass_project_plan(1, 4096, 2048, 1024, 512, dict(gather=binding.GATHER_IN_CTA))["gather"] \
        == binding.GATHER_COOPERATIVE


def test_workspace_queries_are_host_only_and_monotone(lib):
    assert binding.grass_select_workspace_bytes(4096, 256, binding.SEL_TOPR) >= 256
    a = binding.grass_select_workspace_bytes(4096, 256, binding.SEL_MULTINOMIAL_NORM)
    assert a >= 4096 * 12
    small = binding.grass_project_workspace_bytes(1024, 512, 512, 128, binding.BF16)
    big = binding.grass_project_workspace_bytes(32768, 4096, 4096, 1024, binding.BF16)
    assert 1024 * 128 * 2 <= small < big
    assert big >= 32768 * 1024 * 2
    assert binding.grass_project_workspace_bytes(1024, 512, 512, 128, binding.F32) >= 256


def test_plans_are_sane_over_a_sweep_of_shapes(lib):
    """The host plan (tile rows, n-blocks per CTA, pairs, long and short token slices, gather
    mode) for every benchmark shape and a grid of odd ones: structural invariants only."""
    shapes = [(c, T, m, n, r) for c in (1, 2, 4) for T in (31, 512, 4100, 32768, 65536)
              for m, n in ((512, 512), (1376, 512), (2048, 5461), (4096, 4096), (11008, 4096),
                           (4096, 11008), (13824, 5120), (300, 328))
              for r in (1, 64, 100, 256, 600, 1024) if r <= m]
    seen_modes = set()
    for c, T, m, n, r in shapes:
        p = binding.grass_project_plan(c, T, m, n, r)
        assert p["rows_per_tile"] % 64 == 0 and p["rows_per_tile"] * p["row_blocks"] >= r
        assert p["rows_per_tile"] * p["n_blocks_per_cta"] <= 512          # TMEM columns
        assert p["n_blocks_per_cta"] in (1, 2, 4) and p["cta_pair"] in (0, 1)
        assert not p["cta_pair"] or p["rows_per_tile"] % 128 == 0
        assert 1 <= p["token_slices"] <= 64 and 0 <= p["short_slices"] <= 3
        assert p["short_slices"] < p["token_slices"]
        assert 0 < p["long_slice_tokens"] <= T + 127
        assert p["gather"] in (binding.GATHER_PREPASS, binding.GATHER_IN_CTA, binding.GATHER_COOPERATIVE)
        if p["gather"] == binding.GATHER_IN_CTA:
            assert p["rows_per_tile"] <= 128
        if p["gather"] == binding.GATHER_COOPERATIVE:
            assert p["long_slice_tokens"] % 128 == 0 or p["token_slices"] == 1
        gathered = 0 if p["gather"] == binding.GATHER_IN_CTA else T * p["rows_per_tile"] * p["row_blocks"] * 2 * c
        partials = p["token_slices"] * r * n * 4 * c if p["token_slices"] > 1 else 0
        assert p["workspace_bytes"] >= gathered + partials
        slack = p["token_slices"] * r * 3 * 4 * c + 4 * c * (T // 128 + 1) + 1024 * c + 1024   # pitch, counters, alignment
        assert p["workspace_bytes"] <= gathered + partials + slack
        seen_modes.add(p["gather"])
    assert len(seen_modes) == 3
