"""Guard bands around every buffer the library writes.

compute-sanitizer is not available where these tests run, so out-of-bounds writes are looked for
directly: every output, in/out buffer and workspace of a call lives inside a larger allocation
whose bytes before and after it (and the padding between the logical row length and the row
pitch) hold a sentinel pattern.  After the call the sentinels must be untouched.  Shapes are the
awkward ones of the parity suite: n = 5461 with pitch 5464, r = 1, r = m, T not a multiple of the
token block, fewer tokens than one block.
"""
import numpy as np
import pytest
import torch

import paper_2406_17660_b200 as grass
from paper_2406_17660_b200 import synthetic as syn

pytestmark = pytest.mark.gpu
DEV = "cuda"
GUARD = 4096          # bytes on either side; keeps the 256-byte alignment of what lies between
SENTINEL = 0xA5


class Guarded:
    """rows x cols elements with row pitch ld inside a sentinel-filled allocation."""

    def __init__(self, rows, cols, dtype, ld=None, init=None):
        ld = ld or cols
        esize = torch.empty((), dtype=dtype).element_size()
        nbytes = rows * ld * esize
        pad = (-nbytes) % 256
        self.raw = torch.full((GUARD + nbytes + pad + GUARD,), SENTINEL, dtype=torch.uint8, device=DEV)
        self.body = self.raw[GUARD:GUARD + nbytes].view(dtype).view(rows, ld)
        self.t = self.body[:, :cols]
        self.cols, self.esize, self.nbytes = cols, esize, nbytes
        if init is not None:
            self.t.copy_(init)
        elif dtype.is_floating_point:
            self.t.fill_(float("nan"))

    def vec(self):
        return self.t[0]

    def check(self, what):
        assert bool((self.raw[:GUARD] == SENTINEL).all()), f"{what}: bytes before the buffer were written"
        assert bool((self.raw[GUARD + self.nbytes:] == SENTINEL).all()), \
            f"{what}: bytes after the buffer were written"
        if self.body.shape[1] > self.cols:
            padding = self.body[:, self.cols:].contiguous().view(torch.uint8)
            assert bool((padding == SENTINEL).all()), f"{what}: pitch padding was written"


def workspace(nbytes):
    g = Guarded(1, max(int(nbytes), 256), torch.uint8)
    g.t.fill_(0x5A)                                       # not a clean workspace either
    return g


def _idx(m, r, rng, dup=False):
    return torch.tensor(np.sort(rng.choice(m, r, replace=dup)), dtype=torch.int32, device=DEV)


@pytest.mark.parametrize("m,n,ld,dtype", [(37, 1001, 1001, torch.float32), (64, 5461, 5464, torch.bfloat16),
                                          (1, 1, 1, torch.float32)])
def test_row_norms_stays_inside_norms(m, n, ld, dtype):
    G = syn._padded(torch.randn((m, n), device=DEV).to(dtype), ld)
    norms = Guarded(1, m, torch.float32)
    grass.grass_row_norms(G, norms.vec())
    grass.grass_device_status()
    norms.check("norms")
    assert bool(torch.isfinite(norms.vec()).all())


@pytest.mark.parametrize("method", [grass.SEL_TOPR, grass.SEL_MULTINOMIAL_NORM, grass.SEL_UNIFORM_NR])
@pytest.mark.parametrize("m,r", [(300, 1), (300, 300), (13824, 1024), (16384, 77)])
def test_select_stays_inside_idx_rho_and_workspace(method, m, r):
    lam = torch.rand(m, device=DEV) + 0.1
    for static in (False, True):
        idx, rho = Guarded(1, r, torch.int32), Guarded(1, r, torch.float32)
        if static:
            grass.grass_select_static(lam, r, method, 3, 1, 2, idx.vec(), rho.vec())
        else:
            ws = workspace(grass.grass_select_workspace_bytes(m, r, method))
            grass.grass_select(lam, r, method, 3, 1, 2, idx.vec(), rho.vec(), ws.vec())
            ws.check("select workspace")
        grass.grass_device_status()
        idx.check("idx")
        rho.check("rho")
        got = idx.vec().cpu().numpy()
        assert got.min() >= 0 and got.max() < m


PROJECT_SHAPES = [
    # T, m, n, ldx, r
    (777, 2048, 5461, 5464, 512),      # padded pitch, ragged T, n not a tile multiple
    (64, 128, 128, 128, 1),            # r = 1
    (31, 64, 64, 64, 64),              # fewer tokens than one block, r = m
    (1000, 300, 328, 328, 100),        # ragged everything
    (300, 700, 640, 640, 600),         # two row blocks of 320
]


@pytest.mark.parametrize("gather", [grass.GATHER_AUTO, grass.GATHER_PREPASS, grass.GATHER_IN_CTA,
                                    grass.GATHER_COOPERATIVE])
@pytest.mark.parametrize("T,m,n,ldx,r", PROJECT_SHAPES)
def test_project_bf16_stays_inside_gc_and_workspace(T, m, n, ldx, r, gather):
    rng = np.random.default_rng(T + r)
    X = syn._padded(syn.make_X(T, n, torch.bfloat16, seed0=1).to(DEV), ldx)
    dY = syn._padded(syn.make_dY(T, m, torch.bfloat16, seed0=1).to(DEV), syn.pad_to(m, 8))
    idx = _idx(m, r, rng, dup=(r > 1 and r < m))
    rho = torch.rand(r, device=DEV) + 0.5
    ldgc = syn.pad_to(n, 4) + 4                           # Gc with a padded pitch of its own
    for count in (1, 2):
        opts = dict(gather=gather)
        plan = grass.grass_project_plan(count, T, m, n, r, opts)
        ws = workspace(plan["workspace_bytes"])
        Gc = [Guarded(r, n, torch.float32, ld=ldgc) for _ in range(count)]
        grass.grass_project_grad_ex([dY] * count, [X] * count, [idx] * count, [rho] * count, r,
                                    [g.t for g in Gc], ws.vec(), opts)
        grass.grass_device_status()
        ws.check(f"project workspace (count {count})")
        for g in Gc:
            g.check("Gc")
            assert bool(torch.isfinite(g.t).all())
        assert torch.equal(Gc[0].t, Gc[-1].t)
    # the plain entry point and the dense form (idx = NULL, r = m)
    ws = workspace(grass.grass_project_workspace_bytes(T, m, n, r, grass.BF16))
    Gc = Guarded(r, n, torch.float32)
    grass.grass_project_grad(dY, X, idx, rho, r, Gc.t, ws.vec())
    ws.check("project workspace")
    Gc.check("Gc")
    if m <= 700:
        ws = workspace(grass.grass_project_workspace_bytes(T, m, n, m, grass.BF16))
        G = Guarded(m, n, torch.float32)
        grass.grass_project_grad(dY, X, None, None, m, G.t, ws.vec())
        ws.check("dense workspace")
        G.check("dense G")
    grass.grass_device_status()


@pytest.mark.parametrize("T,m,n,ldx", [(777, 1376, 520, 520), (512, 2048, 5461, 5464), (256, 13824, 640, 640),
                                       (100, 50, 72, 72)])
def test_grad_row_norms_stays_inside_norms_and_workspace(T, m, n, ldx):
    X = syn._padded(syn.make_X(T, n, torch.bfloat16, seed0=2).to(DEV), ldx)
    dY = syn._padded(syn.make_dY(T, m, torch.bfloat16, seed0=2).to(DEV), syn.pad_to(m, 8))
    norms = Guarded(1, m, torch.float32)
    ws = workspace(grass.grass_grad_row_norms_workspace_bytes(T, m, n, grass.BF16))
    grass.grass_grad_row_norms(dY, X, norms.vec(), ws.vec())
    grass.grass_device_status()
    norms.check("norms")
    ws.check("row-norm workspace")
    assert bool(torch.isfinite(norms.vec()).all())


def test_fp32_projection_and_norms_stay_inside():
    T, m, n, r = 100, 50, 70, 7
    rng = np.random.default_rng(5)
    X, dY = torch.randn((T, n), device=DEV), torch.randn((T, m), device=DEV)
    idx = _idx(m, r, rng, dup=True)
    ws = workspace(grass.grass_project_workspace_bytes(T, m, n, r, grass.F32))
    Gc = Guarded(r, n, torch.float32, ld=n + 3)
    grass.grass_project_grad(dY, X, idx, None, r, Gc.t, ws.vec())
    ws.check("fp32 workspace")
    Gc.check("Gc")
    norms = Guarded(1, m, torch.float32)
    ws = workspace(grass.grass_grad_row_norms_workspace_bytes(T, m, n, grass.F32))
    grass.grass_grad_row_norms(dY, X, norms.vec(), ws.vec())
    grass.grass_device_status()
    ws.check("fp32 row-norm workspace")
    norms.check("norms")


@pytest.mark.parametrize("m,n,ld,r,wdtype", [
    (64, 5461, 5464, 16, torch.bfloat16), (100, 37, 40, 9, torch.bfloat16), (50, 30, 30, 50, torch.float32),
    (300, 1376, 1376, 1, torch.bfloat16), (4096, 4096, 4096, 256, torch.bfloat16),
])
def test_update_kernels_stay_inside_their_buffers(m, n, ld, r, wdtype):
    rng = np.random.default_rng(m + r)
    idx = _idx(m, r, rng, dup=(1 < r < m))
    rho = torch.rand(r, device=DEV) + 0.5
    g = torch.randn((r, n), device=DEV)
    W0 = syn.make_W(m, n, wdtype, seed0=3).to(DEV)
    lds = syn.pad_to(n, 4) + 4
    hp = (1e-3, 0.9, 0.999, 1e-8)

    def state():
        return (Guarded(r, n, torch.float32, ld=lds, init=torch.zeros((r, n), device=DEV)),
                Guarded(r, n, torch.float32, ld=lds, init=torch.zeros((r, n), device=DEV)),
                Guarded(r, n, torch.float32, ld=lds))

    # separate calls
    M, V, U = state()
    W = Guarded(m, n, wdtype, ld=ld, init=W0)
    grass.grass_subspace_adam(g, M.t, V.t, U.t, *hp, 1)
    grass.grass_scatter_update(W.t, U.t, idx, rho, 0.25)
    grass.grass_device_status()
    for buf, name in ((M, "M"), (V, "V"), (U, "U"), (W, "W")):
        buf.check(name)
    # fused call, with and without U, and the batched form
    for keep_u in (True, False):
        M2, V2, U2 = state()
        W2 = Guarded(m, n, wdtype, ld=ld, init=W0)
        grass.grass_adam_scatter(g, M2.t, V2.t, U2.t if keep_u else None, W2.t, idx, rho, *hp, 1, 0.25)
        grass.grass_device_status()
        for buf, name in ((M2, "M"), (V2, "V"), (U2, "U"), (W2, "W")):
            buf.check(f"fused {name}")
        assert torch.equal(W2.t, W.t) and torch.equal(M2.t, M.t)
    Ms, Vs, Ws = [], [], []
    for _ in range(3):
        a, b, _ = state()
        Ms.append(a)
        Vs.append(b)
        Ws.append(Guarded(m, n, wdtype, ld=ld, init=W0))
    grass.grass_adam_scatter_batched([g] * 3, [x.t for x in Ms], [x.t for x in Vs], None,
                                     [x.t for x in Ws], [idx] * 3, [rho] * 3, *hp, 1, 0.25)
    grass.grass_device_status()
    for group in (Ms, Vs, Ws):
        for buf in group:
            buf.check("batched update")
    assert torch.equal(Ws[2].t, W.t)
    # column form: W is n_out x n_in = m x n, U is r x m, idx picks columns
    if r <= n:
        cidx = _idx(n, r, rng, dup=(1 < r < n))
        Uc = torch.randn((r, m), device=DEV) * 1e-3
        Wc = Guarded(m, n, wdtype, ld=ld, init=W0)
        grass.grass_scatter_update_cols(Wc.t, Uc, cidx, rho, 0.25)
        grass.grass_device_status()
        Wc.check("W (column form)")
