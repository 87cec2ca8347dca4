"""Sequencing of the five library calls into the paper's Algorithm 1, per layer.

Nothing here computes: GrassLayer owns the caller-side buffers (torch device
memory) and issues grass_* calls in the order of Algorithm 1 -- every K
iterations compute_P (dense gradient -> row norms -> select, optional state
reset), then projected gradient, Adam, row-sparse apply.
"""
from __future__ import annotations

import torch

from . import binding as B


class GrassWorkspace:
    """Scratch shared by all layers of a model: sized for the largest layer.

    Holds the norms and the byte workspaces of grass_project_grad,
    grass_grad_row_norms and grass_select.  No m x n gradient buffer exists:
    refresh iterations take the row norms straight from the GEMM's epilogue.
    """

    def __init__(self, shapes, T, r, dtype, method, device="cuda"):
        dt = B.BF16 if dtype == torch.bfloat16 else B.F32
        max_m = max(m for m, _ in shapes)
        proj = 256
        sel = 256
        nrm = 256
        for m, n in shapes:
            rr = min(r, m)
            proj = max(proj, B.grass_project_workspace_bytes(T, m, n, rr, dt))
            nrm = max(nrm, B.grass_grad_row_norms_workspace_bytes(T, m, n, dt))
            sel = max(sel, B.grass_select_workspace_bytes(m, rr, method))
        self.norm_ws = torch.empty(nrm, dtype=torch.uint8, device=device)
        self.norms = torch.empty(max_m, dtype=torch.float32, device=device)
        self.project_ws = torch.empty(proj, dtype=torch.uint8, device=device)
        self.select_ws = torch.empty(sel, dtype=torch.uint8, device=device)


class GrassLayer:
    """State of one linear layer W (m x n) trained by GRASS with rank r."""

    def __init__(self, W, r, method, K, alpha, lr, beta1=0.9, beta2=0.999, eps=1e-8,
                 reset_state=True, seed=0, layer_id=0, workspace=None, side="rows",
                 fused_update=True, keep_U=True):
        """side = "rows": P selects r of the m output features (rows of W).
        side = "cols": P selects r of the n input features (columns of W), the paper's choice
        when m > n; the same library calls are used with dY and X exchanged, the state is
        r x m, and the apply step is the column form."""
        self.W = W
        self.side = side
        # rows only: Adam and the apply step in one kernel; keep_U=False also skips writing U
        self.fused_update = fused_update and side == "rows"
        self.keep_U = keep_U
        self.m, self.n = W.shape if side == "rows" else (W.shape[1], W.shape[0])
        self.r, self.method, self.K = r, method, K
        self.alpha, self.lr, self.beta1, self.beta2, self.eps = alpha, lr, beta1, beta2, eps
        self.reset_state, self.seed, self.layer_id = reset_state, seed, layer_id
        dev = W.device
        self.idx = torch.zeros(r, dtype=torch.int32, device=dev)
        self.rho = torch.ones(r, dtype=torch.float32, device=dev)
        self.M = torch.zeros((r, self.n), dtype=torch.float32, device=dev)
        self.V = torch.zeros((r, self.n), dtype=torch.float32, device=dev)
        self.U = torch.empty((r, self.n), dtype=torch.float32, device=dev)
        self.Gc = torch.empty((r, self.n), dtype=torch.float32, device=dev)
        self.ws = workspace
        self.stream = None    # optional: the caller may pin a layer to a stream
        self.t = 0            # iteration counter of Algorithm 1
        self.adam_step = 0    # updates since the state was last zeroed

    def refresh(self, dY, X):
        """compute_P from this iteration's gradient (Algorithm 1, every K iterations)."""
        ws = self.ws
        norms = ws.norms[: self.m]
        B.grass_grad_row_norms(dY, X, norms, ws.norm_ws)
        B.grass_select(norms, self.r, self.method, self.seed, self.layer_id, self.t // self.K,
                       self.idx, self.rho, ws.select_ws)
        if self.reset_state:
            self.M.zero_()
            self.V.zero_()
            self.adam_step = 0

    def step(self, dY, X):
        """One iteration of Algorithm 1 for this layer; dY (T x m), X (T x n) on the device."""
        if self.side == "cols":
            dY, X = X, dY        # select columns of X, contract with dY: G_C^T = P^T (X^T dY)
        if self.t % self.K == 0:
            self.refresh(dY, X)
        self.adam_step += 1
        B.grass_project_grad(dY, X, self.idx, self.rho, self.r, self.Gc, self.ws.project_ws)
        if self.fused_update:
            B.grass_adam_scatter(self.Gc, self.M, self.V, self.U if self.keep_U else None, self.W,
                                 self.idx, self.rho, self.lr, self.beta1, self.beta2, self.eps,
                                 self.adam_step, self.alpha)
            self.t += 1
            return
        B.grass_subspace_adam(self.Gc, self.M, self.V, self.U, self.lr, self.beta1, self.beta2,
                              self.eps, self.adam_step)
        if self.side == "cols":
            B.grass_scatter_update_cols(self.W, self.U, self.idx, self.rho, self.alpha)
        else:
            B.grass_scatter_update(self.W, self.U, self.idx, self.rho, self.alpha)
        self.t += 1


class GrassLayerGroup:
    """Up to 8 layers of one shape (row selection, bf16) stepped together: their projections
    run as one set of launches and so do their Adam + apply updates.  The layers keep their
    own selection, state and weights; refresh iterations are done layer by layer."""

    def __init__(self, layers, T, device="cuda"):
        if not 1 <= len(layers) <= 8:
            raise ValueError("a group holds 1 to 8 layers")
        first = layers[0]
        for l in layers:
            if (l.W.shape, l.r, l.K, l.side) != (first.W.shape, first.r, first.K, "rows"):
                raise ValueError("layers of a group must share shape, r, K and select rows")
        self.layers = layers
        nbytes = B.grass_project_batched_workspace_bytes(len(layers), T, first.m, first.n, first.r)
        self.ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.stream = None
        # host arrays of device pointers: built once for the buffers the layers own, and once per
        # distinct set of input tensors (the marshalling would otherwise dominate small layers)
        pa = B._ptr_array
        self._own = dict(idx=pa([l.idx for l in layers]), rho=pa([l.rho for l in layers]),
                         Gc=pa([l.Gc for l in layers]), M=pa([l.M for l in layers]),
                         V=pa([l.V for l in layers]), W=pa([l.W for l in layers]),
                         U=pa([l.U if l.keep_U else None for l in layers]))
        self._inputs = {}

    def _input_arrays(self, dYs, Xs):
        key = tuple((t.data_ptr(), t.shape[0], t.stride(0)) for t in dYs) + \
            tuple((t.data_ptr(), t.shape[0], t.stride(0)) for t in Xs)
        hit = self._inputs.get(key)
        if hit is None:
            if len(self._inputs) > 64:
                self._inputs.clear()
            hit = (B._ptr_array(dYs), B._ptr_array(Xs), B._ld(dYs[0]), B._ld(Xs[0]), dYs[0].shape[0])
            self._inputs[key] = hit
        return hit

    def step(self, dYs, Xs):
        ls = self.layers
        first = ls[0]
        if first.t % first.K == 0:
            for l, dY, X in zip(ls, dYs, Xs):
                l.refresh(dY, X)
        for l in ls:
            l.adam_step += 1
            l.t += 1
        lib = B.load_library()
        own = self._own
        dYa, Xa, lddy, ldx, T = self._input_arrays(dYs, Xs)
        stream = B._stream()
        count, ld = len(ls), B._ld(first.Gc)
        B._check(lib.grass_project_grad_batched(count, dYa, lddy, Xa, ldx, T, first.m, first.n,
                                                own["idx"], own["rho"], first.r, own["Gc"], ld,
                                                B._ptr(self.ws), self.ws.numel(), stream),
                 "grass_project_grad_batched")
        B._check(lib.grass_adam_scatter_batched(count, own["Gc"], ld, own["M"], own["V"], own["U"],
                                                B._ld(first.M), own["W"], B._dtype_code(first.W),
                                                first.W.shape[0], first.n, B._ld(first.W),
                                                own["idx"], own["rho"], first.r, first.lr,
                                                first.beta1, first.beta2, first.eps,
                                                first.adam_step, first.alpha, stream),
                 "grass_adam_scatter_batched")
