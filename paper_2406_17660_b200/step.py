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
