"""Run one library call a few times on a seeded synthetic layer: the small case that ncu captures.

    python -m paper_2406_17660_b200.profile_case --op project --T 8192 --m 4096 --n 4096 --r 1024

Ops: project (gather + tcgen05 GEMM + split-K reduce), dense (idx = NULL), gradnorms (dense GEMM
with the row-norm epilogue), adam, scatter, fused (Adam + apply), norms, select (multinomial-norm) / selecttop / selectnr.  Prints the per-kernel event timings of the last repetition so that the plain run leaves a
record next to the capture.
"""
from __future__ import annotations

import argparse
import json

import torch

import paper_2406_17660_b200 as grass
from paper_2406_17660_b200 import synthetic as syn


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="project")
    ap.add_argument("--T", type=int, default=8192)
    ap.add_argument("--m", type=int, default=4096)
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--r", type=int, default=1024)
    ap.add_argument("--reps", type=int, default=3)
    a = ap.parse_args()
    dev = "cuda:0"
    torch.cuda.set_device(0)
    dt = torch.bfloat16
    r = a.m if a.op == "dense" else a.r
    idx = torch.sort(torch.randperm(a.m, device=dev)[:r]).values.to(torch.int32)
    rho = torch.ones(r, device=dev)
    Gc = torch.empty((r, a.n), dtype=torch.float32, device=dev)
    if a.op in ("project", "dense", "gradnorms"):
        X = syn.make_X(a.T, a.n, dt, device=dev, ld=syn.pad_to(a.n, 8))
        dY = syn.make_dY(a.T, a.m, dt, device=dev, ld=syn.pad_to(a.m, 8))
        ws = torch.empty(grass.grass_project_workspace_bytes(a.T, a.m, a.n, r, grass.BF16),
                         dtype=torch.uint8, device=dev)
    if a.op == "gradnorms":
        nws = torch.empty(grass.grass_grad_row_norms_workspace_bytes(a.T, a.m, a.n, grass.BF16),
                          dtype=torch.uint8, device=dev)
    M = torch.zeros_like(Gc)
    V = torch.zeros_like(Gc)
    U = torch.empty_like(Gc)
    W = syn.make_W(a.m, a.n, dt, device=dev, ld=syn.pad_to(a.n, 8))
    G = torch.randn((a.m, a.n), device=dev) if a.op in ("norms", "select", "selecttop", "selectnr") else None
    norms = torch.empty(a.m, device=dev)
    sws = torch.empty(grass.grass_select_workspace_bytes(a.m, r, grass.SEL_MULTINOMIAL_NORM),
                      dtype=torch.uint8, device=dev)
    Gc.normal_()
    recs = []
    for rep in range(a.reps):
        grass.grass_profile_begin(16)
        if a.op == "project":
            grass.grass_project_grad(dY, X, idx, rho, r, Gc, ws)
        elif a.op == "dense":
            grass.grass_project_grad(dY, X, None, None, r, Gc, ws)
        elif a.op == "adam":
            grass.grass_subspace_adam(Gc, M, V, U, 1e-3, 0.9, 0.999, 1e-8, rep + 1)
        elif a.op == "fused":
            grass.grass_adam_scatter(Gc, M, V, None, W, idx, rho, 1e-3, 0.9, 0.999, 1e-8, rep + 1, 0.25)
        elif a.op == "gradnorms":
            grass.grass_grad_row_norms(dY, X, norms, nws)
        elif a.op == "scatter":
            grass.grass_scatter_update(W, Gc, idx, rho, 0.25)
        elif a.op == "norms":
            grass.grass_row_norms(G, norms)
        elif a.op in ("select", "selecttop", "selectnr"):
            method = {"select": grass.SEL_MULTINOMIAL_NORM, "selecttop": grass.SEL_TOPR,
                      "selectnr": grass.SEL_MULTINOMIAL_NORM_NR}[a.op]
            grass.grass_row_norms(G, norms)
            grass.grass_select(norms, r, method, 0, 0, rep, idx, rho, sws)
        else:
            raise SystemExit(f"unknown op {a.op}")
        _, recs = grass.grass_profile_end()
    grass.grass_device_status()
    print(json.dumps({"op": a.op, "T": a.T, "m": a.m, "n": a.n, "r": r,
                      "kernels_us": [(k, round(1e3 * ms, 2)) for k, ms in recs]}))


if __name__ == "__main__":
    main()
