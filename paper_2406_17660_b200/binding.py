"""ctypes binding of include/grass.h: same names, torch tensors in place of pointers.

Argument marshalling only.  Every function enqueues on torch's current CUDA
stream and raises GrassError on a non-zero status; nothing here computes.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_double, c_int, c_int32, c_int64, c_size_t, c_uint32, c_uint64, c_void_p

import torch

F32, BF16 = 0, 1
SEL_TOPR, SEL_MULTINOMIAL_NORM = 0, 1
SEL_MULTINOMIAL_NORM2, SEL_UNIFORM = 2, 3
SEL_MULTINOMIAL_NORM_NR, SEL_MULTINOMIAL_NORM2_NR, SEL_UNIFORM_NR = 4, 5, 6

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class GrassError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {grass_status_string(status)} (status {status})")


def library_path() -> str:
    return os.path.join(_HERE, "libgrass_b200.so")


_SIGNATURES = {
    "grass_row_norms": (c_int, [c_void_p, c_int, c_int64, c_int64, c_int64, c_void_p, c_void_p]),
    "grass_select_workspace_bytes": (c_size_t, [c_int64, c_int32, c_int]),
    "grass_select": (c_int, [c_void_p, c_int64, c_int32, c_int, c_uint64, c_uint32, c_uint32,
                             c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "grass_select_static": (c_int, [c_void_p, c_int64, c_int32, c_int, c_uint64, c_uint32, c_uint32,
                                    c_void_p, c_void_p, c_void_p]),
    "grass_project_workspace_bytes": (c_size_t, [c_int64, c_int64, c_int64, c_int32, c_int]),
    "grass_project_grad": (c_int, [c_void_p, c_int64, c_void_p, c_int64, c_int, c_int64, c_int64,
                                   c_int64, c_void_p, c_void_p, c_int32, c_void_p, c_int64,
                                   c_void_p, c_size_t, c_void_p]),
    "grass_grad_row_norms_workspace_bytes": (c_size_t, [c_int64, c_int64, c_int64, c_int]),
    "grass_grad_row_norms": (c_int, [c_void_p, c_int64, c_void_p, c_int64, c_int, c_int64, c_int64,
                                     c_int64, c_void_p, c_void_p, c_size_t, c_void_p]),
    "grass_subspace_adam": (c_int, [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_int64,
                                    c_int32, c_int64, c_double, c_double, c_double, c_double,
                                    c_int32, c_void_p]),
    "grass_scatter_update": (c_int, [c_void_p, c_int, c_int64, c_int64, c_int64, c_void_p, c_int64,
                                     c_void_p, c_void_p, c_int32, c_double, c_void_p]),
    "grass_adam_scatter": (c_int, [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_int64, c_void_p,
                                   c_int, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_int32,
                                   c_double, c_double, c_double, c_double, c_int32, c_double,
                                   c_void_p]),
    "grass_scatter_update_cols": (c_int, [c_void_p, c_int, c_int64, c_int64, c_int64, c_void_p,
                                          c_int64, c_void_p, c_void_p, c_int32, c_double, c_void_p]),
    "grass_device_status": (c_int, [c_void_p, ctypes.POINTER(c_int32)]),
    "grass_status_string": (ctypes.c_char_p, [c_int]),
    "grass_selftest_bounded_wait": (c_int, [c_int64, c_void_p]),
    "grass_profile_begin": (c_int, [c_int32]),
    "grass_profile_end": (c_int, [ctypes.POINTER(c_int32), ctypes.POINTER(ctypes.c_float),
                                  ctypes.POINTER(c_int32)]),
    "grass_profile_end_timeline": (c_int, [ctypes.POINTER(c_int32), ctypes.POINTER(ctypes.c_float),
                                           ctypes.POINTER(ctypes.c_float), ctypes.POINTER(c_int32)]),
}

KERNEL_NAMES = ["row_norms", "select", "gather", "project_tc", "splitk_reduce", "project_fp32",
                "adam", "scatter", "adam_scatter", "project_tc_dense"]


def load_library():
    """Load libgrass_b200.so (once).  There is no fallback: a missing library is an error."""
    global _LIB
    if _LIB is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2406_17660_b200.build` "
                "(needs nvcc); this package has no other execution path")
        lib = ctypes.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _LIB = lib
    return _LIB


def exported_symbols():
    return sorted(_SIGNATURES)


def grass_status_string(status: int) -> str:
    return load_library().grass_status_string(int(status)).decode()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _ld(t: torch.Tensor) -> int:
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("expected a 2-D tensor with unit inner stride")
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != 0:
        raise GrassError(status, where)


def _require(t, dtype, name):
    if t.dtype != dtype or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor of {dtype}")


def grass_row_norms(G: torch.Tensor, norms: torch.Tensor) -> None:
    m, n = G.shape
    _require(norms, torch.float32, "norms")
    _check(load_library().grass_row_norms(_ptr(G), _dtype_code(G), m, n, _ld(G), _ptr(norms),
                                          _stream()), "grass_row_norms")


def grass_select_workspace_bytes(m: int, r: int, method: int) -> int:
    return int(load_library().grass_select_workspace_bytes(m, r, method))


def grass_select(norms, r, method, seed, layer_id, epoch, idx, rho, ws) -> None:
    _require(norms, torch.float32, "norms")
    _require(idx, torch.int32, "idx")
    _require(rho, torch.float32, "rho")
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(load_library().grass_select(_ptr(norms), norms.numel(), r, method, seed, layer_id, epoch,
                                       _ptr(idx), _ptr(rho), _ptr(ws), ws_bytes, _stream()),
           "grass_select")


def grass_select_static(norms, r, method, seed, layer_id, epoch, idx, rho) -> None:
    """grass_select with the library's built-in scratch: no workspace argument, nothing is
    allocated.  For callers that have tensors but no way to get device memory at this point
    (see include/grass.h for the size limit and the sharing rules)."""
    _require(norms, torch.float32, "norms")
    _require(idx, torch.int32, "idx")
    _require(rho, torch.float32, "rho")
    _check(load_library().grass_select_static(_ptr(norms), norms.numel(), r, method, seed, layer_id,
                                              epoch, _ptr(idx), _ptr(rho), _stream()),
           "grass_select_static")


def grass_project_workspace_bytes(T: int, m: int, n: int, r: int, dt: int) -> int:
    return int(load_library().grass_project_workspace_bytes(T, m, n, r, dt))


def grass_project_grad(dY, X, idx, rho, r, Gc, ws) -> None:
    T, m = dY.shape
    T2, n = X.shape
    if T2 != T or dY.dtype != X.dtype:
        raise ValueError("dY and X must share the token dimension and dtype")
    _require(Gc, torch.float32, "Gc")
    if idx is not None:
        _require(idx, torch.int32, "idx")
    if rho is not None:
        _require(rho, torch.float32, "rho")
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(load_library().grass_project_grad(_ptr(dY), _ld(dY), _ptr(X), _ld(X), _dtype_code(X), T,
                                             m, n, _ptr(idx), _ptr(rho), r, _ptr(Gc), _ld(Gc),
                                             _ptr(ws), ws_bytes, _stream()), "grass_project_grad")


def grass_grad_row_norms_workspace_bytes(T: int, m: int, n: int, dt: int) -> int:
    return int(load_library().grass_grad_row_norms_workspace_bytes(T, m, n, dt))


def grass_grad_row_norms(dY, X, norms, ws) -> None:
    T, m = dY.shape
    T2, n = X.shape
    if T2 != T or dY.dtype != X.dtype:
        raise ValueError("dY and X must share the token dimension and dtype")
    _require(norms, torch.float32, "norms")
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(load_library().grass_grad_row_norms(_ptr(dY), _ld(dY), _ptr(X), _ld(X), _dtype_code(X),
                                               T, m, n, _ptr(norms), _ptr(ws), ws_bytes, _stream()),
           "grass_grad_row_norms")


def grass_subspace_adam(Gc, M, V, U, lr, beta1, beta2, eps, step) -> None:
    r, n = M.shape
    for t, name in ((Gc, "Gc"), (M, "M"), (V, "V"), (U, "U")):
        _require(t, torch.float32, name)
    if _ld(V) != _ld(M) or _ld(U) != _ld(M):
        raise ValueError("M, V and U must share one row pitch")
    _check(load_library().grass_subspace_adam(_ptr(Gc), _ld(Gc), _ptr(M), _ptr(V), _ptr(U), _ld(M),
                                              r, n, lr, beta1, beta2, eps, step, _stream()),
           "grass_subspace_adam")


def grass_scatter_update(W, U, idx, rho, alpha) -> None:
    m, n = W.shape
    r = idx.numel()
    _require(U, torch.float32, "U")
    _require(idx, torch.int32, "idx")
    if rho is not None:
        _require(rho, torch.float32, "rho")
    _check(load_library().grass_scatter_update(_ptr(W), _dtype_code(W), m, n, _ld(W), _ptr(U),
                                               _ld(U), _ptr(idx), _ptr(rho), r, alpha, _stream()),
           "grass_scatter_update")


def grass_adam_scatter(Gc, M, V, U, W, idx, rho, lr, beta1, beta2, eps, step, alpha) -> None:
    """Adam on the r x n state and the row-sparse apply in one kernel; U may be None."""
    r, n = M.shape
    m = W.shape[0]
    for t, name in ((Gc, "Gc"), (M, "M"), (V, "V")):
        _require(t, torch.float32, name)
    if U is not None:
        _require(U, torch.float32, "U")
        if _ld(U) != _ld(M):
            raise ValueError("M, V and U must share one row pitch")
    if _ld(V) != _ld(M):
        raise ValueError("M and V must share one row pitch")
    _require(idx, torch.int32, "idx")
    _check(load_library().grass_adam_scatter(_ptr(Gc), _ld(Gc), _ptr(M), _ptr(V), _ptr(U), _ld(M),
                                             _ptr(W), _dtype_code(W), m, n, _ld(W), _ptr(idx),
                                             _ptr(rho), r, lr, beta1, beta2, eps, step, alpha,
                                             _stream()), "grass_adam_scatter")


def grass_scatter_update_cols(W, U, idx, rho, alpha) -> None:
    m, n = W.shape
    r = idx.numel()
    _require(U, torch.float32, "U")
    _require(idx, torch.int32, "idx")
    if rho is not None:
        _require(rho, torch.float32, "rho")
    _check(load_library().grass_scatter_update_cols(_ptr(W), _dtype_code(W), m, n, _ld(W), _ptr(U),
                                                    _ld(U), _ptr(idx), _ptr(rho), r, alpha,
                                                    _stream()), "grass_scatter_update_cols")


def grass_device_status(raise_on_error: bool = True):
    """Synchronise the current stream and return (status, detail) of the device status word."""
    detail = c_int32(0)
    status = load_library().grass_device_status(_stream(), ctypes.byref(detail))
    if status != 0 and raise_on_error:
        raise GrassError(status, f"device status (detail {detail.value})")
    return status, detail.value


def grass_profile_end_timeline():
    """Returns (launches_seen, [(kernel_name, start_ms, ms), ...]); start_ms counts from the start
    of the first recorded launch, across streams."""
    cap = grass_profile_begin.cap
    kid = (c_int32 * cap)()
    ms = (ctypes.c_float * cap)()
    st = (ctypes.c_float * cap)()
    n = c_int32(0)
    _check(load_library().grass_profile_end_timeline(kid, ms, st, ctypes.byref(n)),
           "grass_profile_end_timeline")
    timed = min(n.value, cap)
    return n.value, [(KERNEL_NAMES[kid[i]], float(st[i]), float(ms[i])) for i in range(timed)]


def grass_selftest_bounded_wait(limit_cycles: int) -> None:
    _check(load_library().grass_selftest_bounded_wait(limit_cycles, _stream()),
           "grass_selftest_bounded_wait")


def grass_profile_begin(max_launches: int) -> None:
    _check(load_library().grass_profile_begin(max_launches), "grass_profile_begin")
    grass_profile_begin.cap = max_launches


def grass_profile_end():
    """Returns (launches_seen, [(kernel_name, ms), ...]) for the launches that were timed."""
    cap = grass_profile_begin.cap
    kid = (c_int32 * cap)()
    ms = (ctypes.c_float * cap)()
    n = c_int32(0)
    _check(load_library().grass_profile_end(kid, ms, ctypes.byref(n)), "grass_profile_end")
    timed = min(n.value, cap)
    return n.value, [(KERNEL_NAMES[kid[i]], float(ms[i])) for i in range(timed)]


# ---- batched calls: `count` layers of one shape per launch ----
_SIGNATURES_BATCHED = {
    "grass_project_batched_workspace_bytes": (c_size_t, [c_int32, c_int64, c_int64, c_int64, c_int32]),
    "grass_project_grad_batched": (c_int, [c_int32, c_void_p, c_int64, c_void_p, c_int64, c_int64,
                                           c_int64, c_int64, c_void_p, c_void_p, c_int32, c_void_p,
                                           c_int64, c_void_p, c_size_t, c_void_p]),
    "grass_adam_scatter_batched": (c_int, [c_int32, c_void_p, c_int64, c_void_p, c_void_p, c_void_p,
                                           c_int64, c_void_p, c_int, c_int64, c_int64, c_int64,
                                           c_void_p, c_void_p, c_int32, c_double, c_double, c_double,
                                           c_double, c_int32, c_double, c_void_p]),
}
_SIGNATURES.update(_SIGNATURES_BATCHED)

GATHER_AUTO, GATHER_PREPASS, GATHER_IN_CTA, GATHER_COOPERATIVE = 0, 1, 2, 3
PAIR_AUTO, PAIR_NEVER, PAIR_ALWAYS = 0, 1, 2


class ProjectOpts(ctypes.Structure):
    """grass_project_opts_t: 0 in a field keeps the library's own choice."""
    _fields_ = [("gather", c_int32), ("n_blocks_per_cta", c_int32), ("cta_pair", c_int32),
                ("token_slices", c_int32), ("gather_warps", c_int32)]


class ProjectPlan(ctypes.Structure):
    """grass_project_plan_t."""
    _fields_ = [("gather", c_int32), ("rows_per_tile", c_int32), ("row_blocks", c_int32),
                ("n_blocks_per_cta", c_int32), ("ctas_per_slice", c_int32), ("cta_pair", c_int32),
                ("token_slices", c_int32), ("short_slices", c_int32), ("long_slice_tokens", c_int32),
                ("tokens_per_stage", c_int32), ("stages", c_int32),
                ("workspace_bytes", c_size_t)]


_SIGNATURES.update({
    "grass_project_plan": (c_int, [c_int32, c_int64, c_int64, c_int64, c_int32,
                                   ctypes.POINTER(ProjectOpts), ctypes.POINTER(ProjectPlan)]),
    "grass_project_grad_ex": (c_int, [c_int32, c_void_p, c_int64, c_void_p, c_int64, c_int64, c_int64,
                                      c_int64, c_void_p, c_void_p, c_int32, c_void_p, c_int64,
                                      c_void_p, c_size_t, ctypes.POINTER(ProjectOpts), c_void_p]),
})


def _opts(opts):
    if opts is None:
        return None
    if isinstance(opts, ProjectOpts):
        return ctypes.byref(opts)
    return ctypes.byref(ProjectOpts(**opts))


def grass_project_plan(count: int, T: int, m: int, n: int, r: int, opts=None) -> dict:
    """What grass_project_grad_ex would do for these arguments (host only, no GPU needed)."""
    plan = ProjectPlan()
    _check(load_library().grass_project_plan(count, T, m, n, r, _opts(opts), ctypes.byref(plan)),
           "grass_project_plan")
    return {name: int(getattr(plan, name)) for name, _ in ProjectPlan._fields_}


def grass_project_grad_ex(dYs, Xs, idxs, rhos, r, Gcs, ws, opts=None) -> None:
    count = len(dYs)
    T, m = dYs[0].shape
    n = Xs[0].shape[1]
    for t in Gcs:
        _require(t, torch.float32, "Gc")
    for t in idxs:
        _require(t, torch.int32, "idx")
    keep = (_ptr_array(dYs), _ptr_array(Xs), _ptr_array(idxs), _ptr_array(rhos), _ptr_array(Gcs))
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(load_library().grass_project_grad_ex(
        count, keep[0], _ld(dYs[0]), keep[1], _ld(Xs[0]), T, m, n, keep[2], keep[3], r, keep[4],
        _ld(Gcs[0]), _ptr(ws), ws_bytes, _opts(opts), _stream()), "grass_project_grad_ex")


def _ptr_array(tensors):
    """Host array of device pointers (None entries become NULL); None -> NULL array."""
    if tensors is None:
        return None
    arr = (c_void_p * len(tensors))(*[None if t is None else t.data_ptr() for t in tensors])
    return arr


def grass_project_batched_workspace_bytes(count: int, T: int, m: int, n: int, r: int) -> int:
    return int(load_library().grass_project_batched_workspace_bytes(count, T, m, n, r))


def grass_project_grad_batched(dYs, Xs, idxs, rhos, r, Gcs, ws) -> None:
    count = len(dYs)
    T, m = dYs[0].shape
    n = Xs[0].shape[1]
    for t in Gcs:
        _require(t, torch.float32, "Gc")
    for t in idxs:
        _require(t, torch.int32, "idx")
    keep = (_ptr_array(dYs), _ptr_array(Xs), _ptr_array(idxs), _ptr_array(rhos), _ptr_array(Gcs))
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(load_library().grass_project_grad_batched(
        count, keep[0], _ld(dYs[0]), keep[1], _ld(Xs[0]), T, m, n, keep[2], keep[3], r, keep[4],
        _ld(Gcs[0]), _ptr(ws), ws_bytes, _stream()), "grass_project_grad_batched")


def grass_adam_scatter_batched(Gcs, Ms, Vs, Us, Ws, idxs, rhos, lr, beta1, beta2, eps, step,
                               alpha) -> None:
    count = len(Gcs)
    r, n = Ms[0].shape
    m = Ws[0].shape[0]
    keep = (_ptr_array(Gcs), _ptr_array(Ms), _ptr_array(Vs), _ptr_array(Us), _ptr_array(Ws),
            _ptr_array(idxs), _ptr_array(rhos))
    _check(load_library().grass_adam_scatter_batched(
        count, keep[0], _ld(Gcs[0]), keep[1], keep[2], keep[3], _ld(Ms[0]), keep[4],
        _dtype_code(Ws[0]), m, n, _ld(Ws[0]), keep[5], keep[6], r, lr, beta1, beta2, eps, step,
        alpha, _stream()), "grass_adam_scatter_batched")
