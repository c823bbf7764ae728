"""Thin ctypes binding of the C ABI in include/meteora.h.

Argument marshalling only: every function takes torch tensors that already live on the
GPU (or pinned host tensors where stated), checks dtype / shape / contiguity, and passes raw
pointers, sizes and the current CUDA stream to the library.  No step of the layer is computed
here, and nothing falls back to PyTorch: if `libmeteora.so` has not been built the first call
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmeteora.so")

METEORA_F32, METEORA_BF16 = 0, 1
STATUS = {0: "METEORA_OK", -1: "METEORA_ERR_INVALID_ARG", -2: "METEORA_ERR_UNSUPPORTED_SHAPE",
          -3: "METEORA_ERR_MISALIGNED", -4: "METEORA_ERR_WORKSPACE_TOO_SMALL", -5: "METEORA_ERR_CUDA",
          -6: "METEORA_ERR_TIMEOUT"}

EXPORTS = ["meteora_gate_topk", "meteora_route", "meteora_lora_delta", "meteora_lora_delta_static",
           "meteora_linear_forward", "meteora_linear_forward_group", "meteora_group_workspace_bytes",
           "meteora_group_workspace_routing", "meteora_group_plan", "meteora_gate_backward",
           "meteora_gate_backward_workspace_bytes", "meteora_gate_backward_bt", "meteora_transpose_adapters_b",
           "meteora_adapters_bt_bytes", "meteora_pad_adapters", "meteora_pad_adapters_bytes",
           "meteora_linear_forward_host", "meteora_workspace_bytes", "meteora_workspace_routing",
           "meteora_workspace_init", "meteora_workspace_status", "meteora_profile_begin", "meteora_profile_end",
           "meteora_describe_plan", "meteora_set_tuning", "meteora_status_string"]


class MeteoraShape(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int), ("d_in", ctypes.c_int), ("d_out", ctypes.c_int), ("N", ctypes.c_int),
                ("r", ctypes.c_int), ("k", ctypes.c_int), ("dtype", ctypes.c_int), ("temperature", ctypes.c_float)]


class MeteoraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS.get(status, status)} ({status})")


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen libmeteora.so (built in-tree by `build.build_library`) and declare its prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2405_13053_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    shp = ctypes.POINTER(MeteoraShape)
    lib.meteora_gate_topk.argtypes = [vp, vp, shp, vp, vp, vp, vp]
    lib.meteora_route.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp]
    lib.meteora_lora_delta.argtypes = [vp, vp, vp, vp, vp, vp, vp, shp, vp, vp, sz, vp]
    lib.meteora_lora_delta_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, shp, vp, vp]
    lib.meteora_linear_forward.argtypes = [vp, vp, vp, vp, vp, shp, vp, vp, sz, vp]
    lib.meteora_linear_forward_host.argtypes = [vp, vp, vp, vp, vp, shp, vp, vp, sz, vp]
    ip = ctypes.POINTER(ci)
    lib.meteora_linear_forward_group.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp),
                                                 ctypes.POINTER(vp), ip, ci, shp, ctypes.POINTER(vp), vp, sz, vp]
    lib.meteora_gate_backward.argtypes = [vp, vp, vp, vp, vp, vp, shp, vp, vp, vp, sz, vp]
    lib.meteora_gate_backward_bt.argtypes = [vp, vp, vp, vp, vp, vp, shp, vp, vp, vp, sz, vp]
    lib.meteora_transpose_adapters_b.argtypes = [vp, shp, vp, vp]
    lib.meteora_pad_adapters_bytes.argtypes = [shp, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.meteora_pad_adapters.argtypes = [vp, vp, shp, vp, vp, vp]
    lib.meteora_adapters_bt_bytes.argtypes = [shp]
    lib.meteora_adapters_bt_bytes.restype = sz
    lib.meteora_gate_backward_workspace_bytes.argtypes = [shp]
    lib.meteora_gate_backward_workspace_bytes.restype = sz
    lib.meteora_group_plan.argtypes = [shp, ip, ci]
    lib.meteora_group_workspace_bytes.argtypes = [shp, ip, ci]
    lib.meteora_group_workspace_bytes.restype = sz
    lib.meteora_group_workspace_routing.argtypes = [shp, ip, ci, ci, vp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.meteora_workspace_bytes.argtypes = [shp]
    lib.meteora_workspace_bytes.restype = sz
    lib.meteora_workspace_routing.argtypes = [shp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.meteora_workspace_init.argtypes = [vp, vp]
    lib.meteora_workspace_status.argtypes = [vp, vp]
    lib.meteora_profile_begin.argtypes = [ci]
    lib.meteora_profile_end.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ci)]
    lib.meteora_describe_plan.argtypes = [shp, ctypes.c_char_p, sz]
    lib.meteora_set_tuning.argtypes = [ctypes.c_char_p, ci]
    lib.meteora_status_string.argtypes = [ci]
    lib.meteora_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("meteora_workspace_bytes", "meteora_group_workspace_bytes",
                        "meteora_gate_backward_workspace_bytes", "meteora_gate_backward_bt", "meteora_transpose_adapters_b",
           "meteora_adapters_bt_bytes", "meteora_pad_adapters", "meteora_pad_adapters_bytes", "meteora_status_string"):
            getattr(lib, name).restype = ci
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != 0:
        raise MeteoraError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return METEORA_F32
    if t.dtype == torch.bfloat16:
        return METEORA_BF16
    raise TypeError(f"unsupported dtype {t.dtype}; the layer runs in float32 or bfloat16")


def _dev(t: torch.Tensor, shape, dtype, name: str) -> int:
    if not (t.is_cuda and t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    if tuple(t.shape) != tuple(shape) or t.dtype != dtype:
        raise ValueError(f"{name}: expected {tuple(shape)} {dtype}, got {tuple(t.shape)} {t.dtype}")
    return t.data_ptr()


def make_shape(T, d_in, d_out, N, r, k, dtype: torch.dtype, temperature: float = 1.0) -> MeteoraShape:
    code = METEORA_F32 if dtype == torch.float32 else METEORA_BF16
    return MeteoraShape(int(T), int(d_in), int(d_out), int(N), int(r), int(k), code, float(temperature))


def meteora_workspace_bytes(shape: MeteoraShape) -> int:
    return int(load_library().meteora_workspace_bytes(ctypes.byref(shape)))


def alloc_workspace(shape: MeteoraShape, device="cuda") -> torch.Tensor:
    """A zeroed byte tensor large enough for any call with this shape."""
    n = meteora_workspace_bytes(shape)
    if n == 0:
        raise MeteoraError(-1, "meteora_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def meteora_gate_topk(x: torch.Tensor, Wg: torch.Tensor, k: int, temperature: float = 1.0,
                      want_logits: bool = False) -> Tuple[torch.Tensor, torch.Tensor, Optional[torch.Tensor]]:
    lib = load_library()
    T, d_in = x.shape
    N = Wg.shape[0]
    shape = make_shape(T, d_in, 1, N, 1, k, x.dtype, temperature)
    _dtype_code(x)
    px, pg = _dev(x, (T, d_in), x.dtype, "x"), _dev(Wg, (N, d_in), x.dtype, "Wg")
    idx = torch.empty((T, k), dtype=torch.int32, device=x.device)
    w = torch.empty((T, k), dtype=torch.float32, device=x.device)
    logits = torch.empty((T, N), dtype=torch.float32, device=x.device) if want_logits else None
    _check(lib.meteora_gate_topk(px, pg, ctypes.byref(shape), idx.data_ptr(), w.data_ptr(),
                                 logits.data_ptr() if want_logits else None, _stream()), "meteora_gate_topk")
    return idx, w, logits


def meteora_route(topk_idx: torch.Tensor, N: int) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    lib = load_library()
    T, k = topk_idx.shape
    p = _dev(topk_idx, (T, k), torch.int32, "topk_idx")
    counts = torch.empty(N, dtype=torch.int32, device=topk_idx.device)
    offsets = torch.empty(N + 1, dtype=torch.int32, device=topk_idx.device)
    perm = torch.empty(T * k, dtype=torch.int32, device=topk_idx.device)
    _check(lib.meteora_route(p, T, k, N, counts.data_ptr(), offsets.data_ptr(), perm.data_ptr(), _stream()),
           "meteora_route")
    return counts, offsets, perm


def meteora_lora_delta(x, A, B, topk_idx, topk_w, offsets, perm, workspace: Optional[torch.Tensor] = None
                       ) -> torch.Tensor:
    lib = load_library()
    T, d_in = x.shape
    N, r, _ = A.shape
    d_out = B.shape[1]
    k = topk_idx.shape[1]
    shape = make_shape(T, d_in, d_out, N, r, k, x.dtype)
    _dtype_code(x)
    if workspace is None:
        workspace = alloc_workspace(shape, x.device)
    delta = torch.empty((T, d_out), dtype=torch.float32, device=x.device)
    _check(lib.meteora_lora_delta(_dev(x, (T, d_in), x.dtype, "x"), _dev(A, (N, r, d_in), x.dtype, "A"),
                                  _dev(B, (N, d_out, r), x.dtype, "B"),
                                  _dev(topk_idx, (T, k), torch.int32, "topk_idx"),
                                  _dev(topk_w, (T, k), torch.float32, "topk_w"),
                                  _dev(offsets, (N + 1,), torch.int32, "offsets"),
                                  _dev(perm, (T * k,), torch.int32, "perm"), ctypes.byref(shape),
                                  delta.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream()),
           "meteora_lora_delta")
    return delta


STATIC_SCRATCH_FLOATS = 65536


def meteora_lora_delta_static(x, A, B, topk_idx, topk_w, offsets, perm, out: Optional[torch.Tensor] = None
                              ) -> torch.Tensor:
    """meteora_lora_delta for callers that cannot allocate: the library's built-in 256 KB device array replaces
    the workspace, so T*k*r must not exceed STATIC_SCRATCH_FLOATS (MeteoraError -2 otherwise).  Pass `out`
    (fp32 [T,d_out]) to keep this wrapper from allocating the result as well.  Calls on one device share
    the array: keep them ordered on the GPU.  Make the first call on a device outside stream capture."""
    lib = load_library()
    T, d_in = x.shape
    N, r, _ = A.shape
    d_out = B.shape[1]
    k = topk_idx.shape[1]
    shape = make_shape(T, d_in, d_out, N, r, k, x.dtype)
    _dtype_code(x)
    delta = out if out is not None else torch.empty((T, d_out), dtype=torch.float32, device=x.device)
    _check(lib.meteora_lora_delta_static(_dev(x, (T, d_in), x.dtype, "x"), _dev(A, (N, r, d_in), x.dtype, "A"),
                                         _dev(B, (N, d_out, r), x.dtype, "B"),
                                         _dev(topk_idx, (T, k), torch.int32, "topk_idx"),
                                         _dev(topk_w, (T, k), torch.float32, "topk_w"),
                                         _dev(offsets, (N + 1,), torch.int32, "offsets"),
                                         _dev(perm, (T * k,), torch.int32, "perm"), ctypes.byref(shape),
                                         _dev(delta, (T, d_out), torch.float32, "delta"), _stream()),
           "meteora_lora_delta_static")
    return delta


def meteora_linear_forward(x, W0, A, B, Wg, k: int, temperature: float = 1.0,
                           workspace: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                           return_routing: bool = False):
    """y = W0 x + sum_{i in topk(x)} w_i B_i A_i x.  Returns y, or (y, topk_idx, topk_w) views of the workspace."""
    lib = load_library()
    T, d_in = x.shape
    d_out = W0.shape[0]
    N, r, _ = A.shape
    shape = make_shape(T, d_in, d_out, N, r, k, x.dtype, temperature)
    _dtype_code(x)
    if workspace is None:
        workspace = alloc_workspace(shape, x.device)
    y = out if out is not None else torch.empty((T, d_out), dtype=x.dtype, device=x.device)
    _check(lib.meteora_linear_forward(_dev(x, (T, d_in), x.dtype, "x"), _dev(W0, (d_out, d_in), x.dtype, "W0"),
                                      _dev(A, (N, r, d_in), x.dtype, "A"), _dev(B, (N, d_out, r), x.dtype, "B"),
                                      _dev(Wg, (N, d_in), x.dtype, "Wg"), ctypes.byref(shape),
                                      _dev(y, (T, d_out), x.dtype, "y"), workspace.data_ptr(), workspace.numel(),
                                      _stream()), "meteora_linear_forward")
    if not return_routing:
        return y
    idx, w = meteora_workspace_routing(shape, workspace)
    return y, idx, w


def meteora_pad_adapters(A, B):
    """(A_pad[N,r8,d_in], B_pad[N,d_out,r8]) with the rank zero-padded to the next multiple of 8, made once for a bf16
    layer whose rank is none: a forward on the padded arrays gives the same bits without padding on every call.
    Returns (A, B) themselves where the library would not pad."""
    lib = load_library()
    N, r, d_in = A.shape
    d_out = B.shape[1]
    shape = make_shape(0, d_in, d_out, N, r, 1, A.dtype)
    a_bytes, b_bytes = ctypes.c_size_t(0), ctypes.c_size_t(0)
    r8 = lib.meteora_pad_adapters_bytes(ctypes.byref(shape), ctypes.byref(a_bytes), ctypes.byref(b_bytes))
    if r8 == 0:
        return A, B
    A_pad = torch.empty((N, r8, d_in), dtype=A.dtype, device=A.device)
    B_pad = torch.empty((N, d_out, r8), dtype=A.dtype, device=A.device)
    assert A_pad.numel() * 2 == a_bytes.value and B_pad.numel() * 2 == b_bytes.value
    _check(lib.meteora_pad_adapters(_dev(A, (N, r, d_in), A.dtype, "A"), _dev(B, (N, d_out, r), A.dtype, "B"),
                                    ctypes.byref(shape), A_pad.data_ptr(), B_pad.data_ptr(), _stream()),
           "meteora_pad_adapters")
    return A_pad, B_pad


def meteora_transpose_adapters_b(B):
    """Bt[N,r,d_out] with Bt[n,p,o] = B[n,o,p]: made once per module for meteora_gate_backward(..., Bt=...)."""
    lib = load_library()
    N, d_out, r = B.shape
    shape = make_shape(0, 1, d_out, N, r, 1, B.dtype)
    Bt = torch.empty((N, r, d_out), dtype=B.dtype, device=B.device)
    _check(lib.meteora_transpose_adapters_b(_dev(B, (N, d_out, r), B.dtype, "B"), ctypes.byref(shape), Bt.data_ptr(),
                                            _stream()), "meteora_transpose_adapters_b")
    return Bt


def meteora_gate_backward(x, A, B, dy, topk_idx, topk_w, temperature: float = 1.0, Bt=None, workspace=None):
    """dWg[N,d_in] (fp32) and dlogit[T,k] (fp32): gradient of the gate through Eq. 3 and Eq. 2 for the routing given.
    With Bt (meteora_transpose_adapters_b(B)) the call skips its own transposition of B."""
    lib = load_library()
    T, d_in = x.shape
    N, r, _ = A.shape
    d_out = B.shape[1] if Bt is None else Bt.shape[2]
    k = topk_idx.shape[1]
    shape = make_shape(T, d_in, d_out, N, r, k, x.dtype, temperature)
    n = lib.meteora_gate_backward_workspace_bytes(ctypes.byref(shape))
    if n == 0:
        raise MeteoraError(-1, "meteora_gate_backward_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=x.device) if workspace is None else workspace
    dWg = torch.empty((N, d_in), dtype=torch.float32, device=x.device)
    dlogit = torch.empty((T, k), dtype=torch.float32, device=x.device)
    fn = lib.meteora_gate_backward if Bt is None else lib.meteora_gate_backward_bt
    b_arg = _dev(B, (N, d_out, r), x.dtype, "B") if Bt is None else _dev(Bt, (N, r, d_out), x.dtype, "Bt")
    _check(fn(_dev(x, (T, d_in), x.dtype, "x"), _dev(A, (N, r, d_in), x.dtype, "A"), b_arg,
              _dev(dy, (T, d_out), x.dtype, "dy"), _dev(topk_idx, (T, k), torch.int32, "topk_idx"),
              _dev(topk_w, (T, k), torch.float32, "topk_w"), ctypes.byref(shape), dlogit.data_ptr(), dWg.data_ptr(),
              ws.data_ptr(), ws.numel(), _stream()), "meteora_gate_backward")
    return dWg, dlogit


def meteora_group_plan(T, d_in, d_outs, N, r, k, dtype: torch.dtype) -> int:
    """1 if meteora_linear_forward_group runs these modules as one kernel launch, 0 if module by module."""
    lib = load_library()
    shape = make_shape(T, d_in, d_outs[0], N, r, k, dtype)
    rc = lib.meteora_group_plan(ctypes.byref(shape), (ctypes.c_int * len(d_outs))(*d_outs), len(d_outs))
    if rc < 0:
        raise MeteoraError(rc, "meteora_group_plan")
    return rc


def meteora_linear_forward_group(x, W0s, As, Bs, Wgs, k: int, temperature: float = 1.0,
                                 workspace: Optional[torch.Tensor] = None, return_routing: bool = False):
    """Several MeteoRA linears on the same x (lists of per-module tensors).  Returns the list of y, or
    (ys, [(topk_idx, topk_w) per module]) with views of the workspace."""
    lib = load_library()
    T, d_in = x.shape
    G = len(W0s)
    N, r, _ = As[0].shape
    d_outs = [int(W0.shape[0]) for W0 in W0s]
    shape = make_shape(T, d_in, d_outs[0], N, r, k, x.dtype, temperature)
    _dtype_code(x)
    c_d_out = (ctypes.c_int * G)(*d_outs)
    if workspace is None:
        n = lib.meteora_group_workspace_bytes(ctypes.byref(shape), c_d_out, G)
        if n == 0:
            raise MeteoraError(-1, "meteora_group_workspace_bytes")
        workspace = torch.zeros(n, dtype=torch.uint8, device=x.device)
    ys = [torch.empty((T, d), dtype=x.dtype, device=x.device) for d in d_outs]
    vpa = ctypes.c_void_p * G
    c_W0 = vpa(*[_dev(W0s[m], (d_outs[m], d_in), x.dtype, "W0") for m in range(G)])
    c_A = vpa(*[_dev(As[m], (N, r, d_in), x.dtype, "A") for m in range(G)])
    c_B = vpa(*[_dev(Bs[m], (N, d_outs[m], r), x.dtype, "B") for m in range(G)])
    c_Wg = vpa(*[_dev(Wgs[m], (N, d_in), x.dtype, "Wg") for m in range(G)])
    c_y = vpa(*[y.data_ptr() for y in ys])
    _check(lib.meteora_linear_forward_group(_dev(x, (T, d_in), x.dtype, "x"), c_W0, c_A, c_B, c_Wg, c_d_out, G,
                                            ctypes.byref(shape), c_y, workspace.data_ptr(), workspace.numel(),
                                            _stream()), "meteora_linear_forward_group")
    if not return_routing:
        return ys
    routing = []
    for m in range(G):
        p_idx, p_w = ctypes.c_void_p(), ctypes.c_void_p()
        _check(lib.meteora_group_workspace_routing(ctypes.byref(shape), c_d_out, G, m, workspace.data_ptr(),
                                                   ctypes.byref(p_idx), ctypes.byref(p_w)),
               "meteora_group_workspace_routing")
        off_i, off_w = p_idx.value - workspace.data_ptr(), p_w.value - workspace.data_ptr()
        idx = workspace[off_i:off_i + T * k * 4].view(torch.int32).view(T, k)
        w = workspace[off_w:off_w + T * k * 4].view(torch.float32).view(T, k)
        routing.append((idx, w))
    return ys, routing


def meteora_linear_forward_host(x_host, W0, A, B, Wg, k: int, y_host: torch.Tensor, workspace: torch.Tensor,
                                temperature: float = 1.0) -> torch.Tensor:
    """x_host / y_host are (pinned) host tensors; weights and workspace are CUDA tensors.  Asynchronous."""
    lib = load_library()
    T, d_in = x_host.shape
    d_out = W0.shape[0]
    N, r, _ = A.shape
    dt = W0.dtype
    shape = make_shape(T, d_in, d_out, N, r, k, dt, temperature)
    for t, n in ((x_host, "x_host"), (y_host, "y_host")):
        if t.is_cuda or not t.is_contiguous() or t.dtype != dt:
            raise ValueError(f"{n} must be a contiguous host tensor of dtype {dt}")
    if tuple(y_host.shape) != (T, d_out):
        raise ValueError("y_host has the wrong shape")
    _check(lib.meteora_linear_forward_host(x_host.data_ptr(), _dev(W0, (d_out, d_in), dt, "W0"),
                                           _dev(A, (N, r, d_in), dt, "A"), _dev(B, (N, d_out, r), dt, "B"),
                                           _dev(Wg, (N, d_in), dt, "Wg"), ctypes.byref(shape), y_host.data_ptr(),
                                           workspace.data_ptr(), workspace.numel(), _stream()),
           "meteora_linear_forward_host")
    return y_host


def meteora_workspace_routing(shape: MeteoraShape, workspace: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """Views of the routing meteora_linear_forward left in the workspace: (topk_idx[T,k], topk_w[T,k])."""
    lib = load_library()
    pi, pw = ctypes.c_void_p(), ctypes.c_void_p()
    _check(lib.meteora_workspace_routing(ctypes.byref(shape), workspace.data_ptr(), ctypes.byref(pi),
                                         ctypes.byref(pw)), "meteora_workspace_routing")
    n = shape.T * shape.k
    off_i, off_w = pi.value - workspace.data_ptr(), pw.value - workspace.data_ptr()
    idx = workspace[off_i:off_i + 4 * n].view(torch.int32).view(shape.T, shape.k)
    w = workspace[off_w:off_w + 4 * n].view(torch.float32).view(shape.T, shape.k)
    return idx, w


def meteora_workspace_init(workspace: torch.Tensor) -> None:
    _check(load_library().meteora_workspace_init(workspace.data_ptr(), _stream()), "meteora_workspace_init")


def meteora_workspace_status(workspace: torch.Tensor) -> int:
    """Synchronises the current stream; returns 0 or METEORA_ERR_TIMEOUT (-6)."""
    return int(load_library().meteora_workspace_status(workspace.data_ptr(), _stream()))


def meteora_profile_begin(max_launches: int) -> None:
    _check(load_library().meteora_profile_begin(int(max_launches)), "meteora_profile_begin")


def meteora_profile_end() -> Tuple[float, int]:
    """Synchronises; returns (summed milliseconds of the timed base-product launches, their count)."""
    ms, n = ctypes.c_float(), ctypes.c_int()
    _check(load_library().meteora_profile_end(ctypes.byref(ms), ctypes.byref(n)), "meteora_profile_end")
    return float(ms.value), int(n.value)


def meteora_describe_plan(shape: MeteoraShape) -> str:
    buf = ctypes.create_string_buffer(640)
    _check(load_library().meteora_describe_plan(ctypes.byref(shape), buf, len(buf)), "meteora_describe_plan")
    return buf.value.decode()


def meteora_set_tuning(name: str, value: int) -> None:
    _check(load_library().meteora_set_tuning(name.encode(), int(value)), f"meteora_set_tuning({name})")


def meteora_status_string(status: int) -> str:
    return load_library().meteora_status_string(int(status)).decode()
