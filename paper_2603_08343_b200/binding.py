"""ctypes binding of libwht_affine.so: same names and argument order as include/wht_affine.h.

Argument marshalling only -- every step of the path runs in the library's CUDA
kernels.  torch is used for device memory and the current stream.  If the shared
library is missing or cannot be loaded, importing this module raises; there is
no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .workloads import WHT_BF16, WHT_BF16_PF32, WHT_F32

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwht_affine.so")

EXPORTS = (
    "wht_affine_fwd", "wht_affine_fwd_residual", "wht_affine_fwd_decode", "wht_affine_bwd", "wht_affine_bwd_ws", "wht_affine_bwd_noalloc", "wht_affine_reduce_grads",
    "wht_affine_fwd_grouped", "wht_affine_bwd_grouped", "wht_affine_bwd_grouped_workspace_bytes",
    "wht_affine_fwd_tp", "wht_affine_bwd_tp", "wht_affine_bwd_tp_workspace_bytes",
    "wht_affine_bwd_workspace_bytes", "wht_affine_set_variant", "wht_affine_get_variant",
    "wht_affine_set_bwd_operand_mode", "wht_affine_get_bwd_operand_mode",
    "wht_copy_rows", "wht_affine_device_status", "wht_affine_selftest_wait_expiry",
    "wht_affine_debug_build", "wht_affine_debug_selftest_guard", "wht_affine_test_fail_allocations",
    "wht_affine_last_cuda_error", "wht_affine_status_string",
    "wht_affine_shutdown",
)


class WhtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.wht_affine_status_string(status).decode()
        cuda = _lib.wht_affine_last_cuda_error()
        super().__init__(f"{where}: {msg} (status {status}, cuda error {cuda})")


def _load(path: str | None = None) -> ctypes.CDLL:
    """Loads the library (the regular build, or another build of it given by path) and declares the
    argument types of every export."""
    path = LIB_PATH if path is None else path
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2603_08343_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    vp, i64, i32, ci, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int, ctypes.c_size_t
    lib.wht_affine_fwd.argtypes = [vp, vp, vp, vp, i64, i32, ci, vp]
    lib.wht_affine_fwd_residual.argtypes = [vp, vp, vp, vp, vp, i64, i32, ci, vp]
    lib.wht_affine_fwd_decode.argtypes = [vp, vp, vp, vp, i64, i32, ci, vp]
    lib.wht_affine_bwd.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, ci, vp]
    lib.wht_affine_bwd_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, ci, vp]
    lib.wht_affine_bwd_ws.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, ci, vp, sz, vp]
    lib.wht_affine_reduce_grads.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.wht_affine_fwd_grouped.argtypes = [vp, vp, vp, vp, i64, i32, i32, ci, vp]
    lib.wht_affine_bwd_grouped.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, i32, ci, vp, sz, vp]
    lib.wht_affine_bwd_grouped_workspace_bytes.argtypes = [i64, i32, i32, ci]
    lib.wht_affine_bwd_grouped_workspace_bytes.restype = sz
    lib.wht_affine_fwd_tp.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, ci, vp]
    lib.wht_affine_bwd_tp.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, i32, i32, ci, vp, sz, vp]
    lib.wht_affine_bwd_tp_workspace_bytes.argtypes = [i64, i32, i32, ci]
    lib.wht_affine_bwd_tp_workspace_bytes.restype = sz
    lib.wht_affine_bwd_workspace_bytes.argtypes = [i64, i32, ci]
    lib.wht_affine_bwd_workspace_bytes.restype = sz
    lib.wht_affine_set_variant.argtypes = [ci]
    lib.wht_affine_get_variant.argtypes = []
    lib.wht_affine_set_bwd_operand_mode.argtypes = [ci]
    lib.wht_affine_get_bwd_operand_mode.argtypes = []
    lib.wht_copy_rows.argtypes = [vp, vp, i64, i32, ci, vp]
    lib.wht_affine_device_status.argtypes = []
    lib.wht_affine_selftest_wait_expiry.argtypes = [ctypes.c_uint32, vp, vp]
    lib.wht_affine_last_cuda_error.argtypes = []
    lib.wht_affine_status_string.argtypes = [ci]
    lib.wht_affine_status_string.restype = ctypes.c_char_p
    lib.wht_affine_shutdown.argtypes = []
    lib.wht_affine_debug_build.argtypes = []
    lib.wht_affine_debug_selftest_guard.argtypes = [ci]
    lib.wht_affine_test_fail_allocations.argtypes = [ci]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is ctypes.c_int or fn.restype is None:
            fn.restype = ctypes.c_int
    return lib


_lib = _load()


def lib() -> ctypes.CDLL:
    """The loaded shared library (for tests that call the C ABI with raw pointers)."""
    return _lib


def load_library(path: str) -> ctypes.CDLL:
    """Another build of the library (the -DWHT_DEBUG one) with the same argument types declared."""
    return _load(path)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(status: int, where: str) -> None:
    if status != 0:
        raise WhtError(status, where)


def _require_cuda(*tensors):
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise ValueError("tensors must live on a CUDA device")
        if t is not None and not t.is_contiguous():
            raise ValueError("tensors must be contiguous")


def wht_affine_fwd(x, a, b, y, T: int, d: int, dtype: int, stream=None) -> None:
    _require_cuda(x, a, b, y)
    _check(_lib.wht_affine_fwd(_ptr(x), _ptr(a), _ptr(b), _ptr(y), T, d, dtype, _stream(stream)),
           "wht_affine_fwd")


def wht_affine_fwd_residual(x, a, b, resid, y, T: int, d: int, dtype: int, stream=None) -> None:
    """y = resid + a (.) (x H)/sqrt(d) + b in one kernel (resid has the layout and type of x)."""
    _require_cuda(x, a, b, resid, y)
    _check(_lib.wht_affine_fwd_residual(_ptr(x), _ptr(a), _ptr(b), _ptr(resid), _ptr(y), T, d, dtype,
                                        _stream(stream)), "wht_affine_fwd_residual")


def wht_affine_fwd_decode(x, a, b, y, T: int, d: int, dtype: int, stream=None) -> None:
    _require_cuda(x, a, b, y)
    _check(_lib.wht_affine_fwd_decode(_ptr(x), _ptr(a), _ptr(b), _ptr(y), T, d, dtype, _stream(stream)),
           "wht_affine_fwd_decode")


class PreparedCall:
    """One call of the C ABI with its arguments marshalled once.

    The plain wrappers look up the current stream, check every tensor and box every pointer on each call,
    about 7 us of Python per call -- several times the device time of a decode-sized forward.  A loop that
    repeats the same call on the same buffers (one decode step after another) prepares it once and then
    pays one foreign call per launch.  The tensors must stay alive and in place; the stream is fixed at
    preparation time.
    """
    __slots__ = ("_fn", "_args", "_where", "_keep")

    def __init__(self, fn, args, where, keep):
        self._fn, self._args, self._where, self._keep = fn, args, where, keep

    def __call__(self) -> None:
        rc = self._fn(*self._args)
        if rc != 0:
            raise WhtError(rc, self._where)


def prepare(name: str, *args, stream=None) -> PreparedCall:
    """Prepares `name(*args, stream)` of the C ABI: tensors become device pointers, integers stay.
    E.g. prepare("wht_affine_fwd_decode", x, a, b, y, T, d, dtype)."""
    if name not in EXPORTS:
        raise ValueError(f"{name} is not an entry point of the library")
    tensors = [t for t in args if isinstance(t, torch.Tensor)]
    _require_cuda(*tensors)
    marshalled = [_ptr(t) if isinstance(t, torch.Tensor) else t for t in args]
    marshalled.append(_stream(stream))
    return PreparedCall(getattr(_lib, name), tuple(marshalled), name, tensors)


def wht_affine_bwd(dy, x, a, dx, da, db, T: int, d: int, dtype: int, stream=None) -> None:
    _require_cuda(dy, x, a, dx, da, db)
    _check(_lib.wht_affine_bwd(_ptr(dy), _ptr(x), _ptr(a), _ptr(dx), _ptr(da), _ptr(db), T, d, dtype,
                               _stream(stream)), "wht_affine_bwd")


def wht_affine_bwd_ws(dy, x, a, dx, da, db, T: int, d: int, dtype: int, workspace, stream=None) -> None:
    _require_cuda(dy, x, a, dx, da, db, workspace)
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.wht_affine_bwd_ws(_ptr(dy), _ptr(x), _ptr(a), _ptr(dx), _ptr(da), _ptr(db), T, d, dtype,
                                  _ptr(workspace), nbytes, _stream(stream)), "wht_affine_bwd_ws")


def wht_affine_bwd_noalloc(dy, x, a, dx, da, db, T: int, d: int, dtype: int, stream=None) -> None:
    """Backward pass that never allocates: its scratch is a fixed 16 MiB array inside the library.

    For callers that cannot let a library call cudaMalloc (a pool that owns all device
    memory, latency-critical loops, allocation banned after start-up).  Same results as
    wht_affine_bwd; raises WhtError(WHT_ERR_WORKSPACE) when the problem needs more scratch
    than the array holds.  Calls on one device share the array: do not overlap them.
    """
    _require_cuda(dy, x, a, dx, da, db)
    _check(_lib.wht_affine_bwd_noalloc(_ptr(dy), _ptr(x), _ptr(a), _ptr(dx), _ptr(da), _ptr(db), T, d, dtype,
                                       _stream(stream)), "wht_affine_bwd_noalloc")


def wht_affine_reduce_grads(parts, n: int, d: int, da, db, stream=None) -> None:
    """da, db = sums over the n (da_p | db_p) pairs stored contiguously in `parts` [n, 2, d] fp32."""
    _require_cuda(parts, da, db)
    _check(_lib.wht_affine_reduce_grads(_ptr(parts), n, d, _ptr(da), _ptr(db), _stream(stream)),
           "wht_affine_reduce_grads")


def wht_affine_fwd_grouped(x, a, b, y, T: int, d: int, block: int, dtype: int, stream=None) -> None:
    """Block-diagonal form: every group of `block` channels is transformed on its own (d = groups*block)."""
    _require_cuda(x, a, b, y)
    _check(_lib.wht_affine_fwd_grouped(_ptr(x), _ptr(a), _ptr(b), _ptr(y), T, d, block, dtype, _stream(stream)),
           "wht_affine_fwd_grouped")


def wht_affine_bwd_grouped(dy, x, a, dx, da, db, T: int, d: int, block: int, dtype: int, workspace,
                           stream=None) -> None:
    _require_cuda(dy, x, a, dx, da, db, workspace)
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.wht_affine_bwd_grouped(_ptr(dy), _ptr(x), _ptr(a), _ptr(dx), _ptr(da), _ptr(db), T, d, block, dtype,
                                       _ptr(workspace), nbytes, _stream(stream)), "wht_affine_bwd_grouped")


def wht_affine_bwd_grouped_workspace_bytes(T: int, d: int, block: int, dtype: int) -> int:
    return int(_lib.wht_affine_bwd_grouped_workspace_bytes(T, d, block, dtype))


def _ptr_array(parts):
    """Host array of device pointers; entries are tensors or integer addresses (peer mappings)."""
    addrs = [p if isinstance(p, int) else p.data_ptr() for p in parts]
    return (ctypes.c_void_p * len(addrs))(*addrs)


def wht_affine_fwd_tp(x_parts, a, b, y, T: int, w: int, g: int, r: int, dtype: int, stream=None) -> None:
    """Column-sharded forward of rank r: x_parts[s] is rank s's [T, w] block (tensor or device address)."""
    _require_cuda(a, b, y, *[p for p in x_parts if not isinstance(p, int)])
    if len(x_parts) != g:
        raise ValueError(f"{len(x_parts)} blocks for g = {g}")
    _check(_lib.wht_affine_fwd_tp(_ptr_array(x_parts), _ptr(a), _ptr(b), _ptr(y), T, w, g, r, dtype,
                                  _stream(stream)), "wht_affine_fwd_tp")


def wht_affine_bwd_tp(dy_parts, x_parts, a_parts, dx, da, db, T: int, w: int, g: int, r: int, dtype: int,
                      workspace, stream=None) -> None:
    _require_cuda(dx, da, db, workspace,
                  *[p for p in (*dy_parts, *x_parts, *a_parts) if not isinstance(p, int)])
    if not len(dy_parts) == len(x_parts) == len(a_parts) == g:
        raise ValueError(f"every list needs g = {g} blocks")
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.wht_affine_bwd_tp(_ptr_array(dy_parts), _ptr_array(x_parts), _ptr_array(a_parts), _ptr(dx),
                                  _ptr(da), _ptr(db), T, w, g, r, dtype, _ptr(workspace), nbytes,
                                  _stream(stream)), "wht_affine_bwd_tp")


def wht_affine_bwd_tp_workspace_bytes(T: int, w: int, g: int, dtype: int) -> int:
    return int(_lib.wht_affine_bwd_tp_workspace_bytes(T, w, g, dtype))


def wht_affine_bwd_workspace_bytes(T: int, d: int, dtype: int) -> int:
    return int(_lib.wht_affine_bwd_workspace_bytes(T, d, dtype))


def wht_affine_set_variant(variant: int) -> None:
    _check(_lib.wht_affine_set_variant(variant), "wht_affine_set_variant")


def wht_affine_get_variant() -> int:
    return int(_lib.wht_affine_get_variant())


def wht_affine_set_bwd_operand_mode(mode: int) -> None:
    """How g = (a/sqrt d) (.) dy enters the tcgen05 backward's second product: 0 = rounded to bf16 once
    (default), 1 = as a bf16 pair hi + lo (dx then is the fp32 result rounded once at the store)."""
    _check(_lib.wht_affine_set_bwd_operand_mode(mode), "wht_affine_set_bwd_operand_mode")


def wht_affine_get_bwd_operand_mode() -> int:
    return int(_lib.wht_affine_get_bwd_operand_mode())


def wht_copy_rows(src, dst, T: int, d: int, dtype: int, stream=None) -> None:
    _require_cuda(src, dst)
    _check(_lib.wht_copy_rows(_ptr(src), _ptr(dst), T, d, dtype, _stream(stream)), "wht_copy_rows")


def wht_affine_device_status() -> None:
    """Synchronises and raises WhtError if a kernel's bounded wait expired since the last query."""
    _check(_lib.wht_affine_device_status(), "wht_affine_device_status")


def wht_affine_selftest_wait_expiry(limit_us: int, out3, stream=None) -> None:
    """Launches the library's one-CTA kernel whose bounded wait runs out after about limit_us microseconds
    (out3: three int32/uint32 words on the device); afterwards wht_affine_device_status() raises once."""
    _require_cuda(out3)
    _check(_lib.wht_affine_selftest_wait_expiry(limit_us, _ptr(out3), _stream(stream)),
           "wht_affine_selftest_wait_expiry")


def wht_affine_test_fail_allocations(n: int) -> int:
    """Test hook: the library's next n allocations of its own fail as out of memory; returns how many
    injected failures were still pending."""
    pending = _lib.wht_affine_test_fail_allocations(n)
    if pending < 0:
        raise WhtError(pending, "wht_affine_test_fail_allocations")
    return pending


def wht_affine_shutdown() -> None:
    _check(_lib.wht_affine_shutdown(), "wht_affine_shutdown")


# ---- convenience wrappers that infer T, d and the dtype code from the tensors ----

def dtype_code(x: torch.Tensor, a: torch.Tensor) -> int:
    if x.dtype == torch.float32 and a.dtype == torch.float32:
        return WHT_F32
    if x.dtype == torch.bfloat16 and a.dtype == torch.bfloat16:
        return WHT_BF16
    if x.dtype == torch.bfloat16 and a.dtype == torch.float32:
        return WHT_BF16_PF32
    raise ValueError(f"unsupported storage types x={x.dtype}, a={a.dtype}")


def forward(x, a, b, out=None, decode: bool = False, stream=None, resid=None):
    """y = [resid +] a (.) (x H)/sqrt(d) + b for x[..., d]; returns `out` (allocated if None)."""
    d = x.shape[-1]
    T = x.numel() // d if d else 0
    y = torch.empty_like(x) if out is None else out
    if resid is not None:
        wht_affine_fwd_residual(x, a, b, resid, y, T, d, dtype_code(x, a), stream)
        return y
    fn = wht_affine_fwd_decode if decode else wht_affine_fwd
    fn(x, a, b, y, T, d, dtype_code(x, a), stream)
    return y


def backward(dy, x, a, stream=None):
    """(dx, da, db) for the forward above; da, db are fp32."""
    d = x.shape[-1]
    T = x.numel() // d if d else 0
    dx = torch.empty_like(x)
    da = torch.empty(d, dtype=torch.float32, device=x.device)
    db = torch.empty(d, dtype=torch.float32, device=x.device)
    wht_affine_bwd(dy, x, a, dx, da, db, T, d, dtype_code(x, a), stream)
    return dx, da, db


class HostPipe:
    """Two copy streams for the host <-> device legs of a step.

    Rows are independent, so the forward pass runs chunk by chunk: chunk i is transformed
    while chunk i+1 is still arriving and chunk i-1 is already on its way back, and the
    copies of the two directions (y going out, dy coming in) share the link.  `join()`
    makes the current stream wait for everything queued on the copy streams.
    """

    def __init__(self, chunk_rows: int = 8192):
        self.chunk_rows = int(chunk_rows)
        self.s_in = torch.cuda.Stream()
        self.s_out = torch.cuda.Stream()

    def chunks(self, T: int):
        return [(r, min(T, r + self.chunk_rows)) for r in range(0, T, self.chunk_rows)]

    def join(self):
        cur = torch.cuda.current_stream()
        cur.wait_stream(self.s_in)
        cur.wait_stream(self.s_out)


def forward_host(x_host, a_host, b_host, y_host, staging, stream=None, pipe: HostPipe | None = None):
    """End-to-end forward from pinned host memory: copy in, transform, copy out.

    `staging` is a dict of preallocated device tensors {"x", "a", "b", "y"}.  Without `pipe`
    all copies are asynchronous on the current stream; with a HostPipe the rows move in chunks
    on its copy streams and the caller ends the step with pipe.join().
    """
    cur = torch.cuda.current_stream() if stream is None else stream
    if pipe is None:
        with torch.cuda.stream(cur):  # copies and kernels on ONE stream: ordered by it
            staging["x"].copy_(x_host, non_blocking=True)
            staging["a"].copy_(a_host, non_blocking=True)
            staging["b"].copy_(b_host, non_blocking=True)
            forward(staging["x"], staging["a"], staging["b"], out=staging["y"], stream=cur)
            y_host.copy_(staging["y"], non_blocking=True)
        return y_host
    xs, ys, a, b = staging["x"], staging["y"], staging["a"], staging["b"]
    d = xs.shape[-1]
    code = dtype_code(xs, a)
    pipe.s_in.wait_stream(cur)   # the staging buffers may still be in use by earlier work
    pipe.s_out.wait_stream(cur)
    cur.wait_stream(pipe.s_out)  # ... and an earlier step's copies out may still be reading staging["y"]
    with torch.cuda.stream(pipe.s_in):
        a.copy_(a_host, non_blocking=True)
        b.copy_(b_host, non_blocking=True)
    for r0, r1 in pipe.chunks(xs.shape[0]):
        with torch.cuda.stream(pipe.s_in):
            xs[r0:r1].copy_(x_host[r0:r1], non_blocking=True)
            arrived = torch.cuda.Event()
            arrived.record(pipe.s_in)
        cur.wait_event(arrived)
        wht_affine_fwd(xs[r0:r1], a, b, ys[r0:r1], r1 - r0, d, code, cur)
        done = torch.cuda.Event()
        done.record(cur)
        pipe.s_out.wait_event(done)
        with torch.cuda.stream(pipe.s_out):
            y_host[r0:r1].copy_(ys[r0:r1], non_blocking=True)
    return y_host


def backward_host(dy_host, x_host, a_host, dx_host, da_host, db_host, staging, stream=None,
                  pipe: HostPipe | None = None, x_resident: bool = False):
    """End-to-end backward from pinned host memory; `staging` holds device tensors
    {"dy", "x", "a", "dx", "da", "db"}.  `x_resident` skips the copy of x and a when the forward
    call of the same step has just put them on the device (as in training)."""
    st = staging
    d = st["x"].shape[-1]
    T = st["x"].numel() // d
    code = dtype_code(st["x"], st["a"])
    cur = torch.cuda.current_stream() if stream is None else stream
    if pipe is None:
        with torch.cuda.stream(cur):  # copies and kernels on ONE stream: ordered by it
            st["dy"].copy_(dy_host, non_blocking=True)
            if not x_resident:
                st["x"].copy_(x_host, non_blocking=True)
                st["a"].copy_(a_host, non_blocking=True)
            wht_affine_bwd(st["dy"], st["x"], st["a"], st["dx"], st["da"], st["db"], T, d, code, cur)
            dx_host.copy_(st["dx"], non_blocking=True)
            da_host.copy_(st["da"], non_blocking=True)
            db_host.copy_(st["db"], non_blocking=True)
        return
    # the staging buffers (and the per-chunk gradient pairs) may still be in use by earlier work on `cur`:
    # a previous step's kernels read st["dy"] / st["x"], its copies out read st["dx"]
    pipe.s_in.wait_stream(cur)
    pipe.s_out.wait_stream(cur)
    cur.wait_stream(pipe.s_out)
    # dy comes in chunk by chunk on the copy stream (sharing the link with the forward's y going
    # out); each chunk is transformed as it lands and its dx leaves on the other copy stream, so the
    # two directions of the link stay busy together.  da, db are sums over rows: every chunk writes
    # its own pair, one small kernel adds them in a fixed order.
    chunks = pipe.chunks(T)
    parts = st.get("grad_parts")
    if parts is None or parts.shape[0] < len(chunks):
        parts = st["grad_parts"] = torch.empty(len(chunks), 2, d, dtype=torch.float32, device=st["x"].device)
    if not x_resident:
        with torch.cuda.stream(pipe.s_in):
            st["x"].copy_(x_host, non_blocking=True)
            st["a"].copy_(a_host, non_blocking=True)
    for i, (r0, r1) in enumerate(chunks):
        with torch.cuda.stream(pipe.s_in):
            st["dy"][r0:r1].copy_(dy_host[r0:r1], non_blocking=True)
            arrived = torch.cuda.Event()
            arrived.record(pipe.s_in)
        cur.wait_event(arrived)
        wht_affine_bwd(st["dy"][r0:r1], st["x"][r0:r1], st["a"], st["dx"][r0:r1], parts[i, 0], parts[i, 1],
                       r1 - r0, d, code, cur)
        done = torch.cuda.Event()
        done.record(cur)
        pipe.s_out.wait_event(done)
        with torch.cuda.stream(pipe.s_out):
            dx_host[r0:r1].copy_(st["dx"][r0:r1], non_blocking=True)
    wht_affine_reduce_grads(parts, len(chunks), d, st["da"], st["db"], cur)
    done = torch.cuda.Event()
    done.record(cur)
    pipe.s_out.wait_event(done)
    with torch.cuda.stream(pipe.s_out):
        da_host.copy_(st["da"], non_blocking=True)
        db_host.copy_(st["db"], non_blocking=True)
