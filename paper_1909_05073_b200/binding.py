"""ctypes binding of libpconv.so: argument marshalling only -- every step of the forward path
runs in the library's CUDA kernels.  Function names mirror the C ABI (include/pconv.h).

There is no CPU fallback: if the shared library is missing or cannot be loaded, every call
raises.  torch is used for device memory and streams only.
"""
import ctypes
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libpconv.so")

OK = 0
F32, F16 = 0, 1
RELU, STRICT4, POOL2X2, REPRODUCIBLE, CHAIN = 1, 2, 4, 8, 0x10
KERNEL_SIMPLE, KERNEL_TILED, KERNEL_GENERIC_TAPS, KERNEL_TENSOR = 0x100, 0x200, 0x400, 0x800
ROWS4, ROWS8, CLUSTER, STAGE_BULK = 0x1000, 0x2000, 0x4000, 0x8000
MAX_PATTERNS = 16

STATUS_NAMES = ["PCONV_OK", "PCONV_ERR_NULL", "PCONV_ERR_SHAPE", "PCONV_ERR_PATTERN_SET",
                "PCONV_ERR_KERNEL_NOT_IN_SET", "PCONV_ERR_RANGE", "PCONV_ERR_UNSUPPORTED",
                "PCONV_ERR_ALIGN", "PCONV_ERR_ALLOC", "PCONV_ERR_CUDA",
                "PCONV_ERR_DEVICE_TIMEOUT", "PCONV_ERR_WORKSPACE"]

EXPORTS = ["pconv_pack", "pconv_forward", "pconv_forward_ws", "pconv_forward_static_ws", "pconv_workspace_bytes", "pconv_plan", "pconv_plan_shape",
           "pconv_free", "pconv_maxpool2x2", "pconv_unpack",
           "pconv_stats", "pconv_filter_order", "pconv_device_status", "pconv_status_str",
           "pconv_stack_create", "pconv_stack_out_shape", "pconv_stack_forward",
           "pconv_stack_forward_host", "pconv_stack_free", "pconv_stack_capture", "pconv_stack_replay", "pconv_stack_status", "pconv_stack_launches",
           "pconv_project", "pconv_project_workspace_bytes"]


class PconvError(RuntimeError):
    def __init__(self, status, what, detail=None):
        self.status = status
        self.detail = detail
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__("%s: %s%s" % (what, name, (" %r" % (detail,)) if detail else ""))


class Stats(ctypes.Structure):
    _fields_ = [("c_out", ctypes.c_int), ("c_in", ctypes.c_int), ("stride", ctypes.c_int),
                ("storage", ctypes.c_int), ("n_patterns", ctypes.c_int),
                ("kept_kernels", ctypes.c_longlong),
                ("per_pattern", ctypes.c_longlong * MAX_PATTERNS),
                ("min_per_filter", ctypes.c_int), ("max_per_filter", ctypes.c_int),
                ("n_groups", ctypes.c_int), ("group_size", ctypes.c_int),
                ("max_group_kernels", ctypes.c_longlong),
                ("min_group_kernels", ctypes.c_longlong),
                ("packed_bytes", ctypes.c_longlong), ("canonical_patterns", ctypes.c_int)]


class Plan(ctypes.Structure):
    _fields_ = [("generic_taps", ctypes.c_int), ("rows_per_lane", ctypes.c_int),
                ("warps_per_unit", ctypes.c_int),
                ("channel_splits", ctypes.c_int), ("groups_per_cta", ctypes.c_int),
                ("pixel_sets", ctypes.c_int), ("tile_width", ctypes.c_int), ("stages", ctypes.c_int),
                ("smem_bytes", ctypes.c_int), ("ctas", ctypes.c_longlong),
                ("staging", ctypes.c_int), ("tensor_path", ctypes.c_int)]


_lib = None


def load(path):
    """Loads a build of the library and declares its entry points' argument types."""
    if not os.path.exists(path):
        raise RuntimeError("%s is missing: run `python -m paper_1909_05073_b200.build`"
                           " (the CUDA library is the only implementation)" % os.path.basename(path))
    L = ctypes.CDLL(path)
    vp, ci, cu = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint
    ip = ctypes.POINTER(ctypes.c_int)
    L.pconv_pack.argtypes = [vp, ci, ci, vp, ci, ci, ci, cu, vp, ctypes.POINTER(vp), ip, ip]
    L.pconv_forward.argtypes = [vp, vp, vp, vp, ci, ci, ci, cu, vp]
    L.pconv_forward_ws.argtypes = [vp, vp, vp, vp, ci, ci, ci, cu, vp, ctypes.c_size_t, vp]
    L.pconv_forward_static_ws.argtypes = [vp, vp, vp, vp, ci, ci, ci, cu, vp]
    L.pconv_workspace_bytes.argtypes = [vp, ci, ci, ci, ctypes.POINTER(ctypes.c_size_t)]
    L.pconv_plan.argtypes = [vp, ci, ci, ci, cu, ci, ctypes.POINTER(Plan)]
    L.pconv_plan_shape.argtypes = [ci, ci, ctypes.c_longlong, ci, ci, ci, ci, ci, ci, cu, ci,
                                   ctypes.POINTER(Plan)]
    L.pconv_free.argtypes = [vp]
    L.pconv_free.restype = None
    L.pconv_maxpool2x2.argtypes = [vp, vp, ci, ci, ci, ci, ci, vp]
    L.pconv_unpack.argtypes = [vp, vp]
    L.pconv_stats.argtypes = [vp, ctypes.POINTER(Stats)]
    L.pconv_filter_order.argtypes = [vp, vp]
    L.pconv_device_status.argtypes = [vp, ip]
    L.pconv_project_workspace_bytes.argtypes = [ctypes.c_longlong, ctypes.POINTER(ctypes.c_size_t)]
    L.pconv_project.argtypes = [vp, ctypes.c_longlong, vp, ci, ctypes.c_double, vp, vp, vp,
                                ctypes.c_size_t, vp]
    if hasattr(L, "pconv_trace_read"):     # development build only (csrc/pconv_dev.h)
        L.pconv_trace_read.argtypes = [vp, ctypes.POINTER(ctypes.c_ulonglong), ci]
        L.pconv_dev_withhold.argtypes = [ci, cu]
        L.pconv_dev_clear_status.argtypes = [vp]
    L.pconv_status_str.argtypes = [ci]
    L.pconv_status_str.restype = ctypes.c_char_p
    L.pconv_stack_create.argtypes = [vp, vp, vp, ci, ci, ci, ci, cu, ctypes.POINTER(vp)]
    L.pconv_stack_out_shape.argtypes = [vp, ip, ip, ip, ip]
    L.pconv_stack_forward.argtypes = [vp, vp, vp, vp]
    L.pconv_stack_forward_host.argtypes = [vp, vp, vp, vp]
    L.pconv_stack_capture.argtypes = [vp, vp, vp, vp]
    L.pconv_stack_replay.argtypes = [vp, vp]
    L.pconv_stack_status.argtypes = [vp, ip]
    L.pconv_stack_launches.argtypes = [vp, ip]
    L.pconv_stack_free.argtypes = [vp]
    L.pconv_stack_free.restype = None
    return L


def lib():
    """The loaded shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        _lib = load(LIB_PATH)
    return _lib


def use_library(path):
    """Makes every call of this module go to another build of the library (the development
    build, in its tests); returns the library that was in use before."""
    global _lib
    old = _lib
    _lib = load(path) if path is not None else None
    return old


def _check(status, what, detail=None):
    if status != OK:
        raise PconvError(status, what, detail)


def _stream_ptr(stream=None):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _storage_of(t):
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.float16:
        return F16
    raise TypeError("activations must be float32 or float16")


def pconv_status_str(status):
    return lib().pconv_status_str(int(status)).decode()


def pconv_pack(w_oihw, patterns, stride=1, storage=F32, flags=0, stream=None):
    """Packs dense OIHW fp32 host weights (numpy) + pattern masks into a device handle."""
    w = np.ascontiguousarray(w_oihw, dtype=np.float32)
    if w.ndim != 4 or w.shape[2:] != (3, 3):
        raise ValueError("weights must be [C_out, C_in, 3, 3]")
    pats = np.ascontiguousarray(patterns, dtype=np.uint16)
    out = ctypes.c_void_p()
    bad_o, bad_c = ctypes.c_int(-1), ctypes.c_int(-1)
    st = lib().pconv_pack(w.ctypes.data, w.shape[0], w.shape[1], pats.ctypes.data, len(pats),
                          int(stride), int(storage), int(flags), _stream_ptr(stream),
                          ctypes.byref(out), ctypes.byref(bad_o), ctypes.byref(bad_c))
    _check(st, "pconv_pack", (bad_o.value, bad_c.value) if bad_o.value >= 0 else None)
    return out


def pconv_free(handle):
    lib().pconv_free(handle)


def pconv_plan(handle, n, h, w, flags=0, with_workspace=False):
    """The launch geometry of a tiled forward of this shape, as a dict."""
    p = Plan()
    _check(lib().pconv_plan(handle, n, h, w, int(flags), int(bool(with_workspace)), ctypes.byref(p)),
           "pconv_plan")
    return {k: int(getattr(p, k)) for k, _ in Plan._fields_}


def pconv_project(w, patterns, keep, out=None, stream=None):
    """Projects a CUDA fp32 tensor [c_out, c_in, 3, 3] onto the pattern set / keep rate.
    Returns (projected weights, int8 pattern ids [c_out, c_in] with -1 = pruned)."""
    import torch
    if not (w.is_cuda and w.is_contiguous() and w.dtype == torch.float32 and tuple(w.shape[2:]) == (3, 3)):
        raise ValueError("w must be a contiguous CUDA float32 tensor [c_out, c_in, 3, 3]")
    n = w.shape[0] * w.shape[1]
    need = ctypes.c_size_t(0)
    _check(lib().pconv_project_workspace_bytes(n, ctypes.byref(need)), "pconv_project_workspace_bytes")
    ws = torch.empty(max(int(need.value), 256), dtype=torch.uint8, device=w.device)
    if out is None:
        out = torch.empty_like(w)
    ids = torch.empty((w.shape[0], w.shape[1]), dtype=torch.int8, device=w.device)
    pats = (ctypes.c_uint16 * len(patterns))(*patterns)
    _check(lib().pconv_project(ctypes.c_void_p(w.data_ptr()), n, pats, len(patterns), float(keep),
                               ctypes.c_void_p(out.data_ptr()), ctypes.c_void_p(ids.data_ptr()),
                               ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream_ptr(stream)),
           "pconv_project")
    return out, ids


TRACE_WORDS = 14


def pconv_trace_read(handle):
    """The handle's trace words (development build of the library only)."""
    buf = (ctypes.c_ulonglong * TRACE_WORDS)()
    _check(lib().pconv_trace_read(handle, buf, TRACE_WORDS), "pconv_trace_read")
    return list(buf)


def pconv_plan_shape(c_out, c_in, kept, stride, storage, canonical, n, h, w, flags=0, with_workspace=False):
    """pconv_plan for a shape alone (host arithmetic; works without a GPU)."""
    p = Plan()
    _check(lib().pconv_plan_shape(c_out, c_in, int(kept), stride, storage, int(bool(canonical)), n, h, w,
                                  int(flags), int(bool(with_workspace)), ctypes.byref(p)), "pconv_plan_shape")
    return {k: int(getattr(p, k)) for k, _ in Plan._fields_}


def pconv_workspace_bytes(handle, n, h, w):
    b = ctypes.c_size_t(0)
    _check(lib().pconv_workspace_bytes(handle, n, h, w, ctypes.byref(b)), "pconv_workspace_bytes")
    return int(b.value)


def pconv_forward(handle, x, bias, y, flags=0, stream=None, workspace=None):
    """x, y: CUDA torch tensors (NCHW, contiguous); bias: CUDA fp32 tensor or None;
    workspace: zeroed CUDA uint8 tensor from pconv_workspace_bytes, or None."""
    if not (x.is_cuda and y.is_cuda and x.is_contiguous() and y.is_contiguous()):
        raise ValueError("x and y must be contiguous CUDA tensors")
    n, _, h, w = x.shape
    bp = None
    if bias is not None:
        if not (bias.is_cuda and bias.is_contiguous()) or bias.dtype.itemsize != 4:
            raise ValueError("bias must be a contiguous CUDA float32 tensor")
        bp = ctypes.c_void_p(bias.data_ptr())
    if workspace is not None:
        st = lib().pconv_forward_ws(handle, ctypes.c_void_p(x.data_ptr()), bp,
                                    ctypes.c_void_p(y.data_ptr()), n, h, w, int(flags),
                                    ctypes.c_void_p(workspace.data_ptr()), workspace.numel(),
                                    _stream_ptr(stream))
    else:
        st = lib().pconv_forward(handle, ctypes.c_void_p(x.data_ptr()), bp,
                                 ctypes.c_void_p(y.data_ptr()), n, h, w, int(flags),
                                 _stream_ptr(stream))
    _check(st, "pconv_forward")


STATIC_WS_BYTES = 8 << 20


def pconv_forward_static_ws(handle, x, bias, y, flags=0, stream=None):
    """pconv_forward_ws on the library's built-in scratch array: for callers that must not
    allocate device memory.  Raises PconvError(PCONV_ERR_WORKSPACE) if the shape needs more than
    STATIC_WS_BYTES.  Calls that overlap on the GPU race on the shared array."""
    if not (x.is_cuda and y.is_cuda and x.is_contiguous() and y.is_contiguous()):
        raise ValueError("x and y must be contiguous CUDA tensors")
    n, _, h, w = x.shape
    bp = ctypes.c_void_p(bias.data_ptr()) if bias is not None else None
    st = lib().pconv_forward_static_ws(handle, ctypes.c_void_p(x.data_ptr()), bp,
                                       ctypes.c_void_p(y.data_ptr()), n, h, w, int(flags),
                                       _stream_ptr(stream))
    _check(st, "pconv_forward_static_ws")


def pconv_maxpool2x2(x, y, stream=None):
    n, c, h, w = x.shape
    st = lib().pconv_maxpool2x2(ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(y.data_ptr()),
                                n, c, h, w, _storage_of(x), _stream_ptr(stream))
    _check(st, "pconv_maxpool2x2")


def pconv_stats(handle):
    s = Stats()
    _check(lib().pconv_stats(handle, ctypes.byref(s)), "pconv_stats")
    return s


def pconv_unpack(handle):
    s = pconv_stats(handle)
    w = np.empty((s.c_out, s.c_in, 3, 3), dtype=np.float32)
    _check(lib().pconv_unpack(handle, w.ctypes.data), "pconv_unpack")
    return w


def pconv_filter_order(handle):
    s = pconv_stats(handle)
    perm = np.empty(s.n_groups * s.group_size, dtype=np.int32)
    _check(lib().pconv_filter_order(handle, perm.ctypes.data), "pconv_filter_order")
    return perm


def pconv_device_status(handle):
    where = ctypes.c_int(0)
    st = lib().pconv_device_status(handle, ctypes.byref(where))
    return st, where.value


class Layer:
    """One packed layer: owns the handle, allocates outputs with torch."""

    def __init__(self, w_oihw, patterns, stride=1, storage=F32, bias=None, strict4=False):
        import torch
        self.handle = pconv_pack(w_oihw, patterns, stride, storage, STRICT4 if strict4 else 0)
        self.stride, self.storage = stride, storage
        self.c_out, self.c_in = int(w_oihw.shape[0]), int(w_oihw.shape[1])
        self.bias = None
        if bias is not None:
            self.bias = torch.as_tensor(np.ascontiguousarray(bias, dtype=np.float32)).cuda()

    def out_shape(self, x_shape):
        n, _, h, w = x_shape
        return (n, self.c_out, (h - 1) // self.stride + 1, (w - 1) // self.stride + 1)

    def workspace(self, x_shape):
        """A zeroed workspace for inputs of this shape (cached), or None if never needed."""
        import torch
        n, _, h, w = x_shape
        need = pconv_workspace_bytes(self.handle, n, h, w)
        if need == 0:
            return None
        ws = getattr(self, "_ws", None)
        if ws is None or ws.numel() < need:
            ws = self._ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
        return ws

    def forward(self, x, relu=True, kernel=0, out=None, split=False, pool=False):
        import torch
        if out is None:
            n, c, h, w = self.out_shape(x.shape)
            shape = (n, c, h // 2, w // 2) if pool else (n, c, h, w)
            out = torch.empty(shape, dtype=x.dtype, device=x.device)
        ws = self.workspace(x.shape) if split else None
        pconv_forward(self.handle, x, self.bias, out,
                      (RELU if relu else 0) | (POOL2X2 if pool else 0) | kernel, workspace=ws)
        return out

    def stats(self):
        return pconv_stats(self.handle)

    def unpack(self):
        return pconv_unpack(self.handle)

    def close(self):
        if self.handle is not None:
            pconv_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Stack:
    """A chain of Layers (+ optional 2x2 max-pools) for a fixed input shape."""

    def __init__(self, layers, pool_after, n, h, w, flags=RELU):
        self.layers = list(layers)          # keeps handles and biases alive
        k = len(self.layers)
        hs = (ctypes.c_void_p * k)(*[l.handle for l in self.layers])
        bs = (ctypes.c_void_p * k)(*[ctypes.c_void_p(l.bias.data_ptr()) if l.bias is not None
                                     else None for l in self.layers])
        ps = (ctypes.c_ubyte * k)(*[1 if p else 0 for p in pool_after])
        out = ctypes.c_void_p()
        _check(lib().pconv_stack_create(hs, bs, ps, k, n, h, w, int(flags), ctypes.byref(out)),
               "pconv_stack_create")
        self.ptr = out
        dims = [ctypes.c_int() for _ in range(4)]
        _check(lib().pconv_stack_out_shape(out, *[ctypes.byref(d) for d in dims]),
               "pconv_stack_out_shape")
        self.out_shape = tuple(d.value for d in dims)
        self.in_shape = (n, self.layers[0].c_in, h, w)

    def forward(self, x, y, stream=None):
        _check(lib().pconv_stack_forward(self.ptr, ctypes.c_void_p(x.data_ptr()),
                                         ctypes.c_void_p(y.data_ptr()), _stream_ptr(stream)),
               "pconv_stack_forward")

    def capture(self, x, y, stream):
        """Captures one forward x -> y into a CUDA graph (stream: a non-default torch stream)."""
        _check(lib().pconv_stack_capture(self.ptr, ctypes.c_void_p(x.data_ptr()),
                                         ctypes.c_void_p(y.data_ptr()), _stream_ptr(stream)),
               "pconv_stack_capture")

    def replay(self, stream=None):
        _check(lib().pconv_stack_replay(self.ptr, _stream_ptr(stream)), "pconv_stack_replay")

    def forward_host(self, x_host, y_host, stream=None):
        """x_host / y_host: CPU torch tensors or numpy arrays (pinned memory makes it async)."""
        xp = x_host.data_ptr() if hasattr(x_host, "data_ptr") else x_host.ctypes.data
        yp = y_host.data_ptr() if hasattr(y_host, "data_ptr") else y_host.ctypes.data
        _check(lib().pconv_stack_forward_host(self.ptr, ctypes.c_void_p(xp), ctypes.c_void_p(yp),
                                              _stream_ptr(stream)), "pconv_stack_forward_host")

    def launches(self):
        """Kernel launches of one forward (a run of layers in one persistent kernel counts once)."""
        k = ctypes.c_int(0)
        _check(lib().pconv_stack_launches(self.ptr, ctypes.byref(k)), "pconv_stack_launches")
        return k.value

    def status(self):
        """(status, wait id): PCONV_ERR_DEVICE_TIMEOUT if a kernel of this stack gave up a bounded
        wait since the last call; the call clears the record and the stack's workspace."""
        where = ctypes.c_int(0)
        st = lib().pconv_stack_status(self.ptr, ctypes.byref(where))
        return st, where.value

    def close(self):
        if self.ptr is not None:
            lib().pconv_stack_free(self.ptr)
            self.ptr = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
