"""ctypes binding of include/mona.h.  Names mirror the C entry points; nothing is computed here."""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MONA_LIBRARY selects another build of the same library (e.g. libmona_debug.so, the -DMONA_DEBUG build with index checks)
_LIB_PATH = os.environ.get("MONA_LIBRARY") or os.path.join(_HERE, "libmona.so")

STATUS_NAMES = {0: "MONA_OK", 1: "MONA_ERR_INVALID_ARG", 2: "MONA_ERR_UNSUPPORTED_SHAPE", 3: "MONA_ERR_ALIGNMENT",
                4: "MONA_ERR_CUDA", 5: "MONA_ERR_TIMEOUT", 6: "MONA_ERR_NONFINITE", 7: "MONA_ERR_ARCH",
                8: "MONA_ERR_BUFFER_TOO_SMALL", 9: "MONA_ERR_BOUNDS", 10: "MONA_ERR_NOT_BUILT"}
TRACE_ROWS, TRACE_SLOTS = 160, 64       # MONA_TRACE_ROWS, MONA_TRACE_SLOTS
MONA_F32, MONA_BF16 = 0, 1
MONA_STATE_COMBINED = 2      # single auxiliary buffer Z = beta_a A - (1 - beta_a) G


class MonaError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {detail}")


class MatrixDesc(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("batch", C.c_int64), ("batch_stride", C.c_int64),
                ("grad_dtype", C.c_int32), ("state_dtype", C.c_int32)]


class Hparams(C.Structure):
    _fields_ = [("lr", C.c_double), ("momentum", C.c_double), ("accel_beta", C.c_double), ("accel_alpha", C.c_double),
                ("weight_decay", C.c_double), ("ns_a", C.c_double), ("ns_b", C.c_double), ("ns_c", C.c_double),
                ("norm_eps", C.c_double), ("scale_value", C.c_double), ("ns_steps", C.c_int32), ("scale_mode", C.c_int32),
                ("ns_precision", C.c_int32), ("algorithm", C.c_int32)]


class Options(C.Structure):
    """mona_options: per-handle tuning knobs (see include/mona.h)."""
    _fields_ = [("chunk_budget_bytes", C.c_size_t), ("chunk_overlap", C.c_int32), ("fuse_update", C.c_int32),
                ("ns_delay", C.c_int32), ("macro_tile_min_k", C.c_int32), ("reserved", C.c_int32 * 4)]


_lib = None


def lib() -> C.CDLL:
    """Loads libmona.so (once).  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2605_26842_b200.build` "
                          "(needs nvcc; the library targets sm_100a and has no CPU fallback)")
    L = C.CDLL(_LIB_PATH)
    vp, vpp = C.c_void_p, C.POINTER(C.c_void_p)
    L.mona_default_hparams.argtypes = [C.POINTER(Hparams)]
    L.mona_set_chunk_budget.argtypes = [C.c_size_t]
    L.mona_set_chunk_overlap.argtypes = [C.c_int]
    L.mona_query_sizes.argtypes = [C.POINTER(MatrixDesc), C.c_int64, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.mona_default_options.argtypes = [C.POINTER(Options)]
    L.mona_query_sizes_opt.argtypes = [C.POINTER(MatrixDesc), C.c_int64, C.POINTER(Options), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.mona_create_opt.argtypes = [C.POINTER(vp), C.POINTER(MatrixDesc), C.c_int64, C.POINTER(Options), vp, C.c_size_t, vp, C.c_size_t, C.c_int]
    L.mona_last_ns_useful_flops.argtypes = [vp, C.POINTER(C.c_double)]
    L.mona_trace_read.argtypes = [C.POINTER(C.c_ulonglong), C.c_size_t, C.c_int]
    L.mona_work_order.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_uint32), C.c_uint32, C.c_uint32,
                                  C.POINTER(C.c_int32), C.c_size_t, C.POINTER(C.c_size_t)]
    L.mona_create.argtypes = [C.POINTER(vp), C.POINTER(MatrixDesc), C.c_int64, vp, C.c_size_t, vp, C.c_size_t, C.c_int]
    L.mona_step.argtypes = [vp, C.POINTER(Hparams), vpp, vpp, vp]
    L.mona_step_ex.argtypes = [vp, C.POINTER(Hparams), vpp, vpp, vpp, C.c_uint32, vp]
    L.mona_step_host.argtypes = [vp, C.POINTER(Hparams), vpp, vpp, vpp, vpp, vp]
    L.mona_poll_status.argtypes = [vp, vp, C.POINTER(C.c_int64)]
    L.mona_selftest_timeout.argtypes = [vp, vp]
    L.mona_selftest_timeout.restype = C.c_int
    L.mona_state_layout.argtypes = [vp, C.c_int64, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.mona_last_launch_count.argtypes = [vp]
    L.mona_last_launch_count.restype = C.c_int64
    L.mona_last_ns_flops.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    L.mona_last_error.argtypes = [vp]
    L.mona_last_error.restype = C.c_char_p
    L.mona_destroy.argtypes = [vp]
    L.mona_destroy.restype = None
    for name in ("mona_default_hparams", "mona_set_chunk_budget", "mona_set_chunk_overlap", "mona_query_sizes", "mona_create", "mona_step",
                 "mona_step_ex", "mona_step_host", "mona_poll_status", "mona_state_layout", "mona_last_ns_flops",
                 "mona_default_options", "mona_query_sizes_opt", "mona_create_opt", "mona_last_ns_useful_flops", "mona_trace_read", "mona_work_order"):
        getattr(L, name).restype = C.c_int
    _lib = L
    return L


def work_order(n_matrices: int, delay: int, items_per_phase: Sequence[int], start: int = 0, stride: int = 1, capacity: Optional[int] = None):
    """mona_work_order(): (matrix, phase, item) of the kernel's work items start, start + stride, ... as a list of tuples."""
    P = len(items_per_phase)
    if capacity is None:
        capacity = (n_matrices * sum(items_per_phase) - start + stride - 1) // stride if n_matrices * sum(items_per_phase) > start else 0
    ipp = (C.c_uint32 * max(1, P))(*items_per_phase)
    out = (C.c_int32 * (3 * max(1, capacity)))()
    n = C.c_size_t(0)
    st = lib().mona_work_order(n_matrices, P, delay, ipp, start, stride, out, capacity, C.byref(n))
    if st:
        raise MonaError(st, "mona_work_order")
    return [(out[3 * i], out[3 * i + 1], out[3 * i + 2]) for i in range(n.value)]


def trace_read(reset: bool = True, rows: int = TRACE_ROWS):
    """mona_trace_read(): the profiling build's table as a list of `rows` lists of TRACE_SLOTS integers (row = CTA).
    Raises MonaError(MONA_ERR_NOT_BUILT) unless the loaded library was compiled with -DMONA_TRACE."""
    buf = (C.c_ulonglong * (rows * TRACE_SLOTS))()
    st = lib().mona_trace_read(buf, rows, 1 if reset else 0)
    if st:
        raise MonaError(st, "mona_trace_read")
    return [list(buf[r * TRACE_SLOTS:(r + 1) * TRACE_SLOTS]) for r in range(rows)]


def default_hparams(**overrides) -> Hparams:
    hp = Hparams()
    st = lib().mona_default_hparams(C.byref(hp))
    if st:
        raise MonaError(st)
    for k, v in overrides.items():
        if not hasattr(hp, k):
            raise AttributeError(k)
        setattr(hp, k, v)
    return hp


def default_options(**overrides) -> Options:
    opt = Options()
    st = lib().mona_default_options(C.byref(opt))
    if st:
        raise MonaError(st)
    for k, v in overrides.items():
        if not hasattr(opt, k):
            raise AttributeError(k)
        setattr(opt, k, v)
    return opt


def set_chunk_budget(nbytes: int) -> None:
    st = lib().mona_set_chunk_budget(nbytes)
    if st:
        raise MonaError(st, "chunk budget must be at least 1 MiB")


def set_chunk_overlap(enabled: bool) -> None:
    st = lib().mona_set_chunk_overlap(1 if enabled else 0)
    if st:
        raise MonaError(st, "mona_set_chunk_overlap")


def _desc_array(descs: Sequence[MatrixDesc]):
    arr = (MatrixDesc * len(descs))()
    for i, d in enumerate(descs):
        arr[i] = d
    return arr


def query_sizes(descs: Sequence[MatrixDesc], options: Optional[Options] = None):
    sb, wb = C.c_size_t(0), C.c_size_t(0)
    st = lib().mona_query_sizes_opt(_desc_array(descs), len(descs), None if options is None else C.byref(options),
                                    C.byref(sb), C.byref(wb))
    if st:
        raise MonaError(st, "mona_query_sizes")
    return sb.value, wb.value


def _ptr_array(tensors: Sequence[Optional[torch.Tensor]]):
    arr = (C.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = None if t is None else t.data_ptr()
    return arr


class MonaOptimizer:
    """Owns the state and workspace tensors (torch device memory) and a mona_handle.

    `params[i]` is an fp32 CUDA tensor of shape (batch, rows, cols) or (rows, cols), contiguous;
    `grads[i]` has the same shape in fp32 or bf16.  step() enqueues one optimizer step on the current
    torch stream."""

    def __init__(self, params: Sequence[torch.Tensor], grad_dtype=torch.float32, device: Optional[int] = None,
                 state_dtype=torch.float32, options: Optional[Options] = None):
        L = lib()
        self.descs: List[MatrixDesc] = []
        for p in params:
            if p.dtype != torch.float32 or not p.is_contiguous() or p.dim() not in (2, 3):
                raise ValueError("parameters must be contiguous fp32 tensors of shape (rows, cols) or (batch, rows, cols)")
            batch = p.shape[0] if p.dim() == 3 else 1
            rows, cols = p.shape[-2], p.shape[-1]
            self.descs.append(MatrixDesc(rows, cols, batch, rows * cols, MONA_BF16 if grad_dtype == torch.bfloat16 else MONA_F32,
                                         state_dtype if isinstance(state_dtype, int) else
                                         (MONA_BF16 if state_dtype == torch.bfloat16 else MONA_F32)))
        self.device = torch.cuda.current_device() if device is None else device
        self.grad_dtype = grad_dtype
        self.options = options if options is not None else default_options()
        sb, wb = query_sizes(self.descs, self.options)
        dev = torch.device("cuda", self.device)
        self.state = torch.empty(sb, dtype=torch.uint8, device=dev)
        self.workspace = torch.empty(wb, dtype=torch.uint8, device=dev)
        self._h = C.c_void_p()
        st = L.mona_create_opt(C.byref(self._h), _desc_array(self.descs), len(self.descs), C.byref(self.options),
                               self.state.data_ptr(), sb, self.workspace.data_ptr(), wb, self.device)
        if st:
            msg = L.mona_last_error(self._h).decode() if self._h else ""
            L.mona_destroy(self._h)
            self._h = None
            raise MonaError(st, msg)

    # -- helpers ---------------------------------------------------------------------------------
    def _check(self, st: int):
        if st:
            raise MonaError(st, lib().mona_last_error(self._h).decode())

    def _stream(self):
        return C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)

    # -- C entry points --------------------------------------------------------------------------
    def step(self, hp: Hparams, params: Sequence[torch.Tensor], grads: Sequence[torch.Tensor]):
        self._check(lib().mona_step(self._h, C.byref(hp), _ptr_array(params), _ptr_array(grads), self._stream()))

    def step_ex(self, hp: Hparams, params, grads, o_out=None, phase_mask: int = 7):
        o_arr = None if o_out is None else _ptr_array(o_out)
        self._check(lib().mona_step_ex(self._h, C.byref(hp), _ptr_array(params), _ptr_array(grads), o_arr, phase_mask,
                                       self._stream()))

    def step_host(self, hp: Hparams, params, grads, grads_host, params_host):
        self._check(lib().mona_step_host(self._h, C.byref(hp), _ptr_array(params), _ptr_array(grads),
                                         _ptr_array(grads_host), _ptr_array(params_host), self._stream()))

    def poll_status(self):
        """Synchronises the current stream; returns (status code, first bad matrix index or -1)."""
        bad = C.c_int64(-1)
        st = lib().mona_poll_status(self._h, self._stream(), C.byref(bad))
        return st, bad.value

    def selftest_timeout(self):
        """Enqueues the launch whose wait must run out; poll_status() then reports MONA_ERR_TIMEOUT once."""
        self._check(lib().mona_selftest_timeout(self._h, self._stream()))

    def state_layout(self, desc: int):
        a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
        self._check(lib().mona_state_layout(self._h, desc, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def state_views(self, desc: int):
        """Views (batch, rows, cols) of M, A, G_prev of descriptor `desc` inside the state block: M fp32,
        A and G_prev in the descriptor's state dtype.  In the single-buffer format the second view is Z and
        the third is None."""
        d = self.descs[desc]
        n = d.batch * d.rows * d.cols
        aux = torch.bfloat16 if d.state_dtype == MONA_BF16 else torch.float32
        offs = self.state_layout(desc)
        out = []
        for off, dt in zip(offs, (torch.float32, aux, aux)):
            if off == C.c_size_t(-1).value:
                out.append(None)
                continue
            sz = 2 if dt == torch.bfloat16 else 4
            out.append(self.state[off: off + n * sz].view(dt).view(d.batch, d.rows, d.cols))
        return tuple(out)

    def last_launch_count(self) -> int:
        return lib().mona_last_launch_count(self._h)

    def last_ns_flops(self):
        e, d = C.c_double(), C.c_double()
        self._check(lib().mona_last_ns_flops(self._h, C.byref(e), C.byref(d)))
        return e.value, d.value

    def last_ns_useful_flops(self) -> float:
        u = C.c_double()
        self._check(lib().mona_last_ns_useful_flops(self._h, C.byref(u)))
        return u.value

    def close(self):
        if getattr(self, "_h", None):
            lib().mona_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def prologue_noalloc(grad: torch.Tensor, M: torch.Tensor, A: torch.Tensor, G_prev: torch.Tensor,
                     inv_norm_out: torch.Tensor, hp: Hparams, xhat: Optional[torch.Tensor] = None):
    """mona_prologue_noalloc on the current device and current torch stream: the fused prologue for one
    (rows, cols) matrix for callers that cannot allocate device memory.  Raises MonaError with the
    library's message on refusal (e.g. a matrix beyond the built-in scratch limit)."""
    L = lib()
    fn = L.mona_prologue_noalloc
    fn.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                   C.POINTER(Hparams), C.c_void_p, C.c_char_p, C.c_size_t]
    fn.restype = C.c_int
    rows, cols = grad.shape[-2], grad.shape[-1]
    err = C.create_string_buffer(256)
    st = fn(grad.data_ptr(), MONA_BF16 if grad.dtype == torch.bfloat16 else MONA_F32, M.data_ptr(), A.data_ptr(),
            G_prev.data_ptr(), None if xhat is None else xhat.data_ptr(), inv_norm_out.data_ptr(), rows, cols, C.byref(hp),
            C.c_void_p(torch.cuda.current_stream().cuda_stream), err, len(err))
    if st:
        raise MonaError(st, err.value.decode())
