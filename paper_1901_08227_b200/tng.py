"""ctypes binding of libtng.so.  Names mirror ``include/tng.h``; the wrappers only
marshal arguments (tensor -> device pointer, current CUDA stream -> void*)."""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libtng.so"

CODEC_SIGN1, CODEC_TERN2, CODEC_QSGD4 = 1, 2, 4
NORM_NONE, NORM_DIFF, NORM_QUOT, NORM_COMB, NORM_MEAN = 0, 1, 2, 3, 4
SCALE_ABSMAX, SCALE_L2 = 0, 1
FUSE_AUTO, FUSE_LAST, FUSE_MEAN, FUSE_LSQ, FUSE_HINDSIGHT = 0, 1, 2, 3, 4
(OPT_BLOCK, OPT_QSGD_LEVELS, OPT_SCALE_KIND, OPT_SEED_LO, OPT_SEED_HI, OPT_FUSE_MODE, OPT_RIDGE, OPT_QUOT_EPS,
 OPT_TIMING, OPT_HOST_STAGING, OPT_REF_EVERY, OPT_COORD_OFFSET) = range(12)
(OK, ERR_INVALID_ARG, ERR_STATE, ERR_ALLOC, ERR_CUDA, ERR_NONFINITE, ERR_UNSUPPORTED) = range(7)
MAX_HISTORY = 16
TILE = 128

# every symbol include/tng.h declares
EXPORTS = [
    "tng_create", "tng_destroy", "tng_set_option", "tng_workspace_bytes", "tng_bind_workspace",
    "tng_push_reference", "tng_step", "tng_step_host", "tng_step_host_async", "tng_host_wait", "tng_fuse", "tng_encode", "tng_decode_aggregate",
    "tng_wire", "tng_wire_means", "tng_reference", "tng_history", "tng_stats", "tng_status_string", "tng_last_cuda_error",
    "tng_logistic_scratch_floats", "tng_logistic_grad", "tng_logistic_loss", "tng_rosenbrock_grad",
    "tng_rosenbrock_value", "tng_sgd_update", "tng_gram_static", "tng_state_bytes", "tng_save_state", "tng_load_state",
    "tng_selftest_bounded_wait", "tng_fuse_local", "tng_local_stats", "tng_local_stats_all", "tng_fuse_finish", "tng_encode_local", "tng_decode_commit",
]


class Stats(C.Structure):
    _fields_ = [
        ("d", C.c_uint64), ("M", C.c_uint32), ("K", C.c_uint32), ("k", C.c_uint32), ("fuse_mode", C.c_uint32),
        ("rounds", C.c_uint64), ("bits_per_coord", C.c_double),
        ("alpha", C.c_double * MAX_HISTORY), ("gram", C.c_double * (MAX_HISTORY * MAX_HISTORY)),
        ("rhs", C.c_double * MAX_HISTORY), ("grad_sq", C.c_double), ("cnz", C.c_double),
        ("solver_fallback", C.c_uint32), ("pipeline_error", C.c_uint32),
        ("nonfinite_scales", C.c_uint64), ("kernel_launches", C.c_uint64), ("timed_rounds", C.c_uint64),
        ("ms_dots", C.c_double), ("ms_solve", C.c_double), ("ms_combine", C.c_double),
        ("ms_encode", C.c_double), ("ms_decode", C.c_double),
    ]


class TngError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status})")


_lib = None


def lib():
    """Load libtng.so; there is no fallback if it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1901_08227_b200.build`")
        L = C.CDLL(str(LIB_PATH))
        vp, u64, u32, f32, f64 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_float, C.c_double
        L.tng_create.argtypes = [C.POINTER(vp), u64, u32, u32, C.c_int, C.c_int]
        L.tng_destroy.argtypes = [vp]
        L.tng_destroy.restype = None
        L.tng_set_option.argtypes = [vp, C.c_int, f64]
        L.tng_workspace_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
        L.tng_bind_workspace.argtypes = [vp, vp, C.c_size_t]
        L.tng_push_reference.argtypes = [vp, vp, vp]
        L.tng_step.argtypes = [vp, vp, u64, vp, vp]
        L.tng_step_host.argtypes = [vp, vp, u64, vp, vp]
        L.tng_step_host_async.argtypes = [vp, vp, u64, vp, vp]
        L.tng_host_wait.argtypes = [vp]
        L.tng_fuse.argtypes = [vp, vp, u64, vp]
        L.tng_encode.argtypes = [vp, vp, u64, vp, u32, vp]
        L.tng_decode_aggregate.argtypes = [vp, vp, vp, vp]
        L.tng_wire.argtypes = [vp, C.POINTER(vp), C.POINTER(C.c_size_t), C.POINTER(vp), C.POINTER(C.c_size_t)]
        L.tng_wire_means.argtypes = [vp, C.POINTER(vp)]
        L.tng_reference.argtypes = [vp, C.POINTER(vp)]
        L.tng_history.argtypes = [vp, u32, C.POINTER(vp)]
        L.tng_stats.argtypes = [vp, C.POINTER(Stats)]
        L.tng_status_string.argtypes = [C.c_int]
        L.tng_status_string.restype = C.c_char_p
        L.tng_last_cuda_error.argtypes = [vp]
        L.tng_logistic_scratch_floats.argtypes = [u64, u64]
        L.tng_logistic_scratch_floats.restype = C.c_size_t
        L.tng_logistic_grad.argtypes = [vp, vp, u64, u64, vp, f32, vp, vp, vp]
        L.tng_logistic_loss.argtypes = [vp, vp, u64, u64, vp, f32, vp, vp, vp]
        L.tng_rosenbrock_grad.argtypes = [vp, u64, vp, u32, u64, vp, vp]
        L.tng_rosenbrock_value.argtypes = [vp, u64, vp, vp]
        L.tng_sgd_update.argtypes = [vp, vp, u64, f32, vp]
        L.tng_state_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
        L.tng_save_state.argtypes = [vp, vp, C.c_size_t, C.POINTER(C.c_size_t), vp]
        L.tng_load_state.argtypes = [vp, vp, C.c_size_t, vp]
        L.tng_fuse_local.argtypes = [vp, vp, u64, u32, vp]
        L.tng_local_stats.argtypes = [vp, C.POINTER(vp), C.POINTER(C.c_size_t)]
        L.tng_local_stats_all.argtypes = [vp, C.POINTER(vp), C.POINTER(C.c_size_t)]
        L.tng_selftest_bounded_wait.argtypes = [vp, C.POINTER(C.c_uint32), vp]
        L.tng_fuse_finish.argtypes = [vp, vp]
        L.tng_encode_local.argtypes = [vp, vp, u64, u32, u32, u32, vp]
        L.tng_decode_commit.argtypes = [vp, vp, vp]
        L.tng_gram_static.argtypes = [C.POINTER(vp), u32, u64, vp, u32, u64, vp, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().tng_status_string(int(status)).decode()


def _check(status, what):
    if status != OK:
        raise TngError(status, what)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t, dtype=torch.float32):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor):
        return int(t)                                  # a raw device address
    if not t.is_cuda or t.dtype != dtype:
        raise TypeError(f"expected a CUDA {dtype} tensor")
    return t.data_ptr()


def _rows(grads):
    """(M, d) CUDA float tensor with unit column stride -> (pointer, ld)."""
    if not grads.is_cuda or grads.dtype != torch.float32 or grads.dim() != 2 or grads.stride(1) != 1:
        raise TypeError("grads must be an (M, d) CUDA float32 tensor with contiguous rows")
    return grads.data_ptr(), grads.stride(0)


class Context:
    """One TNG reducer: d coordinates, M simulated workers, a ring of K past aggregates."""

    _OPTS = {"block": OPT_BLOCK, "qsgd_levels": OPT_QSGD_LEVELS, "scale_kind": OPT_SCALE_KIND,
             "seed_lo": OPT_SEED_LO, "seed_hi": OPT_SEED_HI, "fuse_mode": OPT_FUSE_MODE, "ridge": OPT_RIDGE,
             "quot_eps": OPT_QUOT_EPS, "timing": OPT_TIMING, "host_staging": OPT_HOST_STAGING, "ref_every": OPT_REF_EVERY,
             "coord_offset": OPT_COORD_OFFSET}

    def __init__(self, d, M, K, codec, norm, workspace=None, **options):
        self.d, self.M, self.K, self.codec, self.norm = int(d), int(M), int(K), int(codec), int(norm)
        h = C.c_void_p()
        _check(lib().tng_create(C.byref(h), self.d, self.M, self.K, self.codec, self.norm), "tng_create")
        self._h = h
        for key, val in options.items():
            self.set_option(key, val)
        self._ws = None
        if workspace is not None:
            self.bind_workspace(workspace)

    # -- lifetime
    def close(self):
        if getattr(self, "_h", None):
            lib().tng_destroy(self._h)
            self._h = None
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_option(self, key, value):
        key = self._OPTS[key] if isinstance(key, str) else int(key)
        _check(lib().tng_set_option(self._h, key, float(value)), "tng_set_option")

    def workspace_bytes(self) -> int:
        n = C.c_size_t()
        _check(lib().tng_workspace_bytes(self._h, C.byref(n)), "tng_workspace_bytes")
        return n.value

    def bind_workspace(self, buf: torch.Tensor):
        if not buf.is_cuda or not buf.is_contiguous():
            raise TypeError("workspace must be a contiguous CUDA tensor")
        _check(lib().tng_bind_workspace(self._h, buf.data_ptr(), buf.numel() * buf.element_size()), "tng_bind_workspace")
        self._ws = buf                                  # keep it alive

    # -- the round
    def push_reference(self, vec):
        _check(lib().tng_push_reference(self._h, _dev(vec), _stream()), "tng_push_reference")

    def step(self, grads, out=None):
        p, ld = _rows(grads)
        _check(lib().tng_step(self._h, p, ld, _dev(out), _stream()), "tng_step")
        return out

    def step_host(self, grads_host: torch.Tensor, out_host: torch.Tensor):
        if grads_host.is_cuda or out_host.is_cuda or grads_host.dtype != torch.float32 or grads_host.stride(1) != 1:
            raise TypeError("step_host takes host float32 tensors")
        _check(lib().tng_step_host(self._h, grads_host.data_ptr(), grads_host.stride(0), out_host.data_ptr(), _stream()),
               "tng_step_host")
        return out_host

    def step_host_async(self, grads_host: torch.Tensor, out_host: torch.Tensor):
        """step_host without waiting: out_host holds the aggregate after host_wait()."""
        if grads_host.is_cuda or out_host.is_cuda or grads_host.dtype != torch.float32 or grads_host.stride(1) != 1:
            raise TypeError("step_host_async takes host float32 tensors")
        _check(lib().tng_step_host_async(self._h, grads_host.data_ptr(), grads_host.stride(0), out_host.data_ptr(), _stream()),
               "tng_step_host_async")
        return out_host

    def host_wait(self):
        _check(lib().tng_host_wait(self._h), "tng_host_wait")

    def state_bytes(self) -> int:
        n = C.c_size_t()
        _check(lib().tng_state_bytes(self._h, C.byref(n)), "tng_state_bytes")
        return n.value

    def save_state(self) -> torch.Tensor:
        """The context's state (ring, round counter, held reference) as a host byte tensor."""
        buf = torch.empty(self.state_bytes(), dtype=torch.uint8)
        used = C.c_size_t()
        _check(lib().tng_save_state(self._h, buf.data_ptr(), buf.numel(), C.byref(used), _stream()), "tng_save_state")
        return buf[: used.value].clone()

    def load_state(self, buf: torch.Tensor):
        if buf.is_cuda or buf.dtype != torch.uint8 or not buf.is_contiguous():
            raise TypeError("state must be a contiguous host uint8 tensor")
        _check(lib().tng_load_state(self._h, buf.data_ptr(), buf.numel(), _stream()), "tng_load_state")

    # -- rank-local stages (workers spread over several GPUs)
    def fuse_local(self, grads):
        p, ld = _rows(grads)
        _check(lib().tng_fuse_local(self._h, p, ld, grads.shape[0], _stream()), "tng_fuse_local")

    def local_stats(self) -> torch.Tensor:
        """Zero-copy float64 view of the block to all-reduce (sum) between fuse_local and fuse_finish."""
        p, n = C.c_void_p(), C.c_size_t()
        _check(lib().tng_local_stats(self._h, C.byref(p), C.byref(n)), "tng_local_stats")
        return _view(p.value, (n.value,), torch.float64)

    def selftest_bounded_wait(self) -> bool:
        """True when a wait on a barrier that nothing completes ended by its poll limit (as it must)."""
        out = C.c_uint32(0)
        _check(lib().tng_selftest_bounded_wait(self._h, C.byref(out), _stream()), "tng_selftest_bounded_wait")
        return out.value == 1

    def local_stats_all(self) -> torch.Tensor:
        """The same for ranks that hold slices of the coordinates: Gram, rhs and grad_sq (273 doubles)."""
        p, n = C.c_void_p(), C.c_size_t()
        _check(lib().tng_local_stats_all(self._h, C.byref(p), C.byref(n)), "tng_local_stats_all")
        return _view(p.value, (n.value,), torch.float64)

    def fuse_finish(self):
        _check(lib().tng_fuse_finish(self._h, _stream()), "tng_fuse_finish")

    def encode_local(self, grads, m_first, step):
        p, ld = _rows(grads)
        _check(lib().tng_encode_local(self._h, p, ld, int(m_first), grads.shape[0], int(step), _stream()), "tng_encode_local")

    def decode_commit(self, out=None):
        _check(lib().tng_decode_commit(self._h, _dev(out), _stream()), "tng_decode_commit")
        return out

    def wire_views(self):
        """Zero-copy views of the wire, (M, words) int32 codes and (M, scales) float32, for collectives."""
        cp, wpw, sp, spw = self.wire_pointers()
        return _view(cp, (self.M, wpw), torch.int32), _view(sp, (self.M, spw), torch.float32)

    def fuse(self, grads):
        p, ld = _rows(grads)
        _check(lib().tng_fuse(self._h, p, ld, _stream()), "tng_fuse")

    def encode(self, grads, ref=None, step=0):
        p, ld = _rows(grads)
        _check(lib().tng_encode(self._h, p, ld, _dev(ref), int(step), _stream()), "tng_encode")

    def decode_aggregate(self, out, ref=None):
        _check(lib().tng_decode_aggregate(self._h, _dev(ref), _dev(out), _stream()), "tng_decode_aggregate")
        return out

    # -- views (cloned into fresh tensors on the current stream, so they stay valid)
    def wire(self):
        cp, sp = C.c_void_p(), C.c_void_p()
        wpw, spw = C.c_size_t(), C.c_size_t()
        _check(lib().tng_wire(self._h, C.byref(cp), C.byref(wpw), C.byref(sp), C.byref(spw)), "tng_wire")
        codes = _view(cp.value, (self.M, wpw.value), torch.int32).clone()
        scales = _view(sp.value, (self.M, spw.value), torch.float32).clone()
        return codes, scales

    def wire_pointers(self):
        cp, sp = C.c_void_p(), C.c_void_p()
        wpw, spw = C.c_size_t(), C.c_size_t()
        _check(lib().tng_wire(self._h, C.byref(cp), C.byref(wpw), C.byref(sp), C.byref(spw)), "tng_wire")
        return cp.value, wpw.value, sp.value, spw.value

    def wire_means_view(self):
        """Zero-copy view of the M scalar references (NORM_MEAN), for collectives."""
        p = C.c_void_p()
        _check(lib().tng_wire_means(self._h, C.byref(p)), "tng_wire_means")
        return _view(p.value, (self.M,), torch.float32)

    def wire_means(self):
        return self.wire_means_view().clone()

    def reference(self):
        p = C.c_void_p()
        _check(lib().tng_reference(self._h, C.byref(p)), "tng_reference")
        return _view(p.value, (self.d,), torch.float32).clone()

    def history(self, j):
        p = C.c_void_p()
        _check(lib().tng_history(self._h, int(j), C.byref(p)), "tng_history")
        return _view(p.value, (self.d,), torch.float32).clone()

    def stats(self, raise_on_nonfinite=False) -> Stats:
        s = Stats()
        st = lib().tng_stats(self._h, C.byref(s))
        if st != OK and not (st == ERR_NONFINITE and not raise_on_nonfinite):
            raise TngError(st, "tng_stats")
        return s

    def last_cuda_error(self) -> int:
        return lib().tng_last_cuda_error(self._h)


class _DeviceView:
    """Zero-copy view of library-owned device memory for torch (CUDA array interface)."""

    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (int(ptr), False),
                                         "version": 2}


def _view(ptr, shape, dtype):
    typestr = {torch.float32: "<f4", torch.int32: "<i4", torch.float64: "<f8"}[dtype]
    return torch.as_tensor(_DeviceView(ptr, shape, typestr), device="cuda")


def gram_static(rows, grads, out):
    """tng_gram_static: Gram / rhs / mean squared norm of `rows` (list of (d,) CUDA tensors,
    newest first) against the (M, d) gradient rows, into `out` (k*k+k+1 float64 on the GPU).
    Allocates nothing on the device."""
    k = len(rows)
    arr = (C.c_void_p * max(k, 1))(*[_dev(r) for r in rows])
    p, ld = _rows(grads)
    d = rows[0].numel() if k else 0
    _check(lib().tng_gram_static(arr, k, d, p, grads.shape[0], ld, _dev(out, torch.float64), _stream()), "tng_gram_static")
    return out


# ---- producers -------------------------------------------------------------------------
def logistic_scratch_floats(n, d) -> int:
    return lib().tng_logistic_scratch_floats(int(n), int(d))


def logistic_grad(X, b, w, lambda2, grad, scratch):
    n, d = X.shape
    _check(lib().tng_logistic_grad(_dev(X), _dev(b), n, d, _dev(w), float(lambda2), _dev(grad), _dev(scratch), _stream()),
           "tng_logistic_grad")
    return grad


def logistic_loss(X, b, w, lambda2, loss, scratch):
    n, d = X.shape
    _check(lib().tng_logistic_loss(_dev(X), _dev(b), n, d, _dev(w), float(lambda2), _dev(loss, torch.float64),
                                   _dev(scratch), _stream()), "tng_logistic_loss")
    return loss


def rosenbrock_grad(x, noise, grads):
    p, ld = _rows(grads)
    if noise is not None:
        pn, ldn = _rows(noise)
        if ldn != ld:
            raise ValueError("noise and grads must share the row stride")
    else:
        pn = None
    _check(lib().tng_rosenbrock_grad(_dev(x), x.numel(), pn, grads.shape[0], ld, p, _stream()), "tng_rosenbrock_grad")
    return grads


def rosenbrock_value(x, value):
    _check(lib().tng_rosenbrock_value(_dev(x), x.numel(), _dev(value, torch.float64), _stream()), "tng_rosenbrock_value")
    return value


def sgd_update(w, v, eta):
    _check(lib().tng_sgd_update(_dev(w), _dev(v), w.numel(), float(eta), _stream()), "tng_sgd_update")
    return w
