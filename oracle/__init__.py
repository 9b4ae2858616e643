"""CPU oracle for the TNG step -- TEST INFRASTRUCTURE, not product code.

A thin ctypes layer over ``tng_oracle.c`` (the plain C statement of the method,
arXiv 1901.08227 Sections 3-3.2 and Algorithm 1).  Only tests, the smoke check
and a benchmark's CPU-baseline leg may import this package; the CUDA library
never does, and shares no code with it.

Parity status: stage functions are pinned by ``tests/test_oracle_*.py`` to facts
outside the oracle; the composed multi-step trajectory is "parity unpinned"
(the paper prints no worked numeric example).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tng_oracle.c"
_HDR = _HERE / "tng_oracle.h"
_LIB = _HERE / "libtng_oracle.so"

CODEC_SIGN1, CODEC_TERN2, CODEC_QSGD4 = 1, 2, 4
NORM_NONE, NORM_DIFF, NORM_QUOT, NORM_COMB, NORM_MEAN = 0, 1, 2, 3, 4
SCALE_ABSMAX, SCALE_L2 = 0, 1
FUSE_AUTO, FUSE_LAST, FUSE_MEAN, FUSE_LSQ, FUSE_HINDSIGHT = 0, 1, 2, 3, 4
OPT_BLOCK, OPT_QSGD_LEVELS, OPT_SCALE_KIND, OPT_SEED_LO, OPT_SEED_HI, OPT_FUSE_MODE, OPT_RIDGE, OPT_QUOT_EPS, OPT_REF_EVERY = range(9)
TILE = 128


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no fast-math, no fp contraction)."""
    stale = (not _LIB.exists()) or _LIB.stat().st_mtime < max(_SRC.stat().st_mtime, _HDR.stat().st_mtime)
    if force or stale:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
               "-fPIC", "-Wall", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None

_f32p = C.POINTER(C.c_float)
_f64p = C.POINTER(C.c_double)
_u32p = C.POINTER(C.c_uint32)


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(str(_LIB))
        L.tngo_uniform24.restype = C.c_float
        L.tngo_coord_uniform.restype = C.c_float
        L.tngo_coord_uniform.argtypes = [C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint32, C.c_uint32]
        for name in ("tngo_num_tiles", "tngo_words_per_worker", "tngo_num_blocks"):
            getattr(L, name).restype = C.c_uint64
        L.tngo_num_tiles.argtypes = [C.c_uint64]
        L.tngo_words_per_worker.argtypes = [C.c_uint64, C.c_int]
        L.tngo_num_blocks.argtypes = [C.c_uint64, C.c_uint64]
        L.tngo_fuse_stats.argtypes = [C.POINTER(_f32p), C.c_int, C.c_uint64, _f32p, C.c_int, C.c_uint64, _f64p, _f64p, _f64p]
        L.tngo_fuse_solve.argtypes = [_f64p, _f64p, C.c_int, C.c_double, _f64p, _f32p]
        L.tngo_fuse_solve_hindsight.argtypes = [_f64p, C.c_int, C.c_double, _f64p, _f32p]
        L.tngo_combine.argtypes = [C.POINTER(_f32p), _f32p, C.c_int, C.c_uint64, _f32p]
        L.tngo_quot_den.argtypes = [_f32p, C.c_uint64, C.c_float, _f32p]
        L.tngo_encode.argtypes = [_f32p, C.c_int, C.c_uint64, C.c_uint64, _f32p, C.c_int, C.c_float, C.c_int,
                                  C.c_uint64, C.c_int, C.c_int, C.c_uint32, C.c_uint32, C.c_uint32, _u32p, _f32p]
        L.tngo_encode_at.argtypes = [_f32p, C.c_int, C.c_uint64, C.c_uint64, _f32p, _f32p, _f32p, C.c_int, C.c_float, C.c_int,
                                     C.c_uint64, C.c_int, C.c_int, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64, _u32p, _f32p]
        L.tngo_decode_aggregate.argtypes = [_u32p, _f32p, C.c_int, C.c_uint64, _f32p, C.c_int, C.c_float, C.c_int,
                                            C.c_uint64, C.c_int, _f32p]
        L.tngo_decode_aggregate2.argtypes = [_u32p, _f32p, C.c_int, C.c_uint64, _f32p, _f32p, _f32p, C.c_int, C.c_float, C.c_int,
                                             C.c_uint64, C.c_int, _f32p]
        L.tngo_magnitude_reference.argtypes = [C.POINTER(_f32p), C.c_int, C.c_uint64, _f32p]
        L.tngo_row_mean.argtypes = [_f32p, C.c_uint64]
        L.tngo_row_mean.restype = C.c_float
        L.tngo_mean_of_means.argtypes = [_f32p, C.c_int]
        L.tngo_mean_of_means.restype = C.c_float
        L.tngo_dequant.restype = C.c_float
        L.tngo_dequant.argtypes = [C.c_int, C.c_int, C.c_uint32, C.c_float]
        L.tngo_cnz.restype = C.c_double
        L.tngo_cnz.argtypes = [_f32p, C.c_int, C.c_uint64, C.c_uint64, _f32p]
        L.tngo_bits_per_coord.restype = C.c_double
        L.tngo_bits_per_coord.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_uint64]
        L.tngo_create.restype = C.c_void_p
        L.tngo_create.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_int]
        L.tngo_destroy.argtypes = [C.c_void_p]
        L.tngo_set_option.argtypes = [C.c_void_p, C.c_int, C.c_double]
        L.tngo_push_reference.argtypes = [C.c_void_p, _f32p]
        L.tngo_step.argtypes = [C.c_void_p, _f32p, C.c_uint64, _f32p]
        L.tngo_stage_fuse.argtypes = [C.c_void_p, _f32p, C.c_uint64]
        L.tngo_stage_encode.argtypes = [C.c_void_p, _f32p, C.c_uint64]
        L.tngo_stage_decode_push.argtypes = [C.c_void_p, _f32p]
        for name, rt in (("tngo_ref", _f32p), ("tngo_ref2", _f32p), ("tngo_codes", _u32p), ("tngo_scales", _f32p),
                         ("tngo_means", _f32p), ("tngo_alpha", _f32p), ("tngo_gram", _f64p)):
            getattr(L, name).restype = rt
            getattr(L, name).argtypes = [C.c_void_p]
        L.tngo_history.restype = _f32p
        L.tngo_history.argtypes = [C.c_void_p, C.c_int]
        L.tngo_hist_count.argtypes = [C.c_void_p]
        L.tngo_step_count.restype = C.c_uint32
        L.tngo_step_count.argtypes = [C.c_void_p]
        L.tngo_solver_fallback.argtypes = [C.c_void_p]
        L.tngo_logistic_loss.restype = C.c_double
        L.tngo_logistic_loss.argtypes = [_f32p, _f32p, C.c_uint64, C.c_uint64, _f32p, C.c_double]
        L.tngo_logistic_grad.argtypes = [_f32p, _f32p, C.c_uint64, C.c_uint64, _f32p, C.c_double, _f32p]
        L.tngo_rosenbrock_value.restype = C.c_double
        L.tngo_rosenbrock_value.argtypes = [_f32p, C.c_uint64]
        L.tngo_rosenbrock_grad.argtypes = [_f32p, C.c_uint64, _f32p, C.c_int, C.c_uint64, _f32p]
        L.tngo_sgd_update.argtypes = [_f32p, _f32p, C.c_uint64, C.c_float]
        L.tngo_max_threads.restype = C.c_int
        L.tngo_set_threads.argtypes = [C.c_int]
        _lib = L
    return _lib


def omp_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    return int(lib().tngo_max_threads())


def set_threads(n: int) -> None:
    """Threads for the oracle's parallel loops from now on (timing only: no result depends on it)."""
    lib().tngo_set_threads(int(n))


# --------------------------------------------------------------------------- helpers
def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_f32p)


def _ptr_f32(a):
    return None if a is None else a.ctypes.data_as(_f32p)


def _rows(grads):
    g = np.asarray(grads, dtype=np.float32)
    assert g.ndim == 2 and g.strides[1] == 4
    return g, g.shape[0], g.strides[0] // 4


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    out = (C.c_uint32 * 4)()
    lib().tngo_philox4x32_10(c, k, out)
    return [int(x) for x in out]


def uniform24(x):
    return float(lib().tngo_uniform24(C.c_uint32(int(x))))


def coord_uniform(seed_lo, seed_hi, i, m, t):
    return float(lib().tngo_coord_uniform(seed_lo, seed_hi, i, m, t))


def num_tiles(d):
    return int(lib().tngo_num_tiles(d))


def words_per_worker(d, codec):
    return int(lib().tngo_words_per_worker(d, codec))


def num_blocks(d, B):
    return int(lib().tngo_num_blocks(d, B))


def _hist_ptrs(hist):
    hs = [np.ascontiguousarray(h, dtype=np.float32) for h in hist]
    arr = (_f32p * max(len(hs), 1))(*[h.ctypes.data_as(_f32p) for h in hs])
    return hs, arr


def fuse_stats(hist, grads):
    """hist: list of k vectors, newest first.  Returns (G[k,k], c[k], gg)."""
    hs, arr = _hist_ptrs(hist)
    g, M, ld = _rows(grads)
    k, d = len(hs), g.shape[1]
    G = np.zeros((k, k), dtype=np.float64)
    c = np.zeros(k, dtype=np.float64)
    gg = C.c_double(0.0)
    lib().tngo_fuse_stats(arr, k, d, _ptr_f32(g), M, ld, G.ctypes.data_as(_f64p), c.ctypes.data_as(_f64p), C.byref(gg))
    return G, c, gg.value


def fuse_solve(G, c, ridge):
    G = np.ascontiguousarray(G, dtype=np.float64)
    c = np.ascontiguousarray(c, dtype=np.float64)
    k = len(c)
    a64 = np.zeros(k, dtype=np.float64)
    a32 = np.zeros(k, dtype=np.float32)
    flag = lib().tngo_fuse_solve(G.ctypes.data_as(_f64p), c.ctypes.data_as(_f64p), k, ridge,
                                 a64.ctypes.data_as(_f64p), _ptr_f32(a32))
    return a64, a32, int(flag)


def fuse_solve_hindsight(G, ridge):
    G = np.ascontiguousarray(G, dtype=np.float64)
    k = G.shape[0]
    a64 = np.zeros(k, dtype=np.float64)
    a32 = np.zeros(k, dtype=np.float32)
    flag = lib().tngo_fuse_solve_hindsight(G.ctypes.data_as(_f64p), k, ridge, a64.ctypes.data_as(_f64p), _ptr_f32(a32))
    return a64, a32, int(flag)


def combine(hist, alpha32):
    hs, arr = _hist_ptrs(hist)
    a, ap = _f32(alpha32)
    d = hs[0].shape[0]
    ref = np.zeros(d, dtype=np.float32)
    lib().tngo_combine(arr, ap, len(hs), d, _ptr_f32(ref))
    return ref


def quot_den(ref, quot_eps=2.0 ** -4):
    r, rp = _f32(ref)
    den = np.zeros_like(r)
    lib().tngo_quot_den(rp, r.shape[0], quot_eps, _ptr_f32(den))
    return den


def encode(grads, ref, norm, codec, B=128, s=7, scale_kind=SCALE_ABSMAX, seed=(0, 0), t=0, quot_eps=2.0 ** -4,
           coord_offset=0, ref2=None, means=None):
    """Returns (codes[M, words_per_worker] uint32, scales[M, num_blocks] float32).  With
    coord_offset = i0 the columns handed in are coordinates i0.. of a longer vector.
    NORM_MEAN: `means` are the workers' scalar references (row_means of the whole vectors);
    left out, they are taken from the rows handed in."""
    g, M, ld = _rows(grads)
    d = g.shape[1]
    r = None if ref is None else np.ascontiguousarray(ref, dtype=np.float32)
    r2 = None if ref2 is None else np.ascontiguousarray(ref2, dtype=np.float32)
    mu = None
    if norm == NORM_MEAN:
        mu = row_means(g) if means is None else np.ascontiguousarray(means, dtype=np.float32)
        assert mu.shape == (M,)
    codes = np.zeros((M, words_per_worker(d, codec)), dtype=np.uint32)
    scales = np.zeros((M, num_blocks(d, B)), dtype=np.float32)
    lib().tngo_encode_at(_ptr_f32(g), M, ld, d, _ptr_f32(r), _ptr_f32(r2), _ptr_f32(mu), norm, quot_eps, codec, B, s, scale_kind,
                         seed[0], seed[1], t, int(coord_offset), codes.ctypes.data_as(_u32p), _ptr_f32(scales))
    return codes, scales


def row_means(grads):
    """mean(g^m) of every row: the scalar references of NORM_MEAN (Section 3.1)."""
    g, M, ld = _rows(grads)
    d = g.shape[1]
    return np.array([lib().tngo_row_mean(_ptr_f32(g[m]), d) for m in range(M)], dtype=np.float32)


def mean_of_means(means):
    mu = np.ascontiguousarray(means, dtype=np.float32)
    return np.float32(lib().tngo_mean_of_means(_ptr_f32(mu), mu.shape[0]))


def decode_aggregate(codes, scales, d, ref, norm, codec, B=128, s=7, quot_eps=2.0 ** -4, ref2=None, means=None):
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    scales = np.ascontiguousarray(scales, dtype=np.float32)
    M = codes.shape[0]
    r = None if ref is None else np.ascontiguousarray(ref, dtype=np.float32)
    r2 = None if ref2 is None else np.ascontiguousarray(ref2, dtype=np.float32)
    mu = None if means is None else np.ascontiguousarray(means, dtype=np.float32)
    assert norm != NORM_MEAN or (mu is not None and mu.shape == (M,))
    out = np.zeros(d, dtype=np.float32)
    lib().tngo_decode_aggregate2(codes.ctypes.data_as(_u32p), _ptr_f32(scales), M, d, _ptr_f32(r), _ptr_f32(r2), _ptr_f32(mu), norm,
                                 quot_eps, codec, B, s, _ptr_f32(out))
    return out


def magnitude_reference(hist):
    """r'_d = (1/k) sum_j |h_j,d| (second reference of the combined form)."""
    hs, arr = _hist_ptrs(hist)
    d = hs[0].shape[0]
    ref2 = np.zeros(d, dtype=np.float32)
    lib().tngo_magnitude_reference(arr, len(hs), d, _ptr_f32(ref2))
    return ref2


def dequant(codec, s, symbol, R):
    return float(lib().tngo_dequant(codec, s, symbol, C.c_float(R)))


def cnz(grads, ref):
    g, M, ld = _rows(grads)
    r = None if ref is None else np.ascontiguousarray(ref, dtype=np.float32)
    return float(lib().tngo_cnz(_ptr_f32(g), M, ld, g.shape[1], _ptr_f32(r)))


def bits_per_coord(d, K, codec, B):
    return float(lib().tngo_bits_per_coord(d, K, codec, B))


class State:
    """The round of Algorithm 1 as a state machine (ring of past aggregates)."""

    def __init__(self, d, M, K, codec, norm, **options):
        self.d, self.M, self.K, self.codec, self.norm = d, M, K, codec, norm
        self._h = lib().tngo_create(d, M, K, codec, norm)
        if not self._h:
            raise ValueError("tngo_create rejected the arguments")
        self.B = 128
        names = {"block": OPT_BLOCK, "qsgd_levels": OPT_QSGD_LEVELS, "scale_kind": OPT_SCALE_KIND,
                 "seed_lo": OPT_SEED_LO, "seed_hi": OPT_SEED_HI, "fuse_mode": OPT_FUSE_MODE,
                 "ridge": OPT_RIDGE, "quot_eps": OPT_QUOT_EPS, "ref_every": OPT_REF_EVERY}
        for key, val in options.items():
            if lib().tngo_set_option(self._h, names[key], float(val)):
                raise ValueError(f"bad option {key}={val}")
            if key == "block":
                self.B = int(val)

    def close(self):
        if self._h:
            lib().tngo_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def push_reference(self, vec):
        v, vp = _f32(vec)
        assert v.shape == (self.d,)
        lib().tngo_push_reference(self._h, vp)

    def step(self, grads):
        g, M, ld = _rows(grads)
        assert M == self.M and g.shape[1] == self.d
        out = np.zeros(self.d, dtype=np.float32)
        lib().tngo_step(self._h, _ptr_f32(g), ld, _ptr_f32(out))
        return out

    def fuse(self, grads):
        g, M, ld = _rows(grads)
        lib().tngo_stage_fuse(self._h, _ptr_f32(g), ld)

    def encode(self, grads):
        g, M, ld = _rows(grads)
        lib().tngo_stage_encode(self._h, _ptr_f32(g), ld)

    def decode_push(self):
        out = np.zeros(self.d, dtype=np.float32)
        lib().tngo_stage_decode_push(self._h, _ptr_f32(out))
        return out

    @property
    def k(self):
        return int(lib().tngo_hist_count(self._h))

    @property
    def t(self):
        return int(lib().tngo_step_count(self._h))

    @property
    def fallback(self):
        return int(lib().tngo_solver_fallback(self._h))

    def ref(self):
        return np.ctypeslib.as_array(lib().tngo_ref(self._h), shape=(self.d,)).copy()

    def ref2(self):
        return np.ctypeslib.as_array(lib().tngo_ref2(self._h), shape=(self.d,)).copy()

    def means(self):
        return np.ctypeslib.as_array(lib().tngo_means(self._h), shape=(self.M,)).copy()

    def codes(self):
        w = words_per_worker(self.d, self.codec)
        return np.ctypeslib.as_array(lib().tngo_codes(self._h), shape=(self.M, w)).copy()

    def scales(self):
        nb = num_blocks(self.d, self.B)
        return np.ctypeslib.as_array(lib().tngo_scales(self._h), shape=(self.M, nb)).copy()

    def alpha(self):
        return np.ctypeslib.as_array(lib().tngo_alpha(self._h), shape=(16,)).copy()[: max(self.k, 1)]

    def gram(self):
        k = self.k
        raw = np.ctypeslib.as_array(lib().tngo_gram(self._h), shape=(16 * 16 + 17,)).copy()
        return raw[: k * k].reshape(k, k), raw[k * k: k * k + k], raw[k * k + k]

    def history(self, j):
        return np.ctypeslib.as_array(lib().tngo_history(self._h, j), shape=(self.d,)).copy()


def logistic_loss(X, b, w, lambda2):
    X = np.ascontiguousarray(X, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    n, d = X.shape
    return float(lib().tngo_logistic_loss(_ptr_f32(X), _ptr_f32(b), n, d, _ptr_f32(w), lambda2))


def logistic_grad(X, b, w, lambda2):
    X = np.ascontiguousarray(X, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    n, d = X.shape
    g = np.zeros(d, dtype=np.float32)
    lib().tngo_logistic_grad(_ptr_f32(X), _ptr_f32(b), n, d, _ptr_f32(w), lambda2, _ptr_f32(g))
    return g


def rosenbrock_value(x):
    x = np.ascontiguousarray(x, dtype=np.float32)
    return float(lib().tngo_rosenbrock_value(_ptr_f32(x), x.shape[0]))


def rosenbrock_grad(x, noise=None, M=1):
    x = np.ascontiguousarray(x, dtype=np.float32)
    d = x.shape[0]
    if noise is not None:
        noise = np.ascontiguousarray(noise, dtype=np.float32)
        M = noise.shape[0]
    grads = np.zeros((M, d), dtype=np.float32)
    lib().tngo_rosenbrock_grad(_ptr_f32(x), d, _ptr_f32(noise), M, d, _ptr_f32(grads))
    return grads


def sgd_update(w, v, eta):
    w = np.ascontiguousarray(w, dtype=np.float32).copy()
    v = np.ascontiguousarray(v, dtype=np.float32)
    lib().tngo_sgd_update(_ptr_f32(w), _ptr_f32(v), w.shape[0], C.c_float(eta))
    return w
