"""numpy front end of the CPU oracle (oracle/dat_oracle.c).  TEST INFRASTRUCTURE.

Only tests, the smoke check and the CPU-baseline timing may import this package.
It does not import, and is not imported by, the CUDA path.

All arrays are host numpy arrays.  Element-indexed arrays (gradients, parameters,
codes ...) are addressed by the GLOBAL element index e of the flat parameter vector.
To run a few layers [l0, l1) of a very large problem without materialising the whole
vector, pass arrays that hold only elements offsets[l0] .. offsets[l1]-1 together
with ``window=True``: the wrapper then hands the C code base pointers shifted back
by offsets[l0] elements, so that the C code still indexes with the global e (the
random stream depends on the global index).
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

SCALE_SHARED_MAX = 0
RNG_BITS = (16, 23)      # resolutions of the quantizer's uniform number
SCALE_PER_WORKER = 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _declare(_lib)
    return _lib


_i64 = C.c_int64
_u64 = C.c_uint64
_u32 = C.c_uint32
_f32 = C.c_float
_int = C.c_int
_p = C.c_void_p


def _declare(L):
    L.dat_oracle_philox4x32_10.argtypes = [_p, _p, _p]
    L.dat_oracle_philox4x32_10.restype = None
    L.dat_oracle_random_word.argtypes = [_u64, _u64, _u32, _u64]
    L.dat_oracle_random_word.restype = _u32
    L.dat_oracle_uniform12.argtypes = [_u32]
    L.dat_oracle_uniform12.restype = _f32
    L.dat_oracle_uniform12_at.argtypes = [_u64, _u64, _u32, _u64, _int]
    L.dat_oracle_uniform12_at.restype = _f32
    L.dat_oracle_worker_norms.argtypes = [_i64, _p, _i64, _i64, _int, _p, _p]
    L.dat_oracle_worker_norms.restype = None
    L.dat_oracle_scales.argtypes = [_i64, _i64, _i64, _int, _int, _p, _p]
    L.dat_oracle_scales.restype = None
    L.dat_oracle_quantize.argtypes = [_i64, _p, _i64, _i64, _int, _int, _int, _p, _u64, _u64, _int, _p, _p, _p]
    L.dat_oracle_quantize.restype = None
    L.dat_oracle_requantize.argtypes = [_i64, _p, _i64, _i64, _int, _u64, _u64, _int, _u32, _p, _p, _p, _p, _p]
    L.dat_oracle_requantize.restype = None
    L.dat_oracle_level_plane_bytes.argtypes = [_i64, _int]
    L.dat_oracle_level_plane_bytes.restype = _i64
    L.dat_oracle_sign_plane_bytes.argtypes = [_i64]
    L.dat_oracle_sign_plane_bytes.restype = _i64
    L.dat_oracle_pack.argtypes = [_i64, _int, _p, _p, _p, _p]
    L.dat_oracle_pack.restype = None
    L.dat_oracle_unpack.argtypes = [_i64, _int, _p, _p, _p, _p]
    L.dat_oracle_unpack.restype = None
    L.dat_oracle_aggregate.argtypes = [_i64, _p, _i64, _i64, _int, _int, _int, _p, _p, _p, _p, _p]
    L.dat_oracle_aggregate.restype = None
    L.dat_oracle_average.argtypes = [_p, _i64, _i64, _int, _p, _p]
    L.dat_oracle_average.restype = None
    L.dat_oracle_lalr.argtypes = [_p, _i64, _i64, _p, _p, _p, _f32, _f32, _f32, _f32, _f32, _p]
    L.dat_oracle_lalr.restype = None
    L.dat_oracle_lamb.argtypes = [_p, _i64, _i64, _p, _p, _p, _p, _f32, _f32, _f32, _f32, _f32, _f32, _f32, _i64, _p]
    L.dat_oracle_lamb.restype = None
    L.dat_oracle_step.argtypes = [_i64, _p, _i64, _i64, _int, _int, _int, _p, _p, _p, _u64, _u64, _int, _p,
                                  _f32, _f32, _f32, _f32, _f32, _p, _p, _p]
    L.dat_oracle_step.restype = _int


# ---------------------------------------------------------------- marshalling

def _offsets(offsets):
    o = np.ascontiguousarray(offsets, dtype=np.int64)
    assert o.ndim == 1 and o.size >= 2 and o[0] == 0 and np.all(np.diff(o) > 0)
    return o


def _check(a, dtype, n=None):
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags.c_contiguous, (type(a), getattr(a, "dtype", None))
    if n is not None:
        assert a.size == n, (a.size, n)
    return a


def _addr(a, shift_elems=0):
    """Base address of array a moved back by shift_elems elements (see module doc)."""
    if a is None:
        return None
    return _p(a.ctypes.data - shift_elems * a.itemsize)


def _ptr_array(arrays, shift_elems=0):
    arr = (C.c_void_p * len(arrays))()
    for k, a in enumerate(arrays):
        arr[k] = a.ctypes.data - shift_elems * a.itemsize
    return arr


def _range(o, l0, l1, window):
    h = o.size - 1
    l0 = 0 if l0 is None else int(l0)
    l1 = h if l1 is None else int(l1)
    assert 0 <= l0 < l1 <= h
    n = int(o[l1] - o[l0]) if window else int(o[h])
    shift = int(o[l0]) if window else 0
    return h, l0, l1, n, shift


# ---------------------------------------------------------------- RNG

def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().dat_oracle_philox4x32_10(_addr(c), _addr(k), _addr(out))
    return out


def random_word(seed, step, worker, e):
    return int(lib().dat_oracle_random_word(int(seed), int(step), int(worker), int(e)))


def uniform12(w):
    """1 + u in [1, 2), u from the low 23 bits of w."""
    return float(lib().dat_oracle_uniform12(int(w) & 0xFFFFFFFF))


def uniform12_at(seed, step, worker, e, rng_bits):
    """The quantizer's 1 + u of element e: u has 23 bits (one Philox block per 4 elements) or
    16 bits (one block per 8 elements)."""
    assert rng_bits in RNG_BITS
    return float(lib().dat_oracle_uniform12_at(int(seed), int(step), int(worker), int(e), int(rng_bits)))


# ---------------------------------------------------------------- S1

def worker_norms(offsets, grads, l0=None, l1=None, window=False):
    """float32 [M, h]; rows outside [l0, l1) are left zero."""
    o = _offsets(offsets)
    h, l0, l1, n, shift = _range(o, l0, l1, window)
    grads = [_check(g, np.float32, n) for g in grads]
    M = len(grads)
    out = np.zeros((M, h), dtype=np.float32)
    lib().dat_oracle_worker_norms(h, _addr(o), l0, l1, M, _ptr_array(grads, shift), _addr(out))
    return out


def scales(norms, scale_mode=SCALE_SHARED_MAX, l0=None, l1=None):
    norms = _check(norms, np.float32)
    M, h = norms.shape
    l0 = 0 if l0 is None else l0
    l1 = h if l1 is None else l1
    out = np.zeros((M, h) if scale_mode == SCALE_PER_WORKER else (h,), dtype=np.float32)
    lib().dat_oracle_scales(h, l0, l1, M, scale_mode, _addr(norms), _addr(out))
    return out


# ---------------------------------------------------------------- S2

def quantize(offsets, grads, bits, seed, step, scales_, scale_mode=SCALE_SHARED_MAX,
             l0=None, l1=None, window=False, rng_bits=16):
    """Returns (level uint32 [M, n], neg uint8 [M, n])."""
    o = _offsets(offsets)
    h, l0, l1, n, shift = _range(o, l0, l1, window)
    assert bits in (1, 2, 4, 8, 16) and rng_bits in RNG_BITS
    grads = [_check(g, np.float32, n) for g in grads]
    M = len(grads)
    sc = _check(np.ascontiguousarray(scales_, dtype=np.float32), np.float32,
                M * h if scale_mode == SCALE_PER_WORKER else h)
    level = np.zeros((M, n), dtype=np.uint32)
    neg = np.zeros((M, n), dtype=np.uint8)
    lib().dat_oracle_quantize(h, _addr(o), l0, l1, M, bits, scale_mode, _ptr_array(grads, shift),
                              int(seed), int(step), int(rng_bits), _addr(sc),
                              _ptr_array(list(level), shift), _ptr_array(list(neg), shift))
    return level, neg


def requantize(offsets, g_hat, bits, seed, step, stream, rng_bits=16, scales_in=None):
    """Algorithm A1 Step 10: the server's Q(g_hat).  Returns (g_hat' float32 [d], scales float32 [h],
    level uint32 [d], neg uint8 [d]); the input is untouched.  `stream` = index of the random
    stream (M by convention)."""
    o = _offsets(offsets)
    h, d = o.size - 1, int(o[-1])
    assert bits in (1, 2, 4, 8, 16) and rng_bits in RNG_BITS
    gh = _check(g_hat, np.float32, d).copy()
    sc_in = None if scales_in is None else _check(np.ascontiguousarray(scales_in, dtype=np.float32), np.float32, h)
    sc = np.zeros(h, dtype=np.float32)
    level = np.zeros(d, dtype=np.uint32)
    neg = np.zeros(d, dtype=np.uint8)
    lib().dat_oracle_requantize(h, _addr(o), 0, h, bits, int(seed), int(step), int(rng_bits), int(stream),
                                _addr(sc_in), _addr(gh), _addr(sc), _addr(level), _addr(neg))
    return gh, sc, level, neg


# ---------------------------------------------------------------- S3

def level_plane_bytes(d, bits):
    return int(lib().dat_oracle_level_plane_bytes(int(d), int(bits)))


def sign_plane_bytes(d):
    return int(lib().dat_oracle_sign_plane_bytes(int(d)))


def pack(level, neg, bits):
    level = _check(level, np.uint32)
    d = level.size
    neg = _check(neg, np.uint8, d)
    lp = np.zeros(level_plane_bytes(d, bits), dtype=np.uint8)
    sp = np.zeros(sign_plane_bytes(d), dtype=np.uint8)
    lib().dat_oracle_pack(d, bits, _addr(level), _addr(neg), _addr(lp), _addr(sp))
    return lp, sp


def unpack(level_plane, sign_plane, d, bits):
    lp = _check(level_plane, np.uint8, level_plane_bytes(d, bits))
    sp = _check(sign_plane, np.uint8, sign_plane_bytes(d))
    level = np.zeros(d, dtype=np.uint32)
    neg = np.zeros(d, dtype=np.uint8)
    lib().dat_oracle_unpack(d, bits, _addr(lp), _addr(sp), _addr(level), _addr(neg))
    return level, neg


# ---------------------------------------------------------------- S4-S5

def aggregate(offsets, level, neg, scales_, bits, scale_mode=SCALE_SHARED_MAX,
              l0=None, l1=None, window=False):
    """Returns (code_sum int32 [n] or None in PER_WORKER mode, g_hat float32 [n])."""
    o = _offsets(offsets)
    h, l0, l1, n, shift = _range(o, l0, l1, window)
    level = _check(level, np.uint32)
    M = level.shape[0]
    assert level.shape == (M, n)
    neg = _check(neg, np.uint8, M * n)
    sc = _check(np.ascontiguousarray(scales_, dtype=np.float32), np.float32,
                M * h if scale_mode == SCALE_PER_WORKER else h)
    code_sum = None if scale_mode == SCALE_PER_WORKER else np.zeros(n, dtype=np.int32)
    g_hat = np.zeros(n, dtype=np.float32)
    lib().dat_oracle_aggregate(h, _addr(o), l0, l1, M, bits, scale_mode,
                               _ptr_array(list(level), shift), _ptr_array(list(neg.reshape(M, n)), shift),
                               _addr(sc), _addr(code_sum, shift), _addr(g_hat, shift))
    return code_sum, g_hat


def average(offsets, grads, l0=None, l1=None, window=False):
    o = _offsets(offsets)
    h, l0, l1, n, shift = _range(o, l0, l1, window)
    grads = [_check(g, np.float32, n) for g in grads]
    g_hat = np.zeros(n, dtype=np.float32)
    lib().dat_oracle_average(_addr(o), l0, l1, len(grads), _ptr_array(grads, shift), _addr(g_hat, shift))
    return g_hat


# ---------------------------------------------------------------- S6-S8

def lalr(offsets, theta, mom, g_hat, lr, momentum, weight_decay, c_l=0.0, c_u=10.0,
         l0=None, l1=None, window=False):
    """Returns (theta', m', norms float32 [h, 2] = (||theta_l||, ||u_l||)); inputs untouched."""
    o = _offsets(offsets)
    h, l0, l1, n, shift = _range(o, l0, l1, window)
    th = _check(theta, np.float32, n).copy()
    mo = _check(mom, np.float32, n).copy()
    gh = _check(g_hat, np.float32, n)
    norms = np.zeros((h, 2), dtype=np.float32)
    lib().dat_oracle_lalr(_addr(o), l0, l1, _addr(th, shift), _addr(mo, shift), _addr(gh, shift),
                          lr, momentum, weight_decay, c_l, c_u, _addr(norms))
    return th, mo, norms


def lamb(offsets, theta, mom, var, g_hat, t, lr, beta1=0.9, beta2=0.999, zeta=1e-6, weight_decay=0.0,
         c_l=0.0, c_u=10.0):
    """Algorithm A2 followed by Eq. upth.  Returns (theta', m', v', norms float32 [h, 2] = (||theta_l||, ||u_l||));
    inputs untouched.  t >= 1 is the iteration count of the bias corrections."""
    o = _offsets(offsets)
    h, d = o.size - 1, int(o[-1])
    assert t >= 1
    th = _check(theta, np.float32, d).copy()
    mo = _check(mom, np.float32, d).copy()
    va = _check(var, np.float32, d).copy()
    gh = _check(g_hat, np.float32, d)
    norms = np.zeros((h, 2), dtype=np.float32)
    lib().dat_oracle_lamb(_addr(o), 0, h, _addr(th), _addr(mo), _addr(va), _addr(gh),
                          lr, beta1, beta2, zeta, weight_decay, c_l, c_u, int(t), _addr(norms))
    return th, mo, va, norms


# ---------------------------------------------------------------- whole step

def step(offsets, theta, mom, grads, bits, seed, step_, lr, momentum, weight_decay,
         c_l=0.0, c_u=10.0, scale_mode=SCALE_SHARED_MAX, scales_in=None,
         l0=None, l1=None, window=False, want_code_sum=True, rng_bits=16):
    """One DAT outer-minimisation step.  Returns a dict with theta, mom (new arrays),
    code_sum (int32 or None), layer_norms [h, 2], scales."""
    o = _offsets(offsets)
    h, l0, l1, n, shift = _range(o, l0, l1, window)
    assert bits in (1, 2, 4, 8, 16, 32) and rng_bits in RNG_BITS
    th = _check(theta, np.float32, n).copy()
    mo = _check(mom, np.float32, n).copy()
    grads = [_check(g, np.float32, n) for g in grads]
    M = len(grads)
    n_scales = M * h if scale_mode == SCALE_PER_WORKER else h
    sin = None
    if scales_in is not None:
        sin = _check(np.ascontiguousarray(scales_in, dtype=np.float32).reshape(-1), np.float32, n_scales)
    have_sum = want_code_sum and bits != 32 and scale_mode == SCALE_SHARED_MAX
    code_sum = np.zeros(n, dtype=np.int32) if have_sum else None
    norms = np.zeros((h, 2), dtype=np.float32)
    sout = np.zeros(n_scales, dtype=np.float32)
    rc = lib().dat_oracle_step(h, _addr(o), l0, l1, M, bits, scale_mode,
                               _addr(th, shift), _addr(mo, shift), _ptr_array(grads, shift),
                               int(seed), int(step_), int(rng_bits), _addr(sin), lr, momentum, weight_decay, c_l, c_u,
                               _addr(code_sum, shift), _addr(norms), _addr(sout))
    if rc != 0:
        raise MemoryError("dat_oracle_step")
    return dict(theta=th, mom=mo, code_sum=code_sum, layer_norms=norms, scales=sout)
