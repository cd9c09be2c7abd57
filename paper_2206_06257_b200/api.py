"""ctypes binding of libdat.so: the same names and arguments as include/dat.h.

Argument marshalling only -- every step of the path runs in the library's CUDA kernels.
torch tensors are accepted wherever the C function takes a device (or host) pointer; the
binding passes their data_ptr().  Importing this module loads the library and fails loudly
if it has not been built (python -m paper_2206_06257_b200.build); there is no CPU fallback.
"""
import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# DAT_DEBUG=1 selects the self-checking build (python -m paper_2206_06257_b200.build with the same variable set)
LIB_PATH = os.path.join(_HERE, "libdat_debug.so" if os.environ.get("DAT_DEBUG") == "1" else "libdat.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        os.path.basename(LIB_PATH) + " is missing: build it with `python -m paper_2206_06257_b200.build` "
        "(needs nvcc; the CUDA library is the only implementation of this path)")
_lib = C.CDLL(LIB_PATH)

DAT_MAX_WORKERS = 64
DAT_SCALE_SHARED_MAX, DAT_SCALE_PER_WORKER = 0, 1
DAT_RNG_BITS_16, DAT_RNG_BITS_23 = 16, 23
DAT_OK, DAT_ERR_ARG, DAT_ERR_ALIGN, DAT_ERR_BITS = 0, -1, -2, -3
DAT_ERR_LAYOUT, DAT_ERR_CUDA, DAT_ERR_NOMEM, DAT_ERR_UNSUPPORTED, DAT_ERR_TOO_LARGE = -4, -5, -6, -7, -8
DAT_STATIC_MAX_LAYERS, DAT_STATIC_MAX_TILES = 4096, 32768
DAT_STATUS_NONFINITE, DAT_STATUS_TIMEOUT, DAT_STATUS_BOUNDS = 1, 2, 4

# every symbol include/dat.h declares
EXPORTS = ["dat_plan_create", "dat_plan_set_origin", "dat_plan_destroy", "dat_plan_sizes", "dat_worker_norms", "dat_quantize", "dat_aggregate", "dat_aggregate_gather", "dat_requantize",
           "dat_average", "dat_lalr_step", "dat_lamb_step", "dat_lalr_step_static", "dat_step", "dat_step_lamb", "dat_step_two_sided", "dat_step_lamb_two_sided", "dat_step_passes", "dat_step_pipelined", "dat_plan_test_stall", "dat_step_host", "dat_get_status",
           "dat_plan_launch_count", "dat_strerror", "dat_last_cuda_error"]


class dat_hparams_t(C.Structure):
    _fields_ = [("lr", C.c_float), ("momentum", C.c_float), ("weight_decay", C.c_float),
                ("c_l", C.c_float), ("c_u", C.c_float)]


class dat_lamb_hparams_t(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("zeta", C.c_float),
                ("weight_decay", C.c_float), ("c_l", C.c_float), ("c_u", C.c_float)]


_p, _i64, _u64, _int = C.c_void_p, C.c_int64, C.c_uint64, C.c_int
_lib.dat_plan_create.argtypes = [C.POINTER(_p), _i64, _p, _int, _int, _int, _int]
_lib.dat_plan_destroy.argtypes = [_p]
_lib.dat_plan_set_origin.argtypes = [_p, _i64, _i64]
_lib.dat_worker_norms.argtypes = [_p, _p, _p, _p]
_lib.dat_plan_sizes.argtypes = [_p, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64)]
_lib.dat_quantize.argtypes = [_p, _p, _u64, _u64, _p, _p, _p, _p, _p]
_lib.dat_aggregate.argtypes = [_p, _p, _p, _p, _p, _p, _p]
_lib.dat_aggregate_gather.argtypes = [_p, _p, _p, _p, _p, _p, _p]
_lib.dat_requantize.argtypes = [_p, _p, _u64, _u64, _p, _p, _p, _p, _p]
_lib.dat_average.argtypes = [_p, _p, _p, _p]
_lib.dat_lalr_step.argtypes = [_p, _p, _p, _p, C.POINTER(dat_hparams_t), _p, _p]
_lib.dat_lamb_step.argtypes = [_p, _p, _p, _p, _p, C.POINTER(dat_lamb_hparams_t), _i64, _p, _p]
_lib.dat_lalr_step_static.argtypes = [_i64, _p, _p, _p, _p, C.POINTER(dat_hparams_t), _p, _p]
_lib.dat_step.argtypes = [_p, _p, _p, _p, _u64, _u64, C.POINTER(dat_hparams_t), _p, _p, _p, _p]
_lib.dat_plan_test_stall.argtypes = [_p, _i64, _i64, _p]
_lib.dat_step_lamb.argtypes = [_p, _p, _p, _p, _p, _u64, _u64, C.POINTER(dat_lamb_hparams_t), _i64, _p, _p, _p, _p]
_lib.dat_step_two_sided.argtypes = [_p, _p, _p, _p, _u64, _u64, C.POINTER(dat_hparams_t), _p, _p, _p, _p, _p, _p]
_lib.dat_step_lamb_two_sided.argtypes = [_p, _p, _p, _p, _p, _u64, _u64, C.POINTER(dat_lamb_hparams_t), _i64, _p, _p, _p, _p, _p, _p]
_lib.dat_step_pipelined.argtypes = [_p, _p, _p, _p, _u64, _u64, C.POINTER(dat_hparams_t), _p, _p, _p, _p]
_lib.dat_step_passes.argtypes = [_p, _p, _p, _p, _u64, _u64, C.POINTER(dat_hparams_t), _p, _p, _p, _p]
_lib.dat_step_host.argtypes = [_p, _p, _p, _p, _u64, _u64, C.POINTER(dat_hparams_t), _p]
_lib.dat_get_status.argtypes = [_p, C.POINTER(C.c_uint32), _p]
_lib.dat_plan_launch_count.argtypes = [_p]
_lib.dat_plan_launch_count.restype = _i64
_lib.dat_strerror.argtypes = [_int]
_lib.dat_strerror.restype = C.c_char_p
_lib.dat_last_cuda_error.argtypes = [_p]
for _n in EXPORTS:
    if _n not in ("dat_plan_launch_count", "dat_strerror"):
        getattr(_lib, _n).restype = _int


class DatError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, dat_strerror(code), code))


def _ok(code, where):
    if code != DAT_OK:
        raise DatError(code, where)


def _ptr(x):
    """Address of a tensor / array / int / None, as c_void_p."""
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        return _p(x.data_ptr())
    if isinstance(x, np.ndarray):
        return _p(x.ctypes.data)
    return _p(int(x))


def _ptr_array(xs):
    arr = (C.c_void_p * len(xs))()
    for k, x in enumerate(xs):
        arr[k] = _ptr(x).value if x is not None else None
    return arr


def _stream(stream):
    if stream is None:
        return _p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, torch.cuda.Stream):
        return _p(stream.cuda_stream)
    return _p(int(stream))


def _hp(hp):
    if isinstance(hp, dat_hparams_t):
        return hp
    return dat_hparams_t(*[float(v) for v in hp])


def dat_strerror(code):
    return _lib.dat_strerror(int(code)).decode()


def dat_plan_create(layer_offsets, num_workers, bits, scale_mode=DAT_SCALE_SHARED_MAX, rng_bits=DAT_RNG_BITS_16):
    """Returns the plan handle (an int).  layer_offsets: h+1 int64 values (any sequence)."""
    offs = np.ascontiguousarray(layer_offsets, dtype=np.int64)
    out = _p()
    _ok(_lib.dat_plan_create(C.byref(out), offs.size - 1, _ptr(offs), int(num_workers), int(bits),
                             int(scale_mode), int(rng_bits)), "dat_plan_create")
    return out.value


def dat_plan_set_origin(plan, elem_base, worker_base):
    _ok(_lib.dat_plan_set_origin(_p(plan), int(elem_base), int(worker_base)), "dat_plan_set_origin")


def dat_worker_norms(plan, grads, norms_out, stream=None):
    _ok(_lib.dat_worker_norms(_p(plan), _ptr_array(grads), _ptr(norms_out), _stream(stream)), "dat_worker_norms")


def dat_plan_destroy(plan):
    _ok(_lib.dat_plan_destroy(_p(plan)), "dat_plan_destroy")


def dat_plan_sizes(plan):
    """(level_bytes_per_worker, sign_bytes_per_worker, num_scales, workspace_bytes)"""
    a, b, c, d = _i64(), _i64(), _i64(), _i64()
    _ok(_lib.dat_plan_sizes(_p(plan), C.byref(a), C.byref(b), C.byref(c), C.byref(d)), "dat_plan_sizes")
    return a.value, b.value, c.value, d.value


def dat_quantize(plan, grads, seed, step, levels, signs, scales, scales_in=None, stream=None):
    _ok(_lib.dat_quantize(_p(plan), _ptr_array(grads), int(seed), int(step), _ptr(levels), _ptr(signs),
                          _ptr(scales), _ptr(scales_in), _stream(stream)), "dat_quantize")


def dat_aggregate(plan, levels, signs, scales, code_sum, g_hat, stream=None):
    _ok(_lib.dat_aggregate(_p(plan), _ptr(levels), _ptr(signs), _ptr(scales), _ptr(code_sum), _ptr(g_hat),
                           _stream(stream)), "dat_aggregate")


def dat_aggregate_gather(plan, level_planes, sign_planes, scales, code_sum, g_hat, stream=None):
    """level_planes, sign_planes: M tensors (or addresses), worker i's planes each."""
    _ok(_lib.dat_aggregate_gather(_p(plan), _ptr_array(level_planes), _ptr_array(sign_planes), _ptr(scales),
                                  _ptr(code_sum), _ptr(g_hat), _stream(stream)), "dat_aggregate_gather")


def dat_requantize(plan, g_hat, seed, step, levels, signs, scales, scales_in=None, stream=None):
    _ok(_lib.dat_requantize(_p(plan), _ptr(g_hat), int(seed), int(step), _ptr(levels), _ptr(signs), _ptr(scales),
                            _ptr(scales_in), _stream(stream)), "dat_requantize")


def dat_average(plan, grads, g_hat, stream=None):
    _ok(_lib.dat_average(_p(plan), _ptr_array(grads), _ptr(g_hat), _stream(stream)), "dat_average")


def dat_lalr_step(plan, theta, mom, g_hat, hp, layer_norms_out=None, stream=None):
    h = _hp(hp)
    _ok(_lib.dat_lalr_step(_p(plan), _ptr(theta), _ptr(mom), _ptr(g_hat), C.byref(h), _ptr(layer_norms_out),
                           _stream(stream)), "dat_lalr_step")


def dat_lamb_step(plan, theta, mom, var, g_hat, hp, t, layer_norms_out=None, stream=None):
    """hp: dat_lamb_hparams_t or (lr, beta1, beta2, zeta, weight_decay, c_l, c_u); t >= 1."""
    h = hp if isinstance(hp, dat_lamb_hparams_t) else dat_lamb_hparams_t(*[float(x) for x in hp])
    _ok(_lib.dat_lamb_step(_p(plan), _ptr(theta), _ptr(mom), _ptr(var), _ptr(g_hat), C.byref(h), int(t),
                           _ptr(layer_norms_out), _stream(stream)), "dat_lamb_step")


def dat_lalr_step_static(layer_offsets, theta, mom, g_hat, hp, layer_norms_out=None, stream=None):
    """The LALR update without a plan and without any allocation (see include/dat.h).
    layer_offsets: h+1 int64 values in host memory (any sequence)."""
    offs = np.ascontiguousarray(layer_offsets, dtype=np.int64)
    h = _hp(hp)
    _ok(_lib.dat_lalr_step_static(offs.size - 1, _ptr(offs), _ptr(theta), _ptr(mom), _ptr(g_hat), C.byref(h),
                                  _ptr(layer_norms_out), _stream(stream)), "dat_lalr_step_static")


def dat_step(plan, theta, mom, grads, seed, step, hp, code_sum_out=None, layer_norms_out=None,
             scales_out=None, stream=None):
    h = _hp(hp)
    _ok(_lib.dat_step(_p(plan), _ptr(theta), _ptr(mom), _ptr_array(grads), int(seed), int(step), C.byref(h),
                      _ptr(code_sum_out), _ptr(layer_norms_out), _ptr(scales_out), _stream(stream)), "dat_step")


def dat_step_lamb(plan, theta, mom, var, grads, seed, step, hp, t, code_sum_out=None, layer_norms_out=None,
                  scales_out=None, stream=None):
    """hp: dat_lamb_hparams_t or (lr, beta1, beta2, zeta, weight_decay, c_l, c_u); t >= 1."""
    h = hp if isinstance(hp, dat_lamb_hparams_t) else dat_lamb_hparams_t(*[float(x) for x in hp])
    _ok(_lib.dat_step_lamb(_p(plan), _ptr(theta), _ptr(mom), _ptr(var), _ptr_array(grads), int(seed), int(step), C.byref(h),
                           int(t), _ptr(code_sum_out), _ptr(layer_norms_out), _ptr(scales_out), _stream(stream)), "dat_step_lamb")


def dat_step_two_sided(plan, theta, mom, grads, seed, step, hp, g_hat, code_sum_out=None, layer_norms_out=None,
                       scales_out=None, server_scales_out=None, stream=None):
    """g_hat: fp32[d] workspace; on return the receiver's value of Algorithm A1 Step 10."""
    h = _hp(hp)
    _ok(_lib.dat_step_two_sided(_p(plan), _ptr(theta), _ptr(mom), _ptr_array(grads), int(seed), int(step), C.byref(h),
                                _ptr(g_hat), _ptr(code_sum_out), _ptr(layer_norms_out), _ptr(scales_out),
                                _ptr(server_scales_out), _stream(stream)), "dat_step_two_sided")


def dat_step_lamb_two_sided(plan, theta, mom, var, grads, seed, step, hp, t, g_hat, code_sum_out=None,
                            layer_norms_out=None, scales_out=None, server_scales_out=None, stream=None):
    h = hp if isinstance(hp, dat_lamb_hparams_t) else dat_lamb_hparams_t(*[float(x) for x in hp])
    _ok(_lib.dat_step_lamb_two_sided(_p(plan), _ptr(theta), _ptr(mom), _ptr(var), _ptr_array(grads), int(seed), int(step),
                                     C.byref(h), int(t), _ptr(g_hat), _ptr(code_sum_out), _ptr(layer_norms_out),
                                     _ptr(scales_out), _ptr(server_scales_out), _stream(stream)), "dat_step_lamb_two_sided")


def dat_plan_test_stall(plan, wait_cycles, layer=-1, stream=None):
    """Test hook: wait limit in SM cycles (0: default) and a layer whose norm never completes next call."""
    _ok(_lib.dat_plan_test_stall(_p(plan), int(wait_cycles), int(layer), _stream(stream)), "dat_plan_test_stall")


def dat_step_passes(plan, theta, mom, grads, seed, step, hp, code_sum_out=None, layer_norms_out=None,
                    scales_out=None, stream=None):
    h = _hp(hp)
    _ok(_lib.dat_step_passes(_p(plan), _ptr(theta), _ptr(mom), _ptr_array(grads), int(seed), int(step), C.byref(h),
                             _ptr(code_sum_out), _ptr(layer_norms_out), _ptr(scales_out), _stream(stream)), "dat_step_passes")


def dat_step_pipelined(plan, theta, mom, grads, seed, step, hp, code_sum_out=None, layer_norms_out=None,
                     scales_out=None, stream=None):
    h = _hp(hp)
    _ok(_lib.dat_step_pipelined(_p(plan), _ptr(theta), _ptr(mom), _ptr_array(grads), int(seed), int(step), C.byref(h),
                              _ptr(code_sum_out), _ptr(layer_norms_out), _ptr(scales_out), _stream(stream)), "dat_step_pipelined")


def dat_step_host(plan, theta_host, mom_host, grads_host, seed, step, hp, stream=None):
    h = _hp(hp)
    _ok(_lib.dat_step_host(_p(plan), _ptr(theta_host), _ptr(mom_host), _ptr_array(grads_host), int(seed),
                           int(step), C.byref(h), _stream(stream)), "dat_step_host")


def dat_get_status(plan, stream=None):
    v = C.c_uint32()
    _ok(_lib.dat_get_status(_p(plan), C.byref(v), _stream(stream)), "dat_get_status")
    return v.value


def dat_plan_launch_count(plan):
    return int(_lib.dat_plan_launch_count(_p(plan)))


def dat_last_cuda_error(plan):
    return int(_lib.dat_last_cuda_error(_p(plan)))
