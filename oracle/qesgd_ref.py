"""ctypes binding of the CPU oracle (oracle/qesgd_oracle.c) on numpy arrays.

Test infrastructure: imported by tests/, the smoke check and the benchmark's
CPU leg only.  It shares nothing with the CUDA library or its binding.
"""
import ctypes as C

import numpy as np

from . import build as _build

SCALE_NORM, SCALE_MAX, SCALE_FIXED = 0, 1, 2
STATUS_NONFINITE = 1

_lib = C.CDLL(_build.build())

_u32, _u64, _f32 = C.c_uint32, C.c_uint64, C.c_float
_pf = C.POINTER(C.c_float)
_pu = C.POINTER(C.c_uint32)
_pd = C.POINTER(C.c_double)

_lib.qesgd_ref_philox4x32_10.argtypes = [_pu, _pu, _pu]
_lib.qesgd_ref_philox4x32_10.restype = None
_lib.qesgd_ref_draw16.argtypes = [_u64, _u32, _u32, _u64]
_lib.qesgd_ref_draw16.restype = _u32
_lib.qesgd_ref_bucket_scale.argtypes = [_pf, _u32, _u32, _pd]
_lib.qesgd_ref_bucket_scale.restype = _f32
_lib.qesgd_ref_bucket_sumsq.argtypes = [_pf, _u32, _pd]
_lib.qesgd_ref_bucket_sumsq.restype = C.c_double
_lib.qesgd_ref_inv.argtypes = [_u32, _f32]
_lib.qesgd_ref_inv.restype = _f32
_lib.qesgd_ref_level.argtypes = [_f32, _f32, _u32, _u32]
_lib.qesgd_ref_level.restype = _u32
_lib.qesgd_ref_num_buckets.argtypes = [_u64, _u32]
_lib.qesgd_ref_num_buckets.restype = _u64
_lib.qesgd_ref_code_bytes.argtypes = [_u64, _u32, _u32]
_lib.qesgd_ref_code_bytes.restype = _u64
_lib.qesgd_ref_encode.argtypes = [_pf, _pf, _u64, _u64, _u32, _u32, _u32, _u32, _f32,
                                  _u64, _u32, _u32, _pu, _pf, _pu]
_lib.qesgd_ref_encode.restype = C.c_int
_lib.qesgd_ref_decode.argtypes = [_pu, _pf, _u64, _u32, _u32, _u32, _pf]
_lib.qesgd_ref_decode.restype = C.c_int
_lib.qesgd_ref_decode_average_apply.argtypes = [_pf, _u64, _u32, _pu, _u64, _pf, _u64,
                                                _u32, _u32, _u32]
_lib.qesgd_ref_decode_average_apply.restype = C.c_int
_lib.qesgd_ref_requantize.argtypes = [_pf, _pf, _u64, _u64, _u32, _u32, _u32, _u32, _f32, _u64,
                                      _u32, _u32, _pf, _pu, _pf, _pu]
_lib.qesgd_ref_requantize.restype = C.c_int
_lib.qesgd_ref_decode_average_axpy.argtypes = [_pf, _u64, _u32, _pu, _u64, _pf, _u64,
                                               _u32, _u32, _u32, _f32]
_lib.qesgd_ref_decode_average_axpy.restype = C.c_int
_lib.qesgd_ref_lr_gradient.argtypes = [_pf, _pf, _u32, _u64, _pf, _pf]
_lib.qesgd_ref_lr_gradient.restype = C.c_int
_lib.qesgd_ref_lr_loss.argtypes = [_pf, _pf, _u64, _u64, _pf]
_lib.qesgd_ref_lr_loss.restype = C.c_double
_lib.qesgd_ref_lr_sgd_step.argtypes = [_pf, _pf, _u32, _u64, _f32, _pf]
_lib.qesgd_ref_lr_sgd_step.restype = C.c_int
_lib.qesgd_ref_lr_local_epoch.argtypes = [_pf, _pf, _u64, _u64, _u32, _f32, _pf]
_lib.qesgd_ref_lr_local_epoch.restype = C.c_int


def _f(a):
    assert a.dtype == np.float32 and a.flags.c_contiguous
    return a.ctypes.data_as(_pf)


def _u(a):
    assert a.dtype == np.uint32 and a.flags.c_contiguous
    return a.ctypes.data_as(_pu)


def _check(rc):
    if rc != 0:
        raise ValueError(f"oracle returned {rc}")


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _lib.qesgd_ref_philox4x32_10(_u(c), _u(k), _u(out))
    return out


def draw16(seed, worker, epoch, i):
    return int(_lib.qesgd_ref_draw16(seed, worker, epoch, i))


def bucket_scale(z, scale_mode):
    z = np.ascontiguousarray(z, dtype=np.float32)
    scratch = np.zeros(z.size, dtype=np.float64)
    return np.float32(_lib.qesgd_ref_bucket_scale(_f(z), z.size, scale_mode,
                                                  scratch.ctypes.data_as(_pd)))


def bucket_sumsq(z):
    z = np.ascontiguousarray(z, dtype=np.float32)
    scratch = np.zeros(z.size, dtype=np.float64)
    return float(_lib.qesgd_ref_bucket_sumsq(_f(z), z.size, scratch.ctypes.data_as(_pd)))


def inv(s, scale):
    return np.float32(_lib.qesgd_ref_inv(s, np.float32(scale)))


def level(a, inv, s, h):
    return int(_lib.qesgd_ref_level(np.float32(a), np.float32(inv), s, h))


def num_buckets(d, bucket):
    return int(_lib.qesgd_ref_num_buckets(d, bucket))


def code_words(d, bucket, bits):
    return int(_lib.qesgd_ref_code_bytes(d, bucket, bits)) // 4


def encode(local, anchor, bucket, s, bits, scale_mode, seed, worker, epoch,
           i0=0, fixed_delta=0.0):
    """Returns (codes uint32[nb*B*bits/32], scales float32[nb], status)."""
    local = np.ascontiguousarray(local, dtype=np.float32)
    n = local.size
    nb = num_buckets(n, bucket)
    codes = np.zeros(nb * bucket * bits // 32, dtype=np.uint32)
    scales = np.zeros(nb, dtype=np.float32)
    status = np.zeros(1, dtype=np.uint32)
    if anchor is not None:
        anchor = np.ascontiguousarray(anchor, dtype=np.float32)
        assert anchor.size == n
    _check(_lib.qesgd_ref_encode(_f(local), _f(anchor) if anchor is not None else None,
                                 n, i0, bucket, s, bits, scale_mode, fixed_delta,
                                 seed, worker, epoch, _u(codes), _f(scales), _u(status)))
    return codes, scales, int(status[0])


def decode(codes, scales, n, bucket, s, bits):
    out = np.zeros(n, dtype=np.float32)
    _check(_lib.qesgd_ref_decode(_u(codes), _f(scales), n, bucket, s, bits, _f(out)))
    return out


def decode_average_apply(param, codes, scales, bucket, s, bits):
    """codes: uint32[K, words], scales: float32[K, nb]; returns the new parameter."""
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    scales = np.ascontiguousarray(scales, dtype=np.float32)
    assert codes.ndim == 2 and scales.ndim == 2 and codes.shape[0] == scales.shape[0]
    out = np.array(param, dtype=np.float32, copy=True)
    _check(_lib.qesgd_ref_decode_average_apply(
        _f(out), out.size, codes.shape[0], _u(codes), codes.shape[1] * 4, _f(scales),
        scales.shape[1], bucket, s, bits))
    return out


def requantize(u, anchor, bucket, s, bits, scale_mode, seed, worker, step, zsum=None,
               i0=0, fixed_delta=0.0):
    """Returns (u_new, zsum_new or None, codes, scales, status); inputs are not modified."""
    u = np.array(u, dtype=np.float32, copy=True)
    anchor = np.ascontiguousarray(anchor, dtype=np.float32)
    n = u.size
    nb = num_buckets(n, bucket)
    codes = np.zeros(nb * bucket * bits // 32, dtype=np.uint32)
    scales = np.zeros(nb, dtype=np.float32)
    status = np.zeros(1, dtype=np.uint32)
    z = None if zsum is None else np.array(zsum, dtype=np.float32, copy=True)
    _check(_lib.qesgd_ref_requantize(_f(u), _f(anchor), n, i0, bucket, s, bits, scale_mode,
                                     fixed_delta, seed, worker, step,
                                     _f(z) if z is not None else None, _u(codes), _f(scales),
                                     _u(status)))
    return u, z, codes, scales, int(status[0])


def decode_average_axpy(param, codes, scales, bucket, s, bits, alpha):
    """param + alpha * mean_k decode(stream k); codes uint32[K, words], scales float32[K, nb]."""
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    scales = np.ascontiguousarray(scales, dtype=np.float32)
    out = np.array(param, dtype=np.float32, copy=True)
    _check(_lib.qesgd_ref_decode_average_axpy(
        _f(out), out.size, codes.shape[0], _u(codes), codes.shape[1] * 4, _f(scales),
        scales.shape[1], bucket, s, bits, alpha))
    return out


def lr_gradient(Xb, yb, w):
    Xb = np.ascontiguousarray(Xb, dtype=np.float32)
    g = np.zeros(Xb.shape[1], dtype=np.float32)
    _check(_lib.qesgd_ref_lr_gradient(_f(Xb), _f(np.ascontiguousarray(yb, np.float32)),
                                      Xb.shape[0], Xb.shape[1],
                                      _f(np.ascontiguousarray(w, np.float32)), _f(g)))
    return g


def lr_loss(X, y, w):
    X = np.ascontiguousarray(X, dtype=np.float32)
    return float(_lib.qesgd_ref_lr_loss(_f(X), _f(np.ascontiguousarray(y, np.float32)),
                                        X.shape[0], X.shape[1],
                                        _f(np.ascontiguousarray(w, np.float32))))


def lr_sgd_step(Xb, yb, lr, u):
    Xb = np.ascontiguousarray(Xb, dtype=np.float32)
    out = np.array(u, dtype=np.float32, copy=True)
    _check(_lib.qesgd_ref_lr_sgd_step(_f(Xb), _f(np.ascontiguousarray(yb, np.float32)),
                                      Xb.shape[0], Xb.shape[1], lr, _f(out)))
    return out


def lr_local_epoch(X, y, batch, lr, u):
    X = np.ascontiguousarray(X, dtype=np.float32)
    out = np.array(u, dtype=np.float32, copy=True)
    _check(_lib.qesgd_ref_lr_local_epoch(_f(X), _f(np.ascontiguousarray(y, np.float32)),
                                         X.shape[0], X.shape[1], batch, lr, _f(out)))
    return out
