"""Thin ctypes binding of libqesgd.so (include/qesgd.h) on torch CUDA tensors.

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch supplies device memory and streams.  There is no CPU fallback:
importing this module without the built library raises.
"""
import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
# QESGD_DEBUG=1 in the environment selects the debug build of the same library (index checks in
# the codec kernels, QESGD_STATUS_RANGE); build it with `python -m paper_1901_03040_b200.build --debug`
LIB_PATH = os.path.join(_HERE, "libqesgd_debug.so" if os.environ.get("QESGD_DEBUG") == "1" else "libqesgd.so")

SCALE_NORM, SCALE_MAX, SCALE_FIXED = 0, 1, 2
STATUS_NONFINITE = 1
STATUS_TIMEOUT = 2
STATUS_RANGE = 4
OK, EINVAL, ECUDA, ENOMEM, ELIMIT = 0, -1, -2, -3, -4
MAX_WORKERS, MIN_BUCKET, MAX_BUCKET, MAX_LR_BATCH = 64, 64, 8192, 1024
NOALLOC_MAX_LR_BATCH = 256

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_1901_03040_b200.build` "
        "(nvcc, sm_100a). There is no fallback path.")

lib = C.CDLL(LIB_PATH)

_vp, _u32, _u64, _f32, _int = C.c_void_p, C.c_uint32, C.c_uint64, C.c_float, C.c_int

SIGNATURES = {
    "qesgd_create": (_int, [C.POINTER(_vp), _int, _vp]),
    "qesgd_destroy": (_int, [_vp]),
    "qesgd_set_stream": (_int, [_vp, _vp]),
    "qesgd_set_wait_limit": (_int, [_vp, _u64]),
    "qesgd_debug_drop_signal": (_int, [_vp, C.c_int64]),
    "qesgd_num_buckets": (_u64, [_u64, _u32]),
    "qesgd_code_bytes": (_u64, [_u64, _u32, _u32]),
    "qesgd_encode": (_int, [_vp, _vp, _vp, _u64, _u32, _u32, _u32, _u32, _f32, _u64, _u32, _u32,
                            _vp, _vp]),
    "qesgd_encode_batch": (_int, [_vp, _vp, _u64, _vp, _u64, _u32, _u32, _u32, _u32, _u32, _f32,
                                  _u64, _u32, _u32, _vp, _u64, _vp, _u64]),
    "qesgd_requantize": (_int, [_vp, _vp, _vp, _u64, _u32, _u32, _u32, _u32, _f32, _u64, _u32, _u32,
                                _vp, _vp, _vp]),
    "qesgd_lr_qesgd_step": (_int, [_vp, _vp, _vp, _u32, _u64, _f32, _vp, _vp, _u32, _u32, _u32, _u32, _f32,
                                   _u64, _u32, _u32, _vp, _vp, _vp]),
    "qesgd_decode_average_apply": (_int, [_vp, _vp, _u64, _u32, _vp, _u64, _vp, _u64, _u32, _u32,
                                          _u32]),
    "qesgd_decode_average_axpy": (_int, [_vp, _vp, _u64, _u32, _vp, _u64, _vp, _u64, _u32, _u32,
                                         _u32, _f32]),
    "qesgd_decode": (_int, [_vp, _vp, _vp, _u64, _u32, _u32, _u32, _vp]),
    "qesgd_lr_gradient": (_int, [_vp, _vp, _vp, _u32, _u64, _vp, _vp]),
    "qesgd_lr_sgd_step": (_int, [_vp, _vp, _vp, _u32, _u64, _f32, _vp]),
    "qesgd_lr_local_epoch": (_int, [_vp, _vp, _vp, _u64, _u64, _u32, _f32, _vp]),
    "qesgd_lr_local_epoch_batch": (_int, [_vp, _vp, _vp, _u64, _u64, _u32, _u32, _f32, _vp, _u64]),
    "qesgd_lr_sgd_step_noalloc": (_int, [_vp, _vp, _vp, _u32, _u64, _f32, _vp]),
    "qesgd_status": (_int, [_vp, C.POINTER(_u32)]),
    "qesgd_debug_build": (_int, []),
    "qesgd_debug_range_selftest": (_int, [_vp]),
    "qesgd_launch_count": (_u64, [_vp]),
    "qesgd_last_cuda_error": (_int, [_vp]),
    "qesgd_strerror": (C.c_char_p, [_int]),
}
for _name, (_res, _args) in SIGNATURES.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class QesgdError(RuntimeError):
    def __init__(self, code, cuda_error=0):
        self.code = code
        self.cuda_error = cuda_error
        text = lib.qesgd_strerror(code).decode()
        super().__init__(f"qesgd: {text} (code {code}, cuda error {cuda_error})")


def num_buckets(d, bucket):
    return int(lib.qesgd_num_buckets(d, bucket))


def code_bytes(d, bucket, bits):
    return int(lib.qesgd_code_bytes(d, bucket, bits))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class Context:
    """One qesgd_ctx: a device, a stream, a status word."""

    def __init__(self, device=0, stream=None):
        import torch
        self.device = torch.device("cuda", device) if isinstance(device, int) else torch.device(device)
        index = self.device.index if self.device.index is not None else torch.cuda.current_device()
        handle = C.c_void_p()
        raw = stream.cuda_stream if stream is not None else 0
        rc = lib.qesgd_create(C.byref(handle), index, C.c_void_p(raw))
        if rc != OK:
            raise QesgdError(rc)
        self._h = handle
        self.stream = stream

    def close(self):
        if getattr(self, "_h", None):
            lib.qesgd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != OK:
            raise QesgdError(rc, lib.qesgd_last_cuda_error(self._h))

    def set_stream(self, stream):
        self._check(lib.qesgd_set_stream(self._h, C.c_void_p(stream.cuda_stream if stream else 0)))
        self.stream = stream

    def qesgd_set_wait_limit(self, nanoseconds):
        self._check(lib.qesgd_set_wait_limit(self._h, nanoseconds))

    def qesgd_debug_drop_signal(self, cta):
        self._check(lib.qesgd_debug_drop_signal(self._h, cta))

    # -- worker side ---------------------------------------------------------
    def qesgd_encode(self, local, anchor, d, bucket, s, bits, scale_mode, seed, worker, epoch,
                     codes_out, scales_out, fixed_delta=0.0):
        self._check(lib.qesgd_encode(self._h, _ptr(local), _ptr(anchor), d, bucket, s, bits,
                                     scale_mode, fixed_delta, seed, worker, epoch,
                                     _ptr(codes_out), _ptr(scales_out)))

    def qesgd_encode_batch(self, local, local_stride, anchor, d, K, bucket, s, bits, scale_mode,
                           seed, worker0, epoch, codes_out, code_stride, scales_out, scale_stride,
                           fixed_delta=0.0):
        self._check(lib.qesgd_encode_batch(self._h, _ptr(local), local_stride, _ptr(anchor), d, K,
                                           bucket, s, bits, scale_mode, fixed_delta, seed, worker0,
                                           epoch, _ptr(codes_out), code_stride, _ptr(scales_out),
                                           scale_stride))

    def qesgd_requantize(self, u, anchor, d, bucket, s, bits, scale_mode, seed, worker, step, zsum,
                         codes_out, scales_out, fixed_delta=0.0):
        self._check(lib.qesgd_requantize(self._h, _ptr(u), _ptr(anchor), d, bucket, s, bits,
                                         scale_mode, fixed_delta, seed, worker, step, _ptr(zsum),
                                         _ptr(codes_out), _ptr(scales_out)))

    def qesgd_lr_qesgd_step(self, Xb, yb, m, d, lr, u, anchor, bucket, s, bits, scale_mode, seed, worker,
                            step, zsum, codes_out, scales_out, fixed_delta=0.0):
        self._check(lib.qesgd_lr_qesgd_step(self._h, _ptr(Xb), _ptr(yb), m, d, lr, _ptr(u), _ptr(anchor),
                                            bucket, s, bits, scale_mode, fixed_delta, seed, worker, step,
                                            _ptr(zsum), _ptr(codes_out), _ptr(scales_out)))

    # -- server side ---------------------------------------------------------
    def qesgd_decode_average_apply(self, param, d, K, codes, code_stride, scales, scale_stride,
                                   bucket, s, bits):
        self._check(lib.qesgd_decode_average_apply(self._h, _ptr(param), d, K, _ptr(codes),
                                                   code_stride, _ptr(scales), scale_stride,
                                                   bucket, s, bits))

    def qesgd_decode_average_axpy(self, param, d, K, codes, code_stride, scales, scale_stride,
                                  bucket, s, bits, alpha):
        self._check(lib.qesgd_decode_average_axpy(self._h, _ptr(param), d, K, _ptr(codes),
                                                  code_stride, _ptr(scales), scale_stride,
                                                  bucket, s, bits, alpha))

    def qesgd_decode(self, codes, scales, d, bucket, s, bits, out):
        self._check(lib.qesgd_decode(self._h, _ptr(codes), _ptr(scales), d, bucket, s, bits,
                                     _ptr(out)))

    # -- local epoch ---------------------------------------------------------
    def qesgd_lr_sgd_step(self, Xb, yb, m, d, lr, u):
        self._check(lib.qesgd_lr_sgd_step(self._h, _ptr(Xb), _ptr(yb), m, d, lr, _ptr(u)))

    def qesgd_lr_gradient(self, Xb, yb, m, d, w, g_out):
        self._check(lib.qesgd_lr_gradient(self._h, _ptr(Xb), _ptr(yb), m, d, _ptr(w), _ptr(g_out)))

    def qesgd_lr_local_epoch(self, X, y, n_local, d, batch, lr, u):
        self._check(lib.qesgd_lr_local_epoch(self._h, _ptr(X), _ptr(y), n_local, d, batch, lr,
                                             _ptr(u)))

    def qesgd_lr_local_epoch_batch(self, X, y, n_local, d, K, batch, lr, u, u_stride):
        self._check(lib.qesgd_lr_local_epoch_batch(self._h, _ptr(X), _ptr(y), n_local, d, K, batch,
                                                   lr, _ptr(u), u_stride))

    # -- bookkeeping ---------------------------------------------------------
    def qesgd_status(self):
        flags = C.c_uint32(0)
        self._check(lib.qesgd_status(self._h, C.byref(flags)))
        return int(flags.value)

    def qesgd_launch_count(self):
        return int(lib.qesgd_launch_count(self._h))


def qesgd_lr_sgd_step_noalloc(stream, Xb, yb, m, d, lr, u):
    """One logistic SGD step on the current device without a context and without any
    allocation by the library: for callers that must not allocate device memory when
    they take the step (the scratch is a fixed 64 KB array inside the library; at most
    NOALLOC_MAX_LR_BATCH rows; calls must not overlap on the GPU)."""
    rc = lib.qesgd_lr_sgd_step_noalloc(C.c_void_p(stream.cuda_stream if stream is not None else 0),
                                       _ptr(Xb), _ptr(yb), m, d, lr, _ptr(u))
    if rc != OK:
        raise QesgdError(rc)


def alloc_stream_buffers(K, d, bucket, bits, device):
    """Device buffers for K workers' streams: (codes uint8[K, stride], scales
    float32[K, nb_padded]) with strides that satisfy the library's alignment."""
    import torch
    cb = code_bytes(d, bucket, bits)
    nb = num_buckets(d, bucket)
    nb_pad = (nb + 3) // 4 * 4
    codes = torch.zeros((K, cb), dtype=torch.uint8, device=device)
    scales = torch.zeros((K, nb_pad), dtype=torch.float32, device=device)
    return codes, scales
