"""Helpers for the GPU parity tests: numpy in, numpy out, through the C ABI."""
import numpy as np
import torch

from paper_1901_03040_b200 import qesgd

_CTX = {}


def ctx():
    if "c" not in _CTX:
        _CTX["c"] = qesgd.Context(0, None)
    return _CTX["c"]


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_encode(local, anchor, bucket, s, bits, mode, seed, worker, epoch, fixed_delta=0.0,
               misalign=0):
    """Encode one worker's vector; returns (codes uint32[], scales float32[], status)."""
    c = ctx()
    d = int(local.size)
    nb = qesgd.num_buckets(d, bucket)
    cb = qesgd.code_bytes(d, bucket, bits)
    if misalign:
        buf = torch.zeros(d + misalign, dtype=torch.float32, device="cuda")
        buf[misalign:] = dev(local)
        t_local = buf[misalign:]
    else:
        t_local = dev(local)
    t_anchor = dev(anchor) if anchor is not None else None
    codes = torch.full((cb + 64,), 0xAB, dtype=torch.uint8, device="cuda")   # canary bytes
    scales = torch.full((nb + 16,), -7.0, dtype=torch.float32, device="cuda")
    c.qesgd_encode(t_local, t_anchor, d, bucket, s, bits, mode, seed, worker, epoch, codes,
                   scales, fixed_delta)
    status = c.qesgd_status()
    assert (codes[cb:] == 0xAB).all().item(), "encode wrote past the code stream"
    assert (scales[nb:] == -7.0).all().item(), "encode wrote past the scales"
    return (codes[:cb].cpu().numpy().view(np.uint32).copy(), scales[:nb].cpu().numpy().copy(),
            status)


def gpu_encode_batch(locals_, anchor, bucket, s, bits, mode, seed, worker0, epoch):
    """locals_: float32[K, d].  Returns codes uint32[K, words], scales float32[K, nb], status."""
    c = ctx()
    K, d = locals_.shape
    nb = qesgd.num_buckets(d, bucket)
    cb = qesgd.code_bytes(d, bucket, bits)
    stride_e = (d + 7) // 8 * 8
    buf = torch.zeros((K, stride_e), dtype=torch.float32, device="cuda")
    buf[:, :d] = dev(locals_)
    codes, scales = qesgd.alloc_stream_buffers(K, d, bucket, bits, "cuda")
    c.qesgd_encode_batch(buf, stride_e, dev(anchor) if anchor is not None else None, d, K, bucket,
                         s, bits, mode, seed, worker0, epoch, codes, codes.stride(0), scales,
                         scales.stride(0))
    status = c.qesgd_status()
    return (codes.cpu().numpy().view(np.uint32).reshape(K, cb // 4).copy(),
            scales[:, :nb].cpu().numpy().copy(), status)


def gpu_decode(codes, scales, d, bucket, s, bits):
    c = ctx()
    out = torch.full((d + 8,), 123.0, dtype=torch.float32, device="cuda")
    c.qesgd_decode(dev(codes), dev(scales), d, bucket, s, bits, out)
    torch.cuda.synchronize()
    assert (out[d:] == 123.0).all().item()
    return out[:d].cpu().numpy().copy()


def gpu_decode_average_apply(param, codes, scales, bucket, s, bits):
    """codes uint32[K, words], scales float32[K, nb]."""
    c = ctx()
    K = codes.shape[0]
    d = int(param.size)
    nb = scales.shape[1]
    nb_pad = (nb + 3) // 4 * 4
    t_scales = torch.zeros((K, nb_pad), dtype=torch.float32, device="cuda")
    t_scales[:, :nb] = dev(scales)
    t_codes = dev(codes)
    p = torch.full((d + 8,), 321.0, dtype=torch.float32, device="cuda")
    p[:d] = dev(param)
    c.qesgd_decode_average_apply(p, d, K, t_codes, codes.shape[1] * 4, t_scales, nb_pad, bucket,
                                 s, bits)
    torch.cuda.synchronize()
    assert (p[d:] == 321.0).all().item()
    return p[:d].cpu().numpy().copy()
