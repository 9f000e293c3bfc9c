"""GPU parity at the full sizes of the benchmark configurations, in the launch
configuration bench.py times (one qesgd_encode_batch launch for all workers, one
qesgd_decode_average_apply launch).  Where the oracle cannot run the whole vector in
seconds it checks sampled buckets: a bucket's codes and scale depend only on its own
elements and their global indices, so every sampled bucket is checked exactly."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from oracle import qesgd_ref as ref                         # noqa: E402
from paper_1901_03040_b200 import qesgd, synthetic          # noqa: E402
from tests import gpu_helpers as G                          # noqa: E402


def _sample_buckets(nb, count, seed):
    rng = np.random.default_rng(seed)
    picks = set(rng.integers(0, nb, size=count).tolist())
    picks |= {0, 1, nb - 1, max(0, nb - 2), nb // 2}
    return sorted(picks)


def _run_round(d, K, bits, s, bucket, sigma, outlier, seed, n_samples):
    """Device inputs -> encode_batch -> decode_average_apply; returns the sampled comparison."""
    dev = torch.device("cuda", 0)
    ctx = G.ctx()
    stride = (d + 7) // 8 * 8
    anchor = synthetic.device_normal_f32((d,), synthetic.ANCHOR_SIGMA, seed, dev)
    locs = synthetic.device_normal_f32((K, stride), sigma, seed + 1, dev, outlier_prob=outlier)
    locs[:, :d] += anchor
    param = anchor.clone()
    codes, scales = qesgd.alloc_stream_buffers(K, d, bucket, bits, dev)
    ctx.qesgd_encode_batch(locs, stride, param, d, K, bucket, s, bits, qesgd.SCALE_NORM, 4242, 5, 9,
                           codes, codes.stride(0), scales, scales.stride(0))
    ctx.qesgd_decode_average_apply(param, d, K, codes, codes.stride(0), scales, scales.stride(0),
                                   bucket, s, bits)
    assert ctx.qesgd_status() == 0
    nb = qesgd.num_buckets(d, bucket)
    bpb = bucket * bits // 8                                  # code bytes per bucket
    picks = _sample_buckets(nb, n_samples, seed)
    idx = torch.tensor(picks, device=dev)
    g_scales = scales[:, idx].cpu().numpy()
    byte_idx = (idx[:, None] * bpb + torch.arange(bpb, device=dev)[None, :]).reshape(-1)
    g_codes = codes[:, byte_idx].cpu().numpy().reshape(K, len(picks), bpb)
    bad_codes = bad_scales = bad_param = 0
    for n, j in enumerate(picks):
        lo, hi = j * bucket, min((j + 1) * bucket, d)
        a = anchor[lo:hi].cpu().numpy()
        loc = locs[:, lo:hi].cpu().numpy()
        r_codes, r_scales = [], []
        for k in range(K):
            c, sc, st = ref.encode(loc[k], a, bucket, s, bits, ref.SCALE_NORM, 4242, 5 + k, 9, i0=lo)
            assert st == 0
            r_codes.append(c)
            r_scales.append(sc)
            bad_codes += int((g_codes[k, n].view(np.uint32) != c).any())
            bad_scales += int(g_scales[k, n].view(np.uint32) != sc.view(np.uint32)[0])
        r_codes, r_scales = np.stack(r_codes), np.stack(r_scales)
        want = ref.decode_average_apply(a, r_codes, r_scales, bucket, s, bits)
        got = param[lo:hi].cpu().numpy()
        tol = 1e-6 * np.maximum(np.abs(want), r_scales.max())
        bad_param += int((np.abs(got.astype(np.float64) - want) > tol).any())
    del locs, codes, scales, param, anchor
    torch.cuda.empty_cache()
    return len(picks), bad_codes, bad_scales, bad_param


def test_c2_quantizer_microbench_full_vector():
    """d = 2^24, no anchor, bucket 512, s in {1, 7, 127}: every code word and scale, then the
    decode round trip, against the oracle on the whole vector."""
    d, bucket = 1 << 24, 512
    z = synthetic.delta_vector(d, 1e-3, seed=2)
    for bits, s in ((2, 1), (4, 7), (8, 127)):
        gc, gs, gst = G.gpu_encode(z, None, bucket, s, bits, ref.SCALE_NORM, 77, 0, 3)
        wc, ws, wst = ref.encode(z, None, bucket, s, bits, ref.SCALE_NORM, 77, 0, 3)
        assert gst == wst == 0
        assert (gs.view(np.uint32) == ws.view(np.uint32)).all()
        assert (gc == wc).all()
        got = G.gpu_decode(gc, gs, d, bucket, s, bits)
        want = ref.decode(wc, ws, d, bucket, s, bits)
        assert (got.view(np.uint32) == want.view(np.uint32)).all()
        step = np.repeat(ws.astype(np.float64) / s, bucket)
        assert (np.abs(got - z) < step * (1 + 1e-6)).all()


def test_c3_server_aggregate_resnet18_sized():
    n, bc, bs, bp = _run_round(synthetic.RESNET18_D, 8, 4, 7, 512, 1e-4, 0.0, seed=30, n_samples=600)
    assert n >= 600 * 0.95 and (bc, bs, bp) == (0, 0, 0)


def test_c4_full_round_resnet50_sized():
    n, bc, bs, bp = _run_round(synthetic.RESNET50_D, 16, 2, 1, 256, 1e-4, 0.0, seed=40, n_samples=1024)
    assert n >= 1024 * 0.95 and (bc, bs, bp) == (0, 0, 0)


@pytest.mark.parametrize("bucket", [128, 512, 4096])
def test_c5_large_sweep_two_to_the_thirty(bucket):
    free, _ = torch.cuda.mem_get_info()
    if free < 60 << 30:
        pytest.skip("needs about 45 GB of free device memory")
    n, bc, bs, bp = _run_round(1 << 30, 8, 4, 7, bucket, 1e-3, 0.01, seed=50 + bucket,
                               n_samples=1024 if bucket < 4096 else 256)
    assert (bc, bs, bp) == (0, 0, 0)


def test_c1_end_to_end_logistic_round_with_hand_off():
    """K = 4 workers, one local epoch of minibatch-64 SGD from the anchor, 8-bit encode, apply.
    The local epoch is tolerance-equal; the oracle then encodes the GPU's own u_k, and from
    there codes and scales must be bit-identical and the applied parameter within 1e-6."""
    n, d, K, batch, lr, bucket, s, bits = 8192, 65536, 4, 64, 0.1, 512, 127, 8
    X, y, _ = synthetic.logistic_problem(n, d, seed=0)
    ctx = G.ctx()
    tX, ty = G.dev(X), G.dev(y)
    w0 = np.zeros(d, dtype=np.float32)
    param = torch.zeros(d, dtype=torch.float32, device="cuda")
    u = torch.zeros((K, d), dtype=torch.float32, device="cuda")
    n_local = n // K
    ctx.qesgd_lr_local_epoch_batch(tX, ty, n_local, d, K, batch, lr, u, d)
    u_gpu = u.cpu().numpy()
    for k in (0, K - 1):                       # two workers' epochs against the fp64 oracle
        rows = slice(k * n_local, (k + 1) * n_local)
        want = ref.lr_local_epoch(X[rows], y[rows], batch, lr, w0)
        assert np.linalg.norm(u_gpu[k] - want) <= 1e-5 * np.linalg.norm(want)
        assert np.abs(u_gpu[k] - want).max() <= 1e-5 * np.abs(want).max()
    codes, scales = qesgd.alloc_stream_buffers(K, d, bucket, bits, "cuda")
    ctx.qesgd_encode_batch(u, d, param, d, K, bucket, s, bits, qesgd.SCALE_NORM, 0, 0, 0, codes,
                           codes.stride(0), scales, scales.stride(0))
    ctx.qesgd_decode_average_apply(param, d, K, codes, codes.stride(0), scales, scales.stride(0),
                                   bucket, s, bits)
    assert ctx.qesgd_status() == 0
    nb = qesgd.num_buckets(d, bucket)
    g_codes = codes.cpu().numpy().view(np.uint32)
    g_scales = scales[:, :nb].cpu().numpy()
    r_codes, r_scales = [], []
    for k in range(K):
        c, sc, _ = ref.encode(u_gpu[k], w0, bucket, s, bits, ref.SCALE_NORM, 0, k, 0)
        assert (g_codes[k] == c).all() and (g_scales[k].view(np.uint32) == sc.view(np.uint32)).all()
        r_codes.append(c)
        r_scales.append(sc)
    want = ref.decode_average_apply(w0, np.stack(r_codes), np.stack(r_scales), bucket, s, bits)
    got = param.cpu().numpy()
    tol = 1e-6 * np.maximum(np.abs(want), np.repeat(np.stack(r_scales).max(0), bucket)[:d])
    assert (np.abs(got.astype(np.float64) - want) <= tol).all()
    # the round makes progress, and 8-bit quantisation costs next to nothing (Sec. 4, last paragraph)
    plain_avg = u_gpu.astype(np.float64).mean(axis=0).astype(np.float32)
    sub = slice(0, 1024)
    l0 = ref.lr_loss(X[sub], y[sub], w0)
    lq = ref.lr_loss(X[sub], y[sub], got)
    lp = ref.lr_loss(X[sub], y[sub], plain_avg)
    assert lq < l0 and abs(lq - lp) < 1e-3 * abs(l0 - lp) + 1e-6
