"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded inputs.  Codes and scales must match bit for bit; applied
parameters within 1e-6 relative; the logistic step within 1e-5 relative."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from oracle import qesgd_ref as ref                         # noqa: E402
from paper_1901_03040_b200 import qesgd, synthetic          # noqa: E402
from tests import gpu_helpers as G                          # noqa: E402

BITS_S = [(2, 1), (4, 7), (4, 5), (8, 127), (8, 100)]
BUCKETS = [64, 128, 256, 512, 1024, 2048, 4096, 8192]


def _delta(n, seed, sigma=1e-3, outliers=True):
    return synthetic.delta_vector(n, sigma, seed, 0, 0.01 if outliers else 0.0)


def _assert_streams_equal(got, want):
    gc, gs, gst = got
    wc, ws, wst = want
    assert gs.dtype == ws.dtype == np.float32
    bad = np.nonzero(gs.view(np.uint32) != ws.view(np.uint32))[0]
    assert bad.size == 0, f"{bad.size} scales differ, first bucket {bad[:5]}: {gs[bad[:5]]} vs {ws[bad[:5]]}"
    badc = np.nonzero(gc != wc)[0]
    assert badc.size == 0, f"{badc.size} code words differ, first {badc[:5]}"
    assert gst == wst


# ----------------------------------------------------------------- encode ----
@pytest.mark.parametrize("mode", [ref.SCALE_NORM, ref.SCALE_MAX])
@pytest.mark.parametrize("bucket", BUCKETS)
@pytest.mark.parametrize("bits,s", BITS_S)
def test_encode_matches_oracle_bitwise(bits, s, bucket, mode):
    # several CTA tiles, a ragged tail that is neither a multiple of 8 nor of the bucket
    n = 8192 * 3 + 1000 + 3
    z = _delta(n, seed=bucket + bits)
    args = (bucket, s, bits, mode, 0x1234_5678_9ABC_DEF0, 3, 17)
    _assert_streams_equal(G.gpu_encode(z, None, *args), ref.encode(z, None, *args))


@pytest.mark.parametrize("n", [1, 7, 8, 63, 64, 65, 511, 512, 513, 4095, 8193])
@pytest.mark.parametrize("bucket", [64, 512, 4096])
def test_encode_small_and_ragged_sizes(n, bucket):
    z = _delta(n, seed=n)
    w = synthetic.anchor_vector(n, seed=n + 1)
    u = (w + z).astype(np.float32)
    for mode in (ref.SCALE_NORM, ref.SCALE_MAX):
        args = (bucket, 7, 4, mode, 99, 1, 2)
        _assert_streams_equal(G.gpu_encode(u, w, *args), ref.encode(u, w, *args))


@pytest.mark.parametrize("bits,s", [(2, 1), (4, 7), (8, 127)])
def test_encode_with_anchor_large(bits, s):
    n = (1 << 20) + 40
    w = synthetic.anchor_vector(n, seed=5)
    u = (w + _delta(n, seed=6, sigma=1e-4)).astype(np.float32)
    args = (512, s, bits, ref.SCALE_NORM, 7, 0, 0)
    _assert_streams_equal(G.gpu_encode(u, w, *args), ref.encode(u, w, *args))


def test_encode_unaligned_pointer_takes_the_scalar_path():
    n = 8192 + 77
    z = _delta(n, seed=31)
    args = (256, 7, 4, ref.SCALE_NORM, 5, 0, 1)
    want = ref.encode(z, None, *args)
    for mis in (1, 3, 4):
        _assert_streams_equal(G.gpu_encode(z, None, *args, misalign=mis), want)


def test_encode_batch_uses_worker_ids_and_strides():
    K, n, bucket = 5, 8192 + 520, 128
    w = synthetic.anchor_vector(n, seed=1)
    locs = synthetic.worker_locals(w, K, 1e-4, seed=2)
    gc, gs, gst = G.gpu_encode_batch(locs, w, bucket, 7, 4, ref.SCALE_NORM, 42, 10, 3)
    assert gst == 0
    for k in range(K):
        wc, ws, _ = ref.encode(locs[k], w, bucket, 7, 4, ref.SCALE_NORM, 42, 10 + k, 3)
        assert (gc[k] == wc).all() and (gs[k].view(np.uint32) == ws.view(np.uint32)).all()


def test_encode_batch_with_the_largest_worker_count_and_padded_strides():
    K, n, bucket, bits, s = 64, 2048 + 24, 64, 2, 1
    w = synthetic.anchor_vector(n, seed=3)
    locs = synthetic.worker_locals(w, K, 1e-4, seed=4)
    c = G.ctx()
    stride = n + 40                                          # more than the minimum, multiple of 8
    buf = torch.zeros((K, stride), dtype=torch.float32, device="cuda")
    buf[:, :n] = G.dev(locs)
    cb, nb = qesgd.code_bytes(n, bucket, bits), qesgd.num_buckets(n, bucket)
    codes = torch.full((K, cb + 32), 0xCD, dtype=torch.uint8, device="cuda")
    scales = torch.full((K, nb + 7 + (4 - (nb + 7) % 4) % 4), -1.0, dtype=torch.float32, device="cuda")
    c.qesgd_encode_batch(buf, stride, G.dev(w), n, K, bucket, s, bits, ref.SCALE_MAX, 8, 100, 2,
                         codes, codes.stride(0), scales, scales.stride(0))
    assert c.qesgd_status() == 0
    assert (codes[:, cb:] == 0xCD).all().item() and (scales[:, nb:] == -1.0).all().item()
    gc = codes[:, :cb].contiguous().cpu().numpy().view(np.uint32)
    gs = scales[:, :nb].cpu().numpy()
    for k in (0, 1, 31, 63):
        wc, ws, _ = ref.encode(locs[k], w, bucket, s, bits, ref.SCALE_MAX, 8, 100 + k, 2)
        assert (gc[k] == wc).all() and (gs[k].view(np.uint32) == ws.view(np.uint32)).all()


def test_encode_epoch_and_seed_change_the_draws_but_not_the_scales():
    z = _delta(4096, seed=8)
    a = G.gpu_encode(z, None, 512, 7, 4, ref.SCALE_NORM, 1, 0, 0)
    b = G.gpu_encode(z, None, 512, 7, 4, ref.SCALE_NORM, 1, 0, 1)
    c = G.gpu_encode(z, None, 512, 7, 4, ref.SCALE_NORM, 1, 0, 0)
    assert (a[0] == c[0]).all() and (a[0] != b[0]).any() and (a[1] == b[1]).all()


@pytest.mark.parametrize("mode", [ref.SCALE_NORM, ref.SCALE_MAX])
def test_nonfinite_zero_tiny_and_huge_buckets(mode):
    n = 64 * 8
    z = _delta(n, seed=3)
    z[70] = np.inf
    z[130] = np.nan
    z[192:256] = 0.0
    z[256:320] = np.float32(2.0 ** -120)
    z[320:384] = np.float32(3e38)
    z[384:448] = np.float32(1e-42)        # subnormal inputs
    z[448] = -np.inf
    args = (64, 7, 4, mode, 11, 0, 0)
    got, want = G.gpu_encode(z, None, *args), ref.encode(z, None, *args)
    _assert_streams_equal(got, want)
    assert got[2] == qesgd.STATUS_NONFINITE
    assert G.ctx().qesgd_status() == 0            # reading the status clears it


def test_subnormal_and_mixed_magnitudes_match():
    rng = np.random.default_rng(12)
    n = 4096
    z = (rng.standard_normal(n) * np.exp(rng.uniform(-80, 20, n))).astype(np.float32)
    for bucket in (64, 1024):
        for mode in (ref.SCALE_NORM, ref.SCALE_MAX):
            args = (bucket, 127, 8, mode, 2, 1, 1)
            _assert_streams_equal(G.gpu_encode(z, None, *args), ref.encode(z, None, *args))


def _unpack_levels(words, bits):
    """Levels (codes without their sign bit) of a little-endian packed stream."""
    per = 32 // bits
    shifts = (np.arange(per, dtype=np.uint32) * bits)[None, :]
    fields = (words.astype(np.uint32)[:, None] >> shifts) & np.uint32((1 << bits) - 1)
    return (fields & np.uint32((1 << (bits - 1)) - 1)).reshape(-1)


def test_bucket_maxima_and_huge_scales_stay_at_the_top_level():
    """Buckets whose largest coordinates equal the scale (max mode: many copies of the maximum;
    norm mode: one coordinate carries the whole norm), over many scales, and scales so large that
    the inverse spacing s/scale is subnormal: the product |z| * inv may exceed s by an ulp there,
    and the codes must still be the oracle's (top level s, never s + 1)."""
    rng = np.random.default_rng(99)
    nb, bucket = 256, 64
    for bits, s in ((2, 1), (4, 2), (4, 3), (4, 7), (8, 100), (8, 127)):
        z = np.zeros((nb, bucket), dtype=np.float32)
        mags = np.exp(rng.uniform(-30, 30, nb)).astype(np.float32)
        mags[nb // 2:] = (2.0 ** rng.uniform(126, 127.9, nb - nb // 2)).astype(np.float32)
        signs = rng.choice(np.float32([-1, 1]), (nb, bucket))
        z[:, :16] = mags[:, None] * signs[:, :16]                     # copies of the maximum
        z[:, 16:] = (mags[:, None] * rng.uniform(0, 1, (nb, bucket - 16))).astype(np.float32) * signs[:, 16:]
        flat = z.reshape(-1)
        for epoch in range(3):
            args = (bucket, s, bits, ref.SCALE_MAX, 17, 1, epoch)
            got, want = G.gpu_encode(flat, None, *args), ref.encode(flat, None, *args)
            _assert_streams_equal(got, want)
        levels = _unpack_levels(want[0], bits)[: nb * bucket].reshape(nb, bucket)
        assert (levels[:, :16] == s).all()
        single = np.zeros((nb, bucket), dtype=np.float32)             # one coordinate = the norm
        single[np.arange(nb), rng.integers(0, bucket, nb)] = mags * signs[:, 0]
        args = (bucket, s, bits, ref.SCALE_NORM, 17, 1, 0)
        got, want = G.gpu_encode(single.reshape(-1), None, *args), ref.encode(single.reshape(-1), None, *args)
        _assert_streams_equal(got, want)
        assert got[2] == 0


def test_fixed_delta_mode_matches_and_clips():
    n = 8192 + 100
    z = _delta(n, seed=21)
    z[5] = np.nan
    z[9] = np.inf
    z[10] = -np.inf
    delta = 2.5e-4
    for bits, s in ((4, 7), (8, 127), (2, 1)):
        got = G.gpu_encode(z, None, 512, s, bits, ref.SCALE_FIXED, 3, 2, 1, fixed_delta=delta)
        want = ref.encode(z, None, 512, s, bits, ref.SCALE_FIXED, 3, 2, 1, fixed_delta=delta)
        _assert_streams_equal(got, want)
        assert got[2] == qesgd.STATUS_NONFINITE


def test_negative_zero_and_exact_ties_match_the_oracle():
    """Values whose fractional part times 2^16 is a half-integer sit exactly on the
    boundary between two draws (h + 1/2 = p * 2^16): strict '<' must decide them the same
    way on both sides; negative values that round to level 0 must give the plain 0 code."""
    s, bits, bucket = 7, 4, 64
    delta = 2.0 ** -4
    z = np.zeros(bucket * 2, dtype=np.float32)
    z[0] = s * delta                                   # scale = s * delta, inv = 16 exactly
    ties = [(2 * m + 1) / 131072.0 for m in (0, 1, 5, 1000, 32767, 65535)]
    for n, t in enumerate(ties):
        z[1 + n] = (n % 7 + t) * delta * (-1 if n % 2 else 1)
    z[10:40] = -1e-9
    z[40] = -0.0
    z[64] = -s * delta
    z[65:] = z[1:64]
    for epoch in range(8):
        args = (bucket, s, bits, ref.SCALE_MAX, 31337, 2, epoch)
        got, want = G.gpu_encode(z, None, *args), ref.encode(z, None, *args)
        _assert_streams_equal(got, want)


def test_on_grid_input_round_trips_exactly_on_the_gpu():
    s, bits, bucket = 127, 8, 256
    rng = np.random.default_rng(4)
    n = bucket * 40
    k = rng.integers(-s, s + 1, n)
    k[::bucket] = s
    z = (k * 2.0 ** -14).astype(np.float32)
    codes, scales, status = G.gpu_encode(z, None, bucket, s, bits, ref.SCALE_MAX, 77, 0, 0)
    assert status == 0 and (scales == np.float32(s * 2.0 ** -14)).all()
    assert (G.gpu_decode(codes, scales, n, bucket, s, bits) == z).all()


# ----------------------------------------------------------------- decode ----
@pytest.mark.parametrize("bucket", [64, 512, 8192])
@pytest.mark.parametrize("bits,s", BITS_S)
def test_decode_matches_oracle_bitwise(bits, s, bucket):
    n = 8192 * 2 + 333
    z = _delta(n, seed=bits * 100 + s)
    codes, scales, _ = ref.encode(z, None, bucket, s, bits, ref.SCALE_NORM, 9, 0, 0)
    got = G.gpu_decode(codes, scales, n, bucket, s, bits)
    want = ref.decode(codes, scales, n, bucket, s, bits)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()


# --------------------------------------------------- decode-average-apply ----
def _daa_case(n, K, bucket, bits, s, seed, sigma=1e-4):
    w = synthetic.anchor_vector(n, seed=seed)
    locs = synthetic.worker_locals(w, K, sigma, seed=seed + 1, outlier_prob=0.01)
    codes, scales = [], []
    for k in range(K):
        c, sc, _ = ref.encode(locs[k], w, bucket, s, bits, ref.SCALE_NORM, seed, k, 0)
        codes.append(c)
        scales.append(sc)
    return w, np.stack(codes), np.stack(scales)


def _assert_param_close(got, want, w_before, scales, bucket):
    smax = np.repeat(scales.max(axis=0), bucket)[:want.size]
    tol = 1e-6 * np.maximum(np.abs(want), smax)
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    assert (err <= tol).all(), f"max err/tol {np.max(err / np.maximum(tol, 1e-300))}"
    assert (got != w_before).any()


@pytest.mark.parametrize("K", [1, 2, 3, 4, 5, 8, 16, 33, 64])
@pytest.mark.parametrize("bucket,bits,s", [(64, 2, 1), (64, 4, 7), (64, 8, 127), (128, 2, 1), (256, 2, 1),
                                           (512, 4, 7), (2048, 8, 127), (8192, 4, 7)])
def test_decode_average_apply_matches_oracle(K, bucket, bits, s):
    n = 8192 * 2 + 300 + 5
    w, codes, scales = _daa_case(n, K, bucket, bits, s, seed=K * 7 + bits)
    got = G.gpu_decode_average_apply(w, codes, scales, bucket, s, bits)
    want = ref.decode_average_apply(w, codes, scales, bucket, s, bits)
    _assert_param_close(got, want, w, scales, bucket)


@pytest.mark.parametrize("n", [1, 9, 255, 256, 257, 2049])
def test_decode_average_apply_small_sizes(n):
    w, codes, scales = _daa_case(n, 4, 64, 4, 7, seed=n)
    got = G.gpu_decode_average_apply(w, codes, scales, 64, 7, 4)
    want = ref.decode_average_apply(w, codes, scales, 64, 7, 4)
    _assert_param_close(got, want, w, scales, 64)


def test_k1_on_grid_apply_returns_the_worker_parameter_exactly():
    rng = np.random.default_rng(6)
    n, s, bits, bucket = 512 * 9, 127, 8, 512
    k = rng.integers(-s, s + 1, n)
    k[::bucket] = s
    z = (k * 2.0 ** -10).astype(np.float32)
    w = (rng.integers(-1000, 1000, n) * 2.0 ** -10).astype(np.float32)
    codes, scales, _ = G.gpu_encode(w + z, w, bucket, s, bits, ref.SCALE_MAX, 1, 0, 0)
    out = G.gpu_decode_average_apply(w, codes[None], scales[None], bucket, s, bits)
    assert (out == w + z).all()


# ----------------------------------------------------- logistic regression ---
def _lr_close(got, want):
    dn = np.linalg.norm(got.astype(np.float64) - want)
    assert dn <= 1e-5 * np.linalg.norm(want)
    assert np.abs(got - want).max() <= 1e-5 * np.abs(want).max()


@pytest.mark.parametrize("m,d", [(64, 4096), (64, 65536), (7, 1000), (1, 5), (200, 3001),
                                 (1024, 2048),
                                 (16, 524288),     # 512 column segments: every CTA slot of the margin pass in use
                                 (3, 303108)])     # 297 segments, the last one ragged: one CTA takes two
def test_lr_step_matches_oracle(m, d):
    X, y, _ = synthetic.logistic_problem(m, d, seed=m + d)
    u = (0.3 * synthetic.normal_f32(d, 1.0, 5)).astype(np.float32)
    tu = G.dev(u)
    G.ctx().qesgd_lr_sgd_step(G.dev(X), G.dev(y), m, d, 0.1, tu)
    _lr_close(tu.cpu().numpy(), ref.lr_sgd_step(X, y, 0.1, u))


def test_lr_local_epoch_and_batch_match_oracle():
    K, n_local, d, batch = 3, 150, 2048, 64
    X, y, _ = synthetic.logistic_problem(K * n_local, d, seed=9)
    u0 = np.zeros(d, dtype=np.float32)
    tu = torch.zeros((K, d), dtype=torch.float32, device="cuda")
    G.ctx().qesgd_lr_local_epoch_batch(G.dev(X), G.dev(y), n_local, d, K, batch, 0.5, tu, d)
    got = tu.cpu().numpy()
    for k in range(K):
        rows = slice(k * n_local, (k + 1) * n_local)
        want = ref.lr_local_epoch(X[rows], y[rows], batch, 0.5, u0)
        _lr_close(got[k], want)
    t1 = torch.zeros(d, dtype=torch.float32, device="cuda")
    G.ctx().qesgd_lr_local_epoch(G.dev(X[:n_local]), G.dev(y[:n_local]), n_local, d, batch, 0.5, t1)
    assert (t1.cpu().numpy() == got[0]).all()


@pytest.mark.parametrize("K,n_local,d,batch", [
    (1, 130, 4096, 64),      # one worker: every minibatch waits for the previous update
    (2, 128, 8192, 64),      # even K: a worker's minibatches stay in one consumer group
    (4, 96, 65536, 32),      # the benchmark's width (444 columns per CTA, two TMA boxes)
    (5, 77, 1000, 20),       # odd K, rows not a multiple of 8, ragged last minibatch of 17
    (3, 300, 2048, 256),     # the largest minibatch the persistent kernel takes
    (2, 40, 75776, 8),       # the widest slice (512 columns per CTA)
    (2, 600, 1024, 300),     # minibatch above 256 rows: two-pass steps
    (2, 64, 1002, 32),       # d not a multiple of 4: two-pass steps
    (2, 64, 80000, 32),      # d above 512 columns per SM: two-pass steps
])
def test_lr_local_epoch_shapes_match_oracle(K, n_local, d, batch):
    """The local epoch through the C ABI against the fp64 oracle, over shapes that take the
    persistent kernel (shared-memory tiles, inter-CTA margins) and shapes that fall back to
    one margin pass and one update pass per minibatch."""
    X, y, _ = synthetic.logistic_problem(K * n_local, d, seed=K + n_local + d)
    u0 = (0.1 * synthetic.normal_f32(d, 1.0, 21)).astype(np.float32)
    stride = d + 4 * (K % 2)                       # padded rows for odd K
    tu = torch.zeros((K, stride), dtype=torch.float32, device="cuda")
    tu[:, :d] = G.dev(u0)
    c = G.ctx()
    c.qesgd_lr_local_epoch_batch(G.dev(X), G.dev(y), n_local, d, K, batch, 0.5, tu, stride)
    assert c.qesgd_status() == 0
    got = tu.cpu().numpy()
    for k in range(K):
        rows = slice(k * n_local, (k + 1) * n_local)
        _lr_close(got[k, :d], ref.lr_local_epoch(X[rows], y[rows], batch, 0.5, u0))
    assert (got[:, d:] == 0).all()
    # the same call again gives the same bits (integer sums between the CTAs, fixed order inside them)
    tu2 = torch.zeros((K, stride), dtype=torch.float32, device="cuda")
    tu2[:, :d] = G.dev(u0)
    c.qesgd_lr_local_epoch_batch(G.dev(X), G.dev(y), n_local, d, K, batch, 0.5, tu2, stride)
    assert torch.equal(tu, tu2)


@pytest.mark.parametrize("gain", [2e7, 1e9])
def test_local_epoch_partial_margins_beyond_the_fine_fixed_point_range(gain):
    """The CTAs of the persistent kernel add their partial margins as fixed-point integers: units
    of 2^-28 below 2^17, units of 2^-6 from there on.  With features scaled by 2e7 about half of
    the partial margins of a row take the coarse word and half the fine one; scaled by 1e9 all
    take the coarse one (and the second step's reach 1e13).  The oracle knows no such split."""
    K, n_local, d, batch = 2, 64, 8192, 32
    X, y, _ = synthetic.logistic_problem(K * n_local, d, seed=31)
    X = (X * np.float32(gain)).astype(np.float32)
    u0 = (0.1 * synthetic.normal_f32(d, 1.0, 24)).astype(np.float32)
    c = G.ctx()
    tu = torch.zeros((K, d), dtype=torch.float32, device="cuda")
    tu[:] = G.dev(u0)
    c.qesgd_lr_local_epoch_batch(G.dev(X), G.dev(y), n_local, d, K, batch, 0.5, tu, d)
    assert c.qesgd_status() == 0
    got = tu.cpu().numpy()
    assert np.isfinite(got).all()
    for k in range(K):
        rows = slice(k * n_local, (k + 1) * n_local)
        _lr_close(got[k], ref.lr_local_epoch(X[rows], y[rows], batch, 0.5, u0))


def test_local_epoch_nonfinite_features_spread_as_in_floating_point():
    """A NaN feature makes its row's margin NaN and with it the worker's whole parameter; an
    infinite feature makes the margin that infinity, the step coefficient saturates, and only the
    feature's own column becomes non-finite.  Same pattern as the fp64 oracle; the other worker
    and the finite entries stay within tolerance."""
    K, n_local, d, batch = 2, 96, 8192, 32
    X, y, _ = synthetic.logistic_problem(K * n_local, d, seed=32)
    u0 = (0.1 * synthetic.normal_f32(d, 1.0, 25)).astype(np.float32)
    X[40, 1234] = np.nan                     # worker 0, second minibatch
    X[n_local + 70, 77] = np.inf             # worker 1, last minibatch
    X[n_local + 80, 4000] = -np.inf
    c = G.ctx()
    tu = torch.zeros((K, d), dtype=torch.float32, device="cuda")
    tu[:] = G.dev(u0)
    c.qesgd_lr_local_epoch_batch(G.dev(X), G.dev(y), n_local, d, K, batch, 0.5, tu, d)
    assert c.qesgd_status() == 0
    got = tu.cpu().numpy()
    with np.errstate(all="ignore"):
        want = [ref.lr_local_epoch(X[k * n_local:(k + 1) * n_local], y[k * n_local:(k + 1) * n_local],
                                   batch, 0.5, u0) for k in range(K)]
    assert np.isnan(want[0]).all() and np.isnan(got[0]).all()
    fin = np.isfinite(want[1])
    assert fin.sum() == d - 2 and not fin[77] and not fin[4000]
    assert np.array_equal(np.isnan(got[1]), np.isnan(want[1]))
    assert np.array_equal(got[1][np.isinf(want[1])], want[1][np.isinf(want[1])])
    _lr_close(got[1][fin], want[1][fin])


# ------------------------------ the local-epoch kernel gives up and recovers ---
def _epoch_once(c, X, y, n_local, d, K, batch, u0):
    tu = torch.zeros((K, d), dtype=torch.float32, device="cuda")
    tu[:] = G.dev(u0)
    c.qesgd_lr_local_epoch_batch(X, y, n_local, d, K, batch, 0.5, tu, d)
    return tu, c.qesgd_status()


@pytest.mark.parametrize("K,n_local,d,batch", [
    (2, 96, 8192, 32),       # minibatches stashed in tensor memory between their two uses
    (3, 200, 4096, 100),     # minibatches that stay in shared memory, odd K
])
def test_local_epoch_wait_runs_out_and_the_context_recovers(K, n_local, d, batch):
    """One CTA never announces its partial margins of the first minibatch (a flag nothing
    sets), so every CTA's bounded wait for them runs out: the call returns, the status word
    reports the time-out, nothing faults, and the next call on the same context -- hook off,
    default limit -- matches the oracle and a fresh context bit for bit."""
    X, y, _ = synthetic.logistic_problem(K * n_local, d, seed=5 + K)
    u0 = (0.1 * synthetic.normal_f32(d, 1.0, 22)).astype(np.float32)
    tX, ty = G.dev(X), G.dev(y)
    c = qesgd.Context(0, None)
    c.qesgd_set_wait_limit(3_000_000)              # 3 ms per wait
    c.qesgd_debug_drop_signal(5)
    _, status = _epoch_once(c, tX, ty, n_local, d, K, batch, u0)
    assert status == qesgd.STATUS_TIMEOUT
    assert c.qesgd_status() == 0                   # reading the status word cleared it
    c.qesgd_debug_drop_signal(-1)
    c.qesgd_set_wait_limit(0)                      # back to the default
    after, status = _epoch_once(c, tX, ty, n_local, d, K, batch, u0)
    assert status == 0
    for k in range(K):
        rows = slice(k * n_local, (k + 1) * n_local)
        _lr_close(after[k].cpu().numpy(), ref.lr_local_epoch(X[rows], y[rows], batch, 0.5, u0))
    fresh = qesgd.Context(0, None)
    want, status = _epoch_once(fresh, tX, ty, n_local, d, K, batch, u0)
    assert status == 0 and torch.equal(after, want)
    fresh.close()
    c.close()


def test_local_epoch_with_a_wait_limit_below_the_timer_resolution():
    """A limit under a microsecond means "look once more, then give up": ordinary latency
    between CTAs and of the TMA copies exhausts it at whatever point each CTA happens to be,
    so the give-up path is entered from many places at once.  The call must return either way;
    a run that happened to need no second look is a complete epoch.  The context recovers."""
    K, n_local, d, batch = 4, 256, 16384, 32
    X, y, _ = synthetic.logistic_problem(K * n_local, d, seed=9)
    u0 = (0.1 * synthetic.normal_f32(d, 1.0, 23)).astype(np.float32)
    tX, ty = G.dev(X), G.dev(y)
    want = [ref.lr_local_epoch(X[k * n_local:(k + 1) * n_local], y[k * n_local:(k + 1) * n_local],
                               batch, 0.5, u0) for k in range(K)]
    c = qesgd.Context(0, None)
    for attempt in range(3):
        c.qesgd_set_wait_limit(100)
        got, status = _epoch_once(c, tX, ty, n_local, d, K, batch, u0)
        assert status in (0, qesgd.STATUS_TIMEOUT)
        if status == 0:
            for k in range(K):
                _lr_close(got[k].cpu().numpy(), want[k])
        c.qesgd_set_wait_limit(0)
        got, status = _epoch_once(c, tX, ty, n_local, d, K, batch, u0)
        assert status == 0
        for k in range(K):
            _lr_close(got[k].cpu().numpy(), want[k])
    c.close()


# ----------------------------------------------- per-step QESGD (Algorithm 2) ---
def _gpu_requantize(u, w, zsum, bucket, s, bits, mode, seed, worker, step, fixed_delta=0.0,
                    misalign=0):
    n = u.size
    cb = qesgd.code_bytes(n, bucket, bits)
    nb = qesgd.num_buckets(n, bucket)

    def place(a):
        buf = torch.full((n + misalign + 8,), 55.0, dtype=torch.float32, device="cuda")
        buf[misalign:misalign + n] = G.dev(a)
        return buf, buf[misalign:misalign + n]

    bu, tu = place(u)
    bz, tz = place(zsum) if zsum is not None else (None, None)
    codes = torch.zeros(cb, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(nb + 3, dtype=torch.float32, device="cuda")
    G.ctx().qesgd_requantize(tu, G.dev(w), n, bucket, s, bits, mode, seed, worker, step, tz, codes,
                             scales, fixed_delta)
    st = G.ctx().qesgd_status()
    assert (bu[misalign + n:] == 55.0).all().item() and (bu[:misalign] == 55.0).all().item()
    return (tu.cpu().numpy(), None if tz is None else tz.cpu().numpy(),
            codes.cpu().numpy().view(np.uint32), scales[:nb].cpu().numpy(), st)


@pytest.mark.parametrize("bucket", [64, 256, 1024, 4096])
@pytest.mark.parametrize("bits,s,mode", [(8, 127, 2), (4, 7, 0), (2, 1, 1), (8, 100, 0)])
def test_requantize_matches_oracle_bitwise(bits, s, mode, bucket):
    n = 8192 * 2 + 1000 + 5
    w = synthetic.anchor_vector(n, seed=bucket)
    u = (w + synthetic.delta_vector(n, 1e-3, seed=bucket + 1, outlier_prob=0.01)).astype(np.float32)
    zsum = synthetic.delta_vector(n, 1e-3, seed=bucket + 2)
    delta = 3e-5
    for misalign in (0, 3):
        got = _gpu_requantize(u, w, zsum, bucket, s, bits, mode, 99, 1, 6, delta, misalign)
        want = ref.requantize(u, w, bucket, s, bits, mode, 99, 1, 6, zsum=zsum, fixed_delta=delta)
        assert (got[0].view(np.uint32) == want[0].view(np.uint32)).all()      # u
        assert (got[1].view(np.uint32) == want[1].view(np.uint32)).all()      # running sum
        assert (got[2] == want[2]).all()                                       # codes
        assert (got[3].view(np.uint32) == want[3].view(np.uint32)).all()      # scales
        assert got[4] == want[4]
    got = _gpu_requantize(u, w, None, bucket, s, bits, mode, 99, 1, 6, delta)
    want = ref.requantize(u, w, bucket, s, bits, mode, 99, 1, 6, fixed_delta=delta)
    assert (got[0].view(np.uint32) == want[0].view(np.uint32)).all() and got[1] is None


def test_qesgd_inner_loop_on_the_gpu_follows_the_oracle():
    """Algorithm 2 on a logistic problem: gradient step, requantize, running sum; the GPU's
    u after every step is handed to the oracle's requantize, which must agree bit for bit."""
    m, d, Kt, lr, delta = 64, 4096, 6, 0.5, 2e-4
    X, y, _ = synthetic.logistic_problem(m * Kt, d, seed=17)
    tX, ty = G.dev(X), G.dev(y)
    w = np.zeros(d, dtype=np.float32)
    tw = G.dev(w)
    tu = torch.zeros(d, dtype=torch.float32, device="cuda")
    tz = torch.zeros(d, dtype=torch.float32, device="cuda")
    codes = torch.zeros(qesgd.code_bytes(d, 512, 8), dtype=torch.uint8, device="cuda")
    scales = torch.zeros(qesgd.num_buckets(d, 512), dtype=torch.float32, device="cuda")
    c = G.ctx()
    zsum_ref = np.zeros(d, dtype=np.float32)
    for k in range(Kt):
        rows = slice(k * m, (k + 1) * m)
        c.qesgd_lr_sgd_step(tX[rows].contiguous(), ty[rows].contiguous(), m, d, lr, tu)
        u_hat = tu.cpu().numpy()
        c.qesgd_requantize(tu, tw, d, 512, 127, 8, qesgd.SCALE_FIXED, 3, 0, k, tz, codes, scales, delta)
        u_ref, zsum_ref, c_ref, s_ref, _ = ref.requantize(u_hat, w, 512, 127, 8, ref.SCALE_FIXED, 3, 0, k,
                                                          zsum=zsum_ref, fixed_delta=delta)
        assert (tu.cpu().numpy().view(np.uint32) == u_ref.view(np.uint32)).all()
        assert (tz.cpu().numpy().view(np.uint32) == zsum_ref.view(np.uint32)).all()
        assert (codes.cpu().numpy().view(np.uint32) == c_ref).all()
    assert c.qesgd_status() == 0 and np.abs(zsum_ref).max() > 0


# ------------------------------------------- gradient compression (push side) ---
@pytest.mark.parametrize("m,d,bucket,bits,s,mode,fused", [
    (64, 65536, 512, 8, 127, ref.SCALE_NORM, True),    # the benchmark's logistic shape
    (33, 4100, 64, 4, 7, ref.SCALE_MAX, True),         # ragged last tile, odd row count
    (256, 8192, 1024, 2, 1, ref.SCALE_FIXED, True),    # widest bucket the fused kernel takes
    (16, 524288, 256, 4, 7, ref.SCALE_NORM, True),     # 512 column segments: 296 CTAs in the margin pass
    (64, 8192, 4096, 8, 100, ref.SCALE_NORM, False),   # bucket above 1024: the two calls
    (20, 1002, 128, 4, 7, ref.SCALE_NORM, False),      # d not a multiple of 4: the two calls
])
def test_fused_inner_step_equals_step_then_requantize(m, d, bucket, bits, s, mode, fused):
    """Algorithm 2's inner iteration as one call: gradient step (Eq. 2) on the minibatch, then
    z = Q(z^), u = w_t + z and the running sum.  The gradient step is tolerance-equal to the
    fp64 oracle; from the GPU's own updated parameter on (hand-off) everything must equal the
    oracle's requantisation bit for bit: u, running sum, codes, scales."""
    X, y, _ = synthetic.logistic_problem(m, d, seed=m + d)
    w = synthetic.anchor_vector(d, seed=8)
    u0 = (w + _delta(d, 9, sigma=2e-3)).astype(np.float32)
    zsum0 = _delta(d, 10, sigma=1e-3)
    lr, fixed = 0.3, 4e-3 / s
    c = G.ctx()
    tX, ty = G.dev(X), G.dev(y)
    # the gradient step alone, in the arithmetic the fused call uses
    u1 = G.dev(u0)
    if fused:
        qesgd.qesgd_lr_sgd_step_noalloc(None, tX, ty, m, d, lr, u1)      # always the two-pass form
    else:
        c.qesgd_lr_sgd_step(tX, ty, m, d, lr, u1)
    torch.cuda.synchronize()
    u1 = u1.cpu().numpy()
    _lr_close(u1, ref.lr_sgd_step(X, y, lr, u0))
    want_u, want_zsum, want_codes, want_scales, want_st = ref.requantize(
        u1, w, bucket, s, bits, mode, 21, 3, 7, zsum=zsum0, fixed_delta=fixed)
    # the fused call from the same start
    nb, cb = qesgd.num_buckets(d, bucket), qesgd.code_bytes(d, bucket, bits)
    tu = torch.full((d + 8,), 55.0, dtype=torch.float32, device="cuda")
    tu[:d] = G.dev(u0)
    tz = torch.full((d + 8,), 66.0, dtype=torch.float32, device="cuda")
    tz[:d] = G.dev(zsum0)
    codes = torch.full((cb + 64,), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.full((nb + 16,), -7.0, dtype=torch.float32, device="cuda")
    launches = c.qesgd_launch_count()
    c.qesgd_lr_qesgd_step(tX, ty, m, d, lr, tu[:d], G.dev(w), bucket, s, bits, mode, 21, 3, 7, tz[:d],
                          codes, scales, fixed_delta=fixed)
    assert c.qesgd_status() == want_st
    if fused:
        assert c.qesgd_launch_count() - launches == 2      # margin pass + the fused kernel
    assert (tu[d:] == 55.0).all().item() and (tz[d:] == 66.0).all().item()
    assert (codes[cb:] == 0xAB).all().item() and (scales[nb:] == -7.0).all().item()
    got_u, got_zsum = tu[:d].cpu().numpy(), tz[:d].cpu().numpy()
    assert (scales[:nb].cpu().numpy().view(np.uint32) == want_scales.view(np.uint32)).all()
    assert (codes[:cb].cpu().numpy().view(np.uint32) == want_codes).all()
    assert (got_u.view(np.uint32) == want_u.view(np.uint32)).all()
    assert (got_zsum.view(np.uint32) == want_zsum.view(np.uint32)).all()


@pytest.mark.parametrize("alpha", [-0.1, 1.0, -3.5])
@pytest.mark.parametrize("K,bucket,bits,s", [(4, 128, 4, 7), (16, 256, 2, 1), (3, 1024, 8, 127)])
def test_decode_average_axpy_matches_oracle(K, bucket, bits, s, alpha):
    n = 8192 + 777
    w = synthetic.anchor_vector(n, seed=K)
    codes, scales = [], []
    for k in range(K):
        g = synthetic.delta_vector(n, 1e-2, seed=50 + K, worker=k, outlier_prob=0.01)
        c, sc, _ = ref.encode(g, None, bucket, s, bits, ref.SCALE_NORM, 9, k, 1)
        codes.append(c)
        scales.append(sc)
    codes, scales = np.stack(codes), np.stack(scales)
    nb = scales.shape[1]
    nb_pad = (nb + 3) // 4 * 4
    t_scales = torch.zeros((K, nb_pad), dtype=torch.float32, device="cuda")
    t_scales[:, :nb] = G.dev(scales)
    p = G.dev(w)
    G.ctx().qesgd_decode_average_axpy(p, n, K, G.dev(codes), codes.shape[1] * 4, t_scales, nb_pad,
                                      bucket, s, bits, alpha)
    got = p.cpu().numpy()
    want = ref.decode_average_axpy(w, codes, scales, bucket, s, bits, alpha)
    smax = np.repeat(scales.max(axis=0), bucket)[:n]
    tol = 1e-6 * np.maximum(np.abs(want), abs(alpha) * smax)
    assert (np.abs(got.astype(np.float64) - want) <= tol).all()


@pytest.mark.parametrize("m,d", [(64, 65536), (33, 1001), (256, 4096)])
def test_lr_gradient_matches_oracle_and_quantised_gradient_step(m, d):
    X, y, _ = synthetic.logistic_problem(m, d, seed=3 * m + d)
    w = (0.3 * synthetic.normal_f32(d, 1.0, 8)).astype(np.float32)
    tg = torch.full((d + 4,), 9.0, dtype=torch.float32, device="cuda")
    G.ctx().qesgd_lr_gradient(G.dev(X), G.dev(y), m, d, G.dev(w), tg)
    assert (tg[d:] == 9.0).all().item()
    g = tg[:d].cpu().numpy()
    want = ref.lr_gradient(X, y, w)
    assert np.linalg.norm(g - want) <= 1e-5 * np.linalg.norm(want)
    assert np.abs(g - want).max() <= 1e-5 * np.abs(want).max()
    # the worker pushes the quantised gradient, the server applies -lr * Q(g): hand-off parity
    codes, scales, st = G.gpu_encode(g, None, 256, 127, 8, ref.SCALE_NORM, 5, 0, 0)
    wc, ws, _ = ref.encode(g, None, 256, 127, 8, ref.SCALE_NORM, 5, 0, 0)
    assert st == 0 and (codes == wc).all() and (scales.view(np.uint32) == ws.view(np.uint32)).all()


# ------------------------------------------------------ argument checking ----
def test_quantisation_noise_of_gradient_and_epoch_delta_match_lemma_1():
    """Gradient compression (QSGD baseline of Sec. 5, delta = ||g|| per bucket) against compression
    of the epoch delta (Sec. 2.2) on a logistic problem, same width and bucket: for both vectors
    the library's E||Q(v) - v||^2 over many draws equals Lemma 1's closed form
    sum delta^2 p (1 - p) -- computed here by the CPU oracle's scales and exact fractions -- and
    stays below d * delta^2 / 4; one draw of each is bit-identical to the oracle's."""
    import bench
    n_local, d, batch, lr, bucket = 256, 8192, 32, 0.1, 512
    X, y, _ = synthetic.logistic_problem(n_local, d, seed=77)
    c = G.ctx()
    tX, ty = G.dev(X), G.dev(y)
    w = torch.zeros(d, dtype=torch.float32, device="cuda")
    g = torch.empty(d, dtype=torch.float32, device="cuda")
    u = torch.zeros((1, d), dtype=torch.float32, device="cuda")
    c.qesgd_lr_gradient(tX[:batch].contiguous(), ty[:batch].contiguous(), batch, d, w, g)
    c.qesgd_lr_local_epoch_batch(tX, ty, n_local, d, 1, batch, lr, u, d)
    torch.cuda.synchronize()
    z = (u[0] - w).contiguous()
    for bits, s in ((8, 127), (2, 1)):
        for name, v in (("gradient", g), ("epoch delta", z)):
            got = bench.quantisation_variance(c, v, bucket, s, bits, draws=64)
            hv = v.cpu().numpy()
            # closed form from the oracle's side: its scales, exact fractional parts
            _, r_scales, _ = ref.encode(hv, None, bucket, s, bits, ref.SCALE_NORM, 5, 0, 0)
            delta = np.repeat((r_scales / np.float32(s)).astype(np.float64), bucket)[:d]
            r = np.abs(hv.astype(np.float64)) / delta
            p = r - np.floor(r)
            closed = float((delta ** 2 * p * (1 - p)).sum())
            assert abs(got["closed_form"] - closed) <= 1e-6 * closed, name
            # 64 draws x 8192 coordinates: the standard error of the mean is below 1 % even for 2-bit codes
            assert abs(got["monte_carlo"] - closed) <= 0.04 * closed, (name, bits, got)
            assert got["monte_carlo"] <= got["bound_d_delta2_over_4"]
            gc, gs, _ = G.gpu_encode(hv, None, bucket, s, bits, ref.SCALE_NORM, 5, 0, 3)
            wc, ws, _ = ref.encode(hv, None, bucket, s, bits, ref.SCALE_NORM, 5, 0, 3)
            assert (gc == wc).all() and (gs.view(np.uint32) == ws.view(np.uint32)).all()


def test_invalid_arguments_return_einval_and_launch_nothing():
    c = G.ctx()
    z = torch.zeros(4096, device="cuda")
    codes, scales = qesgd.alloc_stream_buffers(1, 4096, 512, 4, "cuda")
    before = c.qesgd_launch_count()
    bad = [dict(bucket=48), dict(bucket=16384), dict(bits=3), dict(s=8), dict(s=0), dict(mode=3)]
    for kw in bad:
        a = dict(bucket=512, s=7, bits=4, mode=0)
        a.update(kw)
        with pytest.raises(qesgd.QesgdError) as ei:
            c.qesgd_encode(z, None, 4096, a["bucket"], a["s"], a["bits"], a["mode"], 0, 0, 0,
                           codes, scales)
        assert ei.value.code == qesgd.EINVAL
    with pytest.raises(qesgd.QesgdError):
        c.qesgd_encode(z, None, 4096, 512, 7, 4, qesgd.SCALE_FIXED, 0, 0, 0, codes, scales,
                       fixed_delta=0.0)
    with pytest.raises(qesgd.QesgdError):
        c.qesgd_encode(None, None, 4096, 512, 7, 4, 0, 0, 0, 0, codes, scales)
    with pytest.raises(qesgd.QesgdError):
        c.qesgd_decode_average_apply(z, 4096, 65, codes, 0, scales, 0, 512, 7, 4)
    with pytest.raises(qesgd.QesgdError):
        c.qesgd_encode(z, None, 4096, 512, 7, 4, 0, 0, 0, 0, codes.view(-1)[4:], scales)
    c.qesgd_encode(z, None, 0, 512, 7, 4, 0, 0, 0, 0, codes, scales)      # d = 0: no-op
    c.qesgd_decode_average_apply(z, 0, 3, codes, 0, scales, 0, 512, 7, 4)
    assert c.qesgd_launch_count() == before
    assert c.qesgd_status() == 0


# ----------------------------------------------------------- graph replay ----
def test_round_recorded_into_a_cuda_graph_replays_bit_identically():
    """The codec calls only enqueue kernels on the context's stream, so a round (encode of all
    workers, then decode-average-apply) can be recorded by stream capture; replaying the graph
    must give exactly what the direct calls give."""
    K, d, bucket, s, bits = 4, 3 * 4096 + 77, 256, 7, 4
    stream = torch.cuda.Stream()
    ctx = qesgd.Context(0, stream)
    stride = (d + 7) // 8 * 8
    anchor = G.dev(synthetic.anchor_vector(d, seed=5))
    locs = torch.zeros((K, stride), dtype=torch.float32, device="cuda")
    for k in range(K):
        locs[k, :d] = anchor + G.dev(_delta(d, seed=60 + k))
    codes, scales = qesgd.alloc_stream_buffers(K, d, bucket, bits, "cuda")

    def one_round(param):
        ctx.qesgd_encode_batch(locs, stride, anchor, d, K, bucket, s, bits, qesgd.SCALE_NORM, 11, 0, 2,
                               codes, codes.stride(0), scales, scales.stride(0))
        ctx.qesgd_decode_average_apply(param, d, K, codes, codes.stride(0), scales, scales.stride(0),
                                       bucket, s, bits)
    direct = anchor.clone()
    torch.cuda.synchronize()
    one_round(direct)
    stream.synchronize()
    want_codes, want_scales = codes.clone(), scales.clone()
    codes.zero_()
    scales.zero_()
    replayed = anchor.clone()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        one_round(replayed)
    assert (codes == 0).all()                     # capture records, it does not run
    with torch.cuda.stream(stream):
        graph.replay()
    stream.synchronize()
    assert ctx.qesgd_status() == 0
    assert torch.equal(codes, want_codes) and torch.equal(scales, want_scales)
    assert torch.equal(replayed, direct)
    ctx.close()
