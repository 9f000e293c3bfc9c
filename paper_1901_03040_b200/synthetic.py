"""Seeded synthetic inputs for the QESGD hot path.

Only input generation lives here: no quantiser, decoder or SGD arithmetic.
The same arrays are handed to the CUDA library and to whatever checks it.

The vectors stand in for flattened network parameters and their epoch deltas:
only the sizes (a ResNet-18-sized 11 689 512 and a ResNet-50-sized 25 557 032
flat vector) and plausible magnitudes are borrowed; values are i.i.d. normal.
"""
import numpy as np

RESNET18_D = 11_689_512
RESNET50_D = 25_557_032
ANCHOR_SIGMA = 0.05


def _rng(seed, stream=0):
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def normal_f32(n, sigma, seed, stream=0):
    """n i.i.d. N(0, sigma^2) values, drawn in fp32."""
    out = _rng(seed, stream).standard_normal(int(n), dtype=np.float32)
    out *= np.float32(sigma)
    return out


def anchor_vector(d, seed):
    """The server's parameter w_t ~ N(0, 0.05^2)."""
    return normal_f32(d, ANCHOR_SIGMA, seed, stream=1)


def delta_vector(d, sigma, seed, worker=0, outlier_prob=0.0, outlier_gain=100.0):
    """One worker's epoch delta ~ N(0, sigma^2); each element independently
    multiplied by outlier_gain with probability outlier_prob (heavy tail)."""
    z = normal_f32(d, sigma, seed, stream=100 + worker)
    if outlier_prob > 0.0:
        hit = _rng(seed, 10_000 + worker).random(int(d), dtype=np.float32) < outlier_prob
        z[hit] *= np.float32(outlier_gain)
    return z


def worker_locals(anchor, K, sigma, seed, outlier_prob=0.0, outlier_gain=100.0):
    """float32[K, d]: local_k = fl32(anchor + z_k) with independent deltas."""
    d = anchor.size
    out = np.empty((K, d), dtype=np.float32)
    for k in range(K):
        np.add(anchor, delta_vector(d, sigma, seed, k, outlier_prob, outlier_gain), out=out[k])
    return out


def logistic_problem(n, d, seed, flip=0.05):
    """Dense binary classification data: x ~ N(0, 1/d), y = sign(x . w*) with
    w* ~ N(0, 1), a fraction `flip` of the labels negated.  Returns (X, y, w*)."""
    w_star = normal_f32(d, 1.0, seed, stream=2)
    X = np.empty((n, d), dtype=np.float32)
    g = _rng(seed, 3)
    rows = max(1, (1 << 24) // max(1, d))
    inv = np.float32(1.0 / np.sqrt(d))
    for r in range(0, n, rows):
        blk = g.standard_normal((min(rows, n - r), d), dtype=np.float32)
        blk *= inv
        X[r:r + blk.shape[0]] = blk
    y = np.where(X.astype(np.float64) @ w_star.astype(np.float64) >= 0.0, 1.0, -1.0)
    flips = _rng(seed, 4).random(n) < flip
    y[flips] = -y[flips]
    return X, y.astype(np.float32), w_star


def device_normal_f32(shape, sigma, seed, device, outlier_prob=0.0, outlier_gain=100.0):
    """Same distributions drawn directly in device memory with torch's seeded
    generator, for vectors too large to draw on the host in reasonable time."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    out = torch.empty(shape, dtype=torch.float32, device=device)
    flat = out.view(-1)
    step = 1 << 28
    for lo in range(0, flat.numel(), step):
        part = flat[lo:lo + step]
        part.normal_(0.0, float(sigma), generator=g)
        if outlier_prob > 0.0:
            hit = torch.rand(part.shape, device=device, generator=g) < outlier_prob
            part[hit] *= outlier_gain
    return out
