"""The entry point for callers that may not allocate device memory when they take a
logistic SGD step (allocator callbacks, fixed-budget hosts): it must give what the
context-based entry point gives, call after call, through the C ABI.

This file sorts last on purpose: it exercises one extra entry point and, should it
fail, every other test has already run."""
import ctypes as C

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_1901_03040_b200 import qesgd, synthetic          # noqa: E402


def _step_noalloc(X, y, m, d, lr, u):
    rc = qesgd.lib.qesgd_lr_sgd_step_noalloc(None, C.c_void_p(X.data_ptr()), C.c_void_p(y.data_ptr()),
                                             m, d, lr, C.c_void_p(u.data_ptr()))
    assert rc == qesgd.OK, qesgd.lib.qesgd_strerror(rc)


@pytest.mark.parametrize("m,d", [(64, 65536), (100, 3001), (256, 4096), (256, 65536), (16, 524288)])
def test_noalloc_step_matches_the_oracle_and_the_context_entry_point_twice_in_a_row(m, d):
    """Two calls in a row, the second continuing from the first one's result.  Each result is
    compared with the fp64 CPU oracle's step from the same starting point (the tolerance of
    the logistic step, 1e-5) and then with what the context entry point gives.  The last shape
    (256 rows, 64 column segments) uses as many partial-margin slots as the fixed array holds
    (62 of 256 rows beside its counters and margins)."""
    from oracle import qesgd_ref as ref
    torch.cuda.set_device(0)
    X, y, _ = synthetic.logistic_problem(2 * m, d, seed=m + d)
    tX, ty = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    u0 = (0.2 * synthetic.normal_f32(d, 1.0, 3)).astype(np.float32)
    want = torch.from_numpy(u0).cuda()
    got = torch.from_numpy(u0).cuda()
    ctx = qesgd.Context(0, None)
    for call in range(2):
        rows = slice(call * m, (call + 1) * m)
        xb, yb = tX[rows].contiguous(), ty[rows].contiguous()
        start = got.cpu().numpy()
        oracle = ref.lr_sgd_step(X[rows], y[rows], 0.1, start).astype(np.float64)
        ctx.qesgd_lr_sgd_step(xb, yb, m, d, 0.1, want)
        _step_noalloc(xb, yb, m, d, 0.1, got)
        torch.cuda.synchronize()
        w, g = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
        assert np.linalg.norm(g - oracle) <= 1e-5 * np.linalg.norm(oracle)
        assert np.abs(g - oracle).max() <= 1e-5 * np.abs(oracle).max()
        # the step itself (not only the vector it is added to) is right
        step_ref = oracle - start.astype(np.float64)
        assert np.linalg.norm((g - start) - step_ref) <= 1e-3 * np.linalg.norm(step_ref)
        assert np.linalg.norm(g - w) <= 1e-5 * np.linalg.norm(w)
        assert np.abs(g - w).max() <= 1e-5 * np.abs(w).max()
        assert not np.array_equal(g, u0)
    ctx.close()


def test_noalloc_limits_and_arguments():
    torch.cuda.set_device(0)
    d = 512
    x = torch.zeros((qesgd.NOALLOC_MAX_LR_BATCH + 1, d), device="cuda")
    y = torch.ones(qesgd.NOALLOC_MAX_LR_BATCH + 1, device="cuda")
    u = torch.zeros(d, device="cuda")
    lib = qesgd.lib
    args = (C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr()))
    assert lib.qesgd_lr_sgd_step_noalloc(None, *args, qesgd.NOALLOC_MAX_LR_BATCH + 1, d, 0.1,
                                         C.c_void_p(u.data_ptr())) == qesgd.ELIMIT
    assert b"no-allocation" in lib.qesgd_strerror(qesgd.ELIMIT)
    assert lib.qesgd_lr_sgd_step_noalloc(None, *args, 0, d, 0.1, C.c_void_p(u.data_ptr())) == qesgd.EINVAL
    assert lib.qesgd_lr_sgd_step_noalloc(None, None, None, 4, d, 0.1, None) == qesgd.EINVAL
    assert lib.qesgd_lr_sgd_step_noalloc(None, *args, 4, 0, 0.1, C.c_void_p(u.data_ptr())) == qesgd.OK
    with pytest.raises(qesgd.QesgdError):
        qesgd.qesgd_lr_sgd_step_noalloc(None, x, y, qesgd.NOALLOC_MAX_LR_BATCH + 1, d, 0.1, u)
    torch.cuda.synchronize()
    assert (u == 0).all().item()          # nothing was enqueued by the rejected calls
