"""The allocation-free entry point, `la_replica_means_static`, for users who cannot call
cudaMalloc at run time (all device memory already belongs to their own allocator, or their
service forbids allocation once started).  It must give the bits that the ordinary path
(`la_sync` on a context holding the same replicas) gives, on two calls in a row — the second
call reuses the library's one fixed scratch array, which still holds the first call's sums."""
import numpy as np
import pytest

from paper_1911_09030_b200 import local_adaalter as la

pytestmark = pytest.mark.gpu


def _reference_means(x, b2, W, n):
    """The existing entry point: put the replicas into a context, la_sync, read the result."""
    g = la.LocalAdaAlter([n], W, 0.1, 1.0, 4)
    for i in range(W):
        g.write_state(i, x[i, :n].copy(), b2[i, :n].copy(), None)
    g.sync()
    xm, bm, _ = g.read_state(0)
    g.close()
    return xm, bm


@pytest.mark.parametrize("W,n", [(4, 5000), (3, 1), (16, 70001), (8, la.LA_STATIC_SCRATCH_MAX_COORDS)])
def test_static_scratch_means_equal_la_sync_twice_in_a_row(W, n):
    import torch
    stride = (n + 63) // 64 * 64
    rng = np.random.default_rng(W * 1000 + n % 997)
    for call in range(2):                       # second call: scratch is dirty from the first
        x = (rng.standard_normal((W, stride)) * 10.0 ** rng.integers(-3, 3, (W, 1))).astype(np.float32)
        b2 = np.abs(rng.standard_normal((W, stride))).astype(np.float32)
        xd, bd = torch.from_numpy(x).cuda(), torch.from_numpy(b2).cuda()
        xm = torch.full((n,), float("nan"), device="cuda")
        bm = torch.full((n,), float("nan"), device="cuda")
        rc = la.replica_means_static(xd.data_ptr(), bd.data_ptr(), W, n, stride, xm.data_ptr(), bm.data_ptr(),
                                     torch.cuda.current_stream().cuda_stream)
        assert rc == la.LA_OK
        torch.cuda.synchronize()
        ref_x, ref_b = _reference_means(x, b2, W, n)
        assert np.array_equal(xm.cpu().numpy().view(np.uint32), ref_x.view(np.uint32))
        assert np.array_equal(bm.cpu().numpy().view(np.uint32), ref_b.view(np.uint32))
        assert torch.equal(xd.cpu(), torch.from_numpy(x))          # inputs untouched


def test_static_scratch_rejects_what_it_cannot_hold():
    import torch
    big = la.LA_STATIC_SCRATCH_MAX_COORDS + 64
    t = torch.zeros(8, device="cuda")
    p = t.data_ptr()
    assert la.replica_means_static(p, p, 2, big, big, p, p) == la.LA_ETOOBIG
    assert la.replica_means_static(p, p, 0, 4, 4, p, p) == la.LA_EINVAL
    assert la.replica_means_static(p, p, 2, 8, 4, p, p) == la.LA_EINVAL      # stride < n
    assert la.replica_means_static(0, p, 2, 4, 4, p, p) == la.LA_EINVAL
    assert la.replica_means_static(p, p, 2, 4, 4, p, p) == la.LA_OK          # still usable afterwards
    torch.cuda.synchronize()
