"""mpt_softmax_ce_static: the softmax cross-entropy entry point for callers that cannot
allocate device memory (a plugin living on a framework's fixed tensors, or a loop that must
not pay cudaMalloc's device-wide synchronisation) and so have no float[B] scratch to pass.

Its results must equal those of mpt_softmax_ce, which takes the scratch from the caller.
Two calls in a row are checked, the second with fewer rows and different values, so that
whatever the first call left in the library's built-in array cannot leak into the second.
The file name makes pytest collect this test last."""
import numpy as np
import pytest

from gpu_util import dev, host_u16, require_gpu, torch

pytestmark = pytest.mark.gpu


def _both(z16, labels, S, ld):
    from paper_1710_03740_b200 import binding as b
    B, C = z16.shape
    zp = np.zeros((B, ld), dtype=np.uint16)
    zp[:, :C] = z16.view(np.uint16)
    zd, yd = dev(zp), dev(labels.astype(np.int32))
    out = []
    for static in (False, True):
        dz = torch.full((B, ld), 0x5555, dtype=torch.int16, device="cuda")
        loss = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        bad = torch.full((1,), 77, dtype=torch.int32, device="cuda")
        if static:
            b.mpt_softmax_ce_static(zd, ld, yd, B, C, S, dz, ld, loss, bad)
        else:
            rl = torch.zeros(B, dtype=torch.float32, device="cuda")
            b.mpt_softmax_ce(zd, ld, yd, B, C, S, dz, ld, rl, loss, bad)
        torch.cuda.synchronize()
        out.append((host_u16(dz), float(loss.item()), int(bad.item())))
    return out


def test_static_scratch_variant_matches_on_two_calls_in_a_row():
    require_gpu()
    from paper_1710_03740_b200 import binding as b
    rng = np.random.default_rng(99)
    # first call: many rows, one label out of range; second call: fewer rows, other values
    for B, C, ld, S in ((300, 1000, 1000, 1024.0), (37, 10, 16, 8.0)):
        z = (rng.standard_normal((B, C)) * 5).astype(np.float16)
        y = rng.integers(0, C, B)
        if B == 300:
            y[17] = C
        (dz_a, loss_a, bad_a), (dz_b, loss_b, bad_b) = _both(z, y, S, ld)
        # same kernels and arithmetic on both paths: identical bits, well inside the 2-ulp rule
        assert np.array_equal(dz_a, dz_b)
        assert loss_a == loss_b and np.isfinite(loss_a)
        assert bad_a == bad_b == (1 if B == 300 else 0)
    # sizes beyond the built-in array are refused with a clear error and nothing is launched
    zd = torch.zeros((8, 8), dtype=torch.int16, device="cuda")
    yd = torch.zeros(8, dtype=torch.int32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    with pytest.raises(b.MptError) as e:
        b.mpt_softmax_ce_static(zd, 8, yd, 65537, 8, 1.0, zd.clone(), 8, loss)
    assert e.value.code == -2
