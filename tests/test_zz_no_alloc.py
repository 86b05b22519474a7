"""mpt_softmax_ce_static: the softmax cross-entropy entry point for callers that cannot
allocate device memory (a plugin living on a framework's fixed tensors, or a loop that must
not pay cudaMalloc's device-wide synchronisation) and so have no float[B] scratch to pass.

Its results must equal those of mpt_softmax_ce, which takes the scratch from the caller, and
both must agree with the CPU oracle under the tolerance the other softmax tests use (gradient
within 2 FP16 ulp / 1e-2 relative, loss within the summation bound of the row losses).
Calls follow one another without any clean-up in between, with different row counts and values
and through both row kernels (rows held in registers; rows staged in shared memory by bulk
copies), so that whatever one call left in the library's built-in array cannot leak into the
next.  The file name makes pytest collect this test last."""
import numpy as np
import pytest

from oracle import mpo
from parity import gemm_accept
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
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if static:
            b.mpt_softmax_ce_static(zd, ld, yd, B, C, S, dz, ld, loss, bad, status=status)
        else:
            rl = torch.zeros(B, dtype=torch.float32, device="cuda")
            b.mpt_softmax_ce(zd, ld, yd, B, C, S, dz, ld, rl, loss, bad, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        out.append((host_u16(dz)[:, :C], float(loss.item()), int(bad.item())))
    return out


# (rows, classes, pitch, S, rows with a label outside [0, C))
CASES = [
    (300, 1000, 1000, 1024.0, 1),      # rows in registers; one bad label
    (300, 16384, 16384, 8192.0, 0),    # rows staged through shared memory by bulk copies (>= 296 rows, >= 16384 classes)
    (37, 10, 16, 8.0, 0),              # fewer rows than either call before: stale entries must not be read
    (65536, 8, 8, 64.0, 0),            # the largest batch the built-in array holds
    (296, 16392, 16392, 1.0, 2),       # bulk-staged again, after the array was filled to the end
]


def test_static_scratch_variant_matches_on_calls_in_a_row():
    require_gpu()
    from paper_1710_03740_b200 import binding as b
    rng = np.random.default_rng(99)
    for B, C, ld, S, n_bad in CASES:
        z = (rng.standard_normal((B, C)) * 5).astype(np.float16)
        y = rng.integers(0, C, B)
        for k in range(n_bad):
            y[17 + 5 * k] = C + k
        (dz_a, loss_a, bad_a), (dz_b, loss_b, bad_b) = _both(z, y, S, ld)
        # same kernels and arithmetic on both paths: identical bits
        assert np.array_equal(dz_a, dz_b), (B, C)
        assert loss_a == loss_b and np.isfinite(loss_a)
        assert bad_a == bad_b == n_bad
        # and both against the oracle, under the tolerance of the softmax parity tests
        dz_ref, _, loss_ref, bad_ref = mpo.softmax_ce(z, y, S)
        ok, stats = gemm_accept(dz_b, dz_ref)
        assert ok.all(), (B, C, stats)
        assert bad_ref == n_bad
        assert abs(loss_b - loss_ref) <= (C * 2.0 ** -24 + 4e-6) * abs(loss_ref) + 1e-7, (B, C, loss_b, loss_ref)
    # sizes beyond the built-in array are refused with a clear error and nothing is launched
    zd = torch.zeros((8, 8), dtype=torch.int16, device="cuda")
    yd = torch.zeros(8, dtype=torch.int32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    with pytest.raises(b.MptError) as e:
        b.mpt_softmax_ce_static(zd, 8, yd, 65537, 8, 1.0, zd.clone(), 8, loss)
    assert e.value.code == -2
