"""Parity of the fused softmax cross-entropy with the oracle (paper sections 3.2, 3.3)."""
import numpy as np
import pytest

from oracle import mpo
from parity import gemm_accept
from gpu_util import dev, host_u16, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _run(z16, labels, S, ldz=None):
    from paper_1710_03740_b200 import binding as b
    B, C = z16.shape
    ld = C if ldz is None else ldz
    zp = np.zeros((B, ld), dtype=np.uint16)
    zp[:, :C] = z16.view(np.uint16)
    zd = dev(zp)
    dzd = torch.full((B, ld), 0x5555, dtype=torch.int16, device="cuda")
    rl = torch.zeros(B, dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.mpt_softmax_ce(zd, ld, dev(labels.astype(np.int32)), B, C, S, dzd, ld, rl, loss, bad)
    torch.cuda.synchronize()
    out = host_u16(dzd)
    assert np.all(out[:, C:] == 0x5555)            # padding columns untouched
    return out[:, :C], rl.cpu().numpy(), float(loss.item()), int(bad.item())


@pytest.mark.parametrize("B,C,ld", [(64, 10, 16), (256, 10, 10), (7, 1, 8), (33, 1000, 1000), (5, 1003, 1008),
                                    (16, 32000, 32000), (3, 120001, 120008)])
def test_softmax_ce_parity(B, C, ld):
    rng = np.random.default_rng(B * 1000 + C)
    z = (rng.standard_normal((B, C)) * 4).astype(np.float16)
    y = rng.integers(0, C, B)
    S = 1024.0
    dz_ref, rl_ref, loss_ref, _ = mpo.softmax_ce(z, y, S)
    dz, rl, loss, bad = _run(z, y, S, ld)
    assert bad == 0
    ok, stats = gemm_accept(dz, dz_ref)
    assert ok.all(), stats
    assert stats["max_ulp"] <= 2
    # The oracle adds C terms one after the other in FP32: its sum, and with it log(s), may be
    # off by up to C*2^-24 relative; the kernel's pairwise order is closer to the true value.
    assert np.allclose(rl, rl_ref, rtol=2e-6, atol=C * 2.0 ** -24 + 2e-6)
    z64 = z.astype(np.float64)
    m64 = z64.max(1)
    rl64 = m64 + np.log(np.exp(z64 - m64[:, None]).sum(1)) - z64[np.arange(B), y]
    assert np.allclose(rl, rl64, rtol=4e-6, atol=4e-6)
    assert abs(loss - rl64.mean()) <= 4e-6 * max(1.0, abs(rl64.mean()))
    assert abs(loss - loss_ref) <= (C * 2.0 ** -24 + 1e-5) * max(1.0, abs(loss_ref))


def test_softmax_ce_edge_values():
    C = 24
    z = np.zeros((6, C), dtype=np.float16)
    z[1, 3] = 40.0                     # dominant logit
    z[2, :] = 65504.0                  # all at the FP16 maximum
    z[3, 5] = np.nan                   # NaN reaches the whole row
    z[4, 0] = np.inf                   # inf - inf
    z[5, :] = -65504.0
    y = np.array([0, 3, 1, 2, 0, 7])
    dz_ref, rl_ref, loss_ref, _ = mpo.softmax_ce(z, y, 2.0 ** 14)
    dz, rl, loss, bad = _run(z, y, 2.0 ** 14)
    ok, stats = gemm_accept(dz, dz_ref)
    assert ok.all(), stats
    assert np.array_equal(np.isnan(rl), np.isnan(rl_ref))
    fin = ~np.isnan(rl_ref)
    assert np.allclose(rl[fin], rl_ref[fin], rtol=2e-6, atol=2e-6)
    assert np.isnan(loss) and np.isnan(loss_ref)


def test_softmax_ce_bad_labels():
    z = np.zeros((4, 10), dtype=np.float16)
    y = np.array([0, 10, -1, 9])
    dz_ref, rl_ref, loss_ref, bad_ref = mpo.softmax_ce(z, y, 8.0)
    dz, rl, loss, bad = _run(z, y, 8.0, 16)
    assert bad == bad_ref == 2
    assert np.array_equal(dz, dz_ref) or gemm_accept(dz, dz_ref)[0].all()
    assert not dz[1].any() and not dz[2].any()
    assert abs(loss - loss_ref) < 1e-6


@pytest.mark.parametrize("B,C,ld", [(300, 16384, 16384), (457, 32000, 32008), (296, 20480, 20480), (1000, 32768, 32768)])
def test_softmax_ce_bulk_staged_rows(B, C, ld):
    """Many long rows take the persistent kernel whose rows travel through shared memory by bulk
    copies (three buffers per CTA: several rows per CTA, ragged last round, pitched rows).  Edge
    rows (NaN, inf, all-equal maxima, labels outside the range) are mixed in."""
    rng = np.random.default_rng(B + C)
    z = (rng.standard_normal((B, C)) * 4).astype(np.float16)
    y = rng.integers(0, C, B)
    z[3, 5] = np.nan
    z[4, 0] = np.inf
    z[5, :] = 65504.0
    z[6, 17] = 40.0
    y[7] = C            # outside the range
    y[B - 1] = -1
    y[8] = C - 1
    S = 8192.0
    dz_ref, rl_ref, loss_ref, bad_ref = mpo.softmax_ce(z, y, S)
    dz, rl, loss, bad = _run(z, y, S, ld)
    assert bad == bad_ref == 2
    ok, stats = gemm_accept(dz, dz_ref)
    assert ok.all(), stats
    assert stats["max_ulp"] <= 2
    assert not dz[7].any() and not dz[B - 1].any()
    assert np.array_equal(np.isnan(rl), np.isnan(rl_ref))
    fin = ~np.isnan(rl_ref)
    assert np.allclose(rl[fin], rl_ref[fin], rtol=2e-6, atol=C * 2.0 ** -24 + 2e-6)
    # identical bits on a second run
    dz2, rl2, _, _ = _run(z, y, S, ld)
    assert np.array_equal(dz, dz2) and np.array_equal(rl.view(np.uint32), rl2.view(np.uint32))
