"""The failure path of the bounded device-side waits, exercised without hanging anything: a
one-CTA kernel waits for a millisecond on a barrier that nothing signals, gives up, records its
code and returns.  Stateless: the status word is set and the call maps it to MPT_ERR_TIMEOUT.
Through a context: the same expiry poisons the context (only the error message and the
destructor work afterwards) while the CUDA context and other mpt contexts stay usable."""
import time

import numpy as np
import pytest

from paper_1710_03740_b200 import inputs
from gpu_util import dev, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def test_stateless_wait_runs_out_and_is_reported():
    from paper_1710_03740_b200 import binding as b
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = time.time()
    code = b.mpt_selftest_wait_timeout(1000, status)
    dt = time.time() - t0
    assert code == -6                                   # MPT_ERR_TIMEOUT
    word = int(status.item()) & 0xFFFFFFFF
    assert word & 0xFF == (6 | 0x20) and word >> 8 == 0  # KERR_WAIT_SELFTEST, CTA 0
    assert dt < 1.0                                     # it gave up after about a millisecond, not 2 s
    # a longer limit takes correspondingly longer: the limit is what ends the wait
    status.zero_()
    t0 = time.time()
    assert b.mpt_selftest_wait_timeout(200000, status) == -6
    assert 0.15 < time.time() - t0 < 1.5
    # the CUDA context is intact: ordinary work still runs
    x = torch.arange(1024, device="cuda")
    assert int(x.sum().item()) == 1023 * 1024 // 2
    # argument checks
    assert b.mpt_selftest_wait_timeout(0, status) == -1
    assert b.mpt_selftest_wait_timeout(1000, None) == -1


def test_expiry_poisons_the_context_and_only_that_context():
    from paper_1710_03740_b200 import binding as b
    cfg = inputs.MLP_CONFIGS["tiny"]
    masters = inputs.mlp_masters(cfg)
    X, Y = inputs.mlp_batches(cfg, 1)
    nets = []
    for _ in range(2):
        net = b.Context(cfg["layers"], cfg["S"], cfg["lr"], cfg["momentum"], cfg["batch"])
        for l, w in enumerate(masters):
            net.set_master(l, w)
        nets.append(net)
    bad, good = nets
    xd, yd = dev(X[0].view(np.uint16)), dev(Y[0])
    bad.forward(xd)
    with pytest.raises(b.MptError) as e:
        bad.selftest_wait_timeout()
    assert e.value.code == -6
    assert "bounded wait expired" in bad.last_error()
    # poisoned: every further call is refused with MPT_ERR_STATE, the message stays readable
    for call in (lambda: bad.forward(xd), lambda: bad.backward_scaled(yd), lambda: bad.step(),
                 lambda: bad.get_master(0), lambda: bad.get_scale(), lambda: bad.selftest_wait_timeout()):
        with pytest.raises(b.MptError) as e2:
            call()
        assert e2.value.code == -3
    assert "bounded wait expired" in bad.last_error()
    bad.close()
    # the other context is untouched and trains
    good.forward(xd)
    loss = good.backward_scaled(yd)
    assert np.isfinite(loss) and good.step() == 0
    good.close()


def test_softmax_status_word_stays_clear_on_the_bulk_kernel():
    """The stateless softmax launchers take a status word for the row-staging kernel's bounded
    waits; a healthy run leaves it at zero."""
    from paper_1710_03740_b200 import binding as b
    B, C = 300, 16384
    rng = np.random.default_rng(5)
    z = dev(rng.standard_normal((B, C)).astype(np.float16).view(np.uint16))
    y = dev(rng.integers(0, C, B).astype(np.int32))
    dz = torch.empty((B, C), dtype=torch.int16, device="cuda")
    rl = torch.empty(B, dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.mpt_softmax_ce(z, C, y, B, C, 128.0, dz, C, rl, loss, None, status=status)
    b.mpt_softmax_ce_static(z, C, y, B, C, 128.0, dz, C, loss, None, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and np.isfinite(float(loss.item()))


def test_sm_clock_probe_reports_a_plausible_clock():
    from paper_1710_03740_b200 import binding as b
    mhz = torch.zeros(2, dtype=torch.float32, device="cuda")
    b.mpt_sm_clock_probe(50, mhz[0:1])
    b.mpt_sm_clock_probe(200, mhz[1:2])
    torch.cuda.synchronize()
    a, c = mhz.tolist()
    assert 100.0 < a < 2500.0 and 100.0 < c < 2500.0
    with pytest.raises(b.MptError):
        b.mpt_sm_clock_probe(0, mhz)
