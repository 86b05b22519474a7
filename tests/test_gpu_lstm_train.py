"""The LSTM layer with projection as a trained layer (the paper's language-model layer: loss
scale, overflow skip, Adagrad on FP32 masters) against the CPU oracle, through the C ABI:
free-running multi-step loss trajectories within 1e-3, equal skip flags and scales, and the
optimizer step bit for bit when the oracle is fed the device's own gradient bits and the state
the device held before the step."""
import numpy as np
import pytest

from oracle import mpo
from oracle.lstm import OracleLSTMTrainer
from paper_1710_03740_b200 import inputs
from gpu_util import dev, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _case(T, B, I, H, P, seed, steps):
    rng = np.random.default_rng(seed)
    K = I + P
    Wg = inputs.normal_f16(rng, (4 * H, K), K ** -0.5).astype(np.float32)
    bias = inputs.normal_f16(rng, (4 * H,), 0.1).astype(np.float32)
    Wp = inputs.normal_f16(rng, (P, H), 2.0 * H ** -0.5).astype(np.float32)
    xs = [inputs.normal_f16(rng, (T, B, I), 1.0) for _ in range(steps)]
    ys = [rng.integers(0, P, T * B).astype(np.int32) for _ in range(steps)]
    return Wg, bias, Wp, xs, ys


def _pair(dims, S, opt_args, Wg, bias, Wp):
    from paper_1710_03740_b200 import binding as b
    kind, lr, mu, b2, eps, wd, clip = opt_args
    gpu = b.LstmTrainer(*dims, S, b.Optimizer(kind, lr, mu, b2, eps, wd, clip))
    gpu.set_params(Wg, bias, Wp)
    ora = OracleLSTMTrainer(*dims, S, kind, lr, mu=mu, b2=b2, eps=eps, wd=wd, clip=clip)
    ora.set_params(Wg, bias, Wp)
    return gpu, ora


NAMES = ("Wg", "Wp", "bias")


def _state(gpu, with_s1=True):
    st = {k + "32": gpu.get_tensor(k + "32") for k in NAMES}
    if with_s1:
        st.update({"s1_" + k: gpu.get_tensor("s1_%s32" % k) for k in NAMES})
    return st


@pytest.mark.parametrize("dims,kind", [((6, 64, 64, 128, 64), 2), ((4, 256, 128, 256, 128), 2), ((5, 40, 24, 48, 16), 0),
                                        ((3, 64, 32, 64, 32), 3)])
def test_trajectory_flags_and_teacher_forced_update(dims, kind):
    """Adagrad (the paper's language-model optimizer), momentum SGD and Adam; shapes that run on the
    single-CTA and on the CTA-pair tensor-core kernels."""
    from paper_1710_03740_b200 import binding as b
    T, B, I, H, P = dims
    steps = 6
    Wg, bias, Wp, xs, ys = _case(T, B, I, H, P, seed=sum(dims) + kind, steps=steps)
    opt_args = {2: (2, 0.05, 0.0, 0.0, 1e-6, 0.0, 0.0), 0: (0, 0.1, 0.9, 0.0, 0.0, 1e-4, 0.0),
                3: (3, 0.002, 0.9, 0.999, 1e-8, 0.0, 0.5)}[kind]
    S = 128.0
    gpu, ora = _pair(dims, S, opt_args, Wg, bias, Wp)
    chk = OracleLSTMTrainer(T, B, I, H, P, S, *opt_args[:2], mu=opt_args[2], b2=opt_args[3], eps=opt_args[4], wd=opt_args[5],
                            clip=opt_args[6])
    chk.set_params(Wg, bias, Wp)
    for t in range(steps):
        xd, yd = dev(xs[t].view(np.uint16)), dev(ys[t])
        loss_g, flag_g = gpu.train_step(xd, yd)
        loss_o, flag_o = ora.train_step(xs[t], ys[t])
        assert flag_g == flag_o == 0
        assert abs(loss_g - loss_o) <= 1e-3 * abs(loss_o), (t, loss_g, loss_o)
        # teacher-forced step: chk holds the device's state from before this step (bit-identical by
        # induction); give it the device's gradient bits and compare everything the step wrote
        for k in NAMES:
            chk.g16[k] = gpu.get_tensor("d%s16" % k)
        assert chk.step() == 0
        for k in NAMES:
            assert np.array_equal(gpu.get_tensor(k + "32").view(np.uint32), chk.w32[k].view(np.uint32)), (t, k)
            assert np.array_equal(gpu.get_tensor(k + "16"), chk.w16[k]), (t, k)
            assert np.array_equal(gpu.get_tensor("s1_%s32" % k).view(np.uint32), chk.s1[k].view(np.uint32)), (t, k)
    # the logits of the last iteration: the device's r_t against the oracle's, as free-running values
    r_gpu = gpu.get_tensor("xr16")[1:, :, I:].view(np.float16).astype(np.float64)
    r_ora = ora.net.xr[1:, :, I:].view(np.float16).astype(np.float64)
    assert np.abs(r_gpu - r_ora).max() <= 2e-2 * max(1.0, np.abs(r_ora).max())
    gpu.close()


def test_overflowing_scale_skips_and_dynamic_scale_settles_like_the_oracle():
    """Started at S = 2^24 every gradient product overflows on the store: the step is skipped (masters,
    copies and Adagrad state untouched), the dynamic schedule halves S until a step applies; flags
    and scales follow the oracle's, losses stay within 1e-3."""
    dims = (4, 64, 32, 64, 32)
    T, B, I, H, P = dims
    steps = 14
    Wg, bias, Wp, xs, ys = _case(*dims, seed=5, steps=steps)
    opt_args = (2, 0.05, 0.0, 0.0, 1e-6, 0.0, 0.0)
    gpu, ora = _pair(dims, 2.0 ** 24, opt_args, Wg, bias, Wp)
    gpu.set_dynamic_scale(True, 1000, 1.0, 2.0 ** 24)
    ora.set_dynamic_scale(1000, 1.0, 2.0 ** 24)
    before = _state(gpu)
    flags_g, flags_o, scales_g, scales_o = [], [], [], []
    for t in range(steps):
        xd, yd = dev(xs[t].view(np.uint16)), dev(ys[t])
        loss_g, fg = gpu.train_step(xd, yd)
        loss_o, fo = ora.train_step(xs[t], ys[t])
        flags_g.append(fg); flags_o.append(fo)
        scales_g.append(gpu.get_scale()); scales_o.append(float(ora.S))
        assert abs(loss_g - loss_o) <= 1e-3 * abs(loss_o)
        if t == 0:
            assert fg == 1
            after = _state(gpu)
            assert all(np.array_equal(before[k], after[k]) for k in before)      # a skipped step moves nothing
    assert flags_g == flags_o and scales_g == scales_o
    assert flags_g[0] == 1 and flags_g[-1] == 0 and scales_g[-1] < 2.0 ** 24
    gpu.close()


def test_asynchronous_steps_match_synchronous_ones_and_errors():
    from paper_1710_03740_b200 import binding as b
    dims = (3, 32, 16, 32, 16)
    T, B, I, H, P = dims
    Wg, bias, Wp, xs, ys = _case(*dims, seed=9, steps=4)
    opt_args = (2, 0.05, 0.0, 0.0, 1e-6, 0.0, 0.0)
    a, _ = _pair(dims, 128.0, opt_args, Wg, bias, Wp)
    c, _ = _pair(dims, 128.0, opt_args, Wg, bias, Wp)
    keep = []
    for t in range(4):
        xd, yd = dev(xs[t].view(np.uint16)), dev(ys[t])
        keep.append((xd, yd))
        a.train_step(xd, yd)
        c.train_step(xd, yd, want=False)                 # no host read-back: nothing synchronises
    torch.cuda.synchronize()
    for k in NAMES:
        assert np.array_equal(a.get_tensor(k + "32"), c.get_tensor(k + "32"))
    # a label outside [0, P) is reported by a synchronising call and contributes nothing
    bad = ys[0].copy()
    bad[5] = P
    with pytest.raises(b.MptError) as e:
        a.train_step(keep[0][0], dev(bad))
    assert e.value.code == -1
    loss, flag = a.train_step(*keep[1])                  # the context stays usable
    assert np.isfinite(loss) and flag == 0
    # a context without parameters refuses to train
    fresh = b.LstmTrainer(*dims, 128.0, b.Optimizer(2, 0.05, 0.0, 0.0, 1e-6, 0.0, 0.0))
    with pytest.raises(b.MptError) as e:
        fresh.train_step(*keep[0])
    assert e.value.code == -3
    with pytest.raises(b.MptError):
        b.LstmTrainer(3, 32, 15, 32, 16, 128.0, b.Optimizer(2, 0.05, 0.0, 0.0, 1e-6, 0.0, 0.0))   # I not a multiple of 8
    a.close(); c.close(); fresh.close()
