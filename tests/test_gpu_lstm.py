"""GPU parity of the LSTM layer (fused gate epilogue, backward gate arithmetic, bias gradient,
whole layer) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import mpo
from oracle.lstm import OracleLSTM
from paper_1710_03740_b200 import inputs
from gpu_util import dev, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _gpu():
    require_gpu()


def f16(a):
    return np.asarray(a).view(np.float16).astype(np.float64)


def ulp16(x):
    """Spacing of binary16 at |x| (2^-24 in the subnormal range)."""
    ax = np.maximum(np.abs(x), 2.0 ** -14)
    return 2.0 ** (np.floor(np.log2(ax)) - 10)


def host16(t):
    return t.cpu().numpy().view(np.uint16)


def _cell_inputs(B, H, K, seed):
    rng = np.random.default_rng(seed)
    xr = inputs.normal_f16(rng, (B, K), 1.0)
    Wg = inputs.normal_f16(rng, (4 * H, K), 1.0 / np.sqrt(K))
    bias = inputs.normal_f16(rng, (4 * H,), 0.5)
    cp = inputs.normal_f16(rng, (B, H), 1.0)
    return xr, Wg, bias, cp


def _check_cell_forward(B, H, K, flags, seed, rows=None):
    """Gate product + gate arithmetic of one step.  The device sums the products in another order
    than the oracle: a pre-activation may differ by 2*K*2^-23 * sum|a*b| (the GEMM acceptance
    bound), every gate function has slope <= 1, and each stored value carries its own FP16
    rounding plus the few-ulp difference of the exp/tanh implementations."""
    from paper_1710_03740_b200 import binding as b
    xr, Wg, bias, cp = _cell_inputs(B, H, K, seed)
    xd, wd, bd, cd = dev(xr.view(np.uint16)), dev(Wg.view(np.uint16)), dev(bias.view(np.uint16)), dev(cp.view(np.uint16))
    acts = torch.zeros((B, 4 * H), dtype=torch.int16, device="cuda")
    c = torch.zeros((B, H), dtype=torch.int16, device="cuda")
    h = torch.zeros((B, H), dtype=torch.int16, device="cuda")
    status = torch.zeros(16, dtype=torch.int32, device="cuda")
    b.mpt_lstm_cell_forward(B, H, K, xd, K, wd, K, bd, cd, H, acts, 4 * H, c, H, h, H, flags, status)
    torch.cuda.synchronize()
    assert status[3].item() == 0
    sel = slice(None) if rows is None else rows
    a_ref, c_ref, h_ref, pre, ab = mpo.lstm_cell_fwd(xr[sel], Wg, bias, cp[sel], want_pre=True)
    dpre = 2.0 * K * 2.0 ** -23 * ab                                   # [rows, 4H]
    a_got, c_got, h_got = f16(host16(acts)[sel]), f16(host16(c)[sel]), f16(host16(h)[sel])
    assert np.all(np.abs(a_got - f16(a_ref)) <= dpre + 1.01 * ulp16(f16(a_ref)))
    dcell = dpre.reshape(len(a_ref), H, 4)
    # c = f*cp + i*g: |dc| <= |cp| dpre_f + dpre_i + dpre_g; h adds dpre_o and the slope of tanh
    dc = np.abs(f16(cp[sel])) * dcell[:, :, 1] + dcell[:, :, 0] + dcell[:, :, 2]
    assert np.all(np.abs(c_got - f16(c_ref)) <= dc + 1.01 * ulp16(f16(c_ref)))
    assert np.all(np.abs(h_got - f16(h_ref)) <= dc + dcell[:, :, 3] + 2.01 * ulp16(f16(h_ref)) + ulp16(f16(c_ref)))
    # and most values agree exactly
    assert (host16(acts)[sel] == a_ref).mean() > 0.98
    assert (host16(h)[sel] == h_ref).mean() > 0.97


@pytest.mark.parametrize("B,H,K", [(200, 160, 160), (128, 64, 64), (300, 72, 200), (1, 8, 8)])
def test_cell_forward_single_cta_kernel(B, H, K):
    from paper_1710_03740_b200 import binding as b
    _check_cell_forward(B, H, K, b.GEMM_FORCE_TC, seed=B + H)


@pytest.mark.parametrize("B,H,K", [(512, 128, 192), (300, 200, 136), (256, 64, 64)])
def test_cell_forward_pair_kernel(B, H, K):
    from paper_1710_03740_b200 import binding as b
    _check_cell_forward(B, H, K, b.GEMM_FORCE_PAIR, seed=B + H + 1)


@pytest.mark.parametrize("B,H,K", [(37, 13, 29), (64, 16, 40)])
def test_cell_forward_cuda_core_kernel(B, H, K):
    from paper_1710_03740_b200 import binding as b
    _check_cell_forward(B, H, K, b.GEMM_FORCE_SIMT, seed=B + H + 2)


def test_cell_forward_biglstm_shape_sampled_rows():
    """The paper's layer (8192 cells, [x; r] of width 2048, 2048 rows): automatic kernel choice
    (CTA-pair kernel), oracle on 12 sampled rows."""
    _check_cell_forward(2048, 8192, 2048, 0, seed=5, rows=np.array([0, 1, 127, 128, 255, 256, 1000, 1023, 1024, 1999, 2046, 2047]))


@pytest.mark.parametrize("B,H", [(200, 160), (33, 7), (1, 2), (64, 1024)])
def test_cell_backward(B, H):
    """Identical inputs on both sides; only tanh(c) comes from different implementations."""
    from paper_1710_03740_b200 import binding as b
    rng = np.random.default_rng(B * 7 + H)
    acts = np.zeros((B, 4 * H), dtype=np.float16)
    acts[:, 0::4] = rng.uniform(0, 1, (B, H)); acts[:, 1::4] = rng.uniform(0, 1, (B, H))
    acts[:, 2::4] = rng.uniform(-1, 1, (B, H)); acts[:, 3::4] = rng.uniform(0, 1, (B, H))
    cp, c = inputs.normal_f16(rng, (B, H), 1.0), inputs.normal_f16(rng, (B, H), 1.0)
    dh, dcn = inputs.normal_f16(rng, (B, H), 40.0), inputs.normal_f16(rng, (B, H), 40.0)
    for dc_next in (dcn, None):
        dG = torch.zeros((B, 4 * H), dtype=torch.int16, device="cuda")
        dcp = torch.zeros((B, H), dtype=torch.int16, device="cuda")
        b.mpt_lstm_cell_backward(B, H, dev(dh.view(np.uint16)), H, None if dc_next is None else dev(dc_next.view(np.uint16)), H,
                                 dev(acts.view(np.uint16)), 4 * H, dev(cp.view(np.uint16)), H, dev(c.view(np.uint16)), H,
                                 dG, 4 * H, dcp, H)
        torch.cuda.synchronize()
        dG_ref, dcp_ref = mpo.lstm_cell_bwd(dh, dc_next, acts, cp, c)
        # a few FP32 ulps of tanh, amplified by at most |dh| <= a few hundred: far below one FP16 ulp
        assert np.all(np.abs(f16(host16(dG)) - f16(dG_ref)) <= 1.01 * ulp16(f16(dG_ref)))
        assert np.all(np.abs(f16(host16(dcp)) - f16(dcp_ref)) <= 1.01 * ulp16(f16(dcp_ref)))
        assert (host16(dG) == dG_ref).mean() > 0.99


@pytest.mark.parametrize("rows,cols,pad", [(800, 640, 0), (1000, 1000, 0), (77, 24, 8), (5, 3, 0), (4096, 2048, 0)])
def test_bias_grad(rows, cols, pad):
    from paper_1710_03740_b200 import binding as b
    rng = np.random.default_rng(rows + cols)
    ld = cols + pad
    dG = np.zeros((rows, ld), dtype=np.float16)
    dG[:, :cols] = inputs.normal_f16(rng, (rows, cols), 3.0)
    parts = torch.zeros((8, cols), dtype=torch.float32, device="cuda")
    db = torch.zeros(cols, dtype=torch.int16, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.mpt_bias_grad(dev(dG.view(np.uint16)), rows, cols, ld, parts, db, flag)
    torch.cuda.synchronize()
    db16, db32 = mpo.bias_grad(dG[:, :cols])
    bound = rows * 2.0 ** -23 * np.abs(dG[:, :cols].astype(np.float64)).sum(axis=0)
    assert np.all(np.abs(f16(host16(db)) - f16(db16)) <= bound + 1.01 * ulp16(f16(db16)))
    assert flag.item() == 0
    # an infinite entry reaches the flag
    dG[rows // 2, cols // 2] = np.inf
    b.mpt_bias_grad(dev(dG.view(np.uint16)), rows, cols, ld, parts, db, flag)
    torch.cuda.synchronize()
    assert flag.item() == 1


def test_add_f16_bit_exact():
    from paper_1710_03740_b200 import binding as b
    rng = np.random.default_rng(3)
    a, c = inputs.normal_f16(rng, (50, 72), 5.0), inputs.normal_f16(rng, (50, 40), 5.0)
    out = torch.zeros((50, 48), dtype=torch.int16, device="cuda")
    b.mpt_add_f16(dev(a.view(np.uint16)), 72, dev(c.view(np.uint16)), 40, out, 48, 50, 33)
    torch.cuda.synchronize()
    assert np.array_equal(host16(out)[:, :33], mpo.add_f16(a[:, :33], c[:, :33]))
    assert np.all(host16(out)[:, 33:] == 0)


def _run_layer(cfg):
    from paper_1710_03740_b200 import binding as b
    t = inputs.lstm_tensors(cfg)
    T, B, I, H, P = cfg["T"], cfg["B"], cfg["I"], cfg["H"], cfg["P"]
    layer = b.LstmLayer(T, B, I, H, P)
    layer.Wg16.copy_(dev(t["Wg"].view(np.uint16))); layer.Wp16.copy_(dev(t["Wp"].view(np.uint16)))
    layer.bias16.copy_(dev(t["bias16"].view(np.uint16)))
    layer.xr[:T, :, :I] = dev(t["x"].view(np.uint16))
    layer.xr[0, :, I:] = dev(t["r0"].view(np.uint16))
    layer.c[0] = dev(t["c0"].view(np.uint16))
    layer.dr_ext.copy_(dev(t["dr_ext"].view(np.uint16)))
    layer.forward()
    layer.backward()
    torch.cuda.synchronize()
    assert layer.device_error() == 0
    return layer, t


@pytest.mark.parametrize("name", ["small", "medium"])
def test_layer_forward_backward_against_oracle(name):
    """Whole layer, free running over T steps on both sides.  Step-by-step parity is pinned by the
    cell tests above; here the sequencing (recurrent columns, gradient sum of the two consumers of
    r_t, time-summed weight gradients, bias gradient) is checked with a tolerance that absorbs the
    last-ulp differences carried through the recurrence."""
    cfg = inputs.LSTM_CONFIGS[name]
    layer, t = _run_layer(cfg)
    T, B, I, H, P = cfg["T"], cfg["B"], cfg["I"], cfg["H"], cfg["P"]
    ora = OracleLSTM(T, B, I, H, P)
    ora.forward(t["x"], t["r0"], t["c0"], t["Wg"], t["bias16"], t["Wp"])
    ora.backward(t["dr_ext"])

    def close(got, ref, rel):
        got, ref = f16(got), f16(ref)
        # sums over many rows (weight and bias gradients, dxr) cancel: judge their small entries
        # against the typical magnitude of the tensor, not against their own ulp
        near = np.abs(got - ref) <= 4 * ulp16(ref) + 2e-3 * np.abs(ref).mean()
        return np.abs(got - ref).max() <= rel * np.abs(ref).max() and near.mean() > 0.97

    assert close(host16(layer.xr)[1:, :, I:], ora.xr[1:, :, I:], 4e-3)
    assert close(host16(layer.c)[1:], ora.c[1:], 4e-3)
    assert close(host16(layer.h), ora.h, 4e-3)
    assert close(host16(layer.dG), ora.dG, 1e-2)
    assert close(host16(layer.dxr), ora.dxr, 1e-2)
    assert close(host16(layer.dWg16), ora.dWg, 1e-2)
    assert close(host16(layer.dWp16), ora.dWp, 1e-2)
    assert close(host16(layer.dbias16), ora.db16, 1e-2)
    assert layer.nonfinite_flag.item() == 0
    # the left columns of xr (the inputs) are untouched; the first step's gradients exist
    assert np.array_equal(host16(layer.xr)[:T, :, :I], t["x"].view(np.uint16))
    assert np.any(host16(layer.dxr)[0] != 0)


def test_layer_teacher_forced_steps():
    """Each step of the device's forward pass re-derived by the oracle from the device's own
    previous state (so no drift): every step within the single-step bounds."""
    cfg = inputs.LSTM_CONFIGS["small"]
    layer, t = _run_layer(cfg)
    T, B, I, H, P = cfg["T"], cfg["B"], cfg["I"], cfg["H"], cfg["P"]
    xr, c, h = host16(layer.xr), host16(layer.c), host16(layer.h)
    for s in range(T):
        a_ref, c_ref, h_ref, pre, ab = mpo.lstm_cell_fwd(xr[s], t["Wg"], t["bias16"], c[s], want_pre=True)
        tol = 2.0 * (I + P) * 2.0 ** -23 * ab.reshape(B, H, 4).sum(axis=2) * (1.0 + np.abs(f16(c[s])))
        assert np.all(np.abs(f16(c[s + 1]) - f16(c_ref)) <= tol + 1.01 * ulp16(f16(c_ref)))
        assert np.all(np.abs(f16(h[s]) - f16(h_ref)) <= tol + 3.01 * ulp16(f16(h_ref)) + ulp16(f16(c_ref)))
        r_ref = mpo.gemm_f16(mpo.OP_FWD, h[s], t["Wp"])
        assert (np.abs(f16(xr[s + 1][:, I:]) - f16(r_ref)) <= 2.01 * ulp16(f16(r_ref))).mean() > 0.999


def test_layer_rejects_bad_shapes():
    from paper_1710_03740_b200 import binding as b
    layer = b.LstmLayer(2, 16, 8, 8, 8)
    layer.desc.H = 12                       # not a multiple of 8
    with pytest.raises(b.MptError) as e:
        layer.forward()
    assert e.value.code == b.ERR_SHAPE if hasattr(b, "ERR_SHAPE") else True
    layer.desc.H = 8
    layer.tensors.acts = None
    with pytest.raises(b.MptError):
        layer.forward()
