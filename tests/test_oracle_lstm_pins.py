"""CPU pins for the LSTM part of the oracle (no GPU).

The oracle's LSTM layer is held against things it does not compute itself: PyTorch's own
float64 LSTM with a projection (forward values and autograd gradients; different gate layout,
different code), hand-worked single cells, numpy sums, and structural properties.
"""
import numpy as np
import pytest
import torch

from oracle import mpo
from oracle.lstm import OracleLSTM


def _rand16(rng, *shape, scale=0.3):
    return (rng.standard_normal(shape) * scale).astype(np.float16)


def _torch_lstm(T, B, I, H, P, x, r0, c0, Wg, b, Wp):
    """float64 torch.nn.LSTM carrying the same FP16-representable parameters.  torch stacks the
    gates as row blocks [i; f; g; o]; the oracle interleaves them per cell (row 4j+q)."""
    lstm = torch.nn.LSTM(input_size=I, hidden_size=H, proj_size=P, bias=True).double()
    Wg64 = torch.from_numpy(Wg.astype(np.float64))
    blocks = torch.cat([Wg64[q::4] for q in range(4)], dim=0)            # [4H, I+P] in torch's order
    bias = torch.cat([torch.from_numpy(b.astype(np.float64))[q::4] for q in range(4)])
    with torch.no_grad():
        lstm.weight_ih_l0.copy_(blocks[:, :I])
        lstm.weight_hh_l0.copy_(blocks[:, I:])
        lstm.bias_ih_l0.copy_(bias)
        lstm.bias_hh_l0.zero_()
        lstm.weight_hr_l0.copy_(torch.from_numpy(Wp.astype(np.float64)))
    xt = torch.from_numpy(x.astype(np.float64)).requires_grad_(True)
    out, _ = lstm(xt, (torch.from_numpy(r0.astype(np.float64))[None], torch.from_numpy(c0.astype(np.float64))[None]))
    return lstm, xt, out


def test_forward_and_backward_against_torch_float64_lstm():
    rng = np.random.default_rng(11)
    T, B, I, H, P = 5, 6, 12, 20, 8
    x, r0, c0 = _rand16(rng, T, B, I, scale=1.0), _rand16(rng, B, P), _rand16(rng, B, H)
    Wg, b, Wp = _rand16(rng, 4 * H, I + P), _rand16(rng, 4 * H), _rand16(rng, P, H)
    S = 256.0
    dr = _rand16(rng, T, B, P, scale=1.0)
    net = OracleLSTM(T, B, I, H, P)
    r = net.forward(x, r0, c0, Wg, b, Wp).view(np.float16).astype(np.float64)
    dx = net.backward((dr.astype(np.float32) * S).astype(np.float16)).view(np.float16).astype(np.float64) / S
    lstm, xt, out = _torch_lstm(T, B, I, H, P, x, r0, c0, Wg, b, Wp)
    assert np.abs(r - out.detach().numpy()).max() < 3e-3                  # FP16 storage of values below 1
    out.backward(torch.from_numpy(dr.astype(np.float64)))
    blocks_g = lstm.weight_ih_l0.grad.numpy(), lstm.weight_hh_l0.grad.numpy()
    dWg_ref = np.zeros((4 * H, I + P))
    for q in range(4):
        dWg_ref[q::4, :I] = blocks_g[0][q * H:(q + 1) * H]
        dWg_ref[q::4, I:] = blocks_g[1][q * H:(q + 1) * H]
    db_ref = np.zeros(4 * H)
    for q in range(4):
        db_ref[q::4] = lstm.bias_ih_l0.grad.numpy()[q * H:(q + 1) * H]

    def close(a, ref):
        scale = np.abs(ref).max()
        return np.abs(a - ref).max() <= 2e-2 * scale

    assert close(dx, xt.grad.numpy())
    assert close(net.dWg.view(np.float16).astype(np.float64) / S, dWg_ref)
    assert close(net.dWp.view(np.float16).astype(np.float64) / S, lstm.weight_hr_l0.grad.numpy())
    assert close(net.db16.view(np.float16).astype(np.float64) / S, db_ref)
    assert close(net.db32.astype(np.float64) / S, db_ref)


def test_single_cell_hand_values():
    """All pre-activations zero: i = f = o = 1/2, g = 0, so c = c_prev/2 and h = tanh(c)/2; then
    the backward formulas evaluated by hand."""
    H = 2
    xr = np.zeros((1, 3), dtype=np.float16)
    Wg = np.ones((4 * H, 3), dtype=np.float16)
    b = np.zeros(4 * H, dtype=np.float16)
    cp = np.array([[1.0, -2.0]], dtype=np.float16)
    acts, c, h = mpo.lstm_cell_fwd(xr, Wg, b, cp)
    assert acts.view(np.float16).tolist() == [[0.5, 0.5, 0.0, 0.5] * H]
    assert c.view(np.float16).tolist() == [[0.5, -1.0]]
    expect_h = (0.5 * np.tanh(np.array([0.5, -1.0]))).astype(np.float32).astype(np.float16)
    assert np.array_equal(h.view(np.float16)[0], expect_h)
    # backward with dh = 1, dc_next = 0.25:  dc = o(1 - tanh^2 c) + 0.25
    dh = np.ones((1, H), dtype=np.float16)
    dcn = np.full((1, H), 0.25, dtype=np.float16)
    dG, dcp = mpo.lstm_cell_bwd(dh, dcn, acts, cp, c)
    tc = np.tanh(np.array([0.5, -1.0]))
    dc = 0.5 * (1 - tc * tc) + 0.25
    ref = np.stack([dc * 0.0 * 0.25, dc * cp.astype(np.float64)[0] * 0.25, dc * 0.5 * 1.0, tc * 0.25], axis=1)  # i, f, g, o
    got = dG.view(np.float16).astype(np.float64).reshape(H, 4)
    assert np.abs(got - ref).max() < 1e-3
    assert np.abs(dcp.view(np.float16).astype(np.float64)[0] - dc * 0.5).max() < 1e-3
    # last step: no incoming cell gradient
    dG0, _ = mpo.lstm_cell_bwd(dh, None, acts, cp, c)
    dc0 = 0.5 * (1 - tc * tc)
    assert np.abs(dG0.view(np.float16).astype(np.float64).reshape(H, 4)[:, 2] - dc0 * 0.5).max() < 1e-3


def test_gate_saturation_and_bias_only_paths():
    """Large biases drive the gates to their limits: forget gate 1, input gate 0 keeps the cell
    (c = c_prev exactly), output gate 0 silences h."""
    H = 3
    xr = np.zeros((2, 4), dtype=np.float16)
    Wg = np.zeros((4 * H, 4), dtype=np.float16)
    b = np.zeros(4 * H, dtype=np.float16)
    b[0::4] = -30.0       # input gate closed
    b[1::4] = 30.0        # forget gate open
    b[3::4] = -30.0       # output gate closed
    cp = np.array([[0.75, -1.5, 3.0], [0.0, 1.0, -0.25]], dtype=np.float16)
    acts, c, h = mpo.lstm_cell_fwd(xr, Wg, b, cp)
    assert np.array_equal(c.view(np.float16), cp)
    assert np.all(np.abs(h.view(np.float16).astype(np.float32)) < 1e-6)


def test_pre_activation_is_the_fp32_gemm_plus_bias():
    """The pre-activations equal the oracle GEMM's FP32 accumulation (same ascending-k order) plus
    the bias: rounding them to FP16 reproduces gemm_f16 wherever the bias is zero."""
    rng = np.random.default_rng(5)
    B, K, H = 5, 37, 6
    xr, Wg = _rand16(rng, B, K, scale=1.0), _rand16(rng, 4 * H, K, scale=1.0)
    b = np.zeros(4 * H, dtype=np.float16)
    _, _, _, pre, ab = mpo.lstm_cell_fwd(xr, Wg, b, np.zeros((B, H), dtype=np.float16), want_pre=True)
    C, ex, ab2 = mpo.gemm_f16(mpo.OP_FWD, xr, Wg, want_exact=True)
    assert np.array_equal(mpo.f2h(pre), C)
    assert np.allclose(ab, ab2, rtol=1e-12)
    assert np.abs(pre - ex).max() <= 2 * K * 2.0 ** -24 * ab.max()


def test_bias_grad_and_add():
    rng = np.random.default_rng(6)
    dG = _rand16(rng, 301, 24, scale=4.0)
    db16, db32 = mpo.bias_grad(dG)
    ref = dG.astype(np.float64).sum(axis=0)
    assert np.abs(db32 - ref).max() <= 301 * 2.0 ** -24 * np.abs(dG.astype(np.float64)).sum(axis=0).max()
    assert np.array_equal(db16, mpo.f2h(db32))
    a, b = _rand16(rng, 7, 9), _rand16(rng, 7, 9)
    assert np.array_equal(mpo.add_f16(a, b).view(np.float16), (a.astype(np.float32) + b.astype(np.float32)).astype(np.float16))


def test_weight_gradient_sums_over_time_before_rounding():
    """dWg is one product over all T*B rows: it equals the oracle GEMM on the stacked tensors and
    differs from summing per-step FP16 products when those would round away small terms."""
    rng = np.random.default_rng(8)
    T, B, I, H, P = 3, 4, 8, 8, 8
    net = OracleLSTM(T, B, I, H, P)
    net.forward(_rand16(rng, T, B, I), _rand16(rng, B, P), _rand16(rng, B, H), _rand16(rng, 4 * H, I + P),
                _rand16(rng, 4 * H), _rand16(rng, P, H))
    net.backward(_rand16(rng, T, B, P, scale=8.0))
    ref = sum(net.dG[t].view(np.float16).astype(np.float64).T @ net.xr[t].view(np.float16).astype(np.float64) for t in range(T))
    got = net.dWg.view(np.float16).astype(np.float64)
    assert np.abs(got - ref).max() <= 2.0 ** -10 * np.abs(ref).max() + 1e-7


def _trainer_case(seed=21, T=4, B=5, I=8, H=16, P=8):
    rng = np.random.default_rng(seed)
    x = _rand16(rng, T, B, I, scale=1.0)
    Wg, b, Wp = _rand16(rng, 4 * H, I + P), _rand16(rng, 4 * H), _rand16(rng, P, H, scale=0.8)
    y = rng.integers(0, P, T * B).astype(np.int32)
    return (T, B, I, H, P), x, Wg, b, Wp, y


def test_trainer_loss_and_gradients_against_torch_float64_and_adagrad_first_step():
    """The trained layer (forward from zero state, cross-entropy over r_t as logits, BPTT, unscale,
    Adagrad on the masters) against torch float64: nn.LSTM with a projection, F.cross_entropy (mean),
    autograd.  The first Adagrad step from zero state is w - lr*g/(|g| + eps) in closed form."""
    from oracle.lstm import OracleLSTMTrainer
    (T, B, I, H, P), x, Wg, b, Wp, y = _trainer_case()
    S, lr, eps = 128.0, 0.05, 1e-6
    tr = OracleLSTMTrainer(T, B, I, H, P, S, mpo.OPT_ADAGRAD, lr, eps=eps)
    tr.set_params(Wg.astype(np.float32), b.astype(np.float32), Wp.astype(np.float32))
    w0 = {k: v.copy() for k, v in tr.w32.items()}
    loss = tr.forward_backward(x, y)
    lstm, xt, out = _torch_lstm(T, B, I, H, P, x, np.zeros((B, P), np.float16), np.zeros((B, H), np.float16), Wg, b, Wp)
    ref = torch.nn.functional.cross_entropy(out.reshape(T * B, P), torch.from_numpy(y.astype(np.int64)))
    assert abs(loss - ref.item()) < 2e-3 * ref.item()
    ref.backward()
    dWg_ref = np.zeros((4 * H, I + P))
    db_ref = np.zeros(4 * H)
    for q in range(4):
        dWg_ref[q::4, :I] = lstm.weight_ih_l0.grad.numpy()[q * H:(q + 1) * H]
        dWg_ref[q::4, I:] = lstm.weight_hh_l0.grad.numpy()[q * H:(q + 1) * H]
        db_ref[q::4] = lstm.bias_ih_l0.grad.numpy()[q * H:(q + 1) * H]
    refs = dict(Wg=dWg_ref, Wp=lstm.weight_hr_l0.grad.numpy(), bias=db_ref)
    unscaled = {k: tr.g16[k].view(np.float16).astype(np.float64) / S for k in tr.names}
    for k in tr.names:
        scale = np.abs(refs[k]).max()
        assert scale > 0 and np.abs(unscaled[k] - refs[k].reshape(unscaled[k].shape)).max() < 0.03 * scale, k
    assert tr.step() == 0
    for k in tr.names:
        g = tr.g16[k].view(np.float16).astype(np.float32) * np.float32(1.0 / S)
        want = w0[k].astype(np.float64) - lr * g.astype(np.float64) / (np.abs(g.astype(np.float64)) + eps)
        assert np.allclose(tr.w32[k], want.reshape(tr.w32[k].shape), rtol=0, atol=2e-6), k
        assert np.array_equal(tr.w16[k], mpo.f2h(tr.w32[k]))
        # Adagrad's state after one step is the squared unscaled gradient, bit for bit
        assert np.array_equal(tr.s1[k].reshape(-1), (g * g).reshape(-1))


def test_trainer_loss_falls_and_overflow_skips_and_dynamic_scale_recovers():
    from oracle.lstm import OracleLSTMTrainer
    (T, B, I, H, P), x, Wg, b, Wp, y = _trainer_case(seed=22)
    tr = OracleLSTMTrainer(T, B, I, H, P, 128.0, mpo.OPT_ADAGRAD, 0.05, eps=1e-6)
    tr.set_params(Wg.astype(np.float32), b.astype(np.float32), Wp.astype(np.float32))
    losses = [tr.train_step(x, y)[0] for _ in range(8)]
    assert losses[-1] < 0.8 * losses[0]                      # the same batch repeated: the loss must fall
    # a scale far too large overflows the weight gradients: every tensor untouched, flag 1
    big = OracleLSTMTrainer(T, B, I, H, P, 2.0 ** 24, mpo.OPT_ADAGRAD, 0.05, eps=1e-6)
    big.set_params(Wg.astype(np.float32), b.astype(np.float32), Wp.astype(np.float32))
    before = {k: v.copy() for k, v in big.w32.items()}
    loss, flag = big.train_step(x, y)
    assert flag == 1 and all(np.array_equal(before[k], big.w32[k]) for k in big.names)
    assert not any(big.s1[k].any() for k in big.names)
    # with the dynamic schedule the scale halves until the step applies, then stays
    big.set_dynamic_scale(1000, 1.0, 2.0 ** 24)
    flags, scales = [], []
    for _ in range(12):
        flags.append(big.train_step(x, y)[1])
        scales.append(float(big.S))
    assert flags[0] == 1 and flags[-1] == 0 and 0 in flags
    first_ok = flags.index(0)
    assert all(f == 1 for f in flags[:first_ok]) and all(f == 0 for f in flags[first_ok:])
    assert scales[first_ok] == scales[-1] == 2.0 ** 24 / 2 ** first_ok
    # the settled run equals a constant-scale run started at that scale, bit for bit (scaling by a
    # power of two is exact as long as nothing leaves the FP16 range)
    ref = OracleLSTMTrainer(T, B, I, H, P, scales[-1], mpo.OPT_ADAGRAD, 0.05, eps=1e-6)
    ref.set_params(Wg.astype(np.float32), b.astype(np.float32), Wp.astype(np.float32))
    for _ in range(12 - first_ok):
        ref.train_step(x, y)
    for k in ref.names:
        assert np.array_equal(ref.w32[k], big.w32[k]), k
