"""Pins for the oracle's recurrent trunk (two LSTM layers between the depth/proprio feature and the fully connected
layers, Section III-C) over time-major sequence minibatches with done-resets: torch's LSTMCell and autograd in fp64,
special cases of the reset, central differences."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import oracle as orc
from test_oracle_encoder import _theta

SEQ = orc.ModelDesc(H=8, W=10, conv_c=(2, 3), conv_k=(3, 3), fc=(5,), P=2, A=2, n_lstm=2, lstm_h=4)
SEQ1 = orc.ModelDesc(H=6, W=6, conv_c=(2,), conv_k=(3,), fc=(4, 3), P=3, A=1, embed=3, n_lstm=1, lstm_h=5)


def _inputs(md, T, Be, seed, done_rate=0.3):
    g = np.random.default_rng(seed)
    depth = g.uniform(0.1, 2.0, (T, Be, md.H, md.W))
    proprio = g.standard_normal((T, Be, md.P))
    done = (g.random((T, Be)) < done_rate).astype(np.uint8)
    h0 = 0.5 * g.standard_normal((md.n_lstm, Be, md.lstm_h))
    c0 = 0.5 * g.standard_normal((md.n_lstm, Be, md.lstm_h))
    return depth, proprio, done, h0, c0


def _torch_forward(md, lay, th, depth, proprio, done, h0, c0):
    """The same network with torch ops in fp64: conv2d/linear front per row, explicit LSTM cell recurrences."""
    t = torch.tensor(th, dtype=torch.float64, requires_grad=True)
    T, Be = done.shape
    x = torch.tensor(depth, dtype=torch.float64).reshape(T * Be, 1, md.H, md.W)
    i = 0
    for co, k in zip(md.conv_c, md.conv_k):
        Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i]).permute(0, 3, 1, 2)
        b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + co]
        x = F.relu(F.conv2d(x, Wt, b, stride=2, padding=k // 2))
        i += 2
    if md.embed:
        flat = x.permute(0, 2, 3, 1).reshape(x.shape[0], -1)
        We = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
        be = t[lay.offsets[i + 1]:lay.offsets[i + 1] + md.embed]
        feat = F.relu(F.linear(flat, We, be))
        i += 2
    else:
        feat = x.mean(dim=(2, 3))
    seq = torch.cat([feat, torch.tensor(proprio, dtype=torch.float64).reshape(T * Be, md.P)], 1).reshape(T, Be, -1)
    keep = torch.tensor(1.0 - done.astype(np.float64))
    Hn = md.lstm_h
    for l in range(md.n_lstm):
        Wx = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
        Wh = t[lay.offsets[i + 1]:lay.offsets[i + 1] + lay.sizes[i + 1]].reshape(lay.shapes[i + 1])
        b = t[lay.offsets[i + 2]:lay.offsets[i + 2] + 4 * Hn]
        i += 3
        h, c = torch.tensor(h0[l]), torch.tensor(c0[l])
        outs = []
        for s in range(T):
            if s > 0:
                h, c = h * keep[s - 1][:, None], c * keep[s - 1][:, None]
            gates = F.linear(seq[s], Wx) + F.linear(h, Wh) + b
            ig, fg, gg, og = gates.split(Hn, dim=1)          # torch's gate order: input, forget, cell, output
            c = torch.sigmoid(fg) * c + torch.sigmoid(ig) * torch.tanh(gg)
            h = torch.sigmoid(og) * torch.tanh(c)
            outs.append(h)
        seq = torch.stack(outs)
    hcur = seq.reshape(T * Be, Hn)
    for o in md.fc:
        Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
        b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + o]
        hcur = F.relu(F.linear(hcur, Wt, b))
        i += 2
    Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
    b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + md.A + 1]
    out = F.linear(hcur, Wt, b)
    return t, out[:, :md.A], out[:, md.A]


def test_lstm_cell_agrees_with_torch_lstmcell():
    """One layer, one step, no reset: the gate order and the two weight blocks are torch.nn.LSTMCell's."""
    md = orc.ModelDesc(H=4, W=4, conv_c=(2,), conv_k=(3,), fc=(3,), P=2, A=1, n_lstm=1, lstm_h=6)
    th, lay = _theta(md, 1, bias_scale=0.3)
    depth, proprio, done, h0, c0 = _inputs(md, 1, 3, 0, done_rate=0.0)
    _, _, acts, lrec = orc.encoder_fwd_seq(md, th, depth, proprio, done, h0, c0)
    h0w = 2 + 2
    off = md.H * md.W + 2 * 2 * 2
    x = acts[:, off:off + h0w]
    cell = torch.nn.LSTMCell(h0w, 6).double()
    with torch.no_grad():
        cell.weight_ih.copy_(torch.tensor(th[lay.offsets[2]:lay.offsets[2] + lay.sizes[2]].reshape(24, h0w)))
        cell.weight_hh.copy_(torch.tensor(th[lay.offsets[3]:lay.offsets[3] + lay.sizes[3]].reshape(24, 6)))
        cell.bias_ih.copy_(torch.tensor(th[lay.offsets[4]:lay.offsets[4] + 24]))
        cell.bias_hh.zero_()
        h1, c1 = cell(torch.tensor(x), (torch.tensor(h0[0]), torch.tensor(c0[0])))
    assert np.allclose(lrec[:, 5 * 6:6 * 6], h1.numpy(), atol=1e-13)
    assert np.allclose(lrec[:, 4 * 6:5 * 6], c1.numpy(), atol=1e-13)


@pytest.mark.parametrize("md", [SEQ, SEQ1])
def test_forward_and_bptt_match_torch_autograd(md):
    """Catches: wrong gate order, state not reset (or reset one step late) after a done, gradient flowing through a
    reset or into the initial state, the lower layer fed from the wrong step, dropped terms of the cell's backward."""
    th, lay = _theta(md, 3, bias_scale=0.3)
    T, Be = 5, 3
    depth, proprio, done, h0, c0 = _inputs(md, T, Be, 5)
    assert done[:-1].any() and not done.all()
    mu, V, acts, lrec = orc.encoder_fwd_seq(md, th, depth, proprio, done, h0, c0)
    t, mu_t, V_t = _torch_forward(md, lay, th, depth, proprio, done, h0, c0)
    assert np.allclose(mu, mu_t.detach().numpy(), atol=1e-12) and np.allclose(V, V_t.detach().numpy(), atol=1e-12)
    g = np.random.default_rng(7)
    dmu, dV = g.standard_normal(mu.shape), g.standard_normal(V.shape)
    grad = orc.encoder_bwd_seq(md, th, done, acts, lrec, dmu, dV)
    (mu_t * torch.tensor(dmu)).sum().add((V_t * torch.tensor(dV)).sum()).backward()
    assert np.allclose(grad, t.grad.numpy(), atol=1e-11)
    for off, sz in list(zip(lay.offsets, lay.sizes))[:-1]:
        assert np.abs(grad[off:off + sz]).max() > 0


def test_done_resets_cut_the_sequence():
    """All dones set: every step starts from a zero state, so a row's output depends on its own observation only and
    equals the T = 1 result of that row with zero initial state; no dones and T = 1 rows chained by hand agree too."""
    md = SEQ
    th, lay = _theta(md, 2, bias_scale=0.3)
    T, Be = 4, 2
    depth, proprio, _, h0, c0 = _inputs(md, T, Be, 9)
    ones = np.ones((T, Be), np.uint8)
    mu, V, _, _ = orc.encoder_fwd_seq(md, th, depth, proprio, ones, h0, c0)
    z = np.zeros_like(h0)
    for t in range(1, T):
        m1, V1, _, _ = orc.encoder_fwd_seq(md, th, depth[t:t + 1], proprio[t:t + 1], ones[:1], z, z)
        assert np.allclose(mu[t * Be:(t + 1) * Be], m1, atol=1e-13) and np.allclose(V[t * Be:(t + 1) * Be], V1, atol=1e-13)
    zeros = np.zeros((T, Be), np.uint8)
    mu_s, V_s, _, lrec = orc.encoder_fwd_seq(md, th, depth, proprio, zeros, h0, c0)
    h, c = h0.copy(), c0.copy()
    Hn = md.lstm_h
    for t in range(T):
        m1, V1, _, r1 = orc.encoder_fwd_seq(md, th, depth[t:t + 1], proprio[t:t + 1], zeros[:1], h, c)
        assert np.allclose(mu_s[t * Be:(t + 1) * Be], m1, atol=1e-13)
        for l in range(md.n_lstm):
            h[l] = r1[:, l * 8 * Hn + 5 * Hn:l * 8 * Hn + 6 * Hn]
            c[l] = r1[:, l * 8 * Hn + 4 * Hn:l * 8 * Hn + 5 * Hn]


def test_bptt_matches_central_differences():
    md = SEQ
    th, lay = _theta(md, 7, bias_scale=0.3)
    T, Be = 3, 2
    depth, proprio, done, h0, c0 = _inputs(md, T, Be, 11)
    g = np.random.default_rng(1)
    dmu, dV = g.standard_normal((T * Be, md.A)), g.standard_normal(T * Be)

    def f(tt):
        mu, V, _, _ = orc.encoder_fwd_seq(md, tt, depth, proprio, done, h0, c0)
        return float((mu * dmu).sum() + (V * dV).sum())

    _, _, acts, lrec = orc.encoder_fwd_seq(md, th, depth, proprio, done, h0, c0)
    grad = orc.encoder_bwd_seq(md, th, done, acts, lrec, dmu, dV)
    idx = np.concatenate([np.arange(o, o + s) for o, s in list(zip(lay.offsets, lay.sizes))[:-1]])
    for i in np.random.default_rng(0).choice(idx, size=120, replace=False):
        e = np.zeros_like(th)
        e[i] = 1e-6
        fd = (f(th + e) - f(th - e)) / 2e-6
        assert abs(fd - grad[i]) <= 1e-6 * max(1.0, abs(grad[i])) + 2e-7, (i, fd, grad[i])


def test_layout_lists_the_lstm_tensors():
    md = orc.ModelDesc(120, 160, (16, 32, 64, 128), (3, 3, 3, 3), (512, 512, 256), norm=True, embed=32, n_lstm=2, lstm_h=1024)
    lay = orc.param_layout(md)
    assert lay.shapes[18:24] == [(4096, 64), (4096, 1024), (4096,), (4096, 1024), (4096, 1024), (4096,)]
    assert lay.shapes[24] == (512, 1024) and lay.sizes == [int(np.prod(s)) for s in lay.shapes]
