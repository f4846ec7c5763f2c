"""Pins for the oracle's layer-normalised depth CNN with a flatten -> fully connected embedding (Section III-C:
"4-layer CNN ... layer normalization, and ReLU ... fully connected layer which outputs a 32 dimensional embedding"):
torch's layer_norm and autograd in fp64, closed-form special cases of the normalisation, central differences."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import oracle as orc
from test_oracle_encoder import _rnd, _theta

LN_TINY = orc.ModelDesc(H=9, W=11, conv_c=(4, 6), conv_k=(3, 3), fc=(5,), P=2, A=2, norm=True, embed=3)
LN_POOL = orc.ModelDesc(H=8, W=10, conv_c=(4, 4), conv_k=(5, 3), fc=(4,), P=3, A=2, norm=True, embed=0)
EMB_ONLY = orc.ModelDesc(H=8, W=8, conv_c=(2, 3), conv_k=(3, 3), fc=(4,), P=2, A=1, norm=False, embed=5)


def _theta_ln(md, seed):
    """Seeded parameters; the rank-1 tensors (biases, gamma, beta) get noise, gamma around 1."""
    th, lay = _theta(md, seed, bias_scale=0.3)
    i = 0
    for co in md.conv_c:
        i += 2
        if md.norm:
            th[lay.offsets[i]:lay.offsets[i] + co] += 1.0  # gamma
            i += 2
    return th, lay


def _torch_forward(md, lay, th, depth, proprio, act_bf16=False):
    t = torch.tensor(th, dtype=torch.float64, requires_grad=True)
    x = torch.tensor(depth, dtype=torch.float64)[:, None]  # NCHW
    i = 0
    for co, k in zip(md.conv_c, md.conv_k):
        Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i]).permute(0, 3, 1, 2)
        b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + co]
        x = F.conv2d(x, Wt, b, stride=2, padding=k // 2)
        i += 2
        if md.norm:
            gam = t[lay.offsets[i]:lay.offsets[i] + co]
            bet = t[lay.offsets[i + 1]:lay.offsets[i + 1] + co]
            x = F.layer_norm(x.permute(0, 2, 3, 1), (co,), gam, bet, 1e-5).permute(0, 3, 1, 2)
            i += 2
        x = _rnd(F.relu(x), act_bf16)
    if md.embed:
        flat = x.permute(0, 2, 3, 1).reshape(x.shape[0], -1)  # pixel-major, channel innermost
        We = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
        be = t[lay.offsets[i + 1]:lay.offsets[i + 1] + md.embed]
        feat = _rnd(F.relu(F.linear(flat, We, be)), act_bf16)
        i += 2
    else:
        feat = _rnd(x.mean(dim=(2, 3)), act_bf16)
    h = torch.cat([feat, _rnd(torch.tensor(proprio, dtype=torch.float64), act_bf16)], 1)
    for o in md.fc:
        Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
        b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + o]
        h = _rnd(F.relu(F.linear(h, Wt, b)), act_bf16)
        i += 2
    Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
    b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + md.A + 1]
    out = F.linear(h, Wt, b)
    return t, out[:, :md.A], out[:, md.A]


@pytest.mark.parametrize("md", [LN_TINY, LN_POOL, EMB_ONLY])
def test_forward_and_backward_match_torch_layer_norm_autograd(md):
    """Catches: variance over the wrong axis or with the wrong divisor, eps inside/outside the root, gamma/beta
    swapped, normalisation after the ReLU, flatten in the wrong order, a dropped term of the normalisation's backward."""
    th, lay = _theta_ln(md, 3)
    g = np.random.default_rng(5)
    B = 3
    depth = g.uniform(0.1, 2.0, (B, md.H, md.W))
    proprio = g.standard_normal((B, md.P))
    mu, V, acts = orc.encoder_fwd(md, th, depth, proprio, False)
    t, mu_t, V_t = _torch_forward(md, lay, th, depth, proprio)
    assert np.allclose(mu, mu_t.detach().numpy(), atol=1e-11)
    assert np.allclose(V, V_t.detach().numpy(), atol=1e-11)
    dmu = g.standard_normal(mu.shape)
    dV = g.standard_normal(V.shape)
    grad = orc.encoder_bwd(md, th, acts, dmu, dV)
    (mu_t * torch.tensor(dmu)).sum().add((V_t * torch.tensor(dV)).sum()).backward()
    assert np.allclose(grad, t.grad.numpy(), atol=1e-10)
    assert np.abs(grad).max() > 1e-3
    if md is LN_TINY:  # every tensor except log-sigma receives gradient
        for off, sz in list(zip(lay.offsets, lay.sizes))[:-1]:
            assert np.abs(grad[off:off + sz]).max() > 0


def test_layout_lists_gamma_beta_and_the_embedding():
    lay = orc.param_layout(LN_TINY)
    # conv1: W, b, gamma, beta; conv2: W, b, gamma, beta; embed W, b; fc W, b; head W, b; log-sigma
    assert [tuple(s) for s in lay.shapes] == [(4, 3, 3, 1), (4,), (4,), (4,), (6, 3, 3, 4), (6,), (6,), (6,),
                                              (3, 3 * 3 * 6), (3,), (5, 3 + 2), (5,), (3, 5), (3,), (2,)]
    assert lay.sizes == [int(np.prod(s)) for s in lay.shapes]
    # the paper's depth CNN at 160x120: [16, 32, 64, 128] filters, 32-d embedding of the flattened 8x10x128 map
    md = orc.ModelDesc(120, 160, (16, 32, 64, 128), (3, 3, 3, 3), (512, 512, 256), norm=True, embed=32)
    lay = orc.param_layout(md)
    assert orc.conv_shapes(md) == ([60, 30, 15, 8], [80, 40, 20, 10])
    assert lay.shapes[16] == (32, 8 * 10 * 128) and lay.shapes[18] == (512, 32 + 32)


def test_normalisation_special_cases():
    """One conv layer, pooled.  (1) With gamma = 1, beta = 0 the pre-ReLU values of a pixel have mean 0 and variance
    C/(C + eps/var) ~ 1, so sum over channels of ReLU(xhat) - ReLU(-xhat) = 0; checked through the stored xhat: mean 0,
    mean square 1 - eps * rstd^2.  (2) Scaling the conv weights and bias by 7 leaves xhat unchanged up to the eps
    term.  (3) gamma = 0 gives ReLU(beta) everywhere, whatever the image."""
    md = orc.ModelDesc(H=8, W=6, conv_c=(8,), conv_k=(3,), fc=(3,), P=1, A=1, norm=True)
    th, lay = _theta_ln(md, 1)
    g = np.random.default_rng(2)
    depth = g.uniform(0.1, 2.0, (2, md.H, md.W))
    proprio = g.standard_normal((2, 1))
    npx, C = 4 * 3, 8
    _, _, acts = orc.encoder_fwd(md, th, depth, proprio, False)
    main = md.H * md.W + npx * C + (C + 1) + 3
    xh = acts[:, main:main + npx * C].reshape(2, npx, C)
    rstd = acts[:, main + npx * C:main + npx * (C + 1)]
    assert acts.shape[1] == main + npx * (C + 1)
    assert np.abs(xh.mean(-1)).max() < 1e-12
    assert np.allclose((xh ** 2).mean(-1), 1.0 - 1e-5 * rstd ** 2, atol=1e-12)
    th7 = th.copy()
    for i in (0, 1):
        th7[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]] *= 7.0
    _, _, acts7 = orc.encoder_fwd(md, th7, depth, proprio, False)
    xh7 = acts7[:, main:main + npx * C].reshape(2, npx, C)
    assert np.abs(xh7 - xh).max() < 1e-3 and np.allclose(acts7[:, main + npx * C:], rstd / 7.0, rtol=1e-3)
    th0 = th.copy()
    th0[lay.offsets[2]:lay.offsets[2] + C] = 0.0
    beta = th0[lay.offsets[3]:lay.offsets[3] + C]
    _, _, acts0 = orc.encoder_fwd(md, th0, depth, proprio, False)
    a1 = acts0[:, md.H * md.W:md.H * md.W + npx * C].reshape(2, npx, C)
    assert np.allclose(a1, np.maximum(beta, 0.0)[None, None, :], atol=1e-15)


@pytest.mark.parametrize("md", [LN_TINY, LN_POOL])
def test_gradient_matches_central_differences(md):
    """d/dtheta of sum(dmu * mu) + sum(dV * V) by central differences in fp64, every parameter of the small nets."""
    th, lay = _theta_ln(md, 7)
    g = np.random.default_rng(9)
    B = 2
    depth = g.uniform(0.1, 2.0, (B, md.H, md.W))
    proprio = g.standard_normal((B, md.P))
    dmu = g.standard_normal((B, md.A))
    dV = g.standard_normal(B)

    def f(t):
        mu, V, _ = orc.encoder_fwd(md, t, depth, proprio, False)
        return float((mu * dmu).sum() + (V * dV).sum())

    _, _, acts = orc.encoder_fwd(md, th, depth, proprio, False)
    grad = orc.encoder_bwd(md, th, acts, dmu, dV)
    idx = np.concatenate([np.arange(o, o + s) for o, s in list(zip(lay.offsets, lay.sizes))[:-1]])
    rng = np.random.default_rng(0)
    for i in rng.choice(idx, size=min(150, idx.size), replace=False):
        e = np.zeros_like(th)
        e[i] = 1e-6
        fd = (f(th + e) - f(th - e)) / 2e-6
        assert abs(fd - grad[i]) <= 1e-6 * max(1.0, abs(grad[i])) + 2e-7, (i, fd, grad[i])


def test_bf16_storing_mode_rounds_what_is_stored():
    md = LN_TINY
    th, lay = _theta_ln(md, 3)
    g = np.random.default_rng(5)
    depth = g.uniform(0.1, 2.0, (2, md.H, md.W))
    proprio = g.standard_normal((2, md.P))
    mu, V, acts = orc.encoder_fwd(md, th, depth, proprio, True)
    t, mu_t, V_t = _torch_forward(md, lay, th, depth, proprio, True)
    assert np.allclose(mu, mu_t.detach().numpy(), atol=1e-11) and np.allclose(V, V_t.detach().numpy(), atol=1e-11)
    # everything stored behind the image except the reciprocal standard deviations is a bf16 value
    Ho, Wo = orc.conv_shapes(md)
    main = md.H * md.W + sum(h * w * c for h, w, c in zip(Ho, Wo, md.conv_c)) + md.embed + md.P + sum(md.fc)
    stored = [acts[:, md.H * md.W:main]]
    off = main
    for h, w, c in zip(Ho, Wo, md.conv_c):
        stored.append(acts[:, off:off + h * w * c])
        off += h * w * (c + 1)
    for a in stored:
        assert np.array_equal(a, torch.tensor(a).to(torch.bfloat16).to(torch.float64).numpy())
