"""Pins for the oracle's encoder forward/backward: library routines, special cases, finite differences."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import oracle as orc
from paper_2509_16434_b200 import synth

TINY = orc.ModelDesc(H=9, W=11, conv_c=(2, 3), conv_k=(3, 3), fc=(4,), P=2, A=2)
TINY5 = orc.ModelDesc(H=10, W=7, conv_c=(3, 4), conv_k=(5, 3), fc=(5, 3), P=3, A=2)


def _theta(md, seed, bias_scale=0.1):
    lay = orc.param_layout(md)
    th = synth.init_params(lay.total, lay.offsets, lay.shapes, seed).astype(np.float64)
    g = np.random.default_rng(seed + 100)
    for off, sz, shp in zip(lay.offsets, lay.sizes, lay.shapes):
        if len(shp) == 1:
            th[off:off + sz] = bias_scale * g.standard_normal(sz)
    # undo the 0.01 head scale so that head gradients are not tiny
    hw = len(lay.shapes) - 3
    th[lay.offsets[hw]:lay.offsets[hw] + lay.sizes[hw]] *= 100.0
    return th, lay


def _rnd(x, on):
    """bf16 rounding with a straight-through gradient."""
    if not on:
        return x
    return x + (x.detach().to(torch.float32).to(torch.bfloat16).to(torch.float64) - x.detach())


def _torch_forward(md, lay, th, depth, proprio, act_bf16=False):
    """The same network written with torch library ops in fp64 (conv2d is cross-correlation)."""
    t = torch.tensor(th, dtype=torch.float64, requires_grad=True)
    x = torch.tensor(depth, dtype=torch.float64)[:, None]  # NCHW
    i = 0
    for co, k in zip(md.conv_c, md.conv_k):
        shp = lay.shapes[i]
        Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(shp).permute(0, 3, 1, 2)  # [Co,kh,kw,Ci] -> OIHW
        b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + co]
        x = _rnd(F.relu(F.conv2d(x, Wt, b, stride=2, padding=k // 2)), act_bf16)
        i += 2
    h = _rnd(torch.cat([x.mean(dim=(2, 3)), torch.tensor(proprio, dtype=torch.float64)], 1), act_bf16)
    for o in md.fc:
        Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
        b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + o]
        h = _rnd(F.relu(F.linear(h, Wt, b)), act_bf16)
        i += 2
    Wt = t[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]].reshape(lay.shapes[i])
    b = t[lay.offsets[i + 1]:lay.offsets[i + 1] + md.A + 1]
    out = F.linear(h, Wt, b)
    return t, out[:, :md.A], out[:, md.A]


@pytest.mark.parametrize("act_bf16", [False, True])
@pytest.mark.parametrize("md", [TINY, TINY5, orc.ModelDesc(16, 16, (4, 8, 8), (3, 3, 3), (16,), 4, 3)])
def test_forward_and_backward_match_torch_autograd(md, act_bf16):
    """Catches: kernel flip, wrong padding/stride/output size, wrong weight index order, wrong pool divisor,
    concat order, transposed FC weights, missing ReLU mask in the backward."""
    th, lay = _theta(md, 3)
    g = np.random.default_rng(5)
    B = 3
    depth = g.uniform(0.1, 2.0, (B, md.H, md.W))
    proprio = g.standard_normal((B, md.P))
    mu, V, acts = orc.encoder_fwd(md, th, depth, proprio, act_bf16)
    t, mu_t, V_t = _torch_forward(md, lay, th, depth, proprio, act_bf16)
    if act_bf16:  # rounding is on: the stored activations are bf16 values and differ from the unrounded run
        mu_u, _, acts_u = orc.encoder_fwd(md, th, depth, proprio, False)
        n_img = md.H * md.W
        a = acts[:, n_img:]
        assert np.array_equal(a, torch.tensor(a).to(torch.bfloat16).to(torch.float64).numpy())
        assert not np.array_equal(acts, acts_u) and 0 < np.abs(mu - mu_u).max() < 0.05 * np.abs(mu_u).max()
    assert np.allclose(mu, mu_t.detach().numpy(), atol=1e-12)
    assert np.allclose(V, V_t.detach().numpy(), atol=1e-12)
    dmu = g.standard_normal(mu.shape)
    dV = g.standard_normal(V.shape)
    grad = orc.encoder_bwd(md, th, acts, dmu, dV)
    (mu_t * torch.tensor(dmu)).sum().add((V_t * torch.tensor(dV)).sum()).backward()
    assert np.allclose(grad, t.grad.numpy(), atol=1e-11)
    assert np.abs(grad).max() > 1e-3
    # every tensor except log-sigma receives gradient
    for off, sz in list(zip(lay.offsets, lay.sizes))[:-1]:
        assert np.abs(grad[off:off + sz]).max() > 0


def test_output_size_formula():
    """floor((in + 2p - k)/2) + 1: 64->32->16->8, 120->60->30->15->8, 160->80->40->20->10, 240->120 (k=5)."""
    md = orc.ModelDesc(120, 160, (32, 64, 128, 256), (3, 3, 3, 3), (512, 512))
    assert orc.conv_shapes(md) == ([60, 30, 15, 8], [80, 40, 20, 10])
    md = orc.ModelDesc(64, 64, (16, 32, 64), (3, 3, 3), (256,))
    assert orc.conv_shapes(md) == ([32, 16, 8], [32, 16, 8])
    md = orc.ModelDesc(240, 320, (32, 64, 128, 256, 256), (5, 3, 3, 3, 3), (512, 512))
    assert orc.conv_shapes(md) == ([120, 60, 30, 15, 8], [160, 80, 40, 20, 10])


def test_param_counts_of_the_workloads():
    """Unpadded parameter counts worked out by hand from the layer widths."""
    def count(md):
        return sum(orc.param_layout(md).sizes)
    assert count(orc.ModelDesc(64, 64, (16, 32, 64), (3, 3, 3), (256,))) == 51_481
    assert count(orc.ModelDesc(120, 160, (32, 64, 128, 256), (3, 3, 3, 3), (512, 512))) == 805_145
    assert count(orc.ModelDesc(240, 320, (32, 64, 128, 256, 256), (5, 3, 3, 3, 3), (512, 512))) == 1_395_737
    lay = orc.param_layout(TINY)
    assert all(o % 64 == 0 for o in lay.offsets)
    assert all(o2 >= o1 + s1 for o1, s1, o2 in zip(lay.offsets, lay.sizes, lay.offsets[1:]))


def test_conv1_special_cases():
    """All-zero depth gives ReLU(bias); a constant image under a kernel of ones gives 9c inside and 4c/6c where the
    zero padding is hit (top/left only for even sizes; also bottom/right for odd sizes)."""
    for H, W in [(8, 8), (9, 7)]:
        md = orc.ModelDesc(H, W, (2,), (3,), (3,), 1, 1)
        lay = orc.param_layout(md)
        th = np.zeros(lay.total)
        th[lay.offsets[0]:lay.offsets[0] + lay.sizes[0]] = 1.0
        th[lay.offsets[1]:lay.offsets[1] + 2] = [0.25, -0.5]
        Ho, Wo = orc.conv_shapes(md)
        Ho, Wo = Ho[0], Wo[0]
        _, _, acts = orc.encoder_fwd(md, th, np.zeros((1, H, W)), np.zeros((1, 1)))
        a1 = acts[0, H * W:H * W + Ho * Wo * 2].reshape(Ho, Wo, 2)
        assert np.all(a1[..., 0] == 0.25) and np.all(a1[..., 1] == 0.0)
        c = 0.5
        th[lay.offsets[1]:lay.offsets[1] + 2] = 0.0
        _, _, acts = orc.encoder_fwd(md, th, np.full((1, H, W), c), np.zeros((1, 1)))
        a1 = acts[0, H * W:H * W + Ho * Wo * 2].reshape(Ho, Wo, 2)[..., 0]
        rows = np.array([min(H, 2 * oh + 2) - max(0, 2 * oh - 1) for oh in range(Ho)])
        cols = np.array([min(W, 2 * ow + 2) - max(0, 2 * ow - 1) for ow in range(Wo)])
        assert np.array_equal(a1, c * np.outer(rows, cols))
        assert a1[0, 0] == 4 * c and a1[0, 1] == 6 * c and a1[1, 1] == 9 * c
        if H % 2 == 1:
            assert a1[-1, 1] == 6 * c and a1[-1, -1] == 4 * c
        else:
            assert a1[-1, 1] == 9 * c


def test_conv_matches_scipy_correlate():
    """Single layer against scipy.signal.correlate2d('same', zero fill) sampled at even positions."""
    from scipy.signal import correlate2d
    md = orc.ModelDesc(12, 10, (3,), (5,), (2,), 1, 1)
    th, lay = _theta(md, 11)
    g = np.random.default_rng(1)
    x = g.uniform(0.1, 2.0, (1, 12, 10))
    _, _, acts = orc.encoder_fwd(md, th, x, np.zeros((1, 1)))
    Ho, Wo = orc.conv_shapes(md)
    a1 = acts[0, 120:120 + Ho[0] * Wo[0] * 3].reshape(Ho[0], Wo[0], 3)
    Wt = th[lay.offsets[0]:lay.offsets[0] + lay.sizes[0]].reshape(3, 5, 5)
    b = th[lay.offsets[1]:lay.offsets[1] + 3]
    for co in range(3):
        full = correlate2d(x[0], Wt[co], mode="same", boundary="fill")
        assert np.allclose(a1[..., co], np.maximum(full[::2, ::2] + b[co], 0.0), atol=1e-12)


def test_affine_when_relu_inactive():
    """With positive weights, biases and inputs no ReLU clips, so the map is affine: f(a)+f(b)-f(0) = f(a+b)."""
    md = TINY
    lay = orc.param_layout(md)
    g = np.random.default_rng(2)
    th = np.zeros(lay.total)
    for off, sz in zip(lay.offsets[:-1], lay.sizes[:-1]):
        th[off:off + sz] = g.uniform(0.05, 0.3, sz)
    a = g.uniform(0.1, 1.0, (1, md.H, md.W))
    b = g.uniform(0.1, 1.0, (1, md.H, md.W))
    pa, pb = g.uniform(0, 1, (1, md.P)), g.uniform(0, 1, (1, md.P))
    f = lambda d, p: np.concatenate([x.reshape(-1) for x in orc.encoder_fwd(md, th, d, p)[:2]])
    assert np.allclose(f(a, pa) + f(b, pb) - f(0 * a, 0 * pa), f(a + b, pa + pb), atol=1e-12)


def test_weight_rounding_touches_matrices_only():
    md = TINY
    th, lay = _theta(md, 4)
    used = orc.round_weights(md, th)
    for off, sz, mat in zip(lay.offsets, lay.sizes, lay.is_matrix):
        seg, ref = used[off:off + sz], th[off:off + sz]
        if mat:
            want = torch.tensor(ref, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
            assert np.array_equal(seg, want)
        else:
            assert np.array_equal(seg, ref)


@pytest.mark.parametrize("md", [TINY, TINY5])
def test_total_gradient_matches_central_differences(md):
    """d(L_pi + c_v L_V - c_e H)/d(theta) for every parameter, fp64 central differences on a tiny network.

    Weight rounding is bypassed by choosing parameters that are already bf16 values, so the loss is a smooth function
    of the parameters the oracle differentiates (straight-through rounding has no finite-difference counterpart)."""
    th, lay = _theta(md, 21, bias_scale=0.2)
    th = orc.round_weights(md, th)
    g = np.random.default_rng(22)
    B = 3
    depth = g.uniform(0.1, 2.0, (B, md.H, md.W)).astype(np.float16).astype(np.float64)
    proprio = g.standard_normal((B, md.P))
    used_ls = th[lay.offsets[-1]:lay.offsets[-1] + md.A]
    mu0, _, _ = orc.encoder_fwd(md, th, depth, proprio)
    eps = g.standard_normal((B, md.A))
    action, logp0 = orc.sample_action(mu0, used_ls, eps)
    logp_old = logp0 + 0.3 * g.standard_normal(B)
    adv, ret = g.standard_normal(B), g.standard_normal(B)
    clip, cv, ce = 0.2, 0.5, 0.01

    def L_of(theta):
        # no rounding inside: evaluate the pieces directly
        ls = theta[lay.offsets[-1]:lay.offsets[-1] + md.A]
        mu, V, _ = orc.encoder_fwd(md, theta, depth, proprio)
        o, *_ = orc.loss(mu, V, ls, action, logp_old, adv, ret, clip, cv, ce)
        return o[0] + cv * o[1] - ce * o[2]

    L, out, grad, _, _ = orc.total_loss_and_grad(md, th, depth, proprio, action, logp_old, adv, ret, clip, cv, ce)
    assert abs(L - L_of(th)) < 1e-14
    h = 1e-6
    checked = 0
    for off, sz in zip(lay.offsets, lay.sizes):
        for i in range(off, off + sz):
            p, m_ = th.copy(), th.copy()
            p[i] += h
            m_[i] -= h
            fd = (L_of(p) - L_of(m_)) / (2 * h)
            assert abs(fd - grad[i]) <= 1e-8 + 1e-6 * abs(fd), (i, fd, grad[i])
            checked += 1
    assert checked == sum(lay.sizes)
    assert np.abs(grad).max() > 1e-4
