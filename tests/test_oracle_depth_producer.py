"""Pins for the oracle's analytic depth renderer (the stand-in for the simulator's depth rendering): closed forms of
single-primitive scenes, symmetries, equivalences between primitives, and the fp16 rounding."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc

HFOV = 1.2
FAR_PLANE = np.array([[0.0, 0.0, -1.0, -50.0]])  # z = 50: outside every [near, far] used here


def _f(W):
    return 0.5 * W / np.tan(0.5 * HFOV)


def test_fp16_rounding_matches_torch_half():
    g = np.random.default_rng(0)
    xs = np.concatenate([g.uniform(0.05, 3.0, 2000), [0.0, 1.0, 0.1, 2.0, 1 + 2 ** -11, 1 + 3 * 2 ** -11, 6e-8, 1e-7, 6.1e-5]])
    want = torch.tensor(xs, dtype=torch.float64).to(torch.float16).to(torch.float64).numpy()
    got = np.array([orc.round_fp16(x) for x in xs])
    assert np.array_equal(got, want)


def test_plane_facing_the_camera_has_constant_depth():
    pl = np.array([[0.0, 0.0, -1.0, -1.25]])  # -z = -1.25
    d = orc.render_depth(12, 16, HFOV, 0.1, 2.0, pl, np.zeros((1, 0, 8)))
    assert np.all(d == 1.25)
    assert np.all(orc.render_depth(12, 16, HFOV, 0.1, 1.0, pl, np.zeros((1, 0, 8))) == 0.0)  # beyond far: no return


def test_tilted_plane_depth_is_the_closed_form():
    """n . (z d) = off with d = (x, y, 1)  =>  z = off / (n . d)."""
    n = np.array([0.2, -0.9, -0.3])
    n /= np.linalg.norm(n)
    off = -0.45
    H, W = 10, 14
    d = orc.render_depth(H, W, HFOV, 0.05, 5.0, np.array([[*n, off]]), np.zeros((1, 0, 8)))[0]
    f = _f(W)
    for v, u in [(0, 0), (9, 13), (4, 7), (8, 2)]:
        ray = np.array([(u + 0.5 - W / 2) / f, (v + 0.5 - H / 2) / f, 1.0])
        z = off / (n @ ray)
        want = orc.round_fp16(z) if 0.05 <= z <= 5.0 and z > 0 else 0.0
        assert d[v, u] == want


def test_sphere_on_the_axis():
    """Odd image: the centre pixel looks along the axis and sees the front of the sphere at cz - r; the image is
    symmetric under both flips; a pixel whose ray passes the sphere at distance > r sees nothing."""
    H, W = 21, 31
    pr = np.array([[[0, 0.0, 0.0, 1.0, 0.25, 0, 0, 0]]])
    d = orc.render_depth(H, W, HFOV, 0.1, 2.0, FAR_PLANE, pr)[0]
    assert d[H // 2, W // 2] == 0.75
    assert np.array_equal(d, d[::-1, :]) and np.array_equal(d, d[:, ::-1])
    f = _f(W)
    hit = d > 0
    for v in range(H):
        for u in range(W):
            ray = np.array([(u + 0.5 - W / 2) / f, (v + 0.5 - H / 2) / f, 1.0])
            dist = np.linalg.norm(np.cross(ray, [0, 0, 1.0])) / np.linalg.norm(ray)  # of the centre from the ray
            if abs(dist - 0.25) > 1e-9:
                assert hit[v, u] == (dist < 0.25)
    # depth of a hit: the smaller root of |z ray - c|^2 = r^2
    v, u = H // 2 + 2, W // 2 - 3
    ray = np.array([(u + 0.5 - W / 2) / f, (v + 0.5 - H / 2) / f, 1.0])
    a, b, c = ray @ ray, -ray[2] * 1.0, 1.0 - 0.25 ** 2
    z = (-b - np.sqrt(b * b - a * c)) / a
    assert d[v, u] == orc.round_fp16(z)


def test_box_front_face_and_capsule_special_cases():
    H, W = 15, 21
    # a box centred on the axis: every ray that hits it enters through the front face z = cz - hz
    pr = np.array([[[1, 0.0, 0.0, 1.2, 0.2, 0.1, 0.3, 0]]])
    d = orc.render_depth(H, W, HFOV, 0.1, 2.0, FAR_PLANE, pr)[0]
    assert set(np.unique(d)) == {0.0, orc.round_fp16(0.9)}
    f = _f(W)
    for v in range(H):
        for u in range(W):
            x, y = 0.9 * (u + 0.5 - W / 2) / f, 0.9 * (v + 0.5 - H / 2) / f
            if abs(abs(x) - 0.2) > 1e-9 and abs(abs(y) - 0.1) > 1e-9:
                assert (d[v, u] > 0) == (abs(x) < 0.2 and abs(y) < 0.1)
    # a capsule of zero length is a sphere; a capsule along the viewing axis looks like its front sphere
    sph = orc.render_depth(H, W, HFOV, 0.1, 2.0, FAR_PLANE, np.array([[[0, 0.1, -0.05, 1.0, 0.2, 0, 0, 0]]]))
    cap0 = orc.render_depth(H, W, HFOV, 0.1, 2.0, FAR_PLANE, np.array([[[2, 0.1, -0.05, 1.0, 0, 0, 0, 0.2]]]))
    assert np.array_equal(sph, cap0)
    # a capsule across the view: on the image row through its axis the depth is cz - r between the end points
    cap = orc.render_depth(H, W, HFOV, 0.1, 2.0, FAR_PLANE, np.array([[[2, -0.3, 0.0, 1.0, 0.6, 0, 0, 0.1]]]))[0]
    assert H % 2 == 1
    row = cap[H // 2]
    inside = [u for u in range(W) if abs(0.9 * (u + 0.5 - W / 2) / f) < 0.28]
    assert len(inside) >= 3
    for u in inside:  # the centre row's rays have y = 0: they meet the cylinder where x^2 ... at z with (z*0)^2 + (z-1)^2 = r^2
        assert row[u] == orc.round_fp16(0.9)


def test_nearest_primitive_wins_and_order_does_not_matter():
    g = np.random.default_rng(3)
    pr = np.zeros((2, 5, 8))
    pr[:, :, 0] = g.integers(0, 3, (2, 5))
    pr[:, :, 1:3] = g.uniform(-0.4, 0.4, (2, 5, 2))
    pr[:, :, 3] = g.uniform(0.6, 1.6, (2, 5))
    pr[:, :, 4:8] = g.uniform(0.05, 0.2, (2, 5, 4))
    pl = np.array([[0.0, -1.0, 0.0, -0.5]] * 2)
    full = orc.render_depth(24, 32, HFOV, 0.1, 2.0, pl, pr)
    assert np.array_equal(full, orc.render_depth(24, 32, HFOV, 0.1, 2.0, pl, pr[:, ::-1].copy()))
    singles = [orc.render_depth(24, 32, HFOV, 0.1, 2.0, pl, pr[:, k:k + 1]) for k in range(5)]
    stack = np.stack(singles)
    stack[stack == 0] = np.inf
    want = stack.min(0)
    want[np.isinf(want)] = 0.0
    assert np.array_equal(full, want)
