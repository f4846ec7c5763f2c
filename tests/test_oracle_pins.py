"""Pins for the CPU oracle: values fixed by the definitions, not by the oracle itself.

Each test states which mistake it would catch.  Nothing here touches the CUDA path.
"""
import math
import os
from decimal import Decimal, getcontext

import numpy as np
import pytest

from oracle import oracle as orc


# ---------------------------------------------------------------- fixtures --

def _read_gae_fixture(golden_dir):
    rows, norm = [], None
    for line in open(os.path.join(golden_dir, "gae_worked_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("norm"):
            norm = np.array([float(x) for x in line.split()[1:]])
        else:
            rows.append([float(x) for x in line.split()])
    return np.array(rows), norm


def _arrays_from_rows(rows):
    N, T = 2, 3
    r = np.zeros((T, N), np.float32)
    v = np.zeros((T, N), np.float32)
    d = np.zeros((T, N), np.uint8)
    lv = np.zeros(N, np.float32)
    adv = np.zeros((T, N))
    ret = np.zeros((T, N))
    for env, t, rew, val, done, last, a, R in rows:
        env, t = int(env), int(t)
        r[t, env], v[t, env], d[t, env], lv[env], adv[t, env], ret[t, env] = rew, val, done, last, a, R
    return r, v, d, lv, adv, ret


# --------------------------------------------------------------------- GAE --

def test_gae_worked_example_exact(golden_dir):
    """Hand-computed 2 env x 3 step case: catches a wrong done mask, a swapped gamma/lambda, ret != adv + V."""
    rows, norm = _read_gae_fixture(golden_dir)
    r, v, d, lv, adv_want, ret_want = _arrays_from_rows(rows)
    adv, ret = orc.gae(r, v, d, lv, 0.5, 0.5)
    assert np.array_equal(adv, adv_want)
    assert np.array_equal(ret, ret_want)
    a_n, mean, std = orc.adv_normalize(adv)
    assert abs(mean - 1.6197916667) < 1e-9
    assert abs(std - 2.6172815593) < 1e-9  # unbiased; the population value 2.389... would fail
    assert np.allclose(a_n.reshape(-1), norm, atol=2e-10, rtol=0)


def test_gae_gamma_lambda_one_is_return_to_go_minus_value():
    """gamma = lambda = 1, no dones: A_t = sum_{k>=t} r_k + V_T - V_t.  Catches a dropped bootstrap or a wrong scan direction."""
    g = np.random.default_rng(1)
    T, N = 7, 5
    r = g.standard_normal((T, N)).astype(np.float32)
    v = g.standard_normal((T, N)).astype(np.float32)
    lv = g.standard_normal(N).astype(np.float32)
    d = np.zeros((T, N), np.uint8)
    adv, ret = orc.gae(r, v, d, lv, 1.0, 1.0)
    rtg = np.cumsum(r[::-1].astype(np.float64), axis=0)[::-1] + lv.astype(np.float64)
    assert np.allclose(adv, rtg - v, atol=1e-12)
    assert np.allclose(ret, rtg, atol=1e-12)
    # the worked example's env 0 under gamma = lambda = 1
    adv0, _ = orc.gae(np.array([[1], [2], [3]], np.float32), np.array([[0.5], [1], [1.5]], np.float32),
                      np.zeros((3, 1), np.uint8), np.array([2], np.float32), 1.0, 1.0)
    assert np.array_equal(adv0.reshape(-1), [7.5, 6.0, 3.5])


def test_gae_lambda_zero_and_all_done():
    """lambda = 0 gives the one-step TD error; all dones give r - V (no bootstrap, no carry)."""
    g = np.random.default_rng(2)
    T, N = 6, 4
    r = g.standard_normal((T, N)).astype(np.float32)
    v = g.standard_normal((T, N)).astype(np.float32)
    lv = g.standard_normal(N).astype(np.float32)
    d = (g.random((T, N)) < 0.3).astype(np.uint8)
    gamma = 0.9
    adv, _ = orc.gae(r, v, d, lv, gamma, 0.0)
    v_next = np.concatenate([v[1:], lv[None]], 0).astype(np.float64)
    delta = r + gamma * v_next * (1 - d) - v
    assert np.allclose(adv, delta, atol=1e-12)
    adv1, ret1 = orc.gae(r, v, np.ones((T, N), np.uint8), lv, gamma, 0.95)
    assert np.allclose(adv1, r.astype(np.float64) - v, atol=1e-12)
    assert np.allclose(ret1, r, atol=1e-12)


def test_gae_done_blocks_information_flow():
    """A done at step t must make A_0..A_t independent of everything after t."""
    g = np.random.default_rng(3)
    T = 8
    r = g.standard_normal((T, 1)).astype(np.float32)
    v = g.standard_normal((T, 1)).astype(np.float32)
    d = np.zeros((T, 1), np.uint8)
    d[3, 0] = 1
    a1, _ = orc.gae(r, v, d, np.array([0.7], np.float32), 0.99, 0.95)
    r2, v2 = r.copy(), v.copy()
    r2[4:] += 5.0
    v2[4:] -= 3.0
    a2, _ = orc.gae(r2, v2, d, np.array([-9.0], np.float32), 0.99, 0.95)
    assert np.array_equal(a1[:4], a2[:4])
    assert not np.allclose(a1[4:], a2[4:])


def test_adv_normalize_moments():
    g = np.random.default_rng(4)
    a = 3.0 + 2.0 * g.standard_normal(4096)
    an, mean, std = orc.adv_normalize(a)
    assert abs(mean - a.mean()) < 1e-12
    assert abs(std - a.std(ddof=1)) < 1e-12
    assert abs(an.mean()) < 1e-12
    assert abs(an.var(ddof=1) - 1.0) < 1e-7


# ------------------------------------------------------------------ buffer --

def test_depth_bytes_matches_the_papers_example():
    """Section III-B: 512 envs x 320x240 x 16 steps in fp32 is quoted as 2.5 GB."""
    b = orc.depth_bytes(512, 16, 240, 320, 4)
    assert b == 2_516_582_400
    assert round(b / 1e9, 1) == 2.5
    assert orc.depth_bytes(512, 16, 240, 320, 2) == b // 2


# ------------------------------------------------------------- permutation --

def _read_perm_fixture(golden_dir):
    out = []
    for line in open(os.path.join(golden_dir, "perm_vectors.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line.split())
    return out


def test_mix32_constants_are_the_stated_irrationals():
    """The multipliers are floor(2^32/phi) and the fractional parts of sqrt 2, sqrt 3: fixes typos in the constants.

    The constants cannot be read back from the library, so they are recovered from its behaviour:
    mix32(1) = finalise(C1) and the key schedule are compared with an evaluation in Python integers."""
    getcontext().prec = 50
    phi = (Decimal(1) + Decimal(5).sqrt()) / 2
    C1 = int(Decimal(2 ** 32) / phi)
    C2 = int((Decimal(2).sqrt() - 1) * 2 ** 32)
    C3 = int((Decimal(3).sqrt() - 1) * 2 ** 32)
    assert (C1, C2, C3) == (0x9E3779B9, 0x6A09E667, 0xBB67AE85)

    def mix(x):
        x &= 0xFFFFFFFF
        x ^= x >> 16
        x = (x * C1) & 0xFFFFFFFF
        x ^= x >> 15
        x = (x * C2) & 0xFFFFFFFF
        x ^= x >> 16
        return x

    for x in [0, 1, 2, 0xFFFFFFFF, 0x80000000, 123456789]:
        assert orc.mix32(x) == mix(x)
    seed, epoch = 0x1234_5678_9ABC_DEF0, 7
    keys = [mix((seed & 0xFFFFFFFF) ^ mix((seed >> 32) + C1 * (j + 1)) ^ mix(epoch + C3 * (j + 1))) for j in range(6)]
    assert orc.perm_keys(seed, epoch) == keys


def test_perm_golden_vectors(golden_dir):
    for rec in _read_perm_fixture(golden_dir):
        if rec[0] == "mix32":
            assert orc.mix32(int(rec[1], 16)) == int(rec[2], 16)
        elif rec[0] == "keys":
            assert orc.perm_keys(int(rec[1]), int(rec[2])) == [int(x, 16) for x in rec[3:]]
        elif rec[0] == "perm":
            seed, epoch, M, kind = int(rec[1]), int(rec[2]), int(rec[3]), rec[4]
            want = [int(x) for x in rec[5:]]
            got = orc.perm(seed, epoch, M, 0, len(want))
            assert list(got) == want, (M, kind)


@pytest.mark.parametrize("M", [1, 2, 3, 6, 10, 16, 17, 1000, 4096, 4097, 16384, 65536, 100003])
def test_perm_is_a_bijection(M):
    p = orc.perm(5, 2, M)
    assert p.dtype == np.uint32 and p.shape == (M,)
    assert np.array_equal(np.sort(p), np.arange(M, dtype=np.uint32))


def test_perm_half_bits():
    """Domain 2^(2h) must cover M and stay below 4M (cycle walking terminates quickly)."""
    for M in [1, 2, 3, 4, 5, 16, 17, 255, 256, 257, 4096, 65536, 524288, 2 ** 31]:
        h = orc.lib().orc_perm_half_bits(M)
        assert (1 << (2 * h)) >= M
        assert h == 1 or (1 << (2 * h)) < 4 * M


def test_perm_depends_on_seed_and_epoch_and_minibatches_partition():
    M, K = 4096, 4
    base = orc.perm(0, 0, M)
    assert np.array_equal(base, orc.perm(0, 0, M))
    assert not np.array_equal(base, orc.perm(1, 0, M))
    assert not np.array_equal(base, orc.perm(0, 1, M))
    assert not np.array_equal(base, orc.perm(1 << 32, 0, M))  # high seed word matters too
    B = M // K
    parts = [orc.perm(0, 0, M, k * B, B) for k in range(K)]
    assert np.array_equal(np.concatenate(parts), base)
    assert np.array_equal(np.sort(np.concatenate(parts)), np.arange(M))
    # a uniform shuffle puts neighbours within M/100 of each other about 2 % of the time
    p = orc.perm(0, 0, 65536).astype(np.int64)
    near = np.mean(np.abs(np.diff(p)) < 65536 // 100)
    assert 0.01 < near < 0.03


def test_gather_copies_rows():
    g = np.random.default_rng(0)
    T, N = 3, 5
    f = {"x": g.standard_normal((T, N, 4)).astype(np.float32), "y": g.integers(0, 255, (T, N)).astype(np.uint8)}
    idx = np.array([14, 0, 7], np.uint32)
    out = orc.gather(f, idx, N)
    for j, s in enumerate(idx):
        t, n = divmod(int(s), N)
        assert np.array_equal(out["x"][j], f["x"][t, n])
        assert out["y"][j] == f["y"][t, n]


# -------------------------------------------------------------------- loss --

LOG2PI = math.log(2 * math.pi)


def test_gaussian_closed_forms():
    """A=1, a=0.5, mu=0, sigma=1: logp = -0.125 - ln(2 pi)/2; A=12, sigma=1: H = 6 (1 + ln 2 pi)."""
    out, *_ = orc.loss(np.zeros((1, 1)), np.zeros(1), np.zeros(1), np.full((1, 1), 0.5), np.zeros(1), np.ones(1),
                       np.zeros(1), 0.2, 0.5, 0.01)
    logp = -out[3]  # approx_kl = logp_old - logp with logp_old = 0
    assert abs(logp - (-1.0439385332)) < 1e-9
    assert abs(0.5 * LOG2PI - 0.9189385332) < 1e-9
    out, *_ = orc.loss(np.zeros((1, 12)), np.zeros(1), np.zeros(12), np.zeros((1, 12)), np.zeros(1), np.ones(1),
                       np.zeros(1), 0.2, 0.5, 0.01)
    assert abs(out[2] - 17.0272623985) < 1e-9
    # entropy of a Gaussian grows by sum(logsigma)
    out2, *_ = orc.loss(np.zeros((1, 12)), np.zeros(1), np.full(12, 0.25), np.zeros((1, 12)), np.zeros(1), np.ones(1),
                        np.zeros(1), 0.2, 0.5, 0.01)
    assert abs(out2[2] - out[2] - 3.0) < 1e-12
    # logp against scipy's normal density
    from scipy.stats import norm
    g = np.random.default_rng(0)
    mu, ls, a = g.standard_normal((4, 3)), 0.3 * g.standard_normal(3), g.standard_normal((4, 3))
    o, *_ = orc.loss(mu, np.zeros(4), ls, a, np.zeros(4), np.zeros(4), np.zeros(4), 0.2, 0.5, 0.0)
    want = norm.logpdf(a, loc=mu, scale=np.exp(ls)).sum(1)
    assert abs(-o[3] - want.mean()) < 1e-12


def _rand_case(B, A, seed):
    g = np.random.default_rng(seed)
    mu = 0.3 * g.standard_normal((B, A))
    ls = 0.2 * g.standard_normal(A)
    act = mu + np.exp(ls) * g.standard_normal((B, A))
    V = g.standard_normal(B)
    ret = g.standard_normal(B)
    adv = g.standard_normal(B)
    return mu, V, ls, act, adv, ret


def test_ratio_one_when_logp_old_equals_logp():
    """r = 1: surrogate = advantage, nothing clipped, approx_kl = 0, dL/dlogp = -Adv/B."""
    B, A = 16, 12
    mu, V, ls, act, adv, ret = _rand_case(B, A, 1)
    z = (act - mu) / np.exp(ls)
    logp = (-0.5 * z ** 2 - ls - 0.5 * LOG2PI).sum(1)
    out, dmu, dV, dls = orc.loss(mu, V, ls, act, logp, adv, ret, 0.2, 0.5, 0.0)
    assert abs(out[0] + adv.mean()) < 1e-12
    assert abs(out[3]) < 1e-12 and out[4] == 0.0
    assert abs(out[1] - np.mean((V - ret) ** 2)) < 1e-12
    assert np.allclose(dmu, (-adv / B)[:, None] * z / np.exp(ls), atol=1e-14)
    assert np.allclose(dV, 2 * 0.5 * (V - ret) / B, atol=1e-14)
    assert np.allclose(dls, ((-adv / B)[:, None] * (z ** 2 - 1)).sum(0), atol=1e-13)


def test_hand_clip_case():
    """B=2, A=1, eps=0.2, r=1.5: Adv=+1 is clipped (s=1.2, zero gradient); Adv=-1 is not (s=-1.5)."""
    logp = -0.125 - 0.5 * LOG2PI
    lpo = np.full(2, logp - math.log(1.5))
    out, dmu, dV, dls = orc.loss(np.zeros((2, 1)), np.zeros(2), np.zeros(1), np.full((2, 1), 0.5), lpo,
                                 np.array([1.0, -1.0]), np.zeros(2), 0.2, 0.0, 0.0)
    assert abs(out[0] - 0.15) < 1e-12          # -(1.2 - 1.5)/2
    assert out[4] == 1.0                       # both rows have |r-1| > eps
    assert abs(out[3] + math.log(1.5)) < 1e-12
    assert dmu[0, 0] == 0.0
    assert abs(dmu[1, 0] - 0.375) < 1e-12      # dL/dlogp = +0.75, z/sigma = 0.5
    assert abs(dls[0] - (-0.5625)) < 1e-12     # 0.75 * (0.25 - 1)
    # the mirrored case: r = 1/1.5 < 1 - eps clips the negative advantage instead
    lpo2 = np.full(2, logp + math.log(1.5))
    out2, dmu2, _, _ = orc.loss(np.zeros((2, 1)), np.zeros(2), np.zeros(1), np.full((2, 1), 0.5), lpo2,
                                np.array([1.0, -1.0]), np.zeros(2), 0.2, 0.0, 0.0)
    assert abs(out2[0] - (-(1 / 1.5) + 0.8) / 2) < 1e-12
    assert dmu2[1, 0] == 0.0 and dmu2[0, 0] != 0.0


def test_loss_gradients_match_finite_differences():
    """Central differences of L w.r.t. mu, V, logsigma (fp64).  Catches sign and factor mistakes in the fused backward."""
    B, A = 6, 3
    mu, V, ls, act, adv, ret = _rand_case(B, A, 7)
    z = (act - mu) / np.exp(ls)
    lpo = (-0.5 * z ** 2 - ls - 0.5 * LOG2PI).sum(1) + 0.3 * np.random.default_rng(8).standard_normal(B)
    clip, cv, ce = 0.2, 0.5, 0.01

    def L(mu_, V_, ls_):
        o, *_ = orc.loss(mu_, V_, ls_, act, lpo, adv, ret, clip, cv, ce)
        return o[0] + cv * o[1] - ce * o[2], o

    _, o = L(mu, V, ls)
    assert 0.0 < o[4] < 1.0, "case must exercise both clip branches"
    _, dmu, dV, dls = orc.loss(mu, V, ls, act, lpo, adv, ret, clip, cv, ce)
    h = 1e-6
    for i in range(B):
        for j in range(A):
            p, m_ = mu.copy(), mu.copy()
            p[i, j] += h
            m_[i, j] -= h
            fd = (L(p, V, ls)[0] - L(m_, V, ls)[0]) / (2 * h)
            assert abs(fd - dmu[i, j]) < 1e-8 + 1e-6 * abs(fd)
        p, m_ = V.copy(), V.copy()
        p[i] += h
        m_[i] -= h
        fd = (L(mu, p, ls)[0] - L(mu, m_, ls)[0]) / (2 * h)
        assert abs(fd - dV[i]) < 1e-8 + 1e-6 * abs(fd)
    for j in range(A):
        p, m_ = ls.copy(), ls.copy()
        p[j] += h
        m_[j] -= h
        fd = (L(mu, V, p)[0] - L(mu, V, m_)[0]) / (2 * h)
        assert abs(fd - dls[j]) < 1e-8 + 1e-6 * abs(fd)


def test_loss_microbatches_sum_to_minibatch():
    B, A = 12, 4
    mu, V, ls, act, adv, ret = _rand_case(B, A, 9)
    lpo = np.random.default_rng(10).standard_normal(B) * 0.2 - 5.0
    full, dmu, dV, dls = orc.loss(mu, V, ls, act, lpo, adv, ret, 0.2, 0.5, 0.01)
    out = np.zeros(5)
    dls2 = np.zeros(A)
    for lo, hi in [(0, 5), (5, 12)]:
        _, dm, dv, _ = orc.loss(mu[lo:hi], V[lo:hi], ls, act[lo:hi], lpo[lo:hi], adv[lo:hi], ret[lo:hi], 0.2, 0.5,
                                0.01, B_total=B, out=out, dlogsigma=dls2)
        assert np.allclose(dm, dmu[lo:hi], atol=1e-15) and np.allclose(dv, dV[lo:hi], atol=1e-15)
    assert np.allclose(out, full, atol=1e-13) and np.allclose(dls2, dls, atol=1e-13)


def test_sample_action():
    g = np.random.default_rng(0)
    mu, ls, eps = g.standard_normal((5, 3)), 0.1 * g.standard_normal(3), g.standard_normal((5, 3))
    a, lp = orc.sample_action(mu, ls, eps)
    assert np.allclose(a, mu + np.exp(ls) * eps)
    from scipy.stats import norm
    assert np.allclose(lp, norm.logpdf(a, loc=mu, scale=np.exp(ls)).sum(1), atol=1e-12)


# -------------------------------------------------------------------- Adam --

def test_adam_first_step_and_zero_grad():
    g = np.array([0.5, -2.0, 0.0, 1e-3])
    th = np.array([1.0, 1.0, 1.0, 1.0])
    m, v = np.zeros(4), np.zeros(4)
    orc.adam(th, m, v, g, 1e-2, 0.9, 0.999, 1e-8, 1)
    want = 1.0 - 1e-2 * g / (np.abs(g) + 1e-8)
    assert np.allclose(th, want.astype(np.float32), atol=0, rtol=0)
    assert th[2] == 1.0
    assert np.allclose(m, 0.1 * g) and np.allclose(v, 0.001 * g * g)


def test_adam_constant_gradient_and_torch_agreement():
    import torch
    n, steps = 37, 5
    rg = np.random.default_rng(0)
    th0 = rg.standard_normal(n).astype(np.float32).astype(np.float64)
    th, m, v = th0.copy(), np.zeros(n), np.zeros(n)
    p = torch.tensor(th0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=3e-4, betas=(0.9, 0.999), eps=1e-8)
    for s in range(1, steps + 1):
        g = rg.standard_normal(n)
        orc.adam(th, m, v, g, 3e-4, 0.9, 0.999, 1e-8, s)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        # the oracle rounds theta to fp32 every step; torch here does not: agree to fp32 rounding
        assert np.allclose(th, p.detach().numpy(), rtol=0, atol=steps * 1e-7)
    gconst = rg.standard_normal(n)
    m, v = np.zeros(n), np.zeros(n)
    th = th0.copy()
    for s in range(1, 4):
        orc.adam(th, m, v, gconst, 1e-3, 0.9, 0.999, 1e-8, s)
        assert np.allclose(m / (1 - 0.9 ** s), gconst) and np.allclose(v / (1 - 0.999 ** s), gconst ** 2)


# ------------------------------------------------------------------- bf16 ---

def test_round_bf16_ties_to_even_and_torch_agreement():
    import torch
    assert orc.round_bf16(1.0) == 1.0
    assert orc.round_bf16(1.0 + 2 ** -8) == 1.0            # tie, even mantissa below
    assert orc.round_bf16(1.0 + 2 ** -7 + 2 ** -8) == 1.0 + 2 ** -6  # tie, rounds up to even
    assert orc.round_bf16(1.0 + 2 ** -8 + 2 ** -20) == 1.0 + 2 ** -7
    assert orc.round_bf16(-3.1415926) == float(torch.tensor(-3.1415926).to(torch.bfloat16))
    x = np.random.default_rng(0).standard_normal(2000).astype(np.float32)
    want = torch.tensor(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([orc.round_bf16(float(t)) for t in x])
    assert np.array_equal(got, want)
