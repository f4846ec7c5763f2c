"""GPU parity: write_step, GAE + advantage normalisation and the permutation gather against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth
from helpers import max_abs_scaled, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda"
GAE_TOL = 1e-5  # relative L2 and scaled max-abs, fp32 scan vs fp64 oracle


def _fill(buf, roll, action, logp):
    dev = {k: torch.as_tensor(v).to(DEV) for k, v in roll.items()}
    a, lp = torch.as_tensor(action).to(DEV), torch.as_tensor(logp).to(DEV)
    for t in range(buf.desc.T):
        ppo.ppo_buffer_write_step(buf, t, dev["depth"][t], dev["proprio"][t], a[t], lp[t], dev["value"][t],
                                  dev["reward"][t], dev["done"][t])
    return dev


def _small(N, T, H=16, W=24, seed=0, done_rate=0.05):
    w = synth.WORKLOADS["cfg1"].scaled(N, T=T, H=H, W=W, done_rate=done_rate)
    roll = synth.rollout_numpy(w, seed)
    g = np.random.default_rng(seed + 1)
    action = g.standard_normal((T, N, w.A)).astype(np.float32)
    logp = g.standard_normal((T, N)).astype(np.float32)
    return w, roll, action, logp


@pytest.mark.parametrize("N,T", [(37, 5), (256, 16), (1000, 1)])
def test_write_step_is_an_exact_copy(N, T):
    w, roll, action, logp = _small(N, T)
    buf = ppo.Buffer(ppo.buffer_desc(N, T, w.H, w.W, w.P, w.A))
    _fill(buf, roll, action, logp)
    assert ppo.ppo_poll_status() == 0
    want = {ppo.FIELD_DEPTH: roll["depth"], ppo.FIELD_PROPRIO: roll["proprio"], ppo.FIELD_ACTION: action,
            ppo.FIELD_LOGP: logp, ppo.FIELD_VALUE: roll["value"], ppo.FIELD_REWARD: roll["reward"],
            ppo.FIELD_DONE: roll["done"]}
    for f, arr in want.items():
        got = buf.field(f).cpu().numpy()
        assert got.tobytes() == np.ascontiguousarray(arr).tobytes(), f


def test_gae_worked_example_is_exact():
    """2 envs x 3 steps, gamma = lambda = 0.5: dyadic values, so the fp32 scan must be exact."""
    r = np.array([[1, 1], [2, -1], [3, 2]], np.float32)
    v = np.array([[0.5, 0], [1, 2], [1.5, -1]], np.float32)
    d = np.array([[0, 0], [0, 1], [0, 0]], np.uint8)
    lv = np.array([2, 4], np.float32)
    buf = ppo.Buffer(ppo.buffer_desc(2, 3, 4, 8, 32, 12))
    buf.field(ppo.FIELD_REWARD).copy_(torch.as_tensor(r))
    buf.field(ppo.FIELD_VALUE).copy_(torch.as_tensor(v))
    buf.field(ppo.FIELD_DONE).copy_(torch.as_tensor(d))
    stats = torch.zeros(2, device=DEV)
    ppo.ppo_compute_gae(buf, torch.as_tensor(lv).to(DEV), 0.5, 0.5, False, None)
    adv = buf.field(ppo.FIELD_ADV).cpu().numpy()
    ret = buf.field(ppo.FIELD_RET).cpu().numpy()
    assert np.array_equal(adv, [[1.59375, 1.25], [2.375, -3], [2.5, 5]])
    assert np.array_equal(ret, [[2.09375, 1.25], [3.375, -1], [4.0, 4.0]])
    ppo.ppo_compute_gae(buf, torch.as_tensor(lv).to(DEV), 0.5, 0.5, True, stats)
    advn = buf.field(ppo.FIELD_ADV).cpu().numpy().reshape(-1)
    want = [-0.0099498911, -0.1412884540, 0.2885468427, -1.7651106862, 0.3363063201, 1.2914958685]
    assert np.allclose(advn, want, atol=2e-7)
    assert np.allclose(stats.cpu().numpy(), [1.6197916667, 2.6172815593], rtol=1e-6)


@pytest.mark.parametrize("N,T,done_rate", [(1, 1, 0.0), (33, 7, 0.2), (256, 16, 0.01), (1000, 9, 1.0),
                                           (4096, 32, 0.01), (1027, 16, 0.0)])
def test_gae_and_normalisation_match_oracle(N, T, done_rate):
    w, roll, action, logp = _small(N, T, H=4, W=8, done_rate=done_rate, seed=N)
    buf = ppo.Buffer(ppo.buffer_desc(N, T, w.H, w.W, w.P, w.A))
    _fill(buf, roll, action, logp)
    lv = torch.as_tensor(roll["last_value"]).to(DEV)
    adv_o, ret_o = orc.gae(roll["reward"], roll["value"], roll["done"], roll["last_value"], np.float32(0.99),
                           np.float32(0.95))
    ppo.ppo_compute_gae(buf, lv, 0.99, 0.95, False, None)
    adv = buf.field(ppo.FIELD_ADV).cpu().numpy()
    ret = buf.field(ppo.FIELD_RET).cpu().numpy()
    assert rel_l2(adv, adv_o) <= GAE_TOL and max_abs_scaled(adv, adv_o) <= GAE_TOL
    assert rel_l2(ret, ret_o) <= GAE_TOL and max_abs_scaled(ret, ret_o) <= GAE_TOL
    if N * T > 1:
        stats = torch.zeros(2, device=DEV)
        ppo.ppo_compute_gae(buf, lv, 0.99, 0.95, True, stats)
        advn_o, mean_o, std_o = orc.adv_normalize(adv_o)
        advn = buf.field(ppo.FIELD_ADV).cpu().numpy()
        assert rel_l2(advn, advn_o) <= GAE_TOL and max_abs_scaled(advn, advn_o) <= GAE_TOL
        s = stats.cpu().numpy()
        assert abs(s[0] - mean_o) <= 1e-5 * max(1, abs(mean_o)) and abs(s[1] - std_o) <= 1e-5 * std_o
        # returns are not normalised
        assert np.array_equal(buf.field(ppo.FIELD_RET).cpu().numpy(), ret)
        # run twice: the reduction order is fixed, so the result is bit-identical
        ppo.ppo_compute_gae(buf, lv, 0.99, 0.95, True, stats)
        assert np.array_equal(buf.field(ppo.FIELD_ADV).cpu().numpy(), advn)
        # the single-launch variant (scan, grid barrier, normalisation) gives the same bits, twice in a row
        for _ in range(2):
            stats2 = torch.zeros(2, device=DEV)
            ppo.ppo_compute_gae(buf, lv, 0.99, 0.95, 2, stats2)
            assert np.array_equal(buf.field(ppo.FIELD_ADV).cpu().numpy(), advn)
            assert np.array_equal(buf.field(ppo.FIELD_RET).cpu().numpy(), ret)
            assert torch.equal(stats2, stats)
    assert ppo.ppo_poll_status() == 0


@pytest.mark.parametrize("N,T,H,W,K", [(8, 2, 4, 8, 1), (37, 5, 16, 24, 5), (256, 16, 64, 64, 4), (64, 16, 120, 160, 4),
                                       (25, 4, 30, 52, 10)])
def test_gather_is_bit_exact_and_follows_the_permutation(N, T, H, W, K):
    w, roll, action, logp = _small(N, T, H=H, W=W)
    buf = ppo.Buffer(ppo.buffer_desc(N, T, H, W, w.P, w.A))
    _fill(buf, roll, action, logp)
    ppo.ppo_compute_gae(buf, torch.as_tensor(roll["last_value"]).to(DEV), 0.99, 0.95, True, None)
    adv = buf.field(ppo.FIELD_ADV).cpu().numpy()
    ret = buf.field(ppo.FIELD_RET).cpu().numpy()
    M, B = N * T, N * T // K
    fields = {"depth": roll["depth"], "proprio": roll["proprio"], "action": action, "logp_old": logp,
              "value_old": roll["value"], "adv": adv, "ret": ret}
    seen = []
    for seed, epoch in [(0, 0), (0xDEADBEEF12345678, 3)]:
        for k in range(K):
            mb = ppo.MinibatchArrays(buf.desc, B)
            ppo.ppo_shuffle_gather_minibatch(buf, seed, epoch, k, K, mb)
            idx_o = orc.perm(seed, epoch, M, k * B, B)
            idx = mb.index.cpu().numpy().view(np.uint32)
            assert np.array_equal(idx, idx_o)
            want = orc.gather(fields, idx_o, N)
            for name in fields:
                got = getattr(mb, name).cpu().numpy()
                assert got.tobytes() == want[name].tobytes(), name
            if (seed, epoch) == (0, 0):
                seen.append(idx)
    assert np.array_equal(np.sort(np.concatenate(seen)), np.arange(M))
    assert ppo.ppo_poll_status() == 0


def test_gather_requires_gae_after_a_write():
    w, roll, action, logp = _small(8, 2, H=4, W=8)
    buf = ppo.Buffer(ppo.buffer_desc(8, 2, 4, 8, w.P, w.A))
    dev = _fill(buf, roll, action, logp)
    mb = ppo.MinibatchArrays(buf.desc, 16)
    with pytest.raises(ppo.PpoError) as e:
        ppo.ppo_shuffle_gather_minibatch(buf, 0, 0, 0, 1, mb)
    assert e.value.status == 4
    ppo.ppo_compute_gae(buf, dev["last_value"], 0.99, 0.95, True, None)
    ppo.ppo_shuffle_gather_minibatch(buf, 0, 0, 0, 1, mb)
    ppo.ppo_buffer_write_step(buf, 0, dev["depth"][0], dev["proprio"][0], torch.as_tensor(action[0]).to(DEV),
                              torch.as_tensor(logp[0]).to(DEV), dev["value"][0], dev["reward"][0], dev["done"][0])
    with pytest.raises(ppo.PpoError):
        ppo.ppo_shuffle_gather_minibatch(buf, 0, 0, 0, 1, mb)
