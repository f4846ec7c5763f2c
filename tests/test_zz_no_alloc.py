"""GPU check of ppo_gae_static, the GAE entry point that allocates nothing.

It exists for callers that cannot call cudaMalloc (a host application that owns one fixed arena, a fixed
memory budget, code that must not synchronise the device): its scratch lives in a fixed array inside the
library.  The check: on the same inputs it must reproduce what ppo_compute_gae leaves in the buffer slabs,
on two calls in a row with different inputs (the second call finds the first call's leftovers in the shared
scratch), and what the CPU oracle computes; the device's free memory must be the same before and after a call;
and the largest env count it accepts must work.  Collected last on purpose, so that a run that stops at the
first failure has run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth
from helpers import max_abs_scaled, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda"
GAE_TOL = 1e-5  # the tolerance of the GAE parity tests


def _reference(N, T, roll, normalize):
    """The existing entry point: fill a buffer's reward/value/done slabs, run ppo_compute_gae, read the slabs back."""
    buf = ppo.Buffer(ppo.buffer_desc(N, T, 4, 8, 32, 12))
    buf.field(ppo.FIELD_REWARD).copy_(torch.as_tensor(roll["reward"]))
    buf.field(ppo.FIELD_VALUE).copy_(torch.as_tensor(roll["value"]))
    buf.field(ppo.FIELD_DONE).copy_(torch.as_tensor(roll["done"]))
    stats = torch.zeros(2, device=DEV)
    ppo.ppo_compute_gae(buf, torch.as_tensor(roll["last_value"]).to(DEV), 0.99, 0.95, normalize, stats)
    return (buf.field(ppo.FIELD_ADV).cpu().numpy().copy(), buf.field(ppo.FIELD_RET).cpu().numpy().copy(),
            stats.cpu().numpy().copy())


@pytest.mark.parametrize("normalize", [True, False])
def test_static_gae_matches_the_buffer_entry_point_twice_in_a_row(normalize):
    # two different problems back to back: the larger one first, so that the second call sees stale partial sums
    # beyond the part of the scratch it rewrites
    for N, T, seed in [(4099, 16, 3), (257, 7, 4)]:
        w = synth.WORKLOADS["cfg1"].scaled(N, T=T, H=4, W=8, done_rate=0.05)
        roll = synth.rollout_numpy(w, seed)
        want_adv, want_ret, want_stats = _reference(N, T, roll, normalize)
        dev = {k: torch.as_tensor(roll[k]).to(DEV) for k in ("reward", "value", "done", "last_value")}
        adv = torch.full((T, N), float("nan"), device=DEV)
        ret = torch.full((T, N), float("nan"), device=DEV)
        stats = torch.zeros(2, device=DEV)
        ppo.ppo_gae_static(dev["reward"], dev["value"], dev["done"], dev["last_value"], 0.99, 0.95, normalize, adv, ret,
                           stats)
        assert ppo.ppo_poll_status() == 0
        got_adv, got_ret = adv.cpu().numpy(), ret.cpu().numpy()
        assert rel_l2(got_adv, want_adv) <= GAE_TOL and max_abs_scaled(got_adv, want_adv) <= GAE_TOL
        assert rel_l2(got_ret, want_ret) <= GAE_TOL and max_abs_scaled(got_ret, want_ret) <= GAE_TOL
        if normalize:
            assert np.allclose(stats.cpu().numpy(), want_stats, rtol=1e-6, atol=1e-7)
        # and against the CPU oracle directly
        adv_o, ret_o = orc.gae(roll["reward"], roll["value"], roll["done"], roll["last_value"], np.float32(0.99),
                               np.float32(0.95))
        if normalize:
            adv_o, mean_o, std_o = orc.adv_normalize(adv_o)
            st = stats.cpu().numpy()
            assert abs(st[0] - mean_o) <= 1e-5 * max(1, abs(mean_o)) and abs(st[1] - std_o) <= 1e-5 * std_o
        assert rel_l2(got_adv, adv_o) <= GAE_TOL and max_abs_scaled(got_adv, adv_o) <= GAE_TOL
        assert rel_l2(got_ret, ret_o) <= GAE_TOL and max_abs_scaled(got_ret, ret_o) <= GAE_TOL


def test_static_gae_leaves_the_free_device_memory_unchanged_and_takes_its_largest_size():
    """N = 524288 envs is the most the fixed scratch covers (4096 blocks of partial sums).  The first call on a
    device may make the CUDA runtime load the library's module; after that warm-up a call must not change the
    device's free memory, i.e. nothing was allocated on its behalf."""
    N, T = ppo_max_envs(), 1
    g = torch.Generator(device=DEV)
    g.manual_seed(5)
    reward = torch.randn((T, N), generator=g, device=DEV)
    value = torch.randn((T, N), generator=g, device=DEV)
    done = (torch.rand((T, N), generator=g, device=DEV) < 0.05).to(torch.uint8)
    lastv = torch.randn(N, generator=g, device=DEV)
    adv, ret = torch.empty_like(reward), torch.empty_like(reward)
    stats = torch.zeros(2, device=DEV)
    ppo.ppo_gae_static(reward, value, done, lastv, 0.99, 0.95, True, adv, ret, stats)  # warm-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    ppo.ppo_gae_static(reward, value, done, lastv, 0.99, 0.95, True, adv, ret, stats)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert ppo.ppo_poll_status() == 0
    adv_o, ret_o = orc.gae(reward.cpu().numpy(), value.cpu().numpy(), done.cpu().numpy(), lastv.cpu().numpy(),
                           np.float32(0.99), np.float32(0.95))
    adv_o, _, _ = orc.adv_normalize(adv_o)
    assert rel_l2(adv.cpu().numpy(), adv_o) <= GAE_TOL and max_abs_scaled(adv.cpu().numpy(), adv_o) <= GAE_TOL
    assert rel_l2(ret.cpu().numpy(), ret_o) <= GAE_TOL


def ppo_max_envs():
    return 524288  # PPO_GAE_STATIC_MAX_ENVS


def test_static_gae_rejects_more_envs_than_its_scratch_covers():
    # only the size check runs: no array of that size is touched
    t = torch.zeros(1, device=DEV)
    status = ppo.lib().ppo_gae_static(ppo._ptr(t), ppo._ptr(t), ppo._ptr(t), ppo._ptr(t), 1, 524288 + 1, 0.99, 0.95, 1,
                                      ppo._ptr(t), ppo._ptr(t), None, ppo._stream())
    assert status == 7, ppo.ppo_status_string(status)
