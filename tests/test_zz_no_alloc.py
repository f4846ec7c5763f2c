"""GPU check of ppo_gae_static, the GAE entry point that allocates nothing.

It exists for callers that cannot call cudaMalloc (a host application that owns one fixed arena, a fixed
memory budget, code that must not synchronise the device): its scratch lives in a fixed array inside the
library.  The check: on the same inputs it must reproduce what ppo_compute_gae leaves in the buffer slabs,
on two calls in a row with different inputs (the second call finds the first call's leftovers in the shared
scratch).  Collected last on purpose, so that a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

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


def test_static_gae_rejects_more_envs_than_its_scratch_covers():
    # only the size check runs: no array of that size is touched
    t = torch.zeros(1, device=DEV)
    status = ppo.lib().ppo_gae_static(ppo._ptr(t), ppo._ptr(t), ppo._ptr(t), ppo._ptr(t), 1, 524288 + 1, 0.99, 0.95, 1,
                                      ppo._ptr(t), ppo._ptr(t), None, ppo._stream())
    assert status == 7, ppo.ppo_status_string(status)
