"""GPU parity of the synthetic depth producer (ppo_buffer_render_depth) against the oracle's analytic renderer.

The kernel works in fp32, the oracle in fp64, and which primitive a ray meets first (or whether it meets one at all)
is a discrete decision: the two sides may take it differently only for rays that graze a silhouette.  So: every
pixel that is not next to a depth discontinuity of the oracle's image must agree to one fp16 step, and the pixels
that disagree by more must be few and must all sit on such a discontinuity."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
HFOV, NEAR, FAR = 1.2, 0.1, 2.0


def _edges(img, thr=0.02):
    """Pixels with a 4-neighbour whose depth differs by more than thr (or by presence of a return)."""
    e = np.zeros(img.shape, bool)
    dv = np.abs(np.diff(img, axis=-2)) > thr
    dh = np.abs(np.diff(img, axis=-1)) > thr
    e[..., 1:, :] |= dv
    e[..., :-1, :] |= dv
    e[..., :, 1:] |= dh
    e[..., :, :-1] |= dh
    return e


@pytest.mark.parametrize("N,H,W,K", [(5, 33, 47, 6), (16, 120, 160, 8), (3, 240, 320, 32), (4, 16, 24, 0)])
def test_rendered_frames_match_the_oracle(N, H, W, K):
    T = 3
    plane, prims = synth.scenes_numpy(N, max(K, 1), seed=7)
    prims = prims[:, :K]
    buf = ppo.Buffer(ppo.buffer_desc(N, T, H, W, 32, 12))
    buf.field(ppo.FIELD_DEPTH).fill_(-1.0)
    t = 1
    ppo.ppo_buffer_render_depth(buf, t, HFOV, NEAR, FAR, torch.as_tensor(plane).to(DEV),
                                torch.as_tensor(np.ascontiguousarray(prims)).to(DEV).reshape(N, K, 8))
    assert ppo.ppo_poll_status() == 0
    depth = buf.field(ppo.FIELD_DEPTH).cpu().numpy().astype(np.float64)
    assert np.all(depth[0] == -1.0) and np.all(depth[2] == -1.0), "only slab row t is written"
    got = depth[t]
    want = orc.render_depth(H, W, HFOV, NEAR, FAR, plane, prims.reshape(N, K, 8))
    step = np.maximum(np.abs(want), 2.0 ** -14) * 2.0 ** -10  # one fp16 step at the value
    bad = np.abs(got - want) > step
    edge = _edges(want)
    assert not np.any(bad & ~edge), "disagreement away from any silhouette"
    frac = bad.mean()
    print(f"[{N}x{H}x{W}, {K} prims] pixels off by more than one fp16 step: {frac:.2e} (all on silhouettes); "
          f"no-return pixels {np.mean(want == 0):.3f}")
    assert frac <= 2e-3
    if K > 0:
        assert 0.0 < np.mean(want == 0) < 1.0 or np.ptp(want) > 0.1  # the scenes have structure


def test_rendered_rollout_feeds_the_policy_and_the_learner():
    """Rendered frames go through the same path as any other observation: the policy acts on slab row t in place."""
    w = synth.WORKLOADS["cfg1"].scaled(16, T=4, minibatches=2)
    from paper_2509_16434_b200.learner import Learner
    L = Learner(w, 16, DEV)
    shapes, gammas = synth.param_shapes(w)
    theta = synth.init_params(L.model.arena, [o for o, _ in L.model.tensors()], shapes, 0, ones=gammas)
    L.model.load(theta)
    roll = synth.rollout_numpy(w, 0)
    dev = {k: torch.as_tensor(v).to(DEV) for k, v in roll.items()}
    for t in range(w.T):
        plane, prims = synth.scenes_numpy(w.N, 6, seed=100 + t)
        ppo.ppo_buffer_render_depth(L.buffer, t, HFOV, NEAR, FAR, torch.as_tensor(plane).to(DEV), torch.as_tensor(prims).to(DEV))
        L.buffer.field(ppo.FIELD_PROPRIO)[t].copy_(dev["proprio"][t])
        ppo.ppo_policy_act(L.model, L.buffer, t, dev["eps"][t])
        ppo.ppo_buffer_write_outcome(L.buffer, t, dev["reward"][t], dev["done"][t])
    L.train(dev["last_value"], seed=0)
    assert ppo.ppo_poll_status() == 0
    assert bool(torch.isfinite(L.loss).all()) and bool(torch.isfinite(L.model.master).all())
    d = L.buffer.field(ppo.FIELD_DEPTH)
    assert float(d.max()) <= FAR and float(d[d > 0].min()) >= NEAR * 0.999
