"""GPU parity at the workloads' full sizes, in the launch configuration the benchmark times.

The oracle cannot run a whole full-size step in seconds, so: GAE/normalisation are compared in full (cheap),
the permutation indices in full (bit-exact), gathered payload and encoder outputs on sampled rows that the
oracle computes one by one (a forward row depends on its own sample only), and the loss scalars on the
oracle's forward of those same rows via a property: the micro-batched sums equal the one-shot sums.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth
from paper_2509_16434_b200.learner import Learner
from helpers import max_abs_scaled, oracle_model, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda"
GAE_TOL = 1e-5
ENC_TOL = 2e-2
BENCH_MICROBATCH = 4096  # bench.py's default


def _device_rollout(w):
    roll = synth.rollout_torch(w, DEV, w.seed)
    g = torch.Generator(device=DEV)
    g.manual_seed(99)
    action = torch.randn((w.T, w.N, w.A), generator=g, device=DEV)
    logp = torch.randn((w.T, w.N), generator=g, device=DEV)
    return roll, action, logp


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5_1k", "cfg5_4k", "cfg5_16k"])
def test_gae_gather_at_full_size(name):
    w = synth.WORKLOADS[name]
    roll, action, logp = _device_rollout(w)
    buf = ppo.Buffer(ppo.buffer_desc(w.N, w.T, w.H, w.W, w.P, w.A))
    for t in range(w.T):
        ppo.ppo_buffer_write_step(buf, t, roll["depth"][t], roll["proprio"][t], action[t], logp[t], roll["value"][t],
                                  roll["reward"][t], roll["done"][t])
    # write_step is an exact copy (checked on the largest field by equality on the device)
    assert torch.equal(buf.field(ppo.FIELD_DEPTH), roll["depth"])
    stats = torch.zeros(2, device=DEV)
    ppo.ppo_compute_gae(buf, roll["last_value"], w.gamma, w.lam, True, stats)
    host = {k: roll[k].cpu().numpy() for k in ("reward", "value", "done", "last_value")}
    adv_o, ret_o = orc.gae(host["reward"], host["value"], host["done"], host["last_value"], np.float32(w.gamma),
                           np.float32(w.lam))
    advn_o, mean_o, std_o = orc.adv_normalize(adv_o)
    adv = buf.field(ppo.FIELD_ADV).cpu().numpy()
    ret = buf.field(ppo.FIELD_RET).cpu().numpy()
    assert rel_l2(adv, advn_o) <= GAE_TOL and max_abs_scaled(adv, advn_o) <= GAE_TOL
    assert rel_l2(ret, ret_o) <= GAE_TOL and max_abs_scaled(ret, ret_o) <= GAE_TOL
    s = stats.cpu().numpy()
    assert abs(s[0] - mean_o) <= 1e-5 * max(1, abs(mean_o)) and abs(s[1] - std_o) <= 1e-5 * std_o
    # gather: every index of the epoch bit-exact, payload of sampled rows byte-exact
    K, M = w.minibatches, w.M
    B = M // K
    mb = ppo.MinibatchArrays(buf.desc, B)
    seen = torch.zeros(M, dtype=torch.int32, device=DEV)
    rng = np.random.default_rng(0)
    flat = {"depth": roll["depth"].view(M, w.H, w.W), "proprio": roll["proprio"].view(M, w.P),
            "action": action.view(M, w.A), "logp_old": logp.view(M), "value_old": roll["value"].view(M),
            "adv": buf.field(ppo.FIELD_ADV).view(M), "ret": buf.field(ppo.FIELD_RET).view(M)}
    for k in range(K):
        ppo.ppo_shuffle_gather_minibatch(buf, 7, 2, k, K, mb)
        idx_o = orc.perm(7, 2, M, k * B, B)
        idx = mb.index.cpu().numpy().view(np.uint32)
        assert np.array_equal(idx, idx_o)
        seen[torch.as_tensor(idx_o.astype(np.int64), device=DEV)] += 1
        rows = rng.choice(B, size=64, replace=False)
        src = torch.as_tensor(idx_o[rows].astype(np.int64), device=DEV)
        rws = torch.as_tensor(rows, device=DEV)
        for f, arr in flat.items():
            assert torch.equal(getattr(mb, f)[rws], arr[src]), f
        # whole-array check of the biggest field through a checksum that any misplaced row changes
        wts = torch.arange(1, B + 1, device=DEV, dtype=torch.float64)
        got = (mb.depth.view(B, -1)[:, ::97].double().sum(1) * wts).sum()
        want = (flat["depth"].view(M, -1)[torch.as_tensor(idx_o.astype(np.int64), device=DEV)][:, ::97].double().sum(1)
                * wts).sum()
        assert got.item() == want.item()
    assert bool((seen == 1).all()), "the minibatches of an epoch partition the buffer"
    assert ppo.ppo_poll_status() == 0


@pytest.mark.parametrize("name,rows_checked", [("cfg2", 24), ("cfg4", 4)])
def test_encoder_forward_sampled_rows_at_bench_shapes(name, rows_checked):
    """One full micro-batch (the benchmark's launch shapes) through the forward; sampled rows against the oracle."""
    w0 = synth.WORKLOADS[name]
    mbs = min(BENCH_MICROBATCH, w0.B)
    # a buffer with just enough envs for one minibatch of `mbs` rows keeps the test's footprint small
    w = w0.scaled(mbs // w0.T * w0.minibatches, minibatches=w0.minibatches)
    assert w.B == mbs
    md = oracle_model(w)
    lay = orc.param_layout(md)
    theta = synth.init_params(lay.total, lay.offsets, lay.shapes, 0)
    hw = len(lay.offsets) - 3
    theta[lay.offsets[hw]:lay.offsets[hw] + lay.sizes[hw]] *= 20.0  # a head that is not nearly zero
    roll, action, logp = _device_rollout(w)
    L = Learner(w, mbs, DEV, with_index=True)
    L.model.load(theta)
    L.write_rollout(roll, action, logp)
    L.compute_gae(roll["last_value"])
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 0, 0, 1, w.minibatches, L.mb)
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, mbs, L.mean, L.value)
    assert ppo.ppo_poll_status() == 0
    rng = np.random.default_rng(1)
    rows = np.sort(rng.choice(mbs, size=rows_checked, replace=False))
    rows[0], rows[-1] = 0, mbs - 1  # first and last row of the micro-batch
    r = torch.as_tensor(rows, device=DEV)
    depth = L.mb.depth[r].cpu().numpy()
    proprio = L.mb.proprio[r].cpu().numpy()
    mu = L.mean[r].cpu().numpy()
    V = L.value[r].cpu().numpy()
    # against the oracle that stores its activations as bf16 values like the kernels do, and against the one that
    # keeps them in fp64 between layers
    for act_bf16 in (True, False):
        mu_o, V_o, _ = orc.encoder_fwd(md, orc.round_weights(md, theta), depth, proprio, act_bf16)
        print(f"[{name}] bench-shape forward, oracle activations {'bf16' if act_bf16 else 'fp64'}: "
              f"mu {rel_l2(mu, mu_o):.3e}, V {rel_l2(V, V_o):.3e}")
        assert rel_l2(mu, mu_o) <= ENC_TOL, rel_l2(mu, mu_o)
        assert rel_l2(V, V_o) <= ENC_TOL, rel_l2(V, V_o)


def test_microbatched_gradients_add_up_at_bench_shapes():
    """Property at full minibatch size: the gradient accumulated over micro-batches equals the one of a single
    pass over the same minibatch (sums of the same per-sample terms, up to fp32/atomic summation order)."""
    w0 = synth.WORKLOADS["cfg2"]
    w = w0.scaled(256, minibatches=4)  # minibatch of 1024 rows
    md = oracle_model(w)
    lay = orc.param_layout(md)
    theta = synth.init_params(lay.total, lay.offsets, lay.shapes, 0)
    roll, action, logp = _device_rollout(w)
    grads = []
    for mbs in (w.B, 384):  # one pass; three ragged micro-batches (384, 384, 256)
        L = Learner(w, mbs, DEV)
        L.model.load(theta)
        L.write_rollout(roll, action, logp)
        L.compute_gae(roll["last_value"])
        h = L.hyper
        ppo.ppo_shuffle_gather_minibatch(L.buffer, 1, 0, 0, w.minibatches, L.mb)
        ppo.ppo_model_zero_grad(L.model)
        L.loss.zero_()
        for r0 in range(0, w.B, mbs):
            n = min(mbs, w.B - r0)
            ppo.ppo_encoder_fwd(L.model, L.mb, r0, n, L.mean, L.value)
            ppo.ppo_loss_fwd_bwd(L.model, L.mb, r0, n, w.B, L.mean, L.value, h.clip, h.vf_coef, h.ent_coef, L.loss,
                                 L.dmean, L.dvalue)
            ppo.ppo_encoder_bwd(L.model, L.mb, r0, n, L.dmean, L.dvalue, True)
        assert ppo.ppo_poll_status() == 0
        grads.append((L.model.grad.cpu().numpy().copy(), L.loss.cpu().numpy().copy()))
    (g1, l1), (g2, l2) = grads
    assert np.allclose(l1, l2, rtol=1e-4, atol=1e-6)
    for off, sz in zip(lay.offsets, lay.sizes):
        assert rel_l2(g2[off:off + sz], g1[off:off + sz]) <= 1e-3
