"""GPU parity: encoder forward/backward, PPO loss + gradient, Adam and whole minibatch steps against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth
from paper_2509_16434_b200.learner import Hyper, Learner
from helpers import oracle_model, oracle_rollout_actions, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda"
ENC_TOL = 2e-2    # relative L2: bf16 operands / activations with fp32 accumulation vs fp64
LOSS_TOL = 1e-3   # relative error of the loss scalars
ADAM_TOL = 1e-3   # relative L2 of the parameters after one step
# End-to-end gradients (GPU forward feeding GPU backward) against the oracle's own forward+backward.  What separates
# the two sides beyond the arithmetic is the handful of ReLU gates (measured: 0 to 2 in 10^6 of the stored
# activations) that the two forwards decide differently: a flipped gate of a deep layer removes or adds that unit's
# whole contribution, and in a minibatch of a few rows one such unit is a visible share of a tensor's gradient
# (measured: 5.3e-2 of the whole gradient with 4 flipped gates in 4 rows of the cfg4 network, 7e-2 on one tensor in
# 8 rows of cfg2's, 6e-3 of the whole gradient at 1024 rows).  These bounds therefore only catch gross errors;
# test_gpu_parity_wide.py counts the flipped gates and holds the backward pass to 2e-2 per tensor against the
# oracle's backward from the very activations the GPU saved, and on the oracle's activations at up to 1024 rows.
E2E_GRAD_TOL_TOTAL = 1e-1
E2E_GRAD_TOL_TENSOR = 2e-1
SIGN_AGREEMENT = 0.97  # fraction of clearly moved parameters whose Adam update has the oracle's sign


def _setup(w, microbatch, seed=0, jitter=True, theta_scale_head=1.0):
    """Learner with seeded parameters and a buffer filled from the oracle-side rollout policy."""
    md = oracle_model(w)
    lay = orc.param_layout(md)
    theta = synth.init_params(lay.total, lay.offsets, lay.shapes, seed)
    if theta_scale_head != 1.0:
        hw = len(lay.offsets) - 3
        theta[lay.offsets[hw]:lay.offsets[hw] + lay.sizes[hw]] *= theta_scale_head
    g = np.random.default_rng(seed + 7)
    for off, sz, shp in zip(lay.offsets, lay.sizes, lay.shapes):
        if len(shp) == 1:
            theta[off:off + sz] = (0.05 * g.standard_normal(sz)).astype(np.float32)
    for i in synth.param_shapes(w)[1]:  # layer-normalisation scales sit around 1
        theta[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]] += 1.0
    roll = synth.rollout_numpy(w, seed)
    action, logp = oracle_rollout_actions(md, theta, roll)
    if jitter:
        logp = (logp + roll["logp_jitter"]).astype(np.float32)
    L = Learner(w, microbatch, DEV, with_index=True)
    L.model.load(theta)
    dev = {k: torch.as_tensor(v).to(DEV) for k, v in roll.items()}
    L.write_rollout(dev, torch.as_tensor(action).to(DEV), torch.as_tensor(logp).to(DEV))
    return L, md, lay, theta, roll, action, logp, dev


def _oracle_minibatch(md, lay, theta, roll, action, logp, w, hyper, seed, epoch, k, K):
    adv, ret = orc.gae(roll["reward"], roll["value"], roll["done"], roll["last_value"], np.float32(hyper.gamma),
                       np.float32(hyper.lam))
    adv, _, _ = orc.adv_normalize(adv)
    M = w.N * w.T
    B = M // K
    idx = orc.perm(seed, epoch, M, k * B, B)
    f = orc.gather({"depth": roll["depth"], "proprio": roll["proprio"], "action": action, "logp": logp,
                    "adv": adv.astype(np.float32), "ret": ret.astype(np.float32)}, idx, w.N)
    Ltot, out, grad, mu, V = orc.total_loss_and_grad(md, theta, f["depth"], f["proprio"], f["action"], f["logp"],
                                                     f["adv"], f["ret"], np.float32(hyper.clip),
                                                     np.float32(hyper.vf_coef), np.float32(hyper.ent_coef),
                                                     act_bf16=True)
    return f, out, grad, mu, V


def _check_grads(lay, got, want, tol=ENC_TOL, tol_total=None):
    for i, (off, sz) in enumerate(zip(lay.offsets, lay.sizes)):
        e = rel_l2(got[off:off + sz], want[off:off + sz])
        assert e <= tol, f"tensor {i}: rel L2 {e:.3e}"
    assert rel_l2(got, want) <= (tol if tol_total is None else tol_total)


def _upload_oracle_activations(L, md, acts, B):
    """Replaces the activations the GPU forward saved by the oracle's (bf16 values), layer by layer."""
    Ho, Wo = orc.conv_shapes(md)
    off = md.H * md.W
    for l, (h, w_, c) in enumerate(zip(Ho, Wo, md.conv_c), start=1):
        n = h * w_ * c
        L.model.activation(0, l)[:B * n].copy_(torch.as_tensor(acts[:, off:off + n].reshape(-1)).to(torch.bfloat16))
        off += n
    widths = [(md.embed or md.conv_c[-1]) + md.P] + list(md.fc)
    for l, n in enumerate(widths):
        L.model.activation(1, l)[:B * n].copy_(torch.as_tensor(acts[:, off:off + n].reshape(-1)).to(torch.bfloat16))
        off += n
    if md.norm:  # the normalised values and reciprocal standard deviations the backward pass reads
        for l, (h, w_, c) in enumerate(zip(Ho, Wo, md.conv_c), start=1):
            n = h * w_ * c
            L.model.activation(3, l)[:B * n].copy_(torch.as_tensor(acts[:, off:off + n].reshape(-1)).to(torch.bfloat16))
            off += n
            L.model.activation(4, l)[:B * h * w_].copy_(torch.as_tensor(acts[:, off:off + h * w_].reshape(-1)).float())
            off += h * w_
    assert off == acts.shape[1]


@pytest.mark.parametrize("name", ["tiny", "odd", "cfg1_twin", "cfg2_twin", "cfg4_twin"])
def test_backward_matches_oracle_on_identical_activations(name):
    """The backward operator alone: both sides start from the oracle's saved activations, mean and value."""
    w = SHAPES[name]
    B = w.M // w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, B, theta_scale_head=20.0)
    h = L.hyper
    K = w.minibatches
    L.compute_gae(dev["last_value"])
    f, out_o, grad_o, mu_o, V_o = _oracle_minibatch(md, lay, theta, roll, action, logp, w, h, 5, 0, 0, K)
    _, _, acts = orc.encoder_fwd(md, orc.round_weights(md, theta), f["depth"], f["proprio"], True)
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 5, 0, 0, K, L.mb)
    ppo.ppo_model_zero_grad(L.model)
    L.loss.zero_()
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, B, L.mean, L.value)
    _upload_oracle_activations(L, md, acts, B)
    ppo.ppo_model_sync_masks(L.model, B)
    L.mean[:B].copy_(torch.as_tensor(mu_o, dtype=torch.float32))
    L.value[:B].copy_(torch.as_tensor(V_o, dtype=torch.float32))
    ppo.ppo_loss_fwd_bwd(L.model, L.mb, 0, B, B, L.mean, L.value, h.clip, h.vf_coef, h.ent_coef, L.loss, L.dmean,
                         L.dvalue)
    ppo.ppo_encoder_bwd(L.model, L.mb, 0, B, L.dmean, L.dvalue, True)
    assert ppo.ppo_poll_status() == 0
    out = L.loss.cpu().numpy()
    for j in range(5):
        assert abs(out[j] - out_o[j]) <= LOSS_TOL * max(abs(out_o[j]), 1e-2), (j, out[j], out_o[j])
    _check_grads(lay, L.model.grad.cpu().numpy(), grad_o)


SHAPES = {
    "tiny": synth.Workload("tiny", 8, 4, 16, 24, (8, 16), (3, 3), (32,), 1, 2, P=8, A=3),
    "odd": synth.Workload("odd", 6, 5, 17, 23, (8, 16, 24), (5, 3, 3), (40, 24), 1, 3, P=16, A=5),
    "cfg1_twin": synth.WORKLOADS["cfg1"].scaled(16, T=4),
    "cfg2_twin": synth.WORKLOADS["cfg2"].scaled(8, T=2, minibatches=2),
    "cfg4_twin": synth.WORKLOADS["cfg4"].scaled(2, T=2, minibatches=2),
}


@pytest.mark.parametrize("name,microbatch", [("tiny", 16), ("tiny", 5), ("odd", 10), ("cfg1_twin", 16),
                                             ("cfg2_twin", 8), ("cfg2_twin", 3), ("cfg4_twin", 2)])
def test_minibatch_forward_loss_backward_match_oracle(name, microbatch):
    w = SHAPES[name]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, microbatch, theta_scale_head=20.0)
    h = L.hyper
    K = w.minibatches
    B = w.M // K
    L.compute_gae(dev["last_value"])
    k = K - 1
    f, out_o, grad_o, mu_o, V_o = _oracle_minibatch(md, lay, theta, roll, action, logp, w, h, 3, 1, k, K)
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 3, 1, k, K, L.mb)
    ppo.ppo_model_zero_grad(L.model)
    L.loss.zero_()
    mus, Vs = [], []
    for r0 in range(0, B, L.microbatch):
        rows = min(L.microbatch, B - r0)
        ppo.ppo_encoder_fwd(L.model, L.mb, r0, rows, L.mean, L.value)
        mus.append(L.mean[:rows].cpu().numpy().copy())
        Vs.append(L.value[:rows].cpu().numpy().copy())
        ppo.ppo_loss_fwd_bwd(L.model, L.mb, r0, rows, B, L.mean, L.value, h.clip, h.vf_coef, h.ent_coef, L.loss,
                             L.dmean, L.dvalue)
        ppo.ppo_encoder_bwd(L.model, L.mb, r0, rows, L.dmean, L.dvalue, True)
    assert ppo.ppo_poll_status() == 0
    mu, V = np.concatenate(mus), np.concatenate(Vs)
    assert rel_l2(mu, mu_o) <= ENC_TOL, rel_l2(mu, mu_o)
    assert rel_l2(V, V_o) <= ENC_TOL, rel_l2(V, V_o)
    out = L.loss.cpu().numpy()
    assert 0.0 < out_o[4] < 1.0, "both clip branches must be exercised"
    # Entropy (exact arithmetic on log-sigma) to 1e-3 relative.  The value loss is a mean of squared differences V - R
    # and the policy loss and the KL estimate are means of signed terms near zero, so their errors are measured
    # against the mean magnitude of what enters them (V^2 + R^2, |s| ~ |adv|, |log ratio|).  They inherit the encoder's
    # error in mu and V (2e-3 here, inside its 2e-2): over 8 rows and more it averages below 1e-3
    # (test_gpu_parity_wide.py holds that), in a minibatch of 2 to 16 rows it shows almost undiminished, so the
    # bound here is 5e-3 (measured: up to 2e-3).
    small = 5 * LOSS_TOL
    assert abs(out[1] - out_o[1]) <= small * max(abs(out_o[1]), float(np.mean(V_o ** 2 + f["ret"] ** 2)))
    assert abs(out[2] - out_o[2]) <= LOSS_TOL * abs(out_o[2])
    assert abs(out[0] - out_o[0]) <= small * float(np.mean(np.abs(f["adv"])))
    assert abs(out[3] - out_o[3]) <= small * max(1.0, abs(out_o[3]))
    assert abs(out[4] - out_o[4]) <= 2.0 / B + 1e-6
    got = L.model.grad.cpu().numpy()
    errs = [rel_l2(got[o:o + s], grad_o[o:o + s]) for o, s in zip(lay.offsets, lay.sizes)]
    print(f"[{name}-{microbatch}] end-to-end gradients: max per tensor {max(errs):.3e} (tensor {int(np.argmax(errs))}), "
          f"total {rel_l2(got, grad_o):.3e}")
    _check_grads(lay, got, grad_o, E2E_GRAD_TOL_TENSOR, E2E_GRAD_TOL_TOTAL)


def test_loss_kernel_alone_matches_oracle_to_1e3():
    """Same mu and V on both sides: isolates the fused loss/gradient kernel (fp32 vs fp64)."""
    w = SHAPES["cfg1_twin"].scaled(16, minibatches=1)  # one minibatch of 64 rows
    L, md, lay, theta, roll, action, logp, dev = _setup(w, 64)
    g = np.random.default_rng(0)
    B, A = 64, w.A
    mu = (0.3 * g.standard_normal((B, A))).astype(np.float32)
    V = g.standard_normal(B).astype(np.float32)
    ls = (0.2 * g.standard_normal(A)).astype(np.float32)
    act = (mu + np.exp(ls) * g.standard_normal((B, A))).astype(np.float32)
    z = (act - mu) / np.exp(ls)
    lpo = ((-0.5 * z ** 2 - ls - 0.5 * np.log(2 * np.pi)).sum(1) + 0.3 * g.standard_normal(B)).astype(np.float32)
    adv, ret = g.standard_normal(B).astype(np.float32), g.standard_normal(B).astype(np.float32)
    L.model.master[lay.offsets[-1]:lay.offsets[-1] + A] = torch.as_tensor(ls).to(DEV)
    mb = ppo.MinibatchArrays(L.bdesc, B)
    mb.action.copy_(torch.as_tensor(act))
    mb.logp_old.copy_(torch.as_tensor(lpo))
    mb.adv.copy_(torch.as_tensor(adv))
    mb.ret.copy_(torch.as_tensor(ret))
    out_o, dmu_o, dV_o, dls_o = orc.loss(mu, V, ls, act, lpo, adv, ret, np.float32(0.2), 0.5, np.float32(0.01))
    ppo.ppo_model_zero_grad(L.model)
    L.loss.zero_()
    dmean = torch.empty((B, A), device=DEV)
    dvalue = torch.empty(B, device=DEV)
    # two micro-batches of uneven size must add up to the minibatch
    mean_d, value_d = torch.as_tensor(mu).to(DEV), torch.as_tensor(V).to(DEV)
    for r0, rows in [(0, 40), (40, 24)]:
        ppo.ppo_loss_fwd_bwd(L.model, mb, r0, rows, B, mean_d[r0:], value_d[r0:], 0.2, 0.5, 0.01, L.loss,
                             dmean[r0:], dvalue[r0:])
    out = L.loss.cpu().numpy()
    assert 0 < out_o[4] < 1
    for j in range(5):
        assert abs(out[j] - out_o[j]) <= LOSS_TOL * max(abs(out_o[j]), 1e-3), (j, out[j], out_o[j])
    assert rel_l2(dmean.cpu().numpy(), dmu_o) <= LOSS_TOL
    assert rel_l2(dvalue.cpu().numpy(), dV_o) <= LOSS_TOL
    dls = L.model.grad[lay.offsets[-1]:lay.offsets[-1] + A].cpu().numpy()
    assert rel_l2(dls, dls_o) <= LOSS_TOL
    assert ppo.ppo_poll_status() == 0


def test_ratio_is_one_on_the_rollout_policy():
    """Old log-probs from the same weights: r = 1 up to the encoder's rounding, so nothing is clipped."""
    w = SHAPES["cfg1_twin"].scaled(16, minibatches=2)
    L, md, lay, theta, roll, action, logp, dev = _setup(w, 32, jitter=False)
    L.compute_gae(dev["last_value"])
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 0, 0, 0, 2, L.mb)
    L.loss.zero_()
    ppo.ppo_model_zero_grad(L.model)
    B = w.M // 2
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, B, L.mean, L.value)
    ppo.ppo_loss_fwd_bwd(L.model, L.mb, 0, B, B, L.mean, L.value, 0.2, 0.5, 0.01, L.loss, L.dmean, L.dvalue)
    out = L.loss.cpu().numpy()
    assert out[4] == 0.0 and abs(out[3]) < 5e-3
    assert abs(out[0] + L.mb.adv[:B].mean().item()) < 5e-3


def test_adam_step_matches_oracle():
    w = SHAPES["cfg1_twin"]
    L, md, lay, theta, *_ = _setup(w, 16)
    n = lay.total
    g = np.random.default_rng(5)
    grad = (g.standard_normal(n) * (g.random(n) < 0.9)).astype(np.float32)
    m0 = (0.1 * g.standard_normal(n)).astype(np.float32)
    v0 = (0.01 * g.random(n)).astype(np.float32)
    L.model.grad.copy_(torch.as_tensor(grad))
    L.model.adam_m.copy_(torch.as_tensor(m0))
    L.model.adam_v.copy_(torch.as_tensor(v0))
    th, m, v = theta.astype(np.float64), m0.astype(np.float64), v0.astype(np.float64)
    for step in (1, 2, 7):
        orc.adam(th, m, v, grad, np.float32(3e-4), np.float32(0.9), np.float32(0.999), np.float32(1e-8), step)
        ppo.ppo_adam_step(L.model, 3e-4, 0.9, 0.999, 1e-8, step)
        got = L.model.master.cpu().numpy()
        assert rel_l2(got, th) <= ADAM_TOL
        assert rel_l2(got - theta, th - theta) <= ADAM_TOL, "the update itself, not just theta"
        assert rel_l2(L.model.adam_m.cpu().numpy(), m) <= 1e-5
        assert rel_l2(L.model.adam_v.cpu().numpy(), v) <= 1e-5
        sh = L.model.shadow.float().cpu().numpy()
        want = torch.as_tensor(got).to(torch.bfloat16).float().numpy()
        assert np.array_equal(sh, want), "shadow must be the bf16 rounding of the new master"
    assert ppo.ppo_poll_status() == 0


@pytest.mark.parametrize("name,microbatch", [("cfg1_twin", 16), ("cfg2_twin", 8)])
def test_whole_learner_step_parameters_match_oracle(name, microbatch):
    """GAE -> every minibatch of one epoch (gather, fwd, loss, bwd, Adam).  Parameters are compared after the first
    Adam step at ADAM_TOL and after the last one at ADAM_TOL per step taken: Adam's first steps move every
    parameter by ~lr * sign(g), so a gradient whose sign is not settled (|g| below its own error) moves the
    wrong way by the full step and the error grows with the number of steps, not with the gradient error."""
    w = SHAPES[name]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, microbatch, theta_scale_head=20.0)
    h = L.hyper
    L.compute_gae(dev["last_value"])
    th = theta.astype(np.float64)
    m, v = np.zeros_like(th), np.zeros_like(th)
    for k in range(w.minibatches):
        L.minibatch_step(11, 0, k)
        _, _, grad, _, _ = _oracle_minibatch(md, lay, th.astype(np.float32), roll, action, logp, w, h, 11, 0, k,
                                             w.minibatches)
        orc.adam(th, m, v, grad, np.float32(h.lr), np.float32(h.beta1), np.float32(h.beta2), np.float32(h.eps), k + 1)
        got = L.model.master.cpu().numpy()
        assert rel_l2(got, th) <= ADAM_TOL * (k + 1), (k, rel_l2(got, th))
    assert ppo.ppo_poll_status() == 0
    # The update itself: after a few Adam steps from m = v = 0 every parameter has moved by about lr * (steps) *
    # sign(g), so its relative L2 error is sqrt(4 x the fraction of parameters whose gradient sign differs), and a
    # sign differs only where |g| is below the gradient's own error.  Measured as that fraction over the parameters
    # the oracle moved by at least half a step.
    du_g, du_o = got - theta, th - theta
    moved = np.abs(du_o) >= 0.5 * h.lr
    agree = float(np.mean(np.sign(du_g[moved]) == np.sign(du_o[moved])))
    print(f"[{name}] update after {w.minibatches} Adam steps: sign agreement {agree:.4f} over {int(moved.sum())} "
          f"parameters, rel L2 {rel_l2(du_g, du_o):.3e}")
    assert agree >= SIGN_AGREEMENT


def test_policy_act_writes_the_rollout_step_into_its_slab_row():
    """ppo_buffer_write_obs + ppo_policy_act + ppo_buffer_write_outcome fill slab row t like the oracle's rollout:
    observation, reward and done byte-exact, action / log-prob / value from the policy on that observation."""
    w = SHAPES["cfg1_twin"]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, 5, jitter=False)  # 16 envs in micro-batches of 5, 5, 5, 1
    buf = ppo.Buffer(L.bdesc, DEV)
    L.buffer = buf
    for t in range(w.T):
        L.act_into_buffer(t, dev["depth"][t], dev["proprio"][t], dev["eps"][t])
        ppo.ppo_buffer_write_outcome(buf, t, dev["reward"][t], dev["done"][t])
    assert ppo.ppo_poll_status() == 0
    used = orc.round_weights(md, theta)
    _, V_o, _ = orc.encoder_fwd(md, used, roll["depth"].reshape(w.M, w.H, w.W), roll["proprio"].reshape(w.M, w.P), True)
    assert torch.equal(buf.field(ppo.FIELD_DEPTH), dev["depth"])
    assert torch.equal(buf.field(ppo.FIELD_PROPRIO), dev["proprio"])
    assert torch.equal(buf.field(ppo.FIELD_REWARD), dev["reward"])
    assert torch.equal(buf.field(ppo.FIELD_DONE), dev["done"])
    assert rel_l2(buf.field(ppo.FIELD_ACTION).cpu().numpy(), action) <= ENC_TOL
    assert np.abs(buf.field(ppo.FIELD_LOGP).cpu().numpy() - logp).max() <= 1e-4
    assert rel_l2(buf.field(ppo.FIELD_VALUE).cpu().numpy().reshape(-1), V_o) <= ENC_TOL
    # the model and the buffer must agree on the observation's shape
    other = ppo.Buffer(ppo.buffer_desc(w.N, w.T, w.H + 2, w.W, w.P, w.A), DEV)
    assert ppo.lib().ppo_policy_act(L.model.handle, other.handle, 0, ppo._ptr(dev["eps"][0]), ppo._stream()) == 2
    assert ppo.lib().ppo_policy_act(L.model.handle, buf.handle, w.T, ppo._ptr(dev["eps"][0]), ppo._stream()) == 1


def test_a_device_side_wait_that_runs_out_reports_timeout_and_leaves_the_device_usable():
    gave_up = torch.zeros(1, dtype=torch.int32, device=DEV)
    ppo.ppo_selftest_wait_timeout(2_000_000, gave_up)   # ~1 ms
    assert ppo.ppo_poll_status() == 6                   # PPO_ERR_TIMEOUT, cleared by the poll
    assert gave_up.item() == 64
    assert ppo.ppo_poll_status() == 0
    # the context is intact: a real kernel of the library runs and checks out afterwards
    w = SHAPES["tiny"]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, 16)
    L.compute_gae(dev["last_value"])
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 0, 0, 0, w.minibatches, L.mb)
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, w.M // w.minibatches, L.mean, L.value)
    assert ppo.ppo_poll_status() == 0 and bool(torch.isfinite(L.mean).all())


def test_policy_act_matches_oracle():
    w = SHAPES["cfg1_twin"]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, 16, jitter=False)
    a, lp, val = L.act(dev["depth"][0], dev["proprio"][0], dev["eps"][0])
    assert rel_l2(a.cpu().numpy(), action[0]) <= ENC_TOL
    assert np.abs(lp.cpu().numpy() - logp[0]).max() <= 1e-4  # log-prob depends on eps and log-sigma only
    assert ppo.ppo_poll_status() == 0


def test_forward_writes_the_relu_gate_bits_of_its_activations():
    """The one-bit gates the backward pass reads must say exactly act > 0, whether the forward kernels wrote them
    or ppo_model_sync_masks recomputed them."""
    w = SHAPES["cfg2_twin"]
    B = w.M // w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, B)
    L.compute_gae(dev["last_value"])
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 0, 0, 0, w.minibatches, L.mb)
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, B, L.mean, L.value)
    Ho, Wo = orc.conv_shapes(md)
    checked = 0
    for l, (h, w_, c) in enumerate(zip(Ho, Wo, md.conv_c), start=1):
        if l == len(md.conv_c) or c % 32 != 0:
            continue
        n = B * h * w_ * c
        act = L.model.activation(0, l)[:n].float().cpu().numpy().reshape(-1, 32)
        want = (act > 0).astype(np.uint64)
        pos = np.array([(c >> 1) + 16 * (c & 1) for c in range(32)], dtype=np.uint64)  # bit of channel c in its word
        want_words = (want << pos).sum(1).astype(np.uint32)
        got = L.model.activation(2, l)[:n // 32].cpu().numpy().view(np.uint32)
        assert np.array_equal(got, want_words), f"layer {l}: forward-written gates"
        L.model.activation(2, l)[:n // 32].zero_()
        ppo.ppo_model_sync_masks(L.model, B)
        got = L.model.activation(2, l)[:n // 32].cpu().numpy().view(np.uint32)
        assert np.array_equal(got, want_words), f"layer {l}: recomputed gates"
        checked += 1
    assert checked >= 2 and ppo.ppo_poll_status() == 0


def test_backward_on_a_caller_stream_orders_like_one_stream():
    """The backward pass forks a second stream for its weight-gradient leaves and joins it before returning: run on a
    caller's stream (not the default one), twice in a row, it must give the gradients of the default-stream run, and
    work enqueued behind it on the caller's stream (the copy below) must see all of them."""
    w = SHAPES["cfg2_twin"]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, 8)
    h = L.hyper
    K = w.minibatches
    B = w.M // K
    L.compute_gae(dev["last_value"])
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 5, 0, 0, K, L.mb)

    def one_pass(out):
        ppo.ppo_model_zero_grad(L.model)
        L.loss.zero_()
        for r0 in range(0, B, L.microbatch):
            rows = min(L.microbatch, B - r0)
            ppo.ppo_encoder_fwd(L.model, L.mb, r0, rows, L.mean, L.value)
            ppo.ppo_loss_fwd_bwd(L.model, L.mb, r0, rows, B, L.mean, L.value, h.clip, h.vf_coef, h.ent_coef, L.loss,
                                 L.dmean, L.dvalue)
            ppo.ppo_encoder_bwd(L.model, L.mb, r0, rows, L.dmean, L.dvalue, True)
        out.copy_(L.model.grad, non_blocking=True)  # same stream: ordered after the join

    ref = torch.empty_like(L.model.grad)
    one_pass(ref)
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    got = [torch.empty_like(ref), torch.empty_like(ref)]
    with torch.cuda.stream(s):
        one_pass(got[0])
        one_pass(got[1])
    s.synchronize()
    assert ppo.ppo_poll_status() == 0
    r = ref.cpu().numpy()
    assert np.abs(r).max() > 0
    for g in got:  # every reduction adds its partial sums in a fixed order: the same bits on any stream
        assert np.array_equal(g.cpu().numpy(), r)


def test_gradients_are_bit_identical_run_to_run():
    """Every reduction over rows, pixels or splits (weight gradients of all layers, bias gradients, the loss terms)
    adds its partial results in a fixed order: the same minibatch processed twice gives the same bits, also when it
    is accumulated over micro-batches."""
    w = SHAPES["cfg2_twin"]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, 3)
    h = L.hyper
    K = w.minibatches
    B = w.M // K
    L.compute_gae(dev["last_value"])
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 5, 0, 0, K, L.mb)
    runs = []
    for _ in range(3):
        ppo.ppo_model_zero_grad(L.model)
        L.loss.zero_()
        for r0 in range(0, B, L.microbatch):
            rows = min(L.microbatch, B - r0)
            ppo.ppo_encoder_fwd(L.model, L.mb, r0, rows, L.mean, L.value)
            ppo.ppo_loss_fwd_bwd(L.model, L.mb, r0, rows, B, L.mean, L.value, h.clip, h.vf_coef, h.ent_coef, L.loss,
                                 L.dmean, L.dvalue)
            ppo.ppo_encoder_bwd(L.model, L.mb, r0, rows, L.dmean, L.dvalue, True)
        runs.append((L.model.grad.clone(), L.loss.clone()))
    assert ppo.ppo_poll_status() == 0
    assert float(runs[0][0].abs().max()) > 0
    for g, l in runs[1:]:
        assert torch.equal(g, runs[0][0]) and torch.equal(l, runs[0][1])
