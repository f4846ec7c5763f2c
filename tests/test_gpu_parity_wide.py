"""GPU parity at the shapes and in the forms the smaller tests do not reach.

 - the backward operator against the oracle at the launch shapes of a timed micro-batch (1024 rows of the cfg2
   network: many pixel tiles per CTA, split-K weight gradients over hundreds of tiles, multi-tile FC GEMMs; 64 rows
   of the cfg4 network: the 5x5 first layer and the five-layer chain);
 - the forward against the oracle that does NOT round its activations between layers (the 2e-2 budget then covers
   the kernel's bf16 storage as well as its fp32 sums);
 - an audit of what separates end-to-end gradients from the 2e-2 of the backward operator: the ReLU gates that
   differ between the two forwards are counted, and the oracle's backward run from the GPU's own saved
   activations must agree with the GPU's backward to 2e-2;
 - the loss scalars end to end;
 - whole learner steps of the cfg3 and cfg4 twins with their epochs x minibatches (epochs > 0 included).

Measured values are printed (run with -s to see them).
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth
from helpers import oracle_model, rel_l2
from test_gpu_learner import (ADAM_TOL, ENC_TOL, LOSS_TOL, SHAPES, _check_grads, _oracle_minibatch, _setup,
                              _upload_oracle_activations)

pytestmark = pytest.mark.gpu
DEV = "cuda"

WIDE = {
    # one minibatch = one micro-batch of 1024 rows of the cfg2 network (the timed path runs 4096)
    "cfg2_1024": synth.WORKLOADS["cfg2"].scaled(128, T=16, minibatches=2),
    # 64 rows of the cfg4 network: 5x5 first layer on 320x240 frames, five conv layers
    "cfg4_64": synth.WORKLOADS["cfg4"].scaled(32, T=4, minibatches=2),
}


def _download_activations(L, md, B, depth):
    """The activations the GPU forward saved, in the oracle's layout [depth | conv 1..L | h_0..h_F], as float64."""
    Ho, Wo = orc.conv_shapes(md)
    cols = [np.asarray(depth, np.float64).reshape(B, -1)]
    for l, (h, w_, c) in enumerate(zip(Ho, Wo, md.conv_c), start=1):
        n = h * w_ * c
        cols.append(L.model.activation(0, l)[:B * n].float().cpu().numpy().astype(np.float64).reshape(B, n))
    widths = [md.conv_c[-1] + md.P] + list(md.fc)
    for l, n in enumerate(widths):
        cols.append(L.model.activation(1, l)[:B * n].float().cpu().numpy().astype(np.float64).reshape(B, n))
    acts = np.ascontiguousarray(np.concatenate(cols, axis=1))
    assert acts.shape[1] == orc.act_stride(md)
    return acts


@pytest.mark.parametrize("name", ["cfg2_1024", "cfg4_64"])
def test_backward_matches_oracle_at_timed_launch_shapes(name):
    """Teacher-forced (both sides start from the oracle's saved activations, mean and value), 2e-2 per tensor."""
    w = WIDE[name]
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
    mu, V = L.mean[:B].cpu().numpy(), L.value[:B].cpu().numpy()
    assert rel_l2(mu, mu_o) <= ENC_TOL and rel_l2(V, V_o) <= ENC_TOL
    _upload_oracle_activations(L, md, acts, B)
    ppo.ppo_model_sync_masks(L.model, B)
    L.mean[:B].copy_(torch.as_tensor(mu_o, dtype=torch.float32))
    L.value[:B].copy_(torch.as_tensor(V_o, dtype=torch.float32))
    ppo.ppo_loss_fwd_bwd(L.model, L.mb, 0, B, B, L.mean, L.value, h.clip, h.vf_coef, h.ent_coef, L.loss, L.dmean,
                         L.dvalue)
    ppo.ppo_encoder_bwd(L.model, L.mb, 0, B, L.dmean, L.dvalue, True)
    assert ppo.ppo_poll_status() == 0
    got = L.model.grad.cpu().numpy()
    errs = [rel_l2(got[o:o + s], grad_o[o:o + s]) for o, s in zip(lay.offsets, lay.sizes)]
    print(f"[{name}] teacher-forced backward, rel L2 per tensor: max {max(errs):.3e}, total {rel_l2(got, grad_o):.3e}")
    _check_grads(lay, got, grad_o)


@pytest.mark.parametrize("name", ["tiny", "odd", "cfg1_twin", "cfg2_twin", "cfg4_twin", "cfg2_1024"])
def test_forward_matches_the_oracle_that_keeps_its_activations_unrounded(name):
    """mu and V against the oracle with fp64 activations between layers (only the weights are bf16 values there):
    the 2e-2 budget bounds the kernel's bf16 storage of activations together with its fp32 accumulation."""
    w = SHAPES[name] if name in SHAPES else WIDE[name]
    B = w.M // w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, B, theta_scale_head=20.0)
    L.compute_gae(dev["last_value"])
    K = w.minibatches
    idx = orc.perm(9, 0, w.M, 0, B)
    f = orc.gather({"depth": roll["depth"], "proprio": roll["proprio"]}, idx, w.N)
    mu_o, V_o, _ = orc.encoder_fwd(md, orc.round_weights(md, theta), f["depth"], f["proprio"], False)
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 9, 0, 0, K, L.mb)
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, B, L.mean, L.value)
    assert ppo.ppo_poll_status() == 0
    mu, V = L.mean[:B].cpu().numpy(), L.value[:B].cpu().numpy()
    print(f"[{name}] forward vs unrounded oracle: mu {rel_l2(mu, mu_o):.3e}, V {rel_l2(V, V_o):.3e}")
    assert rel_l2(mu, mu_o) <= ENC_TOL
    assert rel_l2(V, V_o) <= ENC_TOL


# Fraction of stored activations whose ReLU gate (act > 0) may differ between the GPU forward and the oracle's
# bf16-storing forward: a gate flips only where a pre-activation lies within the two sides' summation difference
# (fp32 vs fp64 sums of bf16 products, ~1e-7 relative to the typical pre-activation, amplified wherever an
# upstream activation rounds to a different bf16 value) of zero.  Measured: 0 to 9e-7; the bound leaves a decade.
GATE_FLIP_FRACTION = 1e-5


@pytest.mark.parametrize("name", ["cfg1_twin", "cfg2_twin", "cfg4_twin", "cfg2_1024"])
def test_end_to_end_gradient_audit(name):
    """GPU forward -> GPU loss -> GPU backward.  (1) forward outputs within 2e-2 of the oracle; (2) the gates the
    two forwards disagree on are a small counted fraction; (3) the oracle's loss gradient and backward, run from
    the GPU's own mu, V and saved activations, agree with the GPU's gradients to 2e-2 per tensor -- so the whole
    distance between end-to-end gradients and the oracle's comes from the counted gates, not from the kernels."""
    w = SHAPES[name] if name in SHAPES else WIDE[name]
    B = w.M // w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, B, theta_scale_head=20.0)
    h = L.hyper
    K = w.minibatches
    L.compute_gae(dev["last_value"])
    f, out_o, grad_o, mu_o, V_o = _oracle_minibatch(md, lay, theta, roll, action, logp, w, h, 3, 1, 0, K)
    used = orc.round_weights(md, theta)
    _, _, acts_o = orc.encoder_fwd(md, used, f["depth"], f["proprio"], True)
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 3, 1, 0, K, L.mb)
    ppo.ppo_model_zero_grad(L.model)
    L.loss.zero_()
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, B, L.mean, L.value)
    ppo.ppo_loss_fwd_bwd(L.model, L.mb, 0, B, B, L.mean, L.value, h.clip, h.vf_coef, h.ent_coef, L.loss, L.dmean,
                         L.dvalue)
    ppo.ppo_encoder_bwd(L.model, L.mb, 0, B, L.dmean, L.dvalue, True)
    assert ppo.ppo_poll_status() == 0
    mu, V = L.mean[:B].cpu().numpy(), L.value[:B].cpu().numpy()
    assert rel_l2(mu, mu_o) <= ENC_TOL and rel_l2(V, V_o) <= ENC_TOL
    # (2) gates
    acts_g = _download_activations(L, md, B, f["depth"])
    hw0 = md.H * md.W
    gates_g, gates_o = acts_g[:, hw0:] > 0, acts_o[:, hw0:] > 0
    flipped = float(np.mean(gates_g != gates_o))
    print(f"[{name}] ReLU gates that differ between the two forwards: {flipped:.3e} of {gates_o.size}")
    assert flipped <= GATE_FLIP_FRACTION
    # (3) oracle loss gradient + backward from the GPU's forward state
    ls = np.asarray(theta, np.float64)[lay.offsets[-1]:lay.offsets[-1] + md.A]
    out2, dmu2, dV2, dls2 = orc.loss(mu, V, ls, f["action"], f["logp"], f["adv"], f["ret"], np.float32(h.clip),
                                     np.float32(h.vf_coef), np.float32(h.ent_coef))
    grad2 = orc.encoder_bwd(md, used, acts_g, dmu2, dV2)
    grad2[lay.offsets[-1]:lay.offsets[-1] + md.A] += dls2
    got = L.model.grad.cpu().numpy()
    errs = [rel_l2(got[o:o + s], grad2[o:o + s]) for o, s in zip(lay.offsets, lay.sizes)]
    e2e = [rel_l2(got[o:o + s], grad_o[o:o + s]) for o, s in zip(lay.offsets, lay.sizes)]
    print(f"[{name}] gradients vs oracle backward on the GPU's activations: max per tensor {max(errs):.3e}, total "
          f"{rel_l2(got, grad2):.3e}; vs the oracle's own forward+backward: max per tensor {max(e2e):.3e} (tensor "
          f"{int(np.argmax(e2e))} of {len(e2e)}, {lay.sizes[int(np.argmax(e2e))]} elements), total "
          f"{rel_l2(got, grad_o):.3e}")
    _check_grads(lay, got, grad2)
    # end to end against the oracle's own forward and backward the counted gates show: each one removes or adds a
    # unit's whole contribution (measured: 6e-3 of the gradient at 1024 rows, 5e-2 with 4 flipped gates in 4 rows)
    assert rel_l2(got, grad_o) <= (ENC_TOL if B >= 1024 else 1e-1)
    # loss scalars end to end: value loss and entropy relative; the policy loss is a mean of signed terms near zero,
    # so its error is measured against the mean magnitude of its terms (|s| ~ |adv|)
    out = L.loss.cpu().numpy()
    s_scale = float(np.mean(np.abs(f["adv"])))
    print(f"[{name}] loss end to end: L_pi abs err / mean|adv| {abs(out[0] - out_o[0]) / s_scale:.3e}, "
          f"L_V rel {abs(out[1] - out_o[1]) / abs(out_o[1]):.3e}, H rel {abs(out[2] - out_o[2]) / abs(out_o[2]):.3e}")
    v_scale = max(abs(out_o[1]), float(np.mean(V_o ** 2 + f["ret"] ** 2)))  # magnitude of what enters (V - R)^2
    # 1e-3 from 8 rows on; in fewer rows the encoder's own error in mu and V (2e-3, inside its 2e-2) does not average out
    tol = LOSS_TOL if B >= 8 else 5 * LOSS_TOL
    assert abs(out[1] - out_o[1]) <= tol * v_scale
    assert abs(out[2] - out_o[2]) <= LOSS_TOL * abs(out_o[2])
    assert abs(out[0] - out_o[0]) <= tol * s_scale
    # and against the oracle that keeps its activations unrounded between layers
    _, out_u, _, _, _ = orc.total_loss_and_grad(md, theta, f["depth"], f["proprio"], f["action"], f["logp"], f["adv"],
                                                f["ret"], np.float32(h.clip), np.float32(h.vf_coef),
                                                np.float32(h.ent_coef), act_bf16=False)
    print(f"[{name}] loss vs the unrounded oracle: L_pi abs err / mean|adv| {abs(out[0] - out_u[0]) / s_scale:.3e}, "
          f"L_V rel {abs(out[1] - out_u[1]) / abs(out_u[1]):.3e}")
    assert abs(out[1] - out_u[1]) <= tol * v_scale
    assert abs(out[0] - out_u[0]) <= tol * s_scale


@pytest.mark.parametrize("name,twin", [("cfg3", dict(N=8, T=2)), ("cfg4", dict(N=4, T=4))])
def test_whole_step_of_the_multi_epoch_configs(name, twin):
    """GAE, then every minibatch of every epoch (cfg3: 5 x 4, cfg4: 5 x 8) on a twin with few envs: parameters
    against the oracle after every Adam step, with the oracle re-linearised at its own parameters."""
    w0 = synth.WORKLOADS[name]
    w = w0.scaled(twin["N"], T=twin["T"])
    assert w.epochs == 5 and w.M % w.minibatches == 0
    L, md, lay, theta, roll, action, logp, dev = _setup(w, max(1, w.B), theta_scale_head=20.0)
    h = L.hyper
    L.compute_gae(dev["last_value"])
    th = theta.astype(np.float64)
    m, v = np.zeros_like(th), np.zeros_like(th)
    step = 0
    worst = 0.0
    for e in range(w.epochs):
        for k in range(w.minibatches):
            L.minibatch_step(11, e, k)
            _, _, grad, _, _ = _oracle_minibatch(md, lay, th.astype(np.float32), roll, action, logp, w, h, 11, e, k,
                                                 w.minibatches)
            step += 1
            orc.adam(th, m, v, grad, np.float32(h.lr), np.float32(h.beta1), np.float32(h.beta2), np.float32(h.eps),
                     step)
            got = L.model.master.cpu().numpy()
            err = rel_l2(got, th)
            worst = max(worst, err / step)
            assert err <= ADAM_TOL * step, (e, k, err)
    print(f"[{name} twin] {step} Adam steps: worst rel L2 of the parameters per step taken {worst:.3e}")
    assert ppo.ppo_poll_status() == 0
