"""GPU parity of the layer-normalised depth CNN with the flatten -> fully connected embedding (Section III-C) against
the oracle: forward outputs and what the forward saves for the backward pass, the backward operator on the oracle's
activations, and whole minibatch steps."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth
from helpers import rel_l2
from test_gpu_learner import (ADAM_TOL, ENC_TOL, LOSS_TOL, _check_grads, _oracle_minibatch, _setup,
                              _upload_oracle_activations)

pytestmark = pytest.mark.gpu
DEV = "cuda"

LN = {
    # small nets that still cross tile boundaries: first layer of 16 and of 32 channels, pooled and embedded variants
    "ln_small": synth.Workload("ln_small", 8, 4, 16, 24, (16, 32), (3, 3), (32,), 1, 2, P=8, A=3, norm=True, embed=32),
    "ln_pool": synth.Workload("ln_pool", 6, 4, 18, 22, (32, 64, 64), (5, 3, 3), (40,), 1, 2, P=16, A=5, norm=True),
    "embed_only": synth.Workload("embed_only", 8, 4, 16, 24, (16, 32), (3, 3), (32,), 1, 2, P=8, A=3, embed=64),
    # the paper's CNN on 160x120 frames with few envs
    "paper_twin": synth.WORKLOADS["paper_cnn"].scaled(8, T=2, minibatches=2),
    "paper_64": synth.WORKLOADS["paper_cnn"].scaled(32, T=4, minibatches=2),
}


@pytest.mark.parametrize("name", ["ln_small", "ln_pool", "embed_only", "paper_twin"])
def test_forward_and_saved_statistics_match_oracle(name):
    w = LN[name]
    B = w.M // w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, B, theta_scale_head=20.0)
    L.compute_gae(dev["last_value"])
    idx = orc.perm(9, 0, w.M, 0, B)
    f = orc.gather({"depth": roll["depth"], "proprio": roll["proprio"]}, idx, w.N)
    used = orc.round_weights(md, theta)
    ppo.ppo_shuffle_gather_minibatch(L.buffer, 9, 0, 0, w.minibatches, L.mb)
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, B, L.mean, L.value)
    assert ppo.ppo_poll_status() == 0
    mu, V = L.mean[:B].cpu().numpy(), L.value[:B].cpu().numpy()
    for act_bf16 in (True, False):
        mu_o, V_o, acts = orc.encoder_fwd(md, used, f["depth"], f["proprio"], act_bf16)
        print(f"[{name}] forward vs oracle ({'bf16' if act_bf16 else 'fp64'} activations): mu {rel_l2(mu, mu_o):.3e}, "
              f"V {rel_l2(V, V_o):.3e}")
        assert rel_l2(mu, mu_o) <= ENC_TOL and rel_l2(V, V_o) <= ENC_TOL
    if not md.norm:
        return
    # what the forward keeps for the backward pass: xhat and rstd of every layer (bf16-storing oracle)
    _, _, acts = orc.encoder_fwd(md, used, f["depth"], f["proprio"], True)
    Ho, Wo = orc.conv_shapes(md)
    off = md.H * md.W + sum(h * w_ * c for h, w_, c in zip(Ho, Wo, md.conv_c)) + (md.embed or md.conv_c[-1]) + md.P + sum(md.fc)
    for l, (h, w_, c) in enumerate(zip(Ho, Wo, md.conv_c), start=1):
        n = h * w_ * c
        xh = L.model.activation(3, l)[:B * n].float().cpu().numpy()
        rs = L.model.activation(4, l)[:B * h * w_].cpu().numpy()
        xh_o, rs_o = acts[:, off:off + n].reshape(-1), acts[:, off + n:off + n + h * w_].reshape(-1)
        off += n + h * w_
        assert rel_l2(xh, xh_o) <= ENC_TOL, (l, rel_l2(xh, xh_o))
        assert rel_l2(rs, rs_o) <= ENC_TOL, (l, rel_l2(rs, rs_o))


@pytest.mark.parametrize("name", ["ln_small", "ln_pool", "embed_only", "paper_twin", "paper_64"])
def test_backward_matches_oracle_on_identical_activations(name):
    """Both sides start from the oracle's saved activations, normalised values, statistics, mean and value."""
    w = LN[name]
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
    got = L.model.grad.cpu().numpy()
    errs = [rel_l2(got[o:o + s], grad_o[o:o + s]) for o, s in zip(lay.offsets, lay.sizes)]
    print(f"[{name}] teacher-forced backward, rel L2 per tensor: max {max(errs):.3e} (tensor {int(np.argmax(errs))}), "
          f"total {rel_l2(got, grad_o):.3e}")
    _check_grads(lay, got, grad_o)


@pytest.mark.parametrize("name,microbatch", [("ln_small", 16), ("ln_small", 5), ("paper_twin", 8)])
def test_whole_learner_step_parameters_match_oracle(name, microbatch):
    w = LN[name]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, microbatch, theta_scale_head=20.0)
    h = L.hyper
    L.compute_gae(dev["last_value"])
    th = theta.astype(np.float64)
    m, v = np.zeros_like(th), np.zeros_like(th)
    for k in range(w.minibatches):
        L.minibatch_step(11, 0, k)
        _, out_o, grad, _, _ = _oracle_minibatch(md, lay, th.astype(np.float32), roll, action, logp, w, h, 11, 0, k,
                                                 w.minibatches)
        orc.adam(th, m, v, grad, np.float32(h.lr), np.float32(h.beta1), np.float32(h.beta2), np.float32(h.eps), k + 1)
        got = L.model.master.cpu().numpy()
        assert rel_l2(got, th) <= ADAM_TOL * (k + 1), (k, rel_l2(got, th))
    out = L.loss.cpu().numpy()
    assert abs(out[2] - out_o[2]) <= LOSS_TOL * abs(out_o[2])
    assert ppo.ppo_poll_status() == 0
