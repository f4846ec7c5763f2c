"""GPU parity of the recurrent trunk (Section III-C: the joined depth / proprioception feature goes through stacked LSTM
layers before the fully connected layers) against the oracle: the sequence gather, the forward over time-major sequence
minibatches with done-resets, back-propagation through time on the oracle's saved state, and whole minibatch steps."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth
from paper_2509_16434_b200.learner import Learner
from helpers import oracle_model, rel_l2
from test_gpu_learner import ADAM_TOL, ENC_TOL, LOSS_TOL, _check_grads, _upload_oracle_activations

pytestmark = pytest.mark.gpu
DEV = "cuda"

REC = {
    # pooled CNN, one layer; embedded + normalised CNN, two layers; sequences long enough to carry state over resets
    "rec_pool": synth.Workload("rec_pool", 8, 6, 16, 24, (16, 32), (3, 3), (48,), 1, 2, P=32, A=3, n_lstm=1, lstm_h=64),
    "rec_embed": synth.Workload("rec_embed", 12, 5, 16, 24, (16, 32), (3, 3), (40, 24), 1, 2, P=32, A=4, norm=True,
                                embed=32, n_lstm=2, lstm_h=128),
    # the paper's policy (CNN, embedding, 2 x LSTM(1024), fully connected [512, 512, 256]) on few envs
    "paper_twin": synth.WORKLOADS["paper_policy"].scaled(8, T=3, minibatches=2),
    # the same at the paper's horizon of 16 steps: 256-row sequence minibatches (two row tiles in the all-step GEMMs)
    "paper_h16": synth.WORKLOADS["paper_policy"].scaled(32, T=16, minibatches=2),
}


def _states(w, Be, seed, zero=False):
    g = np.random.default_rng(seed + 31)
    shape = (w.n_lstm, Be, w.lstm_h)
    if zero:
        return np.zeros(shape, np.float32), np.zeros(shape, np.float32)
    return (0.5 * g.standard_normal(shape)).astype(np.float32), (0.5 * g.standard_normal(shape)).astype(np.float32)


def _setup(w, microbatch, seed=0, theta_scale_head=20.0):
    """Learner with seeded parameters; the buffer holds a rollout whose actions the oracle's recurrent policy drew."""
    md = oracle_model(w)
    lay = orc.param_layout(md)
    theta = synth.init_params(lay.total, lay.offsets, lay.shapes, seed)
    hw = len(lay.offsets) - 3
    theta[lay.offsets[hw]:lay.offsets[hw] + lay.sizes[hw]] *= theta_scale_head
    g = np.random.default_rng(seed + 7)
    for off, sz, shp in zip(lay.offsets, lay.sizes, lay.shapes):
        if len(shp) == 1:
            theta[off:off + sz] = (0.05 * g.standard_normal(sz)).astype(np.float32)
    for i in synth.param_shapes(w)[1]:
        theta[lay.offsets[i]:lay.offsets[i] + lay.sizes[i]] += 1.0
    roll = synth.rollout_numpy(w, seed)
    roll["done"][1, ::3] = 1  # some episodes end inside every sequence
    h0, c0 = _states(w, w.N, seed, zero=True)
    mu, V, _, _ = orc.encoder_fwd_seq(md, orc.round_weights(md, theta), roll["depth"], roll["proprio"], roll["done"],
                                      h0, c0, True)
    ls = np.asarray(theta, np.float64)[lay.offsets[-1]:lay.offsets[-1] + md.A]
    action, logp = orc.sample_action(mu, ls, roll["eps"].reshape(w.T * w.N, md.A))
    action = action.astype(np.float32).reshape(w.T, w.N, md.A)
    logp = (logp.astype(np.float32).reshape(w.T, w.N) + roll["logp_jitter"]).astype(np.float32)
    L = Learner(w, microbatch, DEV, with_index=True)
    L.model.load(theta)
    dev = {k: torch.as_tensor(v).to(DEV) for k, v in roll.items()}
    L.write_rollout(dev, torch.as_tensor(action).to(DEV), torch.as_tensor(logp).to(DEV))
    return L, md, lay, theta, roll, action, logp, dev


def _oracle_sequences(w, roll, action, logp, hyper, seed, epoch, j, groups):
    """Rows of sequence group j of `groups` (time-major), from the oracle's permutation of the envs."""
    adv, ret = orc.gae(roll["reward"], roll["value"], roll["done"], roll["last_value"], np.float32(hyper.gamma),
                       np.float32(hyper.lam))
    adv, _, _ = orc.adv_normalize(adv)
    per = w.N // groups
    envs = np.asarray(orc.perm(seed, epoch, w.N, j * per, per), dtype=np.int64)
    f = {"depth": roll["depth"][:, envs], "proprio": roll["proprio"][:, envs], "done": roll["done"][:, envs],
         "action": action[:, envs], "logp": logp[:, envs], "adv": adv.astype(np.float32).reshape(w.T, w.N)[:, envs],
         "ret": ret.astype(np.float32).reshape(w.T, w.N)[:, envs], "value": roll["value"][:, envs]}
    return envs, {k: np.ascontiguousarray(v) for k, v in f.items()}


def _gather_group(L, w, seed, epoch, j, groups):
    ppo.ppo_shuffle_gather_sequences(L.buffer, seed, epoch, j, groups, L.mb, L.seq_done)


@pytest.mark.parametrize("name", ["rec_pool", "rec_embed"])
def test_sequence_gather_is_bit_exact(name):
    w = REC[name]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, (w.N // w.minibatches) * w.T)
    L.compute_gae(dev["last_value"])
    Be, K = L.seq_envs, w.N // L.seq_envs
    adv_gpu = L.buffer.field(ppo.FIELD_ADV).cpu().numpy().reshape(w.T, w.N)
    seen = []
    for j in range(K):
        _gather_group(L, w, 3, 1, j, K)
        envs, f = _oracle_sequences(w, roll, action, logp, L.hyper, 3, 1, j, K)
        seen += list(envs)
        R = w.T * Be
        assert np.array_equal(L.mb.depth[:R].cpu().numpy().reshape(w.T, Be, w.H, w.W), f["depth"])
        assert np.array_equal(L.mb.proprio[:R].cpu().numpy().reshape(w.T, Be, w.P), f["proprio"])
        assert np.array_equal(L.mb.action[:R].cpu().numpy().reshape(w.T, Be, w.A), f["action"])
        assert np.array_equal(L.mb.logp_old[:R].cpu().numpy().reshape(w.T, Be), f["logp"])
        assert np.array_equal(L.mb.value_old[:R].cpu().numpy().reshape(w.T, Be), f["value"])
        assert np.array_equal(L.seq_done.cpu().numpy(), f["done"])
        assert np.array_equal(L.mb.adv[:R].cpu().numpy().reshape(w.T, Be), adv_gpu[:, envs])
        want = (np.arange(w.T)[:, None] * w.N + envs[None, :]).reshape(-1)
        assert np.array_equal(L.mb.index[:R].cpu().numpy(), want)
    assert sorted(seen) == list(range(w.N))  # every env in exactly one group


def _forward(L, w, f, h0, c0):
    Be = f["done"].shape[1]
    L.h_init.copy_(torch.as_tensor(h0))
    L.c_init.copy_(torch.as_tensor(c0))
    ppo.ppo_model_set_sequence(L.model, w.T, Be, L.seq_done, L.h_init, L.c_init)
    ppo.ppo_encoder_fwd(L.model, L.mb, 0, w.T * Be, L.mean, L.value)


@pytest.mark.parametrize("name,zero_state", [("rec_pool", False), ("rec_embed", False), ("rec_embed", True),
                                             ("paper_twin", False), ("paper_h16", False)])
def test_forward_through_time_matches_oracle(name, zero_state):
    w = REC[name]
    K = w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, (w.N // K) * w.T)
    L.compute_gae(dev["last_value"])
    Be, R = L.seq_envs, L.seq_envs * w.T
    assert Be == w.N // K
    _gather_group(L, w, 9, 0, 1, K)
    envs, f = _oracle_sequences(w, roll, action, logp, L.hyper, 9, 0, 1, K)
    h0, c0 = _states(w, Be, 1, zero_state)
    _forward(L, w, f, h0, c0)
    assert ppo.ppo_poll_status() == 0
    mu, V = L.mean[:R].cpu().numpy(), L.value[:R].cpu().numpy()
    used = orc.round_weights(md, theta)
    for act_bf16 in (True, False):
        mu_o, V_o, acts, lrec = orc.encoder_fwd_seq(md, used, f["depth"], f["proprio"], f["done"], h0, c0, act_bf16)
        print(f"[{name}] forward vs oracle ({'bf16' if act_bf16 else 'fp64'} activations): mu {rel_l2(mu, mu_o):.3e}, "
              f"V {rel_l2(V, V_o):.3e}")
        assert rel_l2(mu, mu_o) <= ENC_TOL and rel_l2(V, V_o) <= ENC_TOL
    # the state kept for the backward pass, per layer: gates, c, h and the state each step started from
    _, _, _, lrec = orc.encoder_fwd_seq(md, used, f["depth"], f["proprio"], f["done"], h0, c0, True)
    H = w.lstm_h
    for l in range(w.n_lstm):
        rec = lrec[:, l * 8 * H:(l + 1) * 8 * H]
        gates = L.model.activation(7, l)[:R * 4 * H].cpu().numpy().reshape(R, 4 * H)
        cc = L.model.activation(6, l).cpu().numpy()
        c, cprev = cc[:R * H].reshape(R, H), cc[len(cc) // 2:len(cc) // 2 + R * H].reshape(R, H)
        h = L.model.activation(5, l)[:R * H].float().cpu().numpy().reshape(R, H)
        hprev = L.model.activation(8, l)[:R * H].float().cpu().numpy().reshape(R, H)
        for got, want, what in ((gates, rec[:, :4 * H], "gates"), (c, rec[:, 4 * H:5 * H], "c"),
                                (h, rec[:, 5 * H:6 * H], "h"), (hprev, rec[:, 6 * H:7 * H], "h_prev"),
                                (cprev, rec[:, 7 * H:8 * H], "c_prev")):
            assert rel_l2(got, want) <= ENC_TOL, (l, what, rel_l2(got, want))
    # the step after an episode end starts from zeros, whatever the state was
    t_reset = 2
    rows = np.nonzero(f["done"][t_reset - 1])[0]
    assert len(rows) > 0
    hp = L.model.activation(8, 0)[:R * H].float().cpu().numpy().reshape(w.T, Be, H)
    assert np.all(hp[t_reset, rows] == 0.0)


def _upload_oracle_state(L, w, lrec, R):
    H = w.lstm_h
    for l in range(w.n_lstm):
        rec = lrec[:, l * 8 * H:(l + 1) * 8 * H]
        t = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a).reshape(-1)).to(dt)
        L.model.activation(7, l)[:R * 4 * H].copy_(t(rec[:, :4 * H], torch.float32))
        cc = L.model.activation(6, l)
        cc[:R * H].copy_(t(rec[:, 4 * H:5 * H], torch.float32))
        cc[len(cc) // 2:len(cc) // 2 + R * H].copy_(t(rec[:, 7 * H:8 * H], torch.float32))
        L.model.activation(5, l)[:R * H].copy_(t(rec[:, 5 * H:6 * H], torch.bfloat16))
        L.model.activation(8, l)[:R * H].copy_(t(rec[:, 6 * H:7 * H], torch.bfloat16))


def _oracle_step(md, theta, f, h0, c0, h):
    return orc.total_loss_and_grad_seq(md, theta, f["depth"], f["proprio"], f["done"], h0, c0,
                                       f["action"].reshape(-1, md.A), f["logp"].reshape(-1), f["adv"].reshape(-1),
                                       f["ret"].reshape(-1), np.float32(h.clip), np.float32(h.vf_coef),
                                       np.float32(h.ent_coef), act_bf16=True)


@pytest.mark.parametrize("name", ["rec_pool", "rec_embed", "paper_twin", "paper_h16"])
def test_backward_through_time_matches_oracle_on_identical_state(name):
    """Both sides start from the oracle's saved activations, recurrent state, mean and value."""
    w = REC[name]
    K = w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, (w.N // K) * w.T)
    h = L.hyper
    L.compute_gae(dev["last_value"])
    Be, R = L.seq_envs, L.seq_envs * w.T
    _gather_group(L, w, 5, 0, 0, K)
    envs, f = _oracle_sequences(w, roll, action, logp, h, 5, 0, 0, K)
    h0, c0 = _states(w, Be, 2)
    _, out_o, grad_o, mu_o, V_o = _oracle_step(md, theta, f, h0, c0, h)
    _, _, acts, lrec = orc.encoder_fwd_seq(md, orc.round_weights(md, theta), f["depth"], f["proprio"], f["done"], h0,
                                           c0, True)
    ppo.ppo_model_zero_grad(L.model)
    L.loss.zero_()
    _forward(L, w, f, h0, c0)
    _upload_oracle_activations(L, md, acts, R)
    _upload_oracle_state(L, w, lrec, R)
    ppo.ppo_model_sync_masks(L.model, R)
    L.mean[:R].copy_(torch.as_tensor(mu_o, dtype=torch.float32))
    L.value[:R].copy_(torch.as_tensor(V_o, dtype=torch.float32))
    ppo.ppo_loss_fwd_bwd(L.model, L.mb, 0, R, R, L.mean, L.value, h.clip, h.vf_coef, h.ent_coef, L.loss, L.dmean,
                         L.dvalue)
    ppo.ppo_encoder_bwd(L.model, L.mb, 0, R, L.dmean, L.dvalue, True)
    assert ppo.ppo_poll_status() == 0
    got = L.model.grad.cpu().numpy()
    errs = [rel_l2(got[o:o + s], grad_o[o:o + s]) for o, s in zip(lay.offsets, lay.sizes)]
    print(f"[{name}] teacher-forced BPTT, rel L2 per tensor: max {max(errs):.3e} (tensor {int(np.argmax(errs))}), "
          f"total {rel_l2(got, grad_o):.3e}")
    _check_grads(lay, got, grad_o)


@pytest.mark.parametrize("name,microbatch", [("rec_pool", 24), ("rec_embed", 10), ("rec_embed", 30)])
def test_whole_recurrent_step_parameters_match_oracle(name, microbatch):
    """Minibatch steps through the Learner (zero initial state, micro-batches of whole sequences) against the oracle
    taking the same sequences in one piece."""
    w = REC[name]
    K = w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, microbatch)
    h = L.hyper
    L.compute_gae(dev["last_value"])
    Be = w.N // K
    assert Be % L.seq_envs == 0 and L.seq_envs * w.T <= max(microbatch, w.T)
    h0, c0 = _states(w, Be, 0, zero=True)
    th = theta.astype(np.float64)
    m, v = np.zeros_like(th), np.zeros_like(th)
    for k in range(K):
        L.minibatch_step(11, 0, k)
        envs, f = _oracle_sequences(w, roll, action, logp, h, 11, 0, k, K)
        _, out_o, grad, _, _ = _oracle_step(md, th.astype(np.float32), f, h0, c0, h)
        orc.adam(th, m, v, grad, np.float32(h.lr), np.float32(h.beta1), np.float32(h.beta2), np.float32(h.eps), k + 1)
        got = L.model.master.cpu().numpy()
        print(f"[{name}] step {k}: parameters rel L2 {rel_l2(got, th):.3e}")
        assert rel_l2(got, th) <= ADAM_TOL * (k + 1), (k, rel_l2(got, th))
    out = L.loss.cpu().numpy()
    assert abs(out[2] - out_o[2]) <= LOSS_TOL * abs(out_o[2])
    assert ppo.ppo_poll_status() == 0


def test_recurrent_model_rejects_calls_without_a_sequence():
    w = REC["rec_pool"]
    L, md, lay, theta, roll, action, logp, dev = _setup(w, (w.N // w.minibatches) * w.T)
    L.compute_gae(dev["last_value"])
    _gather_group(L, w, 1, 0, 0, w.minibatches)
    with pytest.raises(ppo.PpoError):  # no sequence announced
        ppo.ppo_encoder_fwd(L.model, L.mb, 0, L.microbatch, L.mean, L.value)
    ppo.ppo_model_set_sequence(L.model, w.T, L.seq_envs, L.seq_done, L.h_init, L.c_init)
    with pytest.raises(ppo.PpoError):  # rows that are not T * Be
        ppo.ppo_encoder_fwd(L.model, L.mb, 0, L.microbatch - 1, L.mean, L.value)
    eps = torch.zeros((w.N, w.A), device=DEV)
    with pytest.raises(ppo.PpoError):  # the one-step rollout call has no recurrent state to carry
        ppo.ppo_policy_act(L.model, L.buffer, 0, eps)


def test_state_after_a_sequence_matches_oracle_and_chains():
    """ppo_model_read_state: h and c of the last step (zero where that step was done) against the oracle's record, and
    a sequence run in one piece against the same sequence run step by step through the returned state."""
    w = REC["rec_embed"]
    K = w.minibatches
    L, md, lay, theta, roll, action, logp, dev = _setup(w, (w.N // K) * w.T)
    L.compute_gae(dev["last_value"])
    Be, R, H = L.seq_envs, L.seq_envs * w.T, w.lstm_h
    _gather_group(L, w, 4, 0, 0, K)
    envs, f = _oracle_sequences(w, roll, action, logp, L.hyper, 4, 0, 0, K)
    L.seq_done[w.T - 1, ::2] = 1  # some envs end their episode on the last step
    f["done"][w.T - 1, ::2] = 1
    h0, c0 = _states(w, Be, 3)
    _forward(L, w, f, h0, c0)
    h_out, c_out = torch.empty_like(L.h_init), torch.empty_like(L.c_init)
    ppo.ppo_model_read_state(L.model, h_out, c_out)
    mu_all = L.mean[:R].clone()
    _, _, _, lrec = orc.encoder_fwd_seq(md, orc.round_weights(md, theta), f["depth"], f["proprio"], f["done"], h0, c0, True)
    last = lrec[(w.T - 1) * Be:]
    keep = (f["done"][w.T - 1] == 0)[:, None]
    for l in range(w.n_lstm):
        h_o, c_o = last[:, l * 8 * H + 5 * H:l * 8 * H + 6 * H] * keep, last[:, l * 8 * H + 4 * H:l * 8 * H + 5 * H] * keep
        assert rel_l2(h_out[l].cpu().numpy(), h_o) <= ENC_TOL and rel_l2(c_out[l].cpu().numpy(), c_o) <= ENC_TOL
        assert np.all(h_out[l].cpu().numpy()[::2] == 0) and np.all(c_out[l].cpu().numpy()[::2] == 0)
    # step by step: T one-step sequences, each started from the state the previous one returned
    hs, cs = torch.as_tensor(h0).to(DEV), torch.as_tensor(c0).to(DEV)
    one = ppo.Minibatch(L.mb.depth.data_ptr(), L.mb.proprio.data_ptr(), None, None, None, None, None, None, R)
    for t in range(w.T):
        ppo.ppo_model_set_sequence(L.model, 1, Be, L.seq_done[t], hs, cs)
        ppo.ppo_encoder_fwd(L.model, one, t * Be, Be, L.mean, L.value)
        assert torch.equal(L.mean[:Be], mu_all[t * Be:(t + 1) * Be]), t
        hs, cs = torch.empty_like(hs), torch.empty_like(cs)
        ppo.ppo_model_read_state(L.model, hs, cs)
    assert torch.equal(hs, h_out) and torch.equal(cs, c_out)
    assert ppo.ppo_poll_status() == 0
