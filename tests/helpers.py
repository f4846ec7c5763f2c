"""Shared test utilities: error metrics and the oracle-side composition of a learner step."""
import numpy as np

from oracle import oracle as orc


def rel_l2(x, ref):
    x = np.asarray(x, np.float64).reshape(-1)
    ref = np.asarray(ref, np.float64).reshape(-1)
    d = np.linalg.norm(ref)
    return float(np.linalg.norm(x - ref) / (d if d > 0 else 1.0))


def max_abs_scaled(x, ref):
    """max |x - ref| / max(1, max |ref|): the companion of rel_l2 for arrays that cross zero."""
    x = np.asarray(x, np.float64).reshape(-1)
    ref = np.asarray(ref, np.float64).reshape(-1)
    return float(np.abs(x - ref).max() / max(1.0, np.abs(ref).max()))


def oracle_model(w):
    return orc.ModelDesc(w.H, w.W, tuple(w.conv_c), tuple(w.conv_k), tuple(w.fc), w.P, w.A, norm=w.norm, embed=w.embed,
                         n_lstm=w.n_lstm, lstm_h=w.lstm_h)


def oracle_rollout_actions(md, theta, roll):
    """Actions and old log-probs of the rollout policy (initial weights, sigma from log-sigma) for every env-step."""
    lay = orc.param_layout(md)
    used = orc.round_weights(md, theta)
    T, N = roll["reward"].shape
    depth = roll["depth"].reshape(T * N, md.H, md.W)
    proprio = roll["proprio"].reshape(T * N, md.P)
    mu, V, _ = orc.encoder_fwd(md, used, depth, proprio, True)
    ls = np.asarray(theta, np.float64)[lay.offsets[-1]:lay.offsets[-1] + md.A]
    action, logp = orc.sample_action(mu, ls, roll["eps"].reshape(T * N, md.A))
    return (action.astype(np.float32).reshape(T, N, md.A), logp.astype(np.float32).reshape(T, N))
