"""Seeded synthetic inputs for the PPO learner step.

This module holds workload shapes and random input generators only; none of the
learner's arithmetic lives here.  The frames stand in for a simulator's tiled
depth rendering at 160x120 / 320x240 with a horizon of 16 (Section III-B,
Table I): depth is uniform in [0.1, 2.0] m stored as fp16 with 10 % of the pixels
zeroed (missing returns), proprioception is 32 standard normals, rewards and old
values are standard normals, dones are Bernoulli.

Two back ends produce the same distributions: numpy (Philox, for parity-sized
cases that also feed the CPU checker) and torch on the device (for buffers of
many GB that never visit the host).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Sequence

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    N: int
    T: int
    H: int
    W: int
    conv_c: Sequence[int]
    conv_k: Sequence[int]
    fc: Sequence[int]
    epochs: int
    minibatches: int
    done_rate: float = 0.01
    P: int = 32
    A: int = 12
    gamma: float = 0.99
    lam: float = 0.95
    clip: float = 0.2
    seed: int = 0
    norm: bool = False  # layer normalisation over the channels of every conv output, before its ReLU
    embed: int = 0      # > 0: flatten -> fully connected (embed) -> ReLU instead of the global average pool
    n_lstm: int = 0     # LSTM layers between the joined feature and the fully connected layers
    lstm_h: int = 0     # their width

    @property
    def M(self) -> int:
        return self.N * self.T

    @property
    def B(self) -> int:
        return self.M // self.minibatches

    def scaled(self, N: int, **kw) -> "Workload":
        d = dict(self.__dict__)
        d.update(N=N, **kw)
        return Workload(**d)


WORKLOADS: Dict[str, Workload] = {
    "cfg1": Workload("cfg1", 256, 16, 64, 64, (16, 32, 64), (3, 3, 3), (256,), 1, 4),
    "cfg2": Workload("cfg2", 1024, 16, 120, 160, (32, 64, 128, 256), (3, 3, 3, 3), (512, 512), 1, 4),
    "cfg3": Workload("cfg3", 4096, 16, 120, 160, (32, 64, 128, 256), (3, 3, 3, 3), (512, 512), 5, 4),
    "cfg4": Workload("cfg4", 8192, 16, 240, 320, (32, 64, 128, 256, 256), (5, 3, 3, 3, 3), (512, 512), 5, 8,
                     done_rate=0.005),
    # the depth CNN of Section III-C on 160x120 frames: [16, 32, 64, 128] filters with layer normalisation and ReLU, a
    # 32-d embedding of the flattened map, joined with proprioception, fully connected [512, 512, 256]
    "paper_cnn": Workload("paper_cnn", 1024, 16, 120, 160, (16, 32, 64, 128), (3, 3, 3, 3), (512, 512, 256), 1, 4,
                          norm=True, embed=32),
    # the paper's whole policy: that CNN and embedding, two LSTM layers of 1024 units, fully connected [512, 512, 256];
    # minibatches are sequences (256 envs x 16 steps)
    "paper_policy": Workload("paper_policy", 1024, 16, 120, 160, (16, 32, 64, 128), (3, 3, 3, 3), (512, 512, 256), 1, 4,
                             norm=True, embed=32, n_lstm=2, lstm_h=1024),
    # profiling-sized twin of cfg2: same frames, network and micro-batch shapes, 1/8 of the envs
    "cfg2_prof": Workload("cfg2_prof", 128, 16, 120, 160, (32, 64, 128, 256), (3, 3, 3, 3), (512, 512), 1, 4),
    # profiling-sized twin of cfg4: same frames and network, 64 envs (minibatches of 128 rows)
    "cfg4_prof": Workload("cfg4_prof", 64, 16, 240, 320, (32, 64, 128, 256, 256), (5, 3, 3, 3, 3), (512, 512), 1, 8,
                          done_rate=0.005),
    "cfg5_1k": Workload("cfg5_1k", 1024, 32, 120, 160, (32, 64, 128, 256), (3, 3, 3, 3), (512, 512), 1, 4),
    "cfg5_4k": Workload("cfg5_4k", 4096, 32, 120, 160, (32, 64, 128, 256), (3, 3, 3, 3), (512, 512), 1, 4),
    "cfg5_16k": Workload("cfg5_16k", 16384, 32, 120, 160, (32, 64, 128, 256), (3, 3, 3, 3), (512, 512), 1, 4),
}

_FIELDS = ("depth", "proprio", "reward", "value", "done", "last_value", "eps", "logp_jitter")


def _rng(seed: int, name: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, _FIELDS.index(name) + 1]))


def rollout_numpy(w: Workload, seed: int | None = None) -> Dict[str, np.ndarray]:
    """One rollout's worth of inputs, time-major [T, N, ...], one Philox stream per field.

    `eps` is the standard-normal action noise the rollout policy consumed (the caller turns it into
    actions and old log-probs with its own forward pass); `logp_jitter` is N(0, 0.3^2) noise a test may
    add to the old log-probs so that both branches of the clip are exercised.
    """
    seed = w.seed if seed is None else seed
    T, N = w.T, w.N
    g = _rng(seed, "depth")
    depth = g.uniform(0.1, 2.0, size=(T, N, w.H, w.W)).astype(np.float16)
    depth[g.random(size=depth.shape) < 0.10] = 0
    out = {
        "depth": depth,
        "proprio": _rng(seed, "proprio").standard_normal((T, N, w.P)).astype(np.float32),
        "reward": _rng(seed, "reward").standard_normal((T, N)).astype(np.float32),
        "value": _rng(seed, "value").standard_normal((T, N)).astype(np.float32),
        "done": (_rng(seed, "done").random((T, N)) < w.done_rate).astype(np.uint8),
        "last_value": _rng(seed, "last_value").standard_normal((N,)).astype(np.float32),
        "eps": _rng(seed, "eps").standard_normal((T, N, w.A)).astype(np.float32),
        "logp_jitter": (0.3 * _rng(seed, "logp_jitter").standard_normal((T, N))).astype(np.float32),
    }
    return out


def rollout_torch(w: Workload, device, seed: int | None = None, chunk_t: int = 1):
    """Same distributions generated on `device` with torch's generator (one seed per field and step).

    Returns a dict of device tensors [T, N, ...].  Depth is produced step by step so that the fp32
    temporaries stay small next to a buffer of tens of GB.
    """
    import torch

    seed = w.seed if seed is None else seed
    T, N = w.T, w.N
    gen = torch.Generator(device=device)
    depth = torch.empty((T, N, w.H, w.W), dtype=torch.float16, device=device)
    # generate in slabs of at most ~64M pixels to bound the fp32 temporaries
    rows = max(1, min(N, (64 << 20) // (w.H * w.W)))
    for t in range(T):
        gen.manual_seed(1_000_003 * (seed + 1) + t)
        for n0 in range(0, N, rows):
            n1 = min(N, n0 + rows)
            u = torch.rand((n1 - n0, w.H, w.W), generator=gen, device=device)
            d = (0.1 + 1.9 * u).to(torch.float16)
            z = torch.rand((n1 - n0, w.H, w.W), generator=gen, device=device) < 0.10
            d[z] = 0
            depth[t, n0:n1] = d
            del u, d, z

    def normal(name, shape, scale=1.0):
        gen.manual_seed(7_000_003 * (seed + 1) + _FIELDS.index(name))
        return scale * torch.randn(shape, generator=gen, device=device, dtype=torch.float32)

    gen.manual_seed(7_000_003 * (seed + 1) + _FIELDS.index("done"))
    done = (torch.rand((T, N), generator=gen, device=device) < w.done_rate).to(torch.uint8)
    return {
        "depth": depth,
        "proprio": normal("proprio", (T, N, w.P)),
        "reward": normal("reward", (T, N)),
        "value": normal("value", (T, N)),
        "done": done,
        "last_value": normal("last_value", (N,)),
        "eps": normal("eps", (T, N, w.A)),
        "logp_jitter": normal("logp_jitter", (T, N), 0.3),
    }


def param_shapes(w: Workload):
    """Shapes of the parameter tensors of a workload's network in arena order, and the indices of the layer
    normalisation scales (which start at 1, not 0)."""
    shapes, gammas = [], []
    cin, h, wd = 1, w.H, w.W
    for c, k in zip(w.conv_c, w.conv_k):
        shapes += [(c, k, k, cin), (c,)]
        if w.norm:
            gammas.append(len(shapes))
            shapes += [(c,), (c,)]
        cin = c
        h, wd = (h + 2 * (k // 2) - k) // 2 + 1, (wd + 2 * (k // 2) - k) // 2 + 1
    i = cin + w.P
    if w.embed:
        shapes += [(w.embed, h * wd * cin), (w.embed,)]
        i = w.embed + w.P
    for _ in range(w.n_lstm):
        shapes += [(4 * w.lstm_h, i), (4 * w.lstm_h, w.lstm_h), (4 * w.lstm_h,)]
        i = w.lstm_h
    for o in w.fc:
        shapes += [(o, i), (o,)]
        i = o
    shapes += [(w.A + 1, i), (w.A + 1,), (w.A,)]
    return shapes, gammas


def scenes_numpy(N: int, n_prims: int, seed: int):
    """Seeded scene parameters for the depth producer: per env a table-like plane below the camera and n_prims
    spheres, boxes and capsules in front of it.  Returns (plane [N,4], prims [N,n_prims,8]) as float32."""
    g = np.random.Generator(np.random.Philox(key=[seed, 4242]))
    nrm = np.stack([0.1 * g.standard_normal(N), -np.ones(N), -0.3 + 0.1 * g.standard_normal(N)], 1)
    nrm /= np.linalg.norm(nrm, axis=1, keepdims=True)
    plane = np.concatenate([nrm, -(0.4 + 0.2 * g.random((N, 1)))], 1).astype(np.float32)
    prims = np.zeros((N, n_prims, 8), np.float32)
    prims[:, :, 0] = g.integers(0, 3, (N, n_prims))
    prims[:, :, 1] = g.uniform(-0.5, 0.5, (N, n_prims))
    prims[:, :, 2] = g.uniform(-0.3, 0.4, (N, n_prims))
    prims[:, :, 3] = g.uniform(0.5, 1.8, (N, n_prims))
    size = g.uniform(0.05, 0.2, (N, n_prims, 4)).astype(np.float32)
    prims[:, :, 4:8] = size
    cap = prims[:, :, 0] == 2  # capsules: p0..p2 is the segment vector, p3 the radius
    prims[:, :, 4:7][cap] = g.uniform(-0.25, 0.25, (int(cap.sum()), 3))
    prims[:, :, 7][cap] = g.uniform(0.03, 0.1, int(cap.sum()))
    return plane, prims


def init_params(total: int, offsets: List[int], shapes: List[tuple], seed: int, ones: Sequence[int] = ()) -> np.ndarray:
    """Random initial fp32 parameter vector for a given tensor layout.

    Weight tensors (rank >= 2) ~ U(+-sqrt(6 / fan_in)); the last weight tensor (the mean/value head) is
    scaled by 0.01 so that the initial policy mean is near zero; rank-1 tensors (biases, log-sigma) are 0,
    except those listed in `ones` (layer normalisation scales), which are 1.  Gaps between tensors stay 0.
    """
    theta = np.zeros(total, np.float32)
    for i in ones:
        theta[offsets[i]: offsets[i] + int(np.prod(shapes[i]))] = 1.0
    g = np.random.Generator(np.random.Philox(key=[seed + 1, 99]))
    mats = [i for i, s in enumerate(shapes) if len(s) >= 2]
    for i in mats:
        shp = shapes[i]
        fan_in = int(np.prod(shp[1:]))
        bound = np.sqrt(6.0 / fan_in)
        n = int(np.prod(shp))
        wts = g.uniform(-bound, bound, size=n).astype(np.float32)
        if i == mats[-1]:
            wts *= np.float32(0.01)
        theta[offsets[i]: offsets[i] + n] = wts
    return theta
