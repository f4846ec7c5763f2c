"""ctypes front end of the CPU oracle (oracle/ppo_oracle.c).

TEST INFRASTRUCTURE: only tests/, the smoke check and the bench's CPU-baseline
leg may import this.  It does not import the CUDA package and the CUDA package
does not import it.  All arrays are numpy; floating point is float64 unless a
narrower type is part of the definition (float32 rewards/values as stored in the
buffer, float16 depth).
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field
from typing import List, Sequence

import numpy as np

from . import build as _build

_lib = None


class _Model(C.Structure):
    _fields_ = [
        ("H", C.c_int32), ("W", C.c_int32), ("n_conv", C.c_int32),
        ("conv_c", C.c_int32 * 8), ("conv_k", C.c_int32 * 8),
        ("n_fc", C.c_int32), ("fc", C.c_int32 * 4),
        ("P", C.c_int32), ("A", C.c_int32), ("norm", C.c_int32), ("embed", C.c_int32),
        ("n_lstm", C.c_int32), ("lstm_h", C.c_int32),
    ]


def lib():
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        L.orc_depth_bytes.restype = C.c_uint64
        L.orc_depth_bytes.argtypes = [C.c_uint64] * 5
        L.orc_mix32.restype = C.c_uint32
        L.orc_mix32.argtypes = [C.c_uint32]
        L.orc_perm.restype = C.c_uint32
        L.orc_perm.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
        L.orc_perm_half_bits.restype = C.c_int
        L.orc_perm_half_bits.argtypes = [C.c_uint32]
        L.orc_round_bf16.restype = C.c_double
        L.orc_round_bf16.argtypes = [C.c_double]
        L.orc_param_layout.restype = C.c_int64
        L.orc_act_stride.restype = C.c_int64
        L.orc_num_threads.restype = C.c_int
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def num_threads() -> int:
    return int(lib().orc_num_threads())


@dataclass
class ModelDesc:
    H: int
    W: int
    conv_c: Sequence[int]
    conv_k: Sequence[int]
    fc: Sequence[int]
    P: int = 32
    A: int = 12
    norm: bool = False   # layer normalisation over the channels of every conv output, before its ReLU
    embed: int = 0       # > 0: flatten -> FC(embed) -> ReLU instead of the global average pool
    n_lstm: int = 0      # stacked LSTM layers between h_0 and the fully connected layers
    lstm_h: int = 0      # their width

    def c(self) -> _Model:
        m = _Model()
        m.H, m.W, m.n_conv, m.n_fc, m.P, m.A = self.H, self.W, len(self.conv_c), len(self.fc), self.P, self.A
        m.norm, m.embed = int(self.norm), int(self.embed)
        m.n_lstm, m.lstm_h = int(self.n_lstm), int(self.lstm_h)
        for i, v in enumerate(self.conv_c):
            m.conv_c[i] = v
        for i, v in enumerate(self.conv_k):
            m.conv_k[i] = v
        for i, v in enumerate(self.fc):
            m.fc[i] = v
        return m


@dataclass
class Layout:
    total: int
    offsets: List[int]
    sizes: List[int]
    is_matrix: List[int]
    shapes: List[tuple] = field(default_factory=list)


def depth_bytes(N, T, H, W, elem) -> int:
    return int(lib().orc_depth_bytes(N, T, H, W, elem))


def param_layout(md: ModelDesc) -> Layout:
    n_max = 4 * 8 + 2 * 4 + 3 * 4 + 5
    offs = (C.c_int64 * n_max)()
    szs = (C.c_int64 * n_max)()
    mat = (C.c_int32 * n_max)()
    n = C.c_int32(0)
    m = md.c()
    total = lib().orc_param_layout(C.byref(m), offs, szs, mat, C.byref(n))
    k = n.value
    lay = Layout(int(total), list(offs[:k]), list(szs[:k]), list(mat[:k]))
    cin = 1
    for co, kk in zip(md.conv_c, md.conv_k):
        lay.shapes += [(co, kk, kk, cin), (co,)]
        if md.norm:
            lay.shapes += [(co,), (co,)]
        cin = co
    i = cin + md.P
    if md.embed:
        ho, wo = conv_shapes(md)
        lay.shapes += [(md.embed, ho[-1] * wo[-1] * cin), (md.embed,)]
        i = md.embed + md.P
    for _ in range(md.n_lstm):
        lay.shapes += [(4 * md.lstm_h, i), (4 * md.lstm_h, md.lstm_h), (4 * md.lstm_h,)]
        i = md.lstm_h
    for o in md.fc:
        lay.shapes += [(o, i), (o,)]
        i = o
    lay.shapes += [(md.A + 1, i), (md.A + 1,), (md.A,)]
    return lay


def conv_shapes(md: ModelDesc):
    m = md.c()
    ho = (C.c_int32 * 8)()
    wo = (C.c_int32 * 8)()
    lib().orc_conv_shapes(C.byref(m), ho, wo)
    n = len(md.conv_c)
    return list(ho[:n]), list(wo[:n])


def act_stride(md: ModelDesc) -> int:
    m = md.c()
    return int(lib().orc_act_stride(C.byref(m)))


def round_bf16(x: float) -> float:
    return float(lib().orc_round_bf16(float(x)))


# ------------------------------------------------------------------ GAE ----

def gae(reward, value, done, last_value, gamma, lam):
    """reward, value: float32 [T,N]; done: uint8 [T,N]; last_value float32 [N] -> adv, ret float64 [T,N]."""
    reward = np.ascontiguousarray(reward, dtype=np.float32)
    value = np.ascontiguousarray(value, dtype=np.float32)
    done = np.ascontiguousarray(done, dtype=np.uint8)
    last_value = np.ascontiguousarray(last_value, dtype=np.float32)
    T, N = reward.shape
    adv = np.empty((T, N), np.float64)
    ret = np.empty((T, N), np.float64)
    lib().orc_gae(C.c_int(T), C.c_int(N), _p(reward), _p(value), _p(done), _p(last_value),
                  C.c_double(gamma), C.c_double(lam), _p(adv), _p(ret))
    return adv, ret


def adv_normalize(adv):
    a = _f64(adv).copy()
    mean = C.c_double(0)
    std = C.c_double(0)
    lib().orc_adv_normalize(C.c_size_t(a.size), _p(a), C.byref(mean), C.byref(std))
    return a, mean.value, std.value


# ---------------------------------------------------------- permutation ----

def mix32(x: int) -> int:
    return int(lib().orc_mix32(x & 0xFFFFFFFF))


def perm_keys(seed: int, epoch: int):
    k = (C.c_uint32 * 6)()
    lib().orc_perm_keys(C.c_uint64(seed), C.c_uint32(epoch), k)
    return list(k)


def perm(seed: int, epoch: int, M: int, start: int = 0, count: int | None = None) -> np.ndarray:
    count = M - start if count is None else count
    out = np.empty(count, np.uint32)
    lib().orc_perm_fill(C.c_uint64(seed), C.c_uint32(epoch), C.c_uint32(M), C.c_uint32(start), C.c_uint32(count), _p(out))
    return out


def gather(fields: dict, idx: np.ndarray, N: int) -> dict:
    """Row j of every output is sample idx[j] of the time-major buffer (s = t*N + n): exact copies."""
    out = {}
    for name, arr in fields.items():
        flat = arr.reshape((arr.shape[0] * arr.shape[1],) + arr.shape[2:])
        out[name] = flat[idx.astype(np.int64)].copy()
    return out


# -------------------------------------------------------------- encoder ----

def round_weights(md: ModelDesc, theta) -> np.ndarray:
    theta = _f64(theta)
    out = np.empty_like(theta)
    m = md.c()
    lib().orc_round_weights(C.byref(m), _p(theta), _p(out))
    return out


def encoder_fwd(md: ModelDesc, theta_used, depth, proprio, act_bf16: bool = False):
    """depth [B,H,W] (any float type, values exactly representable), proprio [B,P] -> mu [B,A], V [B], acts.
    act_bf16: round every layer's stored output to bf16 (the next contraction's operand)."""
    depth = _f64(depth)
    proprio = _f64(proprio)
    theta_used = _f64(theta_used)
    B = depth.shape[0]
    acts = np.empty((B, act_stride(md)), np.float64)
    mu = np.empty((B, md.A), np.float64)
    V = np.empty((B,), np.float64)
    m = md.c()
    lib().orc_encoder_fwd(C.byref(m), _p(theta_used), C.c_int(B), _p(depth), _p(proprio), _p(acts), _p(mu), _p(V),
                          C.c_int(int(act_bf16)))
    return mu, V, acts


def encoder_bwd(md: ModelDesc, theta_used, acts, dmu, dV, grad=None) -> np.ndarray:
    theta_used = _f64(theta_used)
    dmu = _f64(dmu)
    dV = _f64(dV)
    B = acts.shape[0]
    if grad is None:
        grad = np.zeros_like(theta_used)
    m = md.c()
    lib().orc_encoder_bwd(C.byref(m), _p(theta_used), C.c_int(B), _p(acts), _p(dmu), _p(dV), _p(grad))
    return grad


# ----------------------------------------------------------------- loss ----

def loss(mu, V, logsigma, action, logp_old, adv, ret, clip, c_v, c_e, B_total=None, out=None, dlogsigma=None):
    mu, V, logsigma, action = _f64(mu), _f64(V), _f64(logsigma), _f64(action)
    logp_old, adv, ret = _f64(logp_old), _f64(adv), _f64(ret)
    B, A = mu.shape
    B_total = B if B_total is None else B_total
    if out is None:
        out = np.zeros(5, np.float64)
    if dlogsigma is None:
        dlogsigma = np.zeros(A, np.float64)
    dmu = np.empty((B, A), np.float64)
    dV = np.empty((B,), np.float64)
    lib().orc_loss(C.c_int(B), C.c_int(B_total), C.c_int(A), _p(mu), _p(V), _p(logsigma), _p(action), _p(logp_old),
                   _p(adv), _p(ret), C.c_double(clip), C.c_double(c_v), C.c_double(c_e), _p(out), _p(dmu), _p(dV),
                   _p(dlogsigma))
    return out, dmu, dV, dlogsigma


def sample_action(mu, logsigma, eps):
    mu, logsigma, eps = _f64(mu), _f64(logsigma), _f64(eps)
    B, A = mu.shape
    action = np.empty((B, A), np.float64)
    logp = np.empty((B,), np.float64)
    lib().orc_sample_action(C.c_int(B), C.c_int(A), _p(mu), _p(logsigma), _p(eps), _p(action), _p(logp))
    return action, logp


# ----------------------------------------------------------------- Adam ----

def adam(theta, m, v, g, lr, beta1, beta2, eps, step):
    """In place on float64 arrays theta, m, v (theta rounded to fp32 values)."""
    for a in (theta, m, v):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    g = _f64(g)
    lib().orc_adam(C.c_int64(theta.size), _p(theta), _p(m), _p(v), _p(g), C.c_double(lr), C.c_double(beta1),
                   C.c_double(beta2), C.c_double(eps), C.c_int64(step))


# ----------------------------------------------------- composed learner ----

def total_loss_and_grad(md: ModelDesc, theta, depth, proprio, action, logp_old, adv, ret, clip, c_v, c_e,
                        act_bf16: bool = False):
    """One minibatch: L = L_pi + c_v L_V - c_e H and dL/dtheta (w.r.t. the fp32 master, straight through the
    bf16 rounding of the weight matrices and, with act_bf16, of the activations).  Returns (L, out[5], grad, mu, V)."""
    lay = param_layout(md)
    theta = _f64(theta)
    used = round_weights(md, theta)
    logsigma = theta[lay.offsets[-1]: lay.offsets[-1] + md.A]
    mu, V, acts = encoder_fwd(md, used, depth, proprio, act_bf16)
    out, dmu, dV, dls = loss(mu, V, logsigma, action, logp_old, adv, ret, clip, c_v, c_e)
    grad = encoder_bwd(md, used, acts, dmu, dV)
    grad[lay.offsets[-1]: lay.offsets[-1] + md.A] += dls
    L = out[0] + c_v * out[1] - c_e * out[2]
    return L, out, grad, mu, V


# -------------------------------------------------------- depth producer ----

def round_fp16(x: float) -> float:
    lib().orc_round_fp16.restype = C.c_double
    lib().orc_round_fp16.argtypes = [C.c_double]
    return float(lib().orc_round_fp16(float(x)))


def render_depth(H: int, W: int, hfov: float, near: float, far: float, plane, prims) -> np.ndarray:
    """plane [N,4] (unit normal, offset), prims [N,K,8] ({type, x, y, z, p0..p3}) -> depth [N,H,W] float64 holding
    fp16 values (0 where nothing is seen within [near, far])."""
    plane = _f64(plane)
    prims = _f64(prims)
    N, K = prims.shape[0], prims.shape[1]
    out = np.empty((N, H, W), np.float64)
    lib().orc_render_depth(C.c_int(N), C.c_int(H), C.c_int(W), C.c_double(hfov), C.c_double(near), C.c_double(far),
                           _p(plane), C.c_int(K), _p(prims), _p(out))
    return out


# ------------------------------------------------------ recurrent trunk ----

def lstm_rec_len(md: ModelDesc) -> int:
    lib().orc_lstm_rec_len.restype = C.c_int64
    m = md.c()
    return int(lib().orc_lstm_rec_len(C.byref(m)))


def encoder_fwd_seq(md: ModelDesc, theta_used, depth, proprio, done, h_init, c_init, act_bf16: bool = False):
    """Sequence minibatch, rows time-major: depth [T,Be,H,W], proprio [T,Be,P], done uint8 [T,Be], h_init / c_init
    [n_lstm,Be,lstm_h] -> mu [T*Be,A], V [T*Be], acts, lrec (the trunk's per-row record, kept for the backward)."""
    T, Be = done.shape
    depth = _f64(depth).reshape(T * Be, md.H, md.W)
    proprio = _f64(proprio).reshape(T * Be, md.P)
    done = np.ascontiguousarray(done, dtype=np.uint8)
    h_init, c_init, theta_used = _f64(h_init), _f64(c_init), _f64(theta_used)
    R = T * Be
    acts = np.zeros((R, act_stride(md)), np.float64)
    lrec = np.zeros((R, lstm_rec_len(md)), np.float64)
    mu = np.empty((R, md.A), np.float64)
    V = np.empty((R,), np.float64)
    m = md.c()
    lib().orc_encoder_fwd_seq(C.byref(m), _p(theta_used), C.c_int(T), C.c_int(Be), _p(depth), _p(proprio), _p(done),
                              _p(h_init), _p(c_init), _p(acts), _p(lrec), _p(mu), _p(V), C.c_int(int(act_bf16)))
    return mu, V, acts, lrec


def encoder_bwd_seq(md: ModelDesc, theta_used, done, acts, lrec, dmu, dV, grad=None) -> np.ndarray:
    T, Be = done.shape
    done = np.ascontiguousarray(done, dtype=np.uint8)
    theta_used, dmu, dV = _f64(theta_used), _f64(dmu), _f64(dV)
    if grad is None:
        grad = np.zeros_like(theta_used)
    m = md.c()
    lib().orc_encoder_bwd_seq(C.byref(m), _p(theta_used), C.c_int(T), C.c_int(Be), _p(done), _p(acts), _p(lrec),
                              _p(dmu), _p(dV), _p(grad))
    return grad


def total_loss_and_grad_seq(md: ModelDesc, theta, depth, proprio, done, h_init, c_init, action, logp_old, adv, ret,
                            clip, c_v, c_e, act_bf16: bool = False):
    """One sequence minibatch (rows time-major, T*Be of them): as total_loss_and_grad, through the recurrent trunk."""
    lay = param_layout(md)
    theta = _f64(theta)
    used = round_weights(md, theta)
    logsigma = theta[lay.offsets[-1]: lay.offsets[-1] + md.A]
    mu, V, acts, lrec = encoder_fwd_seq(md, used, depth, proprio, done, h_init, c_init, act_bf16)
    out, dmu, dV, dls = loss(mu, V, logsigma, action, logp_old, adv, ret, clip, c_v, c_e)
    grad = encoder_bwd_seq(md, used, done, acts, lrec, dmu, dV)
    grad[lay.offsets[-1]: lay.offsets[-1] + md.A] += dls
    L = out[0] + c_v * out[1] - c_e * out[2]
    return L, out, grad, mu, V
