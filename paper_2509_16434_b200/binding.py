"""Thin ctypes binding of libppo_b200.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every computation happens inside the library.
The library must exist (build with `python -m paper_2509_16434_b200.build` or
`__graft_entry__.build()`); there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libppo_b200.so")

PPO_OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "SHAPE", 3: "ALIGN", 4: "STATE", 5: "CUDA", 6: "TIMEOUT", 7: "UNSUPPORTED"}
(FIELD_DEPTH, FIELD_PROPRIO, FIELD_ACTION, FIELD_LOGP, FIELD_VALUE, FIELD_REWARD, FIELD_DONE, FIELD_ADV, FIELD_RET,
 FIELD_SCRATCH, NUM_FIELDS) = range(11)

EXPORTS = [
    "ppo_status_string", "ppo_buffer_field_bytes", "ppo_buffer_bytes", "ppo_buffer_alloc", "ppo_buffer_free",
    "ppo_buffer_field_ptr", "ppo_buffer_write_step", "ppo_compute_gae", "ppo_shuffle_gather_minibatch",
    "ppo_model_create", "ppo_model_destroy", "ppo_model_param_count", "ppo_model_arena_elems",
    "ppo_model_num_tensors", "ppo_model_tensor_info", "ppo_model_workspace_bytes", "ppo_model_bind",
    "ppo_model_sync_shadow", "ppo_encoder_fwd", "ppo_loss_fwd_bwd", "ppo_encoder_bwd", "ppo_model_zero_grad",
    "ppo_adam_step", "ppo_policy_sample", "ppo_poll_status", "ppo_model_activation_ptr", "ppo_gae_static",
    "ppo_model_sync_masks", "ppo_buffer_write_obs", "ppo_buffer_write_outcome", "ppo_policy_act", "ppo_launch_count",
    "ppo_selftest_wait_timeout", "ppo_buffer_render_depth", "ppo_model_set_sequence", "ppo_shuffle_gather_sequences",
    "ppo_model_read_state",
]


class PpoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({status})")


class BufferDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("N", "T", "H", "W", "P", "A")]


class ModelDesc(C.Structure):
    _fields_ = [("H", C.c_int32), ("W", C.c_int32), ("n_conv", C.c_int32), ("conv_c", C.c_int32 * 8),
                ("conv_k", C.c_int32 * 8), ("n_fc", C.c_int32), ("fc", C.c_int32 * 4), ("P", C.c_int32),
                ("A", C.c_int32), ("norm", C.c_int32), ("embed", C.c_int32), ("n_lstm", C.c_int32),
                ("lstm_h", C.c_int32)]


class Minibatch(C.Structure):
    _fields_ = [("depth_f16", C.c_void_p), ("proprio", C.c_void_p), ("action", C.c_void_p),
                ("logp_old", C.c_void_p), ("value_old", C.c_void_p), ("adv", C.c_void_p), ("ret", C.c_void_p),
                ("index", C.c_void_p), ("B", C.c_int32)]


_lib = None


def lib():
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it first (python -m paper_2509_16434_b200.build)")
        L = C.CDLL(LIB_PATH)
        L.ppo_status_string.restype = C.c_char_p
        L.ppo_buffer_bytes.restype = C.c_size_t
        L.ppo_buffer_field_bytes.restype = C.c_size_t
        L.ppo_buffer_field_bytes.argtypes = [C.POINTER(BufferDesc), C.c_int, C.c_int]
        L.ppo_buffer_field_ptr.restype = C.c_void_p
        L.ppo_buffer_field_ptr.argtypes = [C.c_void_p, C.c_int]
        L.ppo_buffer_alloc.argtypes = [C.POINTER(BufferDesc), C.c_void_p, C.c_size_t, C.POINTER(C.c_void_p)]
        L.ppo_buffer_free.argtypes = [C.c_void_p]
        L.ppo_buffer_write_step.argtypes = [C.c_void_p, C.c_int] + [C.c_void_p] * 8
        L.ppo_compute_gae.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_float, C.c_int, C.c_void_p, C.c_void_p]
        L.ppo_shuffle_gather_minibatch.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_int, C.c_int,
                                                   C.POINTER(Minibatch), C.c_void_p]
        L.ppo_model_create.argtypes = [C.POINTER(ModelDesc), C.POINTER(C.c_void_p)]
        L.ppo_model_destroy.argtypes = [C.c_void_p]
        L.ppo_model_param_count.restype = C.c_size_t
        L.ppo_model_param_count.argtypes = [C.c_void_p]
        L.ppo_model_arena_elems.restype = C.c_size_t
        L.ppo_model_arena_elems.argtypes = [C.c_void_p]
        L.ppo_model_num_tensors.argtypes = [C.c_void_p]
        L.ppo_model_tensor_info.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.ppo_model_workspace_bytes.restype = C.c_size_t
        L.ppo_model_workspace_bytes.argtypes = [C.c_void_p, C.c_int]
        L.ppo_model_bind.argtypes = [C.c_void_p] * 7 + [C.c_size_t, C.c_int]
        L.ppo_model_sync_shadow.argtypes = [C.c_void_p, C.c_void_p]
        L.ppo_model_zero_grad.argtypes = [C.c_void_p, C.c_void_p]
        L.ppo_model_sync_masks.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
        L.ppo_encoder_fwd.argtypes = [C.c_void_p, C.POINTER(Minibatch), C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                      C.c_void_p]
        L.ppo_loss_fwd_bwd.argtypes = [C.c_void_p, C.POINTER(Minibatch), C.c_int, C.c_int, C.c_int, C.c_void_p,
                                       C.c_void_p, C.c_float, C.c_float, C.c_float, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_void_p]
        L.ppo_encoder_bwd.argtypes = [C.c_void_p, C.POINTER(Minibatch), C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                      C.c_int, C.c_void_p]
        L.ppo_adam_step.argtypes = [C.c_void_p, C.c_float, C.c_float, C.c_float, C.c_float, C.c_int64, C.c_void_p]
        L.ppo_policy_sample.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p]
        L.ppo_poll_status.argtypes = [C.c_void_p]
        L.ppo_buffer_write_obs.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ppo_buffer_write_outcome.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ppo_policy_act.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.ppo_buffer_render_depth.argtypes = [C.c_void_p, C.c_int, C.c_float, C.c_float, C.c_float, C.c_void_p, C.c_int,
                                              C.c_void_p, C.c_void_p]
        L.ppo_model_set_sequence.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ppo_shuffle_gather_sequences.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_int, C.c_int,
                                                   C.POINTER(Minibatch), C.c_void_p, C.c_void_p]
        L.ppo_model_read_state.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ppo_launch_count.restype = C.c_uint64
        L.ppo_launch_count.argtypes = []
        L.ppo_selftest_wait_timeout.argtypes = [C.c_longlong, C.c_void_p, C.c_void_p]
        L.ppo_gae_static.argtypes = [C.c_void_p] * 4 + [C.c_int, C.c_int, C.c_float, C.c_float, C.c_int] + [C.c_void_p] * 4
        L.ppo_model_activation_ptr.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_void_p),
                                               C.POINTER(C.c_size_t)]
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != PPO_OK:
        raise PpoError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _mbref(mb):
    return C.byref(mb.c if hasattr(mb, "c") else mb)


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def ppo_status_string(status: int) -> str:
    return lib().ppo_status_string(status).decode()


def ppo_poll_status(stream=None) -> int:
    return lib().ppo_poll_status(_stream(stream))


def buffer_desc(N, T, H, W, P=32, A=12) -> BufferDesc:
    return BufferDesc(N, T, H, W, P, A)


def ppo_buffer_bytes(desc: BufferDesc) -> int:
    return lib().ppo_buffer_bytes(C.byref(desc))


def ppo_buffer_field_bytes(desc: BufferDesc, field: int, depth_elem_bytes: int = 2) -> int:
    return lib().ppo_buffer_field_bytes(C.byref(desc), field, depth_elem_bytes)


class Buffer:
    """Handle of the on-device rollout buffer; owns the torch storage the library carves up."""

    _DT = {FIELD_DEPTH: torch.float16, FIELD_DONE: torch.uint8}

    def __init__(self, desc: BufferDesc, device="cuda"):
        self.desc = desc
        nbytes = ppo_buffer_bytes(desc)
        if nbytes == 0:
            raise PpoError(1, "ppo_buffer_bytes")
        self.storage = torch.empty(nbytes, dtype=torch.uint8, device=device)
        h = C.c_void_p()
        _check(lib().ppo_buffer_alloc(C.byref(desc), _ptr(self.storage), nbytes, C.byref(h)), "ppo_buffer_alloc")
        self.handle = h

    def close(self):
        if self.handle:
            lib().ppo_buffer_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def field(self, f: int) -> torch.Tensor:
        """A torch view of one slab (no copy)."""
        d = self.desc
        ptr = lib().ppo_buffer_field_ptr(self.handle, f)
        off = ptr - self.storage.data_ptr()
        nbytes = ppo_buffer_field_bytes(d, f)
        raw = self.storage[off:off + nbytes]
        dt = self._DT.get(f, torch.float32)
        shape = {FIELD_DEPTH: (d.T, d.N, d.H, d.W), FIELD_PROPRIO: (d.T, d.N, d.P), FIELD_ACTION: (d.T, d.N, d.A),
                 FIELD_SCRATCH: (-1,)}.get(f, (d.T, d.N))
        return raw.view(dt).view(shape)


def ppo_buffer_write_step(buf: Buffer, t: int, depth, proprio, action, logp, value, reward, done, stream=None):
    _check(lib().ppo_buffer_write_step(buf.handle, t, _ptr(depth), _ptr(proprio), _ptr(action), _ptr(logp),
                                       _ptr(value), _ptr(reward), _ptr(done), _stream(stream)),
           "ppo_buffer_write_step")


def ppo_buffer_write_obs(buf: Buffer, t: int, depth, proprio, stream=None):
    _check(lib().ppo_buffer_write_obs(buf.handle, t, _ptr(depth), _ptr(proprio), _stream(stream)),
           "ppo_buffer_write_obs")


def ppo_buffer_write_outcome(buf: Buffer, t: int, reward, done, stream=None):
    _check(lib().ppo_buffer_write_outcome(buf.handle, t, _ptr(reward), _ptr(done), _stream(stream)),
           "ppo_buffer_write_outcome")


def ppo_buffer_render_depth(buf: Buffer, t: int, hfov: float, near: float, far: float, plane, prims, stream=None):
    """plane [N,4] fp32, prims [N,K,8] fp32 device tensors: renders the scenes into slab row t of the depth field."""
    _check(lib().ppo_buffer_render_depth(buf.handle, t, hfov, near, far, _ptr(plane), prims.shape[1], _ptr(prims),
                                         _stream(stream)), "ppo_buffer_render_depth")


def ppo_launch_count() -> int:
    return int(lib().ppo_launch_count())


def ppo_selftest_wait_timeout(limit_cycles: int, gave_up, stream=None):
    _check(lib().ppo_selftest_wait_timeout(limit_cycles, _ptr(gave_up), _stream(stream)),
           "ppo_selftest_wait_timeout")


def ppo_compute_gae(buf: Buffer, last_value, gamma: float, lam: float, normalize=True, stats_out=None,
                    stream=None):
    """normalize: False / True (two launches) / 2 (one cooperative launch)."""
    _check(lib().ppo_compute_gae(buf.handle, _ptr(last_value), gamma, lam, int(normalize), _ptr(stats_out),
                                 _stream(stream)), "ppo_compute_gae")


def ppo_gae_static(reward, value, done, last_value, gamma: float, lam: float, normalize: bool, adv, ret,
                   stats_out=None, stream=None):
    """GAE (+ advantage normalisation) on bare [T, N] device tensors without any device allocation by the
    library: for callers that may not call cudaMalloc (fixed arenas, fixed memory budgets).  At most 524288 envs;
    calls that could overlap on the GPU must be serialised (they share one scratch array inside the library)."""
    T, N = reward.shape
    _check(lib().ppo_gae_static(_ptr(reward), _ptr(value), _ptr(done), _ptr(last_value), T, N, gamma, lam,
                                int(normalize), _ptr(adv), _ptr(ret), _ptr(stats_out), _stream(stream)),
           "ppo_gae_static")


class MinibatchArrays:
    """Caller-owned device arrays of one gathered minibatch."""

    def __init__(self, desc: BufferDesc, B: int, device="cuda", with_index: bool = True):
        self.B = B
        self.depth = torch.empty((B, desc.H, desc.W), dtype=torch.float16, device=device)
        self.proprio = torch.empty((B, desc.P), dtype=torch.float32, device=device)
        self.action = torch.empty((B, desc.A), dtype=torch.float32, device=device)
        self.logp_old = torch.empty(B, dtype=torch.float32, device=device)
        self.value_old = torch.empty(B, dtype=torch.float32, device=device)
        self.adv = torch.empty(B, dtype=torch.float32, device=device)
        self.ret = torch.empty(B, dtype=torch.float32, device=device)
        self.index = torch.empty(B, dtype=torch.int32, device=device) if with_index else None
        self.c = Minibatch(self.depth.data_ptr(), self.proprio.data_ptr(), self.action.data_ptr(),
                           self.logp_old.data_ptr(), self.value_old.data_ptr(), self.adv.data_ptr(),
                           self.ret.data_ptr(), self.index.data_ptr() if with_index else None, B)

    def bytes(self) -> int:
        ts = [self.depth, self.proprio, self.action, self.logp_old, self.value_old, self.adv, self.ret]
        return sum(t.numel() * t.element_size() for t in ts)


def ppo_shuffle_gather_minibatch(buf: Buffer, seed: int, epoch: int, mb_index: int, num_minibatches: int,
                                 out: MinibatchArrays, stream=None):
    _check(lib().ppo_shuffle_gather_minibatch(buf.handle, seed, epoch, mb_index, num_minibatches, C.byref(out.c),
                                              _stream(stream)), "ppo_shuffle_gather_minibatch")


def model_desc(H, W, conv_c: Sequence[int], conv_k: Sequence[int], fc: Sequence[int], P=32, A=12, norm=False,
               embed=0, n_lstm=0, lstm_h=0) -> ModelDesc:
    d = ModelDesc()
    d.H, d.W, d.n_conv, d.n_fc, d.P, d.A = H, W, len(conv_c), len(fc), P, A
    d.norm, d.embed, d.n_lstm, d.lstm_h = int(norm), int(embed), int(n_lstm), int(lstm_h)
    for i, v in enumerate(conv_c):
        d.conv_c[i] = v
    for i, v in enumerate(conv_k):
        d.conv_k[i] = v
    for i, v in enumerate(fc):
        d.fc[i] = v
    return d


class Model:
    """Handle of the policy/value network with its torch-owned parameter arena and workspace."""

    def __init__(self, desc: ModelDesc, microbatch: int, device="cuda"):
        self.desc = desc
        h = C.c_void_p()
        _check(lib().ppo_model_create(C.byref(desc), C.byref(h)), "ppo_model_create")
        self.handle = h
        self.microbatch = microbatch
        n = lib().ppo_model_arena_elems(h)
        self.arena = n
        self.master = torch.zeros(n, dtype=torch.float32, device=device)
        self.shadow = torch.zeros(n, dtype=torch.bfloat16, device=device)
        self.grad = torch.zeros(n, dtype=torch.float32, device=device)
        self.adam_m = torch.zeros(n, dtype=torch.float32, device=device)
        self.adam_v = torch.zeros(n, dtype=torch.float32, device=device)
        ws = lib().ppo_model_workspace_bytes(h, microbatch)
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=device)
        _check(lib().ppo_model_bind(h, _ptr(self.master), _ptr(self.shadow), _ptr(self.grad), _ptr(self.adam_m),
                                    _ptr(self.adam_v), _ptr(self.workspace), ws, microbatch), "ppo_model_bind")

    def close(self):
        if self.handle:
            lib().ppo_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def param_count(self) -> int:
        return lib().ppo_model_param_count(self.handle)

    def tensors(self):
        out = []
        for i in range(lib().ppo_model_num_tensors(self.handle)):
            off, sz = C.c_int64(), C.c_int64()
            _check(lib().ppo_model_tensor_info(self.handle, i, C.byref(off), C.byref(sz)), "ppo_model_tensor_info")
            out.append((off.value, sz.value))
        return out

    def activation(self, kind: int, index: int) -> torch.Tensor:
        """A flat bf16 torch view of a saved activation inside the workspace (see ppo_model_activation_ptr)."""
        p, n = C.c_void_p(), C.c_size_t()
        _check(lib().ppo_model_activation_ptr(self.handle, kind, index, C.byref(p), C.byref(n)),
               "ppo_model_activation_ptr")
        off = p.value - self.workspace.data_ptr()
        if kind == 2:
            return self.workspace[off:off + 4 * n.value].view(torch.int32)
        if kind in (4, 6, 7):
            return self.workspace[off:off + 4 * n.value].view(torch.float32)
        return self.workspace[off:off + 2 * n.value].view(torch.bfloat16)

    def load(self, theta, stream=None):
        """Copies an fp32 parameter vector (numpy or torch, arena layout) into master and refreshes the shadow."""
        t = torch.as_tensor(theta, dtype=torch.float32)
        self.master.copy_(t.to(self.master.device))
        ppo_model_sync_shadow(self, stream)


def ppo_model_set_sequence(m: Model, T: int, Be: int, done, h_init, c_init):
    """done uint8 [T,Be], h_init / c_init fp32 [n_lstm,Be,lstm_h]: the tensors must stay alive until the backward pass."""
    _check(lib().ppo_model_set_sequence(m.handle, T, Be, _ptr(done), _ptr(h_init), _ptr(c_init)), "ppo_model_set_sequence")


def ppo_model_read_state(m: Model, h_out, c_out, stream=None):
    """fp32 [n_lstm,Be,lstm_h] each: the state after the last step of the latest forward, zero where that step was done."""
    _check(lib().ppo_model_read_state(m.handle, _ptr(h_out), _ptr(c_out), _stream(stream)), "ppo_model_read_state")


def ppo_shuffle_gather_sequences(buf: Buffer, seed: int, epoch: int, mb_index: int, num_minibatches: int,
                                 out: "MinibatchArrays", done_out, stream=None):
    _check(lib().ppo_shuffle_gather_sequences(buf.handle, seed, epoch, mb_index, num_minibatches, C.byref(out.c),
                                              _ptr(done_out), _stream(stream)), "ppo_shuffle_gather_sequences")


def ppo_model_sync_shadow(m: Model, stream=None):
    _check(lib().ppo_model_sync_shadow(m.handle, _stream(stream)), "ppo_model_sync_shadow")


def ppo_model_sync_masks(m: Model, rows: int, stream=None):
    _check(lib().ppo_model_sync_masks(m.handle, rows, _stream(stream)), "ppo_model_sync_masks")


def ppo_model_zero_grad(m: Model, stream=None):
    _check(lib().ppo_model_zero_grad(m.handle, _stream(stream)), "ppo_model_zero_grad")


def ppo_encoder_fwd(m: Model, mb: MinibatchArrays, row0: int, rows: int, mean, value, stream=None):
    _check(lib().ppo_encoder_fwd(m.handle, _mbref(mb), row0, rows, _ptr(mean), _ptr(value), _stream(stream)),
           "ppo_encoder_fwd")


def ppo_loss_fwd_bwd(m: Model, mb: MinibatchArrays, row0: int, rows: int, B_total: int, mean, value, clip: float,
                     vf_coef: float, ent_coef: float, loss_out, dmean, dvalue, stream=None):
    _check(lib().ppo_loss_fwd_bwd(m.handle, _mbref(mb), row0, rows, B_total, _ptr(mean), _ptr(value), clip,
                                  vf_coef, ent_coef, _ptr(loss_out), _ptr(dmean), _ptr(dvalue), _stream(stream)),
           "ppo_loss_fwd_bwd")


def ppo_encoder_bwd(m: Model, mb: MinibatchArrays, row0: int, rows: int, dmean, dvalue, accumulate: bool,
                    stream=None):
    _check(lib().ppo_encoder_bwd(m.handle, _mbref(mb), row0, rows, _ptr(dmean), _ptr(dvalue), int(accumulate),
                                 _stream(stream)), "ppo_encoder_bwd")


def ppo_adam_step(m: Model, lr: float, beta1: float, beta2: float, eps: float, step: int, stream=None):
    _check(lib().ppo_adam_step(m.handle, lr, beta1, beta2, eps, step, _stream(stream)), "ppo_adam_step")


def ppo_policy_act(m: Model, buf: Buffer, t: int, eps, stream=None):
    _check(lib().ppo_policy_act(m.handle, buf.handle, t, _ptr(eps), _stream(stream)), "ppo_policy_act")


def ppo_policy_sample(m: Model, rows: int, mean, eps, action, logp, stream=None):
    _check(lib().ppo_policy_sample(m.handle, rows, _ptr(mean), _ptr(eps), _ptr(action), _ptr(logp),
                                   _stream(stream)), "ppo_policy_sample")
