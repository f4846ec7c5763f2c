"""CPU-only checks of the CUDA library's host side: it loads, exports what the header declares, sizes and layouts
agree with the definitions, and bad arguments are refused before anything is launched."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2509_16434_b200 import binding as ppo
from paper_2509_16434_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2509_16434_b200 import build
    build.build()
    return ppo.lib()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "ppo_b200.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ppo_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in the header but not exported"
    assert declared == set(ppo.EXPORTS)


def test_status_strings(lib):
    assert ppo.ppo_status_string(0) == "ok"
    assert len({ppo.ppo_status_string(i) for i in range(8)}) == 8


def test_buffer_bytes_closed_forms(lib):
    d = ppo.buffer_desc(512, 16, 240, 320)
    # Section III-B: 512 envs x 320x240 x 16 steps of fp32 depth = 2.5 GB
    assert ppo.ppo_buffer_field_bytes(d, ppo.FIELD_DEPTH, 4) == 2_516_582_400
    assert ppo.ppo_buffer_field_bytes(d, ppo.FIELD_DEPTH, 2) == orc.depth_bytes(512, 16, 240, 320, 2)
    for name, depth_bytes in [("cfg1", 33_554_432), ("cfg2", 629_145_600), ("cfg3", 2_516_582_400),
                              ("cfg4", 20_132_659_200), ("cfg5_16k", 20_132_659_200)]:
        w = synth.WORKLOADS[name]
        d = ppo.buffer_desc(w.N, w.T, w.H, w.W, w.P, w.A)
        assert ppo.ppo_buffer_field_bytes(d, ppo.FIELD_DEPTH) == depth_bytes
        total = ppo.ppo_buffer_bytes(d)
        rec = w.H * w.W * 2 + w.P * 4 + w.A * 4 + 4 * 5 + 1
        assert w.M * rec <= total <= w.M * rec + 11 * 256 + 4096 * 16
    assert ppo.ppo_buffer_bytes(ppo.buffer_desc(0, 16, 8, 8)) == 0
    assert ppo.ppo_buffer_field_bytes(ppo.buffer_desc(4, 4, 8, 8), 99) == 0


def test_buffer_alloc_rejects_bad_arguments(lib):
    d = ppo.buffer_desc(4, 4, 8, 8)
    h = C.c_void_p()
    need = ppo.ppo_buffer_bytes(d)
    assert lib.ppo_buffer_alloc(C.byref(d), None, need, C.byref(h)) == 1
    assert lib.ppo_buffer_alloc(C.byref(d), C.c_void_p(0x1000 + 8), need, C.byref(h)) == 3
    assert lib.ppo_buffer_alloc(C.byref(d), C.c_void_p(0x1000), need - 1, C.byref(h)) == 2
    # a handle over fake (never dereferenced) storage: host-side checks only
    assert lib.ppo_buffer_alloc(C.byref(d), C.c_void_p(0x10000), need, C.byref(h)) == 0
    p = [C.c_void_p(0x20000)] * 7
    assert lib.ppo_buffer_write_step(h, 4, *p, None) == 1      # t out of range
    assert lib.ppo_buffer_write_step(h, -1, *p, None) == 1
    assert lib.ppo_buffer_write_step(h, 0, None, *p[1:], None) == 1
    mb = ppo.Minibatch(*([0x30000] * 8), 4)
    assert lib.ppo_shuffle_gather_minibatch(h, 0, 0, 0, 3, C.byref(mb), None) == 2   # 16 % 3 != 0
    assert lib.ppo_shuffle_gather_minibatch(h, 0, 0, 4, 4, C.byref(mb), None) == 1   # mb_index out of range
    mb.B = 5
    assert lib.ppo_shuffle_gather_minibatch(h, 0, 0, 0, 4, C.byref(mb), None) == 2   # wrong B
    mb.B = 4
    assert lib.ppo_shuffle_gather_minibatch(h, 0, 0, 0, 4, C.byref(mb), None) == 4   # no GAE yet
    assert lib.ppo_compute_gae(h, None, 0.99, 0.95, 1, None, None) == 1
    assert lib.ppo_compute_gae(h, C.c_void_p(0x40000), 1.5, 0.95, 1, None, None) == 1
    assert lib.ppo_buffer_free(h) == 0


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg4", "paper_cnn", "paper_policy"])
def test_model_layout_matches_the_oracles(lib, name):
    w = synth.WORKLOADS[name]
    md = ppo.model_desc(w.H, w.W, w.conv_c, w.conv_k, w.fc, w.P, w.A, norm=w.norm, embed=w.embed, n_lstm=w.n_lstm,
                        lstm_h=w.lstm_h)
    h = C.c_void_p()
    assert lib.ppo_model_create(C.byref(md), C.byref(h)) == 0
    lay = orc.param_layout(orc.ModelDesc(w.H, w.W, w.conv_c, w.conv_k, w.fc, w.P, w.A, norm=w.norm, embed=w.embed,
                                         n_lstm=w.n_lstm, lstm_h=w.lstm_h))
    assert [tuple(s) for s in lay.shapes] == [tuple(s) for s in synth.param_shapes(w)[0]]
    assert lib.ppo_model_param_count(h) == sum(lay.sizes)
    assert lib.ppo_model_arena_elems(h) == lay.total
    assert lib.ppo_model_num_tensors(h) == len(lay.offsets)
    for i, (o, s) in enumerate(zip(lay.offsets, lay.sizes)):
        off, sz = C.c_int64(), C.c_int64()
        assert lib.ppo_model_tensor_info(h, i, C.byref(off), C.byref(sz)) == 0
        assert (off.value, sz.value) == (o, s)
    closed = {"cfg1": 51_481, "cfg2": 805_145, "cfg4": 1_395_737}
    if name in closed:
        assert lib.ppo_model_param_count(h) == closed[name]
    if w.n_lstm:  # W_x, W_h and b of each layer: 4H (in + H + 1)
        H, ins = w.lstm_h, [w.embed + w.P] + [w.lstm_h] * (w.n_lstm - 1)
        i0 = len(lay.sizes) - 3 - 2 * len(w.fc) - 3 * w.n_lstm
        assert sum(lay.sizes[i0:i0 + 3 * w.n_lstm]) == sum(4 * H * (i + H + 1) for i in ins)
        # a sequence must be announced with sane arguments
        assert lib.ppo_model_set_sequence(h, 4, 4, C.c_void_p(0x100), C.c_void_p(0x100), C.c_void_p(0x100)) == 4  # unbound
        assert lib.ppo_model_set_sequence(h, 4, 4, None, C.c_void_p(0x100), C.c_void_p(0x100)) == 1
        assert lib.ppo_model_read_state(h, C.c_void_p(0x100), C.c_void_p(0x100), None) == 4  # nothing was run yet
        assert lib.ppo_model_read_state(h, None, C.c_void_p(0x100), None) == 1
    else:
        assert lib.ppo_model_set_sequence(h, 4, 4, C.c_void_p(0x100), C.c_void_p(0x100), C.c_void_p(0x100)) != 0
    ws1, ws2 = lib.ppo_model_workspace_bytes(h, 64), lib.ppo_model_workspace_bytes(h, 128)
    assert 0 < ws1 < ws2
    # calls before bind are refused
    mb = ppo.Minibatch(*([0x30000] * 8), 16)
    assert lib.ppo_encoder_fwd(h, C.byref(mb), 0, 8, C.c_void_p(0x1000), C.c_void_p(0x1000), None) == 4
    assert lib.ppo_adam_step(h, 1e-3, 0.9, 0.999, 1e-8, 1, None) == 4
    assert lib.ppo_model_bind(h, C.c_void_p(0x1000), C.c_void_p(0x2000), C.c_void_p(0x3000), C.c_void_p(0x4000),
                              C.c_void_p(0x5000), C.c_void_p(0x6001), ws1, 64) == 3
    assert lib.ppo_model_bind(h, C.c_void_p(0x1000), C.c_void_p(0x2000), C.c_void_p(0x3000), C.c_void_p(0x4000),
                              C.c_void_p(0x5000), C.c_void_p(0x10000), ws1 - 1, 64) == 2
    assert lib.ppo_model_bind(h, C.c_void_p(0x1000), C.c_void_p(0x2000), C.c_void_p(0x3000), C.c_void_p(0x4000),
                              C.c_void_p(0x5000), C.c_void_p(0x10000), ws1, 64) == 0
    assert lib.ppo_encoder_fwd(h, C.byref(mb), 0, 65, C.c_void_p(0x1000), C.c_void_p(0x1000), None) == 2  # > microbatch
    assert lib.ppo_encoder_fwd(h, C.byref(mb), 10, 8, C.c_void_p(0x1000), C.c_void_p(0x1000), None) == 2  # past B
    assert lib.ppo_encoder_bwd(h, C.byref(mb), 0, 8, C.c_void_p(0x1000), C.c_void_p(0x1000), 1, None) == 4  # no fwd
    assert lib.ppo_adam_step(h, 1e-3, 0.9, 0.999, 1e-8, 0, None) == 1                                       # step < 1
    assert lib.ppo_model_destroy(h) == 0


def test_model_create_rejects_unsupported_shapes(lib):
    h = C.c_void_p()
    bad = [ppo.model_desc(64, 64, (16, 30), (3, 3), (64,)),      # channels not a multiple of 8
           ppo.model_desc(64, 64, (16, 32), (3, 4), (64,)),      # even kernel
           ppo.model_desc(64, 64, (16, 32), (3, 3), (60,)),      # fc width
           ppo.model_desc(64, 64, (16, 32), (3, 3), (64,), P=3),  # pooled + proprio width
           ppo.model_desc(64, 64, (16, 32), (3, 3), (64,), n_lstm=1, lstm_h=48),   # LSTM width
           ppo.model_desc(64, 64, (16, 32), (3, 3), (64,), P=8, n_lstm=1, lstm_h=64),]  # LSTM input width
    for md in bad:
        assert lib.ppo_model_create(C.byref(md), C.byref(h)) == 7
    assert lib.ppo_model_create(None, C.byref(h)) == 1
    many = ppo.model_desc(64, 64, (16, 32), (3, 3), (64,), n_lstm=5, lstm_h=64)  # more layers than the descriptor holds
    assert lib.ppo_model_create(C.byref(many), C.byref(h)) == 1


def test_synth_is_seeded_and_shaped():
    w = synth.WORKLOADS["cfg1"].scaled(8, T=4)
    a, b = synth.rollout_numpy(w), synth.rollout_numpy(w)
    for k in a:
        assert np.array_equal(a[k], b[k])
    c = synth.rollout_numpy(w, seed=1)
    assert not np.array_equal(a["reward"], c["reward"])
    d = a["depth"]
    assert d.dtype == np.float16 and d.shape == (4, 8, 64, 64)
    nz = d[d > 0]
    assert 0.07 < np.mean(d == 0) < 0.13 and nz.min() >= 0.1 and nz.max() <= 2.0
    assert a["done"].dtype == np.uint8 and a["proprio"].shape == (4, 8, 32) and a["eps"].shape == (4, 8, 12)
