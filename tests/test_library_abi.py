"""Host-side checks: the shared library builds, exports every declared symbol, and rejects
bad arguments before touching the GPU."""
import ctypes
import os
import re

import pytest

from paper_2305_14152_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "peqa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(peqa_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared()
    assert "peqa_qlinear_fwd" in names and "peqa_scale_adamw" in names and len(names) >= 12
    for n in names:
        assert hasattr(L, n), n


def test_version(L):
    assert L.peqa_version() >= 100


def test_argument_validation_needs_no_gpu(L):
    buf = ctypes.create_string_buffer(4096)
    p = ctypes.addressof(buf)
    p16 = (p + 15) & ~15
    assert L.peqa_quantize_rtn(0, 4, 64, 4, 0, p16, p16, p16, 0) == -1
    assert L.peqa_quantize_rtn(p16, 4, 64, 5, 0, p16, p16, p16, 0) == -2
    assert L.peqa_quantize_rtn(p16, 4, 48, 4, 0, p16, p16, p16, 0) == -3
    assert L.peqa_quantize_rtn(p16, 4, 64, 4, 24, p16, p16, p16, 0) == -3
    assert L.peqa_quantize_rtn(p16, 0, 64, 4, 0, p16, p16, p16, 0) == -3
    assert L.peqa_quantize_rtn(p16 + 4, 4, 64, 4, 0, p16, p16, p16, 0) == -4
    assert L.peqa_quantize_rtn(p16, 4, 1 << 17, 4, 0, p16, p16, p16, 0) == -9
    assert L.peqa_pack(0, 1, 32, 4, p16, 0) == -1
    assert L.peqa_unpack(p16, 1, 32, 2, p16, 0) == -2
    assert L.peqa_scale_adamw(p16, p16, p16, 0, 4, 1e-3, 0.9, 0.999, 1e-8, 0.0, 1, 0) == -1
    assert L.peqa_scale_adamw(p16, p16, p16, p16, 4, 1e-3, 0.9, 0.999, 1e-8, 0.0, 0, 0) == -3
    w = binding._QWeight(4, 128, 256, 0, p16, p16, p16)
    assert L.peqa_qlinear_fwd(ctypes.byref(w), 0, 8, p16, 0, 0, 0) == -1
    assert L.peqa_qlinear_fwd(ctypes.byref(w), p16, 0, p16, 0, 0, 0) == -3
    w2 = binding._QWeight(4, 128, 96, 0, p16, p16, p16)
    assert L.peqa_qlinear_fwd(ctypes.byref(w2), p16, 8, p16, 0, 0, 0) == -3      # K % 64
    w3 = binding._QWeight(4, 100, 256, 0, p16, p16, p16)
    assert L.peqa_qlinear_fwd(ctypes.byref(w3), p16, 8, p16, 0, 0, 0) == -3      # N % 8
    assert L.peqa_qlinear_decode(ctypes.byref(w), p16, 17, p16, 0, 0, 0) == -3
    assert L.peqa_qlinear_bwd(ctypes.byref(w), p16, 0, 8, p16, 0, 0, 0, 0) == -1
    # the entry points beyond the basic five: null pointers, shapes and modes they do not take
    wg = binding._QWeight(4, 128, 256, 128, p16, p16, p16)           # two groups per row
    assert L.peqa_qlinear_bwd_ds_from_y(ctypes.byref(w), p16, 0, 8, p16, p16, 4096, 0) == -1
    assert L.peqa_qlinear_bwd_ds_from_y(ctypes.byref(wg), p16, p16, 8, p16, p16, 4096, 0) == -3
    assert L.peqa_qlinear_bwd_ds_from_y(ctypes.byref(w), p16, p16, 0, p16, p16, 4096, 0) == -3
    assert L.peqa_qlinear_bwd_dsdz(ctypes.byref(w), p16, p16, 8, p16, 0, 0, 0, 0) == -1
    assert L.peqa_qlinear_bwd_dsdz(ctypes.byref(w2), p16, p16, 8, p16, p16, 0, 0, 0) == -3
    assert L.peqa_qlinear_bwd_ds_adamw(ctypes.byref(w), p16, p16, 8, p16, p16, 0, 1e-3, 0.9, 0.999,
                                       1e-8, 0.0, 1, 0, 0, 0) == -1
    assert L.peqa_qlinear_bwd_ds_adamw(ctypes.byref(w), p16, p16, 8, p16, p16, p16, 1e-3, 0.9, 0.999,
                                       1e-8, 0.0, 0, 0, 0, 0) == -3             # step counts from 1
    assert L.peqa_qlinear_decode_multitask(ctypes.byref(w), p16, 2, 0, p16, 1, p16, 0) == -1
    assert L.peqa_qlinear_decode_multitask(ctypes.byref(wg), p16, 2, p16, p16, 1, p16, 0) == -3
    assert L.peqa_qlinear_decode_multitask(ctypes.byref(w), p16, 0, p16, p16, 1, p16, 0) == -3
    assert L.peqa_qlinear_decode_multitask(ctypes.byref(w), p16, 2, p16, p16, 17, p16, 0) == -3
    # the host-buffer layer step: null list, empty list, a linear without host buffers, and two
    # linears whose device staging buffers overlap
    f = (1e-3, 0.9, 0.999, 1e-8, 0.0)
    assert L.peqa_layer_train_step_host(None, 1, 8, *f, 1, 0) == -1
    one = (binding._LayerHostLinear * 1)()
    assert L.peqa_layer_train_step_host(one, 0, 8, *f, 1, 0) == -3
    one[0].w = w
    assert L.peqa_layer_train_step_host(one, 1, 8, *f, 1, 0) == -1
    big = ctypes.create_string_buffer(1 << 16)
    q = (ctypes.addressof(big) + 255) & ~255
    two = (binding._LayerHostLinear * 2)()
    for i in range(2):
        two[i].w = w
        two[i].workspace, two[i].workspace_bytes = q + 40960, 8192
        for name in ("h_X", "h_dY", "h_Y", "h_dX", "h_dS", "d_dS", "d_m", "d_v"):
            setattr(two[i], name, q)
        # T = 8 tokens: X, dX take 8*256*2 = 4096 bytes, dY, Y 8*128*2 = 2048 bytes
        two[i].d_X, two[i].d_dX, two[i].d_dY, two[i].d_Y = (q + i * 16384, q + i * 16384 + 4096,
                                                             q + i * 16384 + 8192, q + i * 16384 + 10240)
    two[1].d_dY = two[0].d_X + 4080                                  # 16 bytes into linear 0's d_X
    assert L.peqa_layer_train_step_host(two, 2, 8, *f, 1, 0) == -3


def test_workspace_query(L):
    w = binding._QWeight(4, 4096, 4096, 0, 16, 16, 16)
    assert L.peqa_workspace_bytes(binding.OP_BWD, 2048, ctypes.byref(w)) == 4096 * (4096 // 128) * 4
    w = binding._QWeight(3, 4096, 4096, 128, 16, 16, 16)
    assert L.peqa_workspace_bytes(binding.OP_BWD, 2048, ctypes.byref(w)) == 0
    assert L.peqa_workspace_bytes(binding.OP_FWD, 2048, ctypes.byref(w)) == 0
    assert L.peqa_workspace_bytes(binding.OP_BWD_DSDZ, 2048, ctypes.byref(w)) == 0
    assert L.peqa_workspace_bytes(binding.OP_BWD_DS_FROM_Y, 2048, ctypes.byref(w)) == 0   # grouped: not served
    w = binding._QWeight(4, 4096, 4096, 0, 16, 16, 16)
    assert L.peqa_workspace_bytes(binding.OP_BWD_DSDZ, 2048, ctypes.byref(w)) == 2 * 4096 * (4096 // 128) * 4
    n = L.peqa_workspace_bytes(binding.OP_BWD_DS_FROM_Y, 2048, ctypes.byref(w))
    assert n > 0 and n % (4096 * 4) == 0
