"""GPU parity: peqa_train_step_host (forward, dX, dS of Eq. 2 and one AdamW step, host buffers in
and out) against the oracle, including token counts that split into several chunks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import adamw_scale_tol, assert_close, oracle_layer, to_qweight

pytestmark = pytest.mark.gpu


def _bf16_host(bits16, pin):
    t = torch.from_numpy(bits16.view(np.int16).copy()).view(torch.bfloat16)
    return t.pin_memory() if pin else t


def _f64(t):
    return t.view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("bits,g,T,pin", [(4, 0, 300, True), (3, 64, 1100, True), (3, 0, 2049, True),
                                          (4, 128, 700, False)])
def test_step_matches_oracle(bits, g, T, pin):
    N, K = 264, 384
    d = synth.custom(900 + bits + g + T, N, K, T, bits, g, outliers=True, sigma_dy=1e-2)
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    qw = to_qweight(packed, zeros, scales, bits, g, K)
    G = scales.shape[1]
    hX, hdY = _bf16_host(d["X"], pin), _bf16_host(d["dY"], pin)
    hY = torch.empty((T, N), dtype=torch.bfloat16)
    hdX = torch.empty((T, K), dtype=torch.bfloat16)
    hdS = torch.empty((N, G), dtype=torch.float32)
    if pin:
        hY, hdX, hdS = hY.pin_memory(), hdX.pin_memory(), hdS.pin_memory()
    dev = "cuda"
    dXin = torch.empty((T, K), dtype=torch.bfloat16, device=dev)
    ddY = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
    dY_ = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
    ddX = torch.empty((T, K), dtype=torch.bfloat16, device=dev)
    ddS = torch.empty((N, G), dtype=torch.float32, device=dev)
    m = torch.zeros((N, G), dtype=torch.float32, device=dev)
    v = torch.zeros((N, G), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(binding.OP_BWD, T, qw)
    lr = float(np.float32(1e-5))
    for step in (1, 2):      # the second call reuses the library's streams and events
        s_before = qw.scales.cpu().numpy().copy()
        m_before, v_before = m.cpu().numpy().copy(), v.cpu().numpy().copy()
        binding.train_step_host(qw, hX, hdY, hY, hdX, hdS, dXin, ddY, dY_, ddX, ddS, m, v, lr,
                                step=step, workspace=ws)
        binding.check_status()
        Y = synth.bf16_bits_to_f32(_f64(hY)).astype(np.float64)
        dX = synth.bf16_bits_to_f32(_f64(hdX)).astype(np.float64)
        assert_close(Y, oracle.fwd(d["X"], packed, zeros, s_before, bits, g), "Y")
        assert_close(dX, oracle.bwd_dx(d["dY"], packed, zeros, s_before, K, bits, g), "dX")
        dS = hdS.numpy().astype(np.float64)
        assert_close(dS, oracle.bwd_ds(d["X"], d["dY"], packed, zeros, bits, g), "dS")
        # AdamW acted on the dS that came back
        # the C ABI takes binary32 hyper-parameters: the oracle gets exactly those values
        so, mo, vo = oracle.adamw(s_before, hdS.numpy(), m_before, v_before, lr, float(np.float32(0.9)),
                                  float(np.float32(0.999)), float(np.float32(1e-8)), 0.0, step)
        got = qw.scales.cpu().numpy().astype(np.float64).ravel()
        assert np.all(np.abs(got - so) <= adamw_scale_tol(s_before, hdS.numpy(), m_before, v_before, lr,
                                                          float(np.float32(0.9)), float(np.float32(0.999)),
                                                          float(np.float32(1e-8)), 0.0, step))
