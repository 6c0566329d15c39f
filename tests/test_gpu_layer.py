"""GPU parity: peqa_layer_train_step, one call for several linears (forward, dX, dS of Eq. 2 and
App. A's AdamW step on the scales), against the oracle and against the single calls."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, dp, synth
from gpu_util import adamw_scale_tol, assert_close, bf16_to_dev, dev_to_f64, oracle_layer, to_qweight

pytestmark = pytest.mark.gpu

SHAPES = [(264, 384, 3, 64), (384, 264 + 56, 4, 0), (128, 384, 3, 128), (392, 128, 4, 32)]   # N, K, bits, g
LR = float(np.float32(1e-3))


def _build(T, with_state=True, bucket=None):
    layers, host = [], []
    ds_shapes = []
    for i, (N, K, bits, g) in enumerate(SHAPES):
        d = synth.custom(300 + i, N, K, T, bits, g, outliers=True, sigma_dy=1e-2)
        codes, zeros, scales, packed = oracle_layer(d, bits, g)
        host.append((d, zeros, scales, packed, bits, g))
        ds_shapes.append(scales.shape)
    views = None
    if bucket:
        flat, views = dp.bucket_views([torch.empty(s, device="cuda") for s in ds_shapes])
    for i, (d, zeros, scales, packed, bits, g) in enumerate(host):
        N, K = d["W"].shape
        qw = to_qweight(packed, zeros, scales, bits, g, K)
        G = scales.shape[1]
        L = binding.LayerLinear(
            w=qw, X=bf16_to_dev(d["X"]), dY=bf16_to_dev(d["dY"]),
            Y=torch.empty((T, N), dtype=torch.bfloat16, device="cuda"),
            dX=torch.empty((T, K), dtype=torch.bfloat16, device="cuda"),
            dS=views[i] if views else torch.empty((N, G), dtype=torch.float32, device="cuda"),
            m=torch.zeros((N, G), dtype=torch.float32, device="cuda") if with_state else None,
            v=torch.zeros((N, G), dtype=torch.float32, device="cuda") if with_state else None,
            workspace=binding.alloc_workspace(binding.OP_BWD, T, qw))
        layers.append(L)
    return layers, host


@pytest.mark.parametrize("T", [300, 1024])
def test_layer_step_matches_oracle_and_single_calls(T):
    layers, host = _build(T)
    ref_layers, _ = _build(T)
    binding.layer_train_step(layers, LR, step=1)
    binding.check_status()
    for L, R, (d, zeros, scales, packed, bits, g) in zip(layers, ref_layers, host):
        K = d["W"].shape[1]
        assert_close(dev_to_f64(L.Y), oracle.fwd(d["X"], packed, zeros, scales, bits, g), "Y")
        assert_close(dev_to_f64(L.dX), oracle.bwd_dx(d["dY"], packed, zeros, scales, K, bits, g), "dX")
        ds_ref = oracle.bwd_ds(d["X"], d["dY"], packed, zeros, bits, g)
        assert_close(dev_to_f64(L.dS), ds_ref, "dS")
        # the optimizer step, from the dS the kernel produced
        ds_gpu = L.dS.cpu().numpy()
        zero = np.zeros_like(scales)
        s_ref, m_ref, v_ref = oracle.adamw(scales, ds_gpu, zero, zero, LR, float(np.float32(0.9)),
                                           float(np.float32(0.999)), float(np.float32(1e-8)), 0.0, 1)
        tol = adamw_scale_tol(scales, ds_gpu, zero, zero, LR, 0.9, 0.999, 1e-8, 0.0, 1)
        assert np.all(np.abs(L.w.scales.cpu().numpy().ravel().astype(np.float64) - s_ref) <= tol)
        # bit-identical to the single calls
        Y = binding.qlinear_fwd(R.w, R.X)
        dX, _ = binding.qlinear_bwd(R.w, R.X, R.dY, need_ds=False)
        dS = binding.qlinear_bwd_ds_adamw(R.w, R.X, R.dY, R.m, R.v, LR, step=1, workspace=R.workspace)
        torch.cuda.synchronize()
        assert torch.equal(Y, L.Y) and torch.equal(dX, L.dX) and torch.equal(dS, L.dS)
        assert torch.equal(R.w.scales, L.w.scales) and torch.equal(R.m, L.m) and torch.equal(R.v, L.v)


def test_gradients_only_into_a_bucket_then_optimizer():
    """apply_adamw = 0 leaves the scales alone; dS lands in views of one flat bucket (what a
    data-parallel step all-reduces), and the AdamW call afterwards gives the fused result."""
    T = 512
    layers, host = _build(T, bucket=True)
    fused, _ = _build(T)
    before = [L.w.scales.clone() for L in layers]
    dp.layer_train_step_dp(layers, LR, step=1)          # no process group: the all-reduce is the identity
    binding.layer_train_step(fused, LR, step=1)
    binding.check_status()
    for L, F, b in zip(layers, fused, before):
        assert not torch.equal(L.w.scales, b)
        assert torch.equal(L.dS, F.dS) and torch.equal(L.w.scales, F.w.scales)
        assert torch.equal(L.m, F.m) and torch.equal(L.v, F.v)
    # and without optimizer state at all
    plain, _ = _build(T, with_state=False)
    binding.layer_train_step(plain, apply_adamw=False)
    binding.check_status()
    for L, F, b in zip(plain, fused, before):
        assert torch.equal(L.w.scales, b) and torch.equal(L.dS, F.dS)


def test_arguments_are_checked_before_anything_runs():
    layers, _ = _build(64)
    sentinel = layers[0].Y.fill_(3.0).clone()
    layers[2].workspace = None if layers[2].workspace is None else layers[2].workspace
    bad = layers[3]
    bad.m = None
    with pytest.raises(binding.PeqaError):
        binding.layer_train_step(layers, LR, step=1)
    torch.cuda.synchronize()
    assert torch.equal(layers[0].Y, sentinel)           # the first linear did not run either
    with pytest.raises(binding.PeqaError):
        binding.layer_train_step(layers[:3], LR, step=0)


def _host_linears(layers, T, shared_staging=False):
    out = []
    stage = None
    for L in layers:
        N, K, G = L.w.N, L.w.K, L.w.G
        pin = lambda t: t.cpu().pin_memory()
        if shared_staging and stage is not None:
            d_X = stage                                   # the first linear's buffer again
        else:
            d_X = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
            stage = stage if stage is not None else d_X
        out.append(binding.HostLinear(
            w=L.w, h_X=pin(L.X), h_dY=pin(L.dY),
            h_Y=torch.empty((T, N), dtype=torch.bfloat16).pin_memory(),
            h_dX=torch.empty((T, K), dtype=torch.bfloat16).pin_memory(),
            h_dS=torch.empty((N, G), dtype=torch.float32).pin_memory(),
            d_X=d_X, d_dY=torch.empty((T, N), dtype=torch.bfloat16, device="cuda"),
            d_Y=torch.empty((T, N), dtype=torch.bfloat16, device="cuda"),
            d_dX=torch.empty((T, K), dtype=torch.bfloat16, device="cuda"),
            d_dS=torch.empty((N, G), dtype=torch.float32, device="cuda"),
            d_m=L.m, d_v=L.v, workspace=L.workspace))
    return out


@pytest.mark.parametrize("T", [300, 1100])
def test_layer_step_with_host_buffers(T):
    """peqa_layer_train_step_host: every linear's Y, dX, dS come back to the host and its scales
    take the AdamW step, bit-identical to the device-buffer layer call (chunking the tokens
    changes neither the forward nor dX; dS runs once over all tokens)."""
    layers, host = _build(T)
    ref, _ = _build(T)
    hl = _host_linears(layers, T)
    binding.layer_train_step_host(hl, LR, step=1)
    binding.check_status()
    binding.layer_train_step(ref, LR, step=1)
    torch.cuda.synchronize()
    for H, R, (d, zeros, scales, packed, bits, g) in zip(hl, ref, host):
        assert torch.equal(H.h_Y, R.Y.cpu()) and torch.equal(H.h_dX, R.dX.cpu())
        assert torch.equal(H.h_dS, R.dS.cpu())
        assert torch.equal(H.w.scales, R.w.scales) and torch.equal(H.d_m, R.m) and torch.equal(H.d_v, R.v)
        assert_close(H.h_Y.double().numpy(), oracle.fwd(d["X"], packed, zeros, scales, bits, g), "Y")


def test_layer_host_step_rejects_shared_staging_buffers():
    """The copies of a linear run ahead of the kernels of the one before: staging buffers that
    overlap between linears are refused before anything is enqueued."""
    T = 64
    layers, _ = _build(T)
    layers = [layers[0], layers[2]]                       # both K = 384: the same d_X size
    hl = _host_linears(layers, T, shared_staging=True)
    before = [L.w.scales.clone() for L in layers]
    with pytest.raises(binding.PeqaError):
        binding.layer_train_step_host(hl, LR, step=1)
    torch.cuda.synchronize()
    for L, b in zip(layers, before):
        assert torch.equal(L.w.scales, b)
