"""Helpers shared by the GPU parity tests: buffer conversion and the error metrics."""
import numpy as np
import torch

import oracle
from paper_2305_14152_b200 import binding

REL_L2_TOL = 5e-3       # per output tensor
MAX_ABS_TOL = 1e-2      # times max|ref|


def bf16_to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def dev_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def u32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint32)


def assert_close(got: np.ndarray, ref: np.ndarray, what: str):
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.all(np.isfinite(got)), what
    denom = np.linalg.norm(ref.ravel())
    rel = np.linalg.norm((got - ref).ravel()) / max(denom, 1e-300)
    mx = np.abs(got - ref).max()
    assert rel <= REL_L2_TOL, f"{what}: rel-L2 {rel:.3e} > {REL_L2_TOL}"
    assert mx <= MAX_ABS_TOL * np.abs(ref).max(), f"{what}: max-abs {mx:.3e} vs max|ref| {np.abs(ref).max():.3e}"
    return rel, mx


def oracle_layer(d, bits, g):
    """Quantize with the oracle; returns (codes, zeros, scales, packed)."""
    codes, zeros, scales = oracle.quantize_rtn(d["W"], bits, g)
    return codes, zeros, scales, oracle.pack(codes, bits)


def to_qweight(packed, zeros, scales, bits, g, K) -> binding.QWeight:
    N = packed.shape[0]
    q = torch.from_numpy(packed.view(np.int32)).cuda()
    z = torch.from_numpy(np.ascontiguousarray(zeros)).cuda()
    s = torch.from_numpy(np.ascontiguousarray(scales)).cuda()
    return binding.QWeight(bits, N, K, g, q, z, s)
