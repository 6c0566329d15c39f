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


def adamw_scale_tol(s_old, grad, m_old, v_old, lr, b1, b2, eps, wd, step):
    """Bound on |s_kernel - s_oracle| for one AdamW step evaluated in binary32 (the oracle works
    in binary64 on the same binary32 inputs).  With h = 2^-24 (half an ulp, the relative error of
    one rounded operation):
      * the update u = lr * (m'/c1) / (sqrt(v'/c2) + eps) goes through twelve roundings -- the
        constants 1-b1 and 1/c1 (2), the two products and the fused multiply-add that form m'
        and its bias correction (4), and the denominator chain 1-b2, 1/c2, three operations for
        v', one product, halved by the square root (3), the root itself, + eps and the division
        (3).  The errors of m' scale with the sizes of its two terms, which may cancel, so the
        bound uses U = lr * (b1|m| + (1-b1)|g|) / c1 / (sqrt(v'/c2) + eps) rather than |u|;
        16 h U leaves a third of slack over the linear count;
      * s' = s * (1 - lr*wd) - u rounds the decay constant, the product and the difference:
        3 h |s|.
    """
    h = 2.0 ** -24
    s_old, grad, m_old, v_old = (np.asarray(a, dtype=np.float64).ravel() for a in (s_old, grad, m_old, v_old))
    c1, c2 = 1.0 - b1 ** step, 1.0 - b2 ** step
    v_new = b2 * v_old + (1.0 - b2) * grad * grad
    U = lr * (b1 * np.abs(m_old) + (1.0 - b1) * np.abs(grad)) / c1 / (np.sqrt(v_new / c2) + eps)
    return 16 * h * U + 3 * h * np.abs(s_old) + 1e-45
