"""Shared helpers of the GPU parity tests: tolerances and error measures."""
import numpy as np
import torch

# Tolerances stated by the benchmark spec: bf16 inputs, fp32 accumulation.
# The bound on O is element-wise: |dO| <= 1e-2 wherever |O_ref| <= 1 and 1e-2 * |O_ref| for the
# larger elements (the output is rounded to bf16, whose half-ulp is 2^-9 relative: 0.0156 for an
# element of magnitude 4, which an absolute 1e-2 could not admit).  No element borrows slack from
# another: a small output next to a large one is still held to 1e-2.
TOL_O_MAXABS = 1e-2
TOL_LSE_ABS = 1e-3
TOL_O_REL_L2 = 1e-2     # per (row set, head): guards against a kernel that ignores keys when |O| is tiny


def to_dev_ids(ids: np.ndarray, dev) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(ids).view(np.int32)).to(dev)


def check_attention(O_gpu, LSE_gpu, O_ref, LSE_ref, what=""):
    """O_gpu bf16/f32 tensor [n,H,d], O_ref float64 ndarray, same for LSE [n,H]."""
    o = O_gpu.float().cpu().numpy().astype(np.float64)
    err = np.abs(o - O_ref)
    max_abs = err.max()
    num = np.sqrt((err ** 2).sum(axis=(0, 2)))
    den = np.sqrt((O_ref ** 2).sum(axis=(0, 2))) + 1e-30
    rel = (num / den).max()
    msg = f"{what}: max|dO|={max_abs:.3e} relL2={rel:.3e}"
    if LSE_gpu is not None:
        le = np.abs(LSE_gpu.cpu().numpy().astype(np.float64) - LSE_ref).max()
        msg += f" max|dLSE|={le:.3e}"
        assert le <= TOL_LSE_ABS, msg
    assert np.isfinite(o).all(), msg + " (non-finite output)"
    bound = TOL_O_MAXABS * np.maximum(1.0, np.abs(O_ref))
    worst = float((err / bound).max())
    assert worst <= 1.0, msg + f" (worst element at {worst:.2f} of its bound)"
    assert rel <= TOL_O_REL_L2, msg
    return msg
