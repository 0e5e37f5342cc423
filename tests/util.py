"""Shared helpers of the GPU parity tests (metrics, layout conversion, oracle-side composition)."""
import numpy as np

# Tolerances of the parity bar: relative L2 for the fp32 path; relative L2 and max-abs on
# output pixels for the bf16 path (bf16 operands and storage, fp32 accumulation).
F32_REL_L2 = 1e-4
BF16_REL_L2 = 1e-2
BF16_MAX_ABS = 3e-2


def rel_l2(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))


def max_abs(got, ref) -> float:
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - np.asarray(ref, dtype=np.float64))))


def nchw_to_dev_nhwc(a: np.ndarray, dtype, device="cuda:0"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a.transpose(0, 2, 3, 1))).to(device=device, dtype=dtype).contiguous()


def dev_nhwc_to_nchw(t) -> np.ndarray:
    return t.float().permute(0, 3, 1, 2).contiguous().cpu().numpy()
