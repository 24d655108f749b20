"""Helpers shared by the GPU parity tests: numpy <-> device tensors and the parity metric."""
import numpy as np

from paper_2406_08128_b200 import inputs


def to_device(a: np.ndarray, dtype: str):
    """float32 numpy array (already rounded to ``dtype``) -> CUDA tensor of that storage dtype."""
    import torch
    if dtype == "bf16":
        bits = inputs.bf16_bits(a).astype(np.int16)
        return torch.from_numpy(bits).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def to_numpy(t) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |err| / RMS(reference output): the parity metric of the benchmark spec."""
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    return float(np.abs(got.astype(np.float64) - ref).max() / max(rms, 1e-300))
