"""Helpers for the GPU parity tests: torch is used for device memory only."""
import numpy as np
import torch


def dev(a: np.ndarray) -> torch.Tensor:
    """Copy a numpy array (float32 / complex64 / uint8 / float64) to the GPU."""
    if np.iscomplexobj(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.float32)).cuda()
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t: torch.Tensor, complex64: bool = False) -> np.ndarray:
    a = t.detach().cpu().numpy()
    return a.view(np.complex64) if complex64 else a


def normwise(a, b):
    """max |a - b| / max |b| (the error measure used for every sum in these tests)."""
    return float(np.abs(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64)).max()
                 / max(np.abs(np.asarray(b, dtype=np.float64)).max(), 1e-300))


def fp32_sequential_sum(rows: np.ndarray) -> np.ndarray:
    """rows[0] + rows[1] + ... in fp32, left to right (no fused or pairwise order)."""
    acc = np.zeros(rows.shape[1], dtype=np.float32)
    for r in rows:
        acc = (acc + r.astype(np.float32)).astype(np.float32)
    return acc
