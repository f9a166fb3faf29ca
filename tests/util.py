"""Helpers shared by the tests (no method arithmetic)."""
import numpy as np
import torch


def to_np(t: torch.Tensor) -> np.ndarray:
    """torch tensor -> numpy; bf16 becomes its uint16 bit pattern."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def as_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def mask_to_dense(keep_mask: np.ndarray, E: int) -> np.ndarray:
    """[N, W] uint64 words -> [N, E] 0/1."""
    N, W = keep_mask.shape
    out = np.zeros((N, E), np.uint8)
    for e in range(E):
        out[:, e] = ((keep_mask[:, e >> 6] >> np.uint64(e & 63)) & np.uint64(1)).astype(np.uint8)
    return out


def rel_err(a: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.max(np.abs(ref)))
    return float(np.max(np.abs(a - ref))) / (den if den > 0 else 1.0)
