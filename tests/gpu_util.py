"""Helpers shared by the GPU parity tests (test code only)."""
import numpy as np
import torch

DEV = "cuda:0"


def dbf16(a):
    """numpy uint16 bf16 bit patterns -> device bf16 tensor"""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(DEV).view(torch.bfloat16)


def bits16(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bits8(t):
    return t.contiguous().view(torch.uint8).cpu().numpy()


def rel_fro(a, ref):
    a = np.asarray(a, np.float64)
    return float(np.linalg.norm(a - ref) / max(np.linalg.norm(ref), 1e-300))


def canonical_meta(ctx, meta, rows, k, dt):
    out = torch.empty((rows, k // 16), dtype=torch.int16, device=DEV)
    ctx.meta_to_canonical(meta, rows, k, dt, out)
    return out.cpu().numpy().view(np.uint16)
