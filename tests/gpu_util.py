"""Helpers of the GPU parity tests: host <-> device movement and bit views."""
import numpy as np
import torch


def to_dev(x, dtype):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if t.dtype == torch.float32 and dtype == "bf16":
        t = t.to(torch.bfloat16)
    return t.cuda()


def to_host_f32(t):
    return t.detach().to(torch.float32).cpu().numpy()


def bits_host(t):
    """uint32 / uint16 bit patterns of a float32 / bf16 device tensor."""
    if t.dtype == torch.bfloat16:
        return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)
    return t.detach().view(torch.int32).cpu().numpy().view(np.uint32)


def u32(t):
    return t.detach().cpu().numpy().view(np.uint32)


def rel_err(g, ref):
    """(Frobenius relative error, max-abs relative error) of g against ref."""
    g = np.asarray(g, np.float64)
    ref = np.asarray(ref, np.float64)
    fro = np.linalg.norm(g - ref) / max(np.linalg.norm(ref), 1e-300)
    mx = np.abs(g - ref).max() / max(np.abs(ref).max(), 1e-300)
    return fro, mx


TOL = {"f32": 1e-5, "bf16": 2e-2}
