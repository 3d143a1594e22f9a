"""Helpers shared by the GPU parity tests: run library calls on seeded inputs and fetch results."""
import numpy as np
import torch

import paper_2302_06058_b200 as bm


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.cuda()


def bits_dev(a_u16):
    """uint16 bf16 bit patterns -> CUDA bf16 tensor."""
    return torch.from_numpy(np.ascontiguousarray(a_u16).view(np.int16)).cuda().view(torch.bfloat16)


def u32(t):
    return t.cpu().numpy().view(np.uint32)


def u16(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def rel_err(got, ref):
    """max |got - ref| / max(|ref|, rms(ref)): element-wise relative error with an rms floor."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref))) or 1.0
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), rms)))


def run_fwd_mask(W, N, M=4):
    I, J = W.shape
    b = bm.alloc_layer_buffers(1, I, J, 1)
    Wd = dev(W)
    bm.bimask_fwd_mask(Wd, I, J, N, M, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
    torch.cuda.synchronize()
    return Wd, b


def run_layer_step(W, X, dY, N, M, P, seed, do_search=True, perm=None, cands=None):
    I, J = W.shape
    T = X.shape[0]
    b = bm.alloc_layer_buffers(T, I, J, P)
    b["W"], b["X"], b["dY"] = dev(W), bits_dev(X), bits_dev(dY)
    if perm is not None:
        b["perm"] = dev(np.asarray(perm, dtype=np.int32))
    if cands is not None:
        b["cands"] = dev(np.asarray(cands, dtype=np.int32))
    args = bm.make_layer_args(T, I, J, N, M, P, seed, do_search, b)
    bm.bimask_layer_step(args)
    torch.cuda.synchronize()
    return b
