"""ctypes binding of libbimask.so: the same entry points as include/bimask.h, taking torch CUDA
tensors (or raw integer addresses) and doing argument marshalling only.  Every step of the path
runs in the library's kernels; if the library cannot be loaded the calls raise -- there is no
fallback of any kind."""
from __future__ import annotations

import ctypes
import os
from ctypes import c_float, c_int, c_int32, c_int64, c_size_t, c_uint64, c_void_p, c_char_p, POINTER, Structure

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# BIMASK_LIBRARY=debug loads the bounds-reporting build (libbimask_debug.so) instead
LIB_PATH = os.path.join(_HERE, "libbimask_debug.so" if os.environ.get("BIMASK_LIBRARY") == "debug" else "libbimask.so")

BIMASK_OK, BIMASK_EINVAL, BIMASK_EUNSUPPORTED, BIMASK_ECUDA, BIMASK_ETIMEOUT, BIMASK_EBOUNDS = 0, -1, -2, -3, -4, -5

EXPORTS = ("bimask_last_error", "bimask_launch_count", "bimask_hw_meta_bytes", "bimask_workspace_bytes", "bimask_fwd_mask",
           "bimask_perm_search", "bimask_bwd_mask", "bimask_spmm_fwd", "bimask_spmm_dgrad", "bimask_wgrad",
           "bimask_layer_step", "bimask_layer_step_host", "bimask_layer_step_host_async", "bimask_host_sync",
           "bimask_check_perms", "bimask_debug_wait_probe", "bimask_perm_search_static",
           "bimask_perm_search_static_max_entries", "bimask_sgd_fwd_mask", "bimask_train_step",
           "bimask_bwd_mask_criterion", "bimask_conv_workspace_bytes", "bimask_conv_layer_step",
           "bimask_refine_workspace_bytes", "bimask_perm_refine", "bimask_debug_gen_candidates", "bimask_debug_status")


class BimaskError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"bimask status {code}: {text}")
        self.code = code


class LayerArgs(Structure):
    """Mirror of bimask_layer_args."""
    _fields_ = [("T", c_int), ("I", c_int), ("J", c_int), ("N", c_int), ("M", c_int), ("P", c_int),
                ("seed", c_uint64), ("do_search", c_int),
                ("W", c_void_p), ("X", c_void_p), ("dY", c_void_p), ("cands", c_void_p),
                ("perm", c_void_p), ("best_idx", c_void_p), ("counts", c_void_p),
                ("maskbits_f", c_void_p), ("vals_f", c_void_p), ("meta_f", c_void_p), ("hw_meta_f", c_void_p),
                ("maskbits_b", c_void_p), ("vals_b", c_void_p), ("meta_b", c_void_p), ("hw_meta_b", c_void_p),
                ("Y", c_void_p), ("dX", c_void_p), ("dW", c_void_p),
                ("ws", c_void_p), ("ws_bytes", c_size_t), ("status_word", c_void_p), ("stream", c_void_p)]


class TrainArgs(Structure):
    """Mirror of bimask_train_args."""
    _fields_ = [("layer", LayerArgs), ("mom", c_void_p), ("lr", c_float), ("momentum", c_float),
                ("weight_decay", c_float), ("t", c_int64), ("delta_t", c_int32), ("premasked", c_int32)]


class ConvArgs(Structure):
    """Mirror of bimask_conv_args."""
    _fields_ = [("layer", LayerArgs), ("NB", c_int), ("H", c_int), ("W", c_int), ("C", c_int), ("mode", c_int),
                ("stride", c_int)]


CONV_AUTO, CONV_EXPLICIT, CONV_IMPLICIT = 0, 1, 2

_lib = None


def lib() -> ctypes.CDLL:
    """Load the library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2302_06058_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        L.bimask_last_error.restype = c_char_p
        L.bimask_launch_count.restype = c_uint64
        L.bimask_hw_meta_bytes.restype = c_size_t
        L.bimask_hw_meta_bytes.argtypes = [c_int, c_int]
        L.bimask_workspace_bytes.restype = c_size_t
        L.bimask_workspace_bytes.argtypes = [c_int, c_int, c_int, c_int]
        L.bimask_fwd_mask.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.bimask_perm_search.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_uint64, c_void_p,
                                         c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.bimask_bwd_mask.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_int,
                                      c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.bimask_spmm_fwd.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p]
        L.bimask_spmm_dgrad.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p,
                                        c_void_p, c_size_t, c_void_p, c_void_p]
        L.bimask_wgrad.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
        L.bimask_layer_step.argtypes = [POINTER(LayerArgs)]
        L.bimask_layer_step_host.argtypes = [POINTER(LayerArgs), POINTER(LayerArgs), c_void_p]
        L.bimask_layer_step_host_async.argtypes = [POINTER(LayerArgs), POINTER(LayerArgs), c_void_p]
        L.bimask_host_sync.argtypes = []
        L.bimask_refine_workspace_bytes.restype = c_size_t
        L.bimask_refine_workspace_bytes.argtypes = [c_int, c_int, c_int]
        L.bimask_perm_refine.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_uint64, c_void_p, c_void_p, c_void_p,
                                         c_size_t, c_void_p]
        L.bimask_conv_workspace_bytes.restype = c_size_t
        L.bimask_conv_workspace_bytes.argtypes = [c_int, c_int, c_int, c_int, c_int, c_int, c_int]
        L.bimask_conv_layer_step.argtypes = [POINTER(ConvArgs)]
        L.bimask_bwd_mask_criterion.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_int,
                                                c_uint64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.bimask_sgd_fwd_mask.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_float, c_float,
                                          c_float, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.bimask_train_step.argtypes = [POINTER(TrainArgs)]
        L.bimask_check_perms.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p, c_size_t, c_void_p]
        L.bimask_debug_wait_probe.argtypes = [c_void_p, c_void_p]
        L.bimask_debug_status.argtypes = [c_void_p]
        L.bimask_debug_gen_candidates.argtypes = [c_uint64, c_int, c_int, c_int, c_void_p, c_void_p]
        L.bimask_perm_search_static.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_uint64,
                                                c_void_p, c_void_p, c_void_p, c_void_p]
        L.bimask_perm_search_static_max_entries.restype = c_size_t
        for name in EXPORTS:
            if name not in ("bimask_last_error", "bimask_launch_count", "bimask_hw_meta_bytes", "bimask_workspace_bytes",
                            "bimask_perm_search_static_max_entries", "bimask_conv_workspace_bytes",
                            "bimask_refine_workspace_bytes"):
                getattr(L, name).restype = c_int
        _lib = L
    return _lib


def _ptr(x):
    """Address of a tensor's storage (device or pinned host), an int address, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, torch.Tensor):
        if not x.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return x.data_ptr()
    raise TypeError(type(x))


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream
    return int(stream)


def _check(rc: int) -> int:
    if rc < 0:
        raise BimaskError(rc, bimask_last_error())
    return rc


def bimask_last_error() -> str:
    return lib().bimask_last_error().decode()


def bimask_launch_count() -> int:
    return int(lib().bimask_launch_count())


def bimask_hw_meta_bytes(rows: int, K: int) -> int:
    return lib().bimask_hw_meta_bytes(rows, K)


def bimask_workspace_bytes(T: int, I: int, J: int, P: int) -> int:
    return lib().bimask_workspace_bytes(T, I, J, P)


def bimask_fwd_mask(W, I, J, N, M, maskbits_f, vals_f, meta_f, hw_meta_f, stream=None):
    return _check(lib().bimask_fwd_mask(_ptr(W), I, J, N, M, _ptr(maskbits_f), _ptr(vals_f), _ptr(meta_f),
                                        _ptr(hw_meta_f), _stream(stream)))


def bimask_perm_search(maskbits_f, I, J, N, M, P, seed, cands_or_null, best_perm, best_idx, counts, ws, ws_bytes,
                       stream=None):
    return _check(lib().bimask_perm_search(_ptr(maskbits_f), I, J, N, M, P, seed, _ptr(cands_or_null), _ptr(best_perm),
                                           _ptr(best_idx), _ptr(counts), _ptr(ws), ws_bytes, _stream(stream)))


def bimask_bwd_mask(W, maskbits_f, perm, I, J, N, M, maskbits_b, vals_b, meta_b, hw_meta_b, stream=None):
    return _check(lib().bimask_bwd_mask(_ptr(W), _ptr(maskbits_f), _ptr(perm), I, J, N, M, _ptr(maskbits_b),
                                        _ptr(vals_b), _ptr(meta_b), _ptr(hw_meta_b), _stream(stream)))


CRIT_WEIGHT, CRIT_SCORE, CRIT_MULTINOMIAL, CRIT_RANDOM = 0, 1, 2, 3


def bimask_refine_workspace_bytes(I, M, rounds) -> int:
    return lib().bimask_refine_workspace_bytes(I, M, rounds)


def bimask_perm_refine(maskbits_f, I, J, N, M, rounds, seed, perm_inout, count_out, ws, ws_bytes, stream=None):
    return _check(lib().bimask_perm_refine(_ptr(maskbits_f), I, J, N, M, rounds, seed, _ptr(perm_inout), _ptr(count_out),
                                           _ptr(ws), ws_bytes, _stream(stream)))


def bimask_bwd_mask_criterion(W, S_or_null, maskbits_f, perm, I, J, N, M, criterion, seed, maskbits_b, vals_b, meta_b,
                              hw_meta_b, stream=None):
    return _check(lib().bimask_bwd_mask_criterion(_ptr(W), _ptr(S_or_null), _ptr(maskbits_f), _ptr(perm), I, J, N, M,
                                                  criterion, seed, _ptr(maskbits_b), _ptr(vals_b), _ptr(meta_b),
                                                  _ptr(hw_meta_b), _stream(stream)))


def bimask_spmm_fwd(X, vals_f, hw_meta_f, T, I, J, Y, status_word, stream=None):
    return _check(lib().bimask_spmm_fwd(_ptr(X), _ptr(vals_f), _ptr(hw_meta_f), T, I, J, _ptr(Y), _ptr(status_word),
                                        _stream(stream)))


def bimask_spmm_dgrad(dY, perm, vals_b, hw_meta_b, T, I, J, dX, ws, ws_bytes, status_word, stream=None):
    return _check(lib().bimask_spmm_dgrad(_ptr(dY), _ptr(perm), _ptr(vals_b), _ptr(hw_meta_b), T, I, J, _ptr(dX),
                                          _ptr(ws), ws_bytes, _ptr(status_word), _stream(stream)))


def bimask_wgrad(dY, X, T, I, J, dW, ws, ws_bytes, status_word, stream=None):
    return _check(lib().bimask_wgrad(_ptr(dY), _ptr(X), T, I, J, _ptr(dW), _ptr(ws), ws_bytes, _ptr(status_word),
                                     _stream(stream)))


def make_layer_args(T, I, J, N, M, P, seed, do_search, bufs: dict, stream=None) -> LayerArgs:
    """Fill a bimask_layer_args from a dict of tensors keyed by field name (missing keys -> NULL)."""
    a = LayerArgs()
    a.T, a.I, a.J, a.N, a.M, a.P = T, I, J, N, M, P
    a.seed, a.do_search = seed, int(do_search)
    for name in ("W", "X", "dY", "cands", "perm", "best_idx", "counts", "maskbits_f", "vals_f", "meta_f", "hw_meta_f",
                 "maskbits_b", "vals_b", "meta_b", "hw_meta_b", "Y", "dX", "dW", "ws", "status_word"):
        setattr(a, name, _ptr(bufs.get(name)))
    ws = bufs.get("ws")
    a.ws_bytes = ws.numel() * ws.element_size() if isinstance(ws, torch.Tensor) else int(bufs.get("ws_bytes", 0))
    a.stream = _stream(stream)
    return a


def bimask_layer_step(args: LayerArgs):
    return _check(lib().bimask_layer_step(ctypes.byref(args)))


def bimask_sgd_fwd_mask(W, dW, mom_or_null, I, J, N, M, lr, momentum, weight_decay, maskbits_f, vals_f, meta_f, hw_meta_f,
                        stream=None):
    return _check(lib().bimask_sgd_fwd_mask(_ptr(W), _ptr(dW), _ptr(mom_or_null), I, J, N, M, lr, momentum, weight_decay,
                                            _ptr(maskbits_f), _ptr(vals_f), _ptr(meta_f), _ptr(hw_meta_f),
                                            _stream(stream)))


def bimask_conv_workspace_bytes(NB, H, W, C, I, P, stride=1) -> int:
    return lib().bimask_conv_workspace_bytes(NB, H, W, C, I, P, stride)


def make_conv_args(layer: LayerArgs, NB, H, W, C, mode=CONV_AUTO, stride=1) -> ConvArgs:
    a = ConvArgs()
    ctypes.memmove(ctypes.byref(a.layer), ctypes.byref(layer), ctypes.sizeof(LayerArgs))
    a.NB, a.H, a.W, a.C, a.mode, a.stride = NB, H, W, C, mode, stride
    return a


def bimask_conv_layer_step(args: ConvArgs):
    return _check(lib().bimask_conv_layer_step(ctypes.byref(args)))


def make_train_args(layer: LayerArgs, mom, lr, momentum, weight_decay, t, delta_t, premasked) -> TrainArgs:
    a = TrainArgs()
    ctypes.memmove(ctypes.byref(a.layer), ctypes.byref(layer), ctypes.sizeof(LayerArgs))
    a.mom = _ptr(mom)
    a.lr, a.momentum, a.weight_decay = lr, momentum, weight_decay
    a.t, a.delta_t, a.premasked = t, delta_t, int(bool(premasked))
    return a


def bimask_train_step(args: TrainArgs):
    return _check(lib().bimask_train_step(ctypes.byref(args)))


def bimask_layer_step_host(dev: LayerArgs, host: LayerArgs, host_status_word=None):
    return _check(lib().bimask_layer_step_host(ctypes.byref(dev), ctypes.byref(host), _ptr(host_status_word)))


def bimask_layer_step_host_async(dev: LayerArgs, host: LayerArgs, host_status_word=None):
    return _check(lib().bimask_layer_step_host_async(ctypes.byref(dev), ctypes.byref(host), _ptr(host_status_word)))


def bimask_host_sync():
    return _check(lib().bimask_host_sync())


def bimask_debug_wait_probe(status_word, stream=None):
    return _check(lib().bimask_debug_wait_probe(_ptr(status_word), _stream(stream)))


def bimask_debug_status():
    """[code, site, index, bound] of the first out-of-range row index the debug build's kernels met (all zero when
    none); raises BimaskError(BIMASK_EUNSUPPORTED) on the release build."""
    out = (c_int32 * 4)()
    _check(lib().bimask_debug_status(ctypes.cast(out, c_void_p)))
    return [int(v) for v in out]


def bimask_debug_gen_candidates(seed, P, I, part_cap, cands, stream=None):
    return _check(lib().bimask_debug_gen_candidates(seed, P, I, part_cap, _ptr(cands), _stream(stream)))


def bimask_check_perms(cands, P, I, ok, ws, ws_bytes, stream=None):
    return _check(lib().bimask_check_perms(_ptr(cands), P, I, _ptr(ok), _ptr(ws), ws_bytes, _stream(stream)))


def bimask_perm_search_static(maskbits_f, I, J, N, M, P, seed, best_perm, best_idx, counts, stream=None):
    """Permutation search without a workspace: the candidates live in the library's built-in
    8 MiB device array (P * I <= bimask_perm_search_static_max_entries()).  Allocates nothing."""
    return _check(lib().bimask_perm_search_static(_ptr(maskbits_f), I, J, N, M, P, seed, _ptr(best_perm),
                                                  _ptr(best_idx), _ptr(counts), _stream(stream)))


def bimask_perm_search_static_max_entries() -> int:
    return int(lib().bimask_perm_search_static_max_entries())


def alloc_layer_buffers(T, I, J, P, device="cuda", dense=False) -> dict:
    """Device buffers for every output of a layer step plus scratch (torch is the allocator).
    dense: size vals_f / vals_b for the dense masked operands of a pattern that does not fit the
    2:4 container (I*J bf16 each instead of half that)."""
    d = torch.device(device)
    b = {
        "perm": torch.arange(I, dtype=torch.int32, device=d),
        "best_idx": torch.zeros(1, dtype=torch.int32, device=d),
        "counts": torch.zeros(max(P, 1), dtype=torch.int64, device=d),
        "maskbits_f": torch.empty(I, J // 32, dtype=torch.int32, device=d),
        "vals_f": torch.empty(I, J if dense else J // 2, dtype=torch.bfloat16, device=d),
        "meta_f": torch.empty(I, J // 32, dtype=torch.int32, device=d),
        "hw_meta_f": torch.empty(bimask_hw_meta_bytes(I, J), dtype=torch.uint8, device=d),
        "maskbits_b": torch.empty(I, J // 32, dtype=torch.int32, device=d),
        "vals_b": torch.empty(J, I if dense else I // 2, dtype=torch.bfloat16, device=d),
        "meta_b": torch.empty(J, I // 32, dtype=torch.int32, device=d),
        "hw_meta_b": torch.empty(bimask_hw_meta_bytes(J, I), dtype=torch.uint8, device=d),
        "Y": torch.empty(T, I, dtype=torch.bfloat16, device=d),
        "dX": torch.empty(T, J, dtype=torch.bfloat16, device=d),
        "dW": torch.empty(I, J, dtype=torch.float32, device=d),
        "ws": torch.empty(bimask_workspace_bytes(T, I, J, P), dtype=torch.uint8, device=d),
        "status_word": torch.zeros(1, dtype=torch.int32, device=d),
    }
    return b
