"""Device-side fills (workloads/fill.cu): the same tensors as rng.py, produced on the GPU."""
import ctypes as C
import os
import subprocess

import torch

from .rng import stream_key, NORMAL_SCALE_F32

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fill.cu")
_SO = os.path.join(_HERE, "libcbfill.so")
_lib = None


def build(force=False):
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-shared",
                               "-Xcompiler", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.wl_fill_normal.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_float, C.c_int, C.c_void_p]
        _lib.wl_fill_normal.restype = C.c_int
        _lib.wl_stream_targets.argtypes = [C.c_void_p, C.c_longlong, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                           C.c_int32, C.c_void_p, C.c_void_p]
        _lib.wl_stream_targets.restype = C.c_int
        _lib.wl_plant_logits.argtypes = [C.c_void_p, C.c_longlong, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p,
                                         C.c_int, C.c_void_p]
        _lib.wl_plant_logits.restype = C.c_int
    return _lib


def fill_normal(t: torch.Tensor, seed: int, tid: int):
    """In-place: t.flatten()[i] = normal(seed, tid, i); t is a contiguous CUDA tensor, bf16 or float32."""
    assert t.is_cuda and t.is_contiguous() and t.dtype in (torch.bfloat16, torch.float32)
    rc = _load().wl_fill_normal(t.data_ptr(), t.numel(), stream_key(seed, tid), float(NORMAL_SCALE_F32),
                                int(t.dtype == torch.bfloat16), torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise RuntimeError("wl_fill_normal failed with CUDA error %d" % rc)
    return t


def normal_tensor(shape, dtype, seed, tid, device="cuda:0"):
    return fill_normal(torch.empty(shape, dtype=dtype, device=device), seed, tid)


def stream_targets(tokens: torch.Tensor, seq_len: torch.Tensor, tree: dict, junk_base: int, out: torch.Tensor):
    """Closed-loop stand-in for the target model (input generation): out[b, i] = the token of the stream `tokens[b]` that follows
    node i's path if that path equals the stream's continuation after position seq_len[b] - 1 (the tree's root), else
    junk_base + i.  All int32 CUDA tensors; tree = dict(tokens, parent, depth, n_nodes) as cb_draft_tree writes it."""
    B, T = tree["tokens"].shape
    rc = _load().wl_stream_targets(tokens.data_ptr(), tokens.stride(0), seq_len.data_ptr(), tree["tokens"].data_ptr(), tree["parent"].data_ptr(),
                                   tree["depth"].data_ptr(), tree["n_nodes"].data_ptr(), B, T, junk_base, out.data_ptr(),
                                   torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise RuntimeError("wl_stream_targets failed with CUDA error %d" % rc)
    return out


def plant_logits(logits: torch.Tensor, target: torch.Tensor, n_nodes: torch.Tensor, saved: torch.Tensor, restore: bool = False, value: float = 32.0):
    """Closed-loop stand-in for an LM head (input generation): fp32 logits [B, T, V] get `value` at column target[b, i] of every
    valid row whose target is a vocabulary id, the entries they replace are kept in saved [B, T]; restore=True puts them back."""
    B, T, V = logits.shape
    assert logits.dtype == torch.float32 and logits.stride(2) == 1 and logits.stride(0) == T * logits.stride(1)
    rc = _load().wl_plant_logits(logits.data_ptr(), logits.stride(1), target.data_ptr(), n_nodes.data_ptr(), B, T, V, float(value),
                                 saved.data_ptr(), 1 if restore else 0, torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise RuntimeError("wl_plant_logits failed with CUDA error %d" % rc)
