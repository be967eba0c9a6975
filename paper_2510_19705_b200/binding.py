"""Thin ctypes binding over the C-ABI library (include/hsd.h).

Argument marshalling only: torch supplies device memory and streams, every step of the path runs
in the library's own CUDA kernels.  There is no CPU fallback: if the shared library has not been
built, or a call returns an error status, this module raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhsd.so")
HSD_F32, HSD_BF16 = 0, 1
_lib = None


class HsdError(RuntimeError):
    pass


def library():
    """Load libhsd.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise HsdError("libhsd.so is missing: run `python -m paper_2510_19705_b200.build` "
                           "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        _declare(lib)
        _lib = lib
    return _lib


def _declare(lib):
    c = ctypes
    vp, i32, u64, sz = c.c_void_p, c.c_int, c.c_uint64, c.c_size_t
    lib.hsd_strerror.restype = c.c_char_p
    lib.hsd_strerror.argtypes = [i32]
    lib.hsd_draft_sample.restype = i32
    lib.hsd_draft_sample.argtypes = [vp, i32, i32, i32, i32, u64, u64, vp, vp]
    lib.hsd_verify_workspace_bytes.restype = sz
    lib.hsd_verify_workspace_bytes.argtypes = [i32, i32]
    lib.hsd_verify_level.restype = i32
    lib.hsd_verify_level.argtypes = [i32, vp, vp, vp, i32, i32, i32, i32, u64, u64, vp, sz, vp, vp, vp]


def _check(status):
    if status != 0:
        raise HsdError("hsd call failed: %s (%d)" % (library().hsd_strerror(status).decode(), status))


def _dtype_code(t):
    if t.dtype == torch.float32:
        return HSD_F32
    if t.dtype == torch.bfloat16:
        return HSD_BF16
    raise HsdError("unsupported logits dtype %s" % t.dtype)


def _dev(t):
    if not (t.is_cuda and t.is_contiguous()):
        raise HsdError("expected a contiguous CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def hsd_draft_sample(logits, seed, call_serial, out_tokens=None):
    """logits [batch, rows, vocab] (CUDA, fp32/bf16) -> int32 tokens [batch, rows]."""
    batch, rows, vocab = logits.shape
    if out_tokens is None:
        out_tokens = torch.empty(batch, rows, dtype=torch.int32, device=logits.device)
    _check(library().hsd_draft_sample(_dev(logits), batch, rows, vocab, _dtype_code(logits), seed, call_serial,
                                      _stream(), _dev(out_tokens)))
    return out_tokens


def hsd_verify_workspace_bytes(batch, t):
    return int(library().hsd_verify_workspace_bytes(batch, t))


def hsd_verify_level(level, target_logits, draft_logits, draft_tokens, seed, call_serial, workspace=None,
                     out_tokens=None, out_n_accepted=None):
    """target_logits [batch, t+1, vocab], draft_logits [batch, t, vocab], draft_tokens int32 [batch, t]
    -> (out_tokens int32 [batch, t+1] padded with -1, n_accepted int32 [batch])."""
    batch, tp1, vocab = target_logits.shape
    t = tp1 - 1
    dev = target_logits.device
    if workspace is None:
        workspace = torch.empty(max(16, hsd_verify_workspace_bytes(batch, t)), dtype=torch.uint8, device=dev)
    if out_tokens is None:
        out_tokens = torch.empty(batch, t + 1, dtype=torch.int32, device=dev)
    if out_n_accepted is None:
        out_n_accepted = torch.empty(batch, dtype=torch.int32, device=dev)
    _check(library().hsd_verify_level(level, _dev(target_logits), _dev(draft_logits) if t > 0 else None,
                                      _dev(draft_tokens) if t > 0 else None, batch, t, vocab,
                                      _dtype_code(target_logits), seed, call_serial, _dev(workspace),
                                      workspace.numel(), _stream(), _dev(out_tokens), _dev(out_n_accepted)))
    return out_tokens, out_n_accepted
