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
    lib.hsd_verify_level_static.restype = i32
    lib.hsd_verify_level_static.argtypes = [i32, vp, vp, vp, i32, i32, i32, i32, u64, u64, vp, vp, vp]


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


def hsd_verify_level_static(level, target_logits, draft_logits, draft_tokens, seed, call_serial, out_tokens,
                            out_n_accepted):
    """hsd_verify_level for callers that cannot allocate: the library's built-in scratch is used and
    the caller supplies the outputs (out_tokens int32 [batch, t+1], out_n_accepted int32 [batch]).
    This wrapper allocates nothing either.  Limit: batch * (2 t + 1) <= 4096.  Calls must not
    overlap on the GPU (they share the scratch)."""
    batch, tp1, vocab = target_logits.shape
    t = tp1 - 1
    _check(library().hsd_verify_level_static(level, _dev(target_logits), _dev(draft_logits) if t > 0 else None,
                                             _dev(draft_tokens) if t > 0 else None, batch, t, vocab,
                                             _dtype_code(target_logits), seed, call_serial, _stream(),
                                             _dev(out_tokens), _dev(out_n_accepted)))
    return out_tokens, out_n_accepted


# ------------------------------------------------------------------------------------- engine
class _ModelDesc(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("d_model", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("d_ff", ctypes.c_int32),
                ("vocab", ctypes.c_int32), ("dtype", ctypes.c_int32), ("rms_eps", ctypes.c_float),
                ("rope_theta", ctypes.c_float), ("max_batch", ctypes.c_int32), ("max_seq", ctypes.c_int32),
                ("page_size", ctypes.c_int32), ("embed", ctypes.c_void_p), ("final_norm", ctypes.c_void_p),
                ("lm_head", ctypes.c_void_p), ("layer_weights", ctypes.POINTER(ctypes.c_void_p))]


class LevelStats(ctypes.Structure):
    _fields_ = [("calls", ctypes.c_int64), ("rows", ctypes.c_int64), ("drafted", ctypes.c_int64),
                ("tested", ctypes.c_int64), ("accepted", ctypes.c_int64), ("emitted", ctypes.c_int64),
                ("forwards", ctypes.c_int64), ("ms", ctypes.c_double)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "wg", "wu", "wd")


def _declare_engine(lib):
    c = ctypes
    vp, i32, u64, sz = c.c_void_p, c.c_int, c.c_uint64, c.c_size_t
    lib.hsd_workspace_bytes.restype = sz
    lib.hsd_workspace_bytes.argtypes = [c.POINTER(_ModelDesc), c.POINTER(c.c_int32), i32, c.POINTER(c.c_int32)]
    lib.hsd_create.restype = i32
    lib.hsd_create.argtypes = [c.POINTER(_ModelDesc), c.POINTER(c.c_int32), i32, c.POINTER(c.c_int32), vp, sz,
                               c.POINTER(vp)]
    lib.hsd_models_workspace_bytes.restype = sz
    lib.hsd_models_workspace_bytes.argtypes = [c.POINTER(_ModelDesc), i32, c.POINTER(c.c_int32)]
    lib.hsd_create_models.restype = i32
    lib.hsd_create_models.argtypes = [c.POINTER(_ModelDesc), i32, c.POINTER(c.c_int32), vp, sz, c.POINTER(vp)]
    lib.hsd_set_phase_folding.restype = i32
    lib.hsd_set_phase_folding.argtypes = [vp, i32, i32, i32]
    lib.hsd_set_tensor_attention.restype = i32
    lib.hsd_set_tensor_attention.argtypes = [vp, i32]
    lib.hsd_generate.restype = i32
    lib.hsd_generate.argtypes = [vp, vp, i32, i32, i32, u64, vp, vp, c.POINTER(LevelStats), c.POINTER(c.c_double)]
    lib.hsd_set_trace.restype = i32
    lib.hsd_set_trace.argtypes = [vp, c.c_char_p, i32]
    lib.hsd_set_iid_acceptance.restype = i32
    lib.hsd_set_iid_acceptance.argtypes = [vp, c.POINTER(c.c_double)]
    lib.hsd_set_exit_heads.restype = i32
    lib.hsd_set_exit_heads.argtypes = [vp, c.POINTER(vp), c.POINTER(vp)]
    lib.hsd_destroy.restype = None
    lib.hsd_destroy.argtypes = [vp]
    lib.hsd_expected_latency.restype = i32
    lib.hsd_expected_latency.argtypes = [c.POINTER(c.c_double), c.POINTER(c.c_double), i32, c.POINTER(c.c_int32),
                                         c.POINTER(c.c_double)]
    lib.hsd_expected_latency_literal.restype = i32
    lib.hsd_expected_latency_literal.argtypes = lib.hsd_expected_latency.argtypes
    lib.hsd_search_T.restype = i32
    lib.hsd_search_T.argtypes = [c.POINTER(c.c_double), c.POINTER(c.c_double), i32, i32, i32, c.POINTER(c.c_int32),
                                 c.POINTER(c.c_double)]
    lib.hsd_search_hierarchy.restype = i32
    lib.hsd_search_hierarchy.argtypes = [c.POINTER(c.c_double), c.POINTER(c.c_double), i32, i32, c.POINTER(c.c_int32),
                                         c.POINTER(c.c_int32), c.POINTER(c.c_int32), c.POINTER(c.c_double)]
    lib.hsd_pairwise_alpha_workspace_bytes.restype = sz
    lib.hsd_pairwise_alpha_workspace_bytes.argtypes = [i32, i32, i32]
    lib.hsd_pairwise_alpha.restype = i32
    lib.hsd_pairwise_alpha.argtypes = [vp, i32, i32, i32, i32, c.c_longlong, vp, sz, vp, vp]
    lib.hsd_layer_logits.restype = i32
    lib.hsd_layer_logits.argtypes = [vp, vp, i32, c.POINTER(c.c_int32), i32, vp, vp]
    lib.hsd_stream_read.restype = i32
    lib.hsd_stream_read.argtypes = [vp, sz, vp, vp]
    lib.hsd_kernel_launches.restype = c.c_uint64
    lib.hsd_kernel_launches.argtypes = []
    lib.hsd_gemm_workspace_bytes.restype = sz
    lib.hsd_gemm_workspace_bytes.argtypes = [i32, i32, i32]
    lib.hsd_gemm_bf16.restype = i32
    lib.hsd_gemm_bf16.argtypes = [vp, i32, i32, vp, i32, vp, vp, sz, vp]
    lib.hsd_gemm_status.restype = i32
    lib.hsd_gemm_status.argtypes = [vp, vp]


def _model_desc(cfg, weights, max_batch, max_seq, page_size):
    """(hsd_model_desc, the host pointer array it refers to) for one decoder."""
    n_layers = cfg["n_layers"]
    ptrs = (ctypes.c_void_p * (n_layers * 9))()
    for l, layer in enumerate(weights["layers"]):
        for k, name in enumerate(_LAYER_KEYS):
            t = layer[name]
            assert t.is_cuda and t.is_contiguous()
            ptrs[l * 9 + k] = t.data_ptr()
    d = _ModelDesc(n_layers, cfg["d_model"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["d_ff"],
                   cfg["vocab"], HSD_BF16 if cfg["dtype"] == "bf16" else HSD_F32, cfg["rms_eps"],
                   cfg["rope_theta"], max_batch, max_seq, page_size, weights["embed"].data_ptr(),
                   weights["final_norm"].data_ptr(), weights["lm_head"].data_ptr(), ptrs)
    return d, ptrs


class Hsd:
    """A hierarchy M_0..M_K (hsd_create / hsd_create_models, hsd_generate, hsd_destroy).

    Early exits of one decoder: cfg = dict as produced by inputs.model_cfg, weights = dict of CUDA tensors
    (inputs.make_weights), exits = exit layer per level (last == n_layers).
    Separate models: cfg and weights are LISTS with one entry per level (the last is the target), exits = None.
    T: T_0..T_{K-1}."""

    def __init__(self, cfg, weights, exits, T, max_batch, max_seq, page_size=16):
        lib = library()
        _declare_engine(lib)
        self._lib = lib
        self.T = list(T)
        self.weights = weights                      # keep the device buffers alive
        tt = (ctypes.c_int32 * max(1, len(self.T)))(*(self.T or [1]))
        ctx = ctypes.c_void_p()
        if exits is None:
            cfgs, ws = list(cfg), list(weights)
            n_levels = len(cfgs)
            descs = (_ModelDesc * n_levels)()
            self._ptrs = []
            for i in range(n_levels):
                descs[i], ptrs = _model_desc(cfgs[i], ws[i], max_batch, max_seq, page_size)
                self._ptrs.append(ptrs)
            self._desc = descs
            self.cfg, self.exits = dict(cfgs[-1]), [c["n_layers"] for c in cfgs]
            need = lib.hsd_models_workspace_bytes(descs, n_levels, tt)
            dev = ws[-1]["embed"].device
        else:
            self.cfg, self.exits = dict(cfg), list(exits)
            n_levels = len(self.exits)
            d, self._ptrs = _model_desc(cfg, weights, max_batch, max_seq, page_size)
            self._desc = d
            ex = (ctypes.c_int32 * n_levels)(*self.exits)
            need = lib.hsd_workspace_bytes(ctypes.byref(d), ex, n_levels, tt)
            dev = weights["embed"].device
        if need == 0:
            raise HsdError("the workspace-size call rejected the configuration")
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=dev)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        if exits is None:
            _check(lib.hsd_create_models(self._desc, n_levels, tt, ctypes.c_void_p(base), need, ctypes.byref(ctx)))
        else:
            _check(lib.hsd_create(ctypes.byref(self._desc), ex, n_levels, tt, ctypes.c_void_p(base), need, ctypes.byref(ctx)))
        self._ctx = ctx
        self.n_levels = n_levels
        self.workspace_bytes = need

    def set_phase_folding(self, fold_qkv=True, fold_gate_up=True, early_norm=True):
        """hsd_set_phase_folding: keep (False) or fold (True) the two finish phases of decode passes; keep (False) or
        drop (True) the grid barrier between a residual projection and its norm."""
        _check(self._lib.hsd_set_phase_folding(self._ctx, int(bool(fold_qkv)), int(bool(fold_gate_up)), int(bool(early_norm))))

    def set_tensor_attention(self, enabled=True):
        """hsd_set_tensor_attention: long key ranges on the tensor-memory attention path (True) or on the warp-level
        path like the short ones (False); "prefer": on, and key splits never shorter than that path takes."""
        _check(self._lib.hsd_set_tensor_attention(self._ctx, 2 if enabled == "prefer" else int(bool(enabled))))

    def set_exit_heads(self, heads):
        """heads: list over levels of None (shared head) or dict(lm_head[, final_norm]) of CUDA tensors in the
        model's dtype (hsd_set_exit_heads); None restores the shared head everywhere."""
        n = self.n_levels
        norms = (ctypes.c_void_p * n)()
        mats = (ctypes.c_void_p * n)()
        for i in range(n):
            h = heads[i] if heads is not None else None
            if h is not None:
                assert h["lm_head"].is_cuda and h["lm_head"].is_contiguous()
                mats[i] = h["lm_head"].data_ptr()
                if h.get("final_norm") is not None:
                    norms[i] = h["final_norm"].data_ptr()
        self._exit_heads = heads                    # keep the device buffers alive
        _check(self._lib.hsd_set_exit_heads(self._ctx, norms, mats))

    def set_iid_acceptance(self, alphas):
        """Ablation mode (hsd_set_iid_acceptance): alphas[i] = coin probability of level i+1's accept tests; None
        restores Algorithm 2's rule."""
        if alphas is None:
            _check(self._lib.hsd_set_iid_acceptance(self._ctx, None))
        else:
            assert len(alphas) == self.n_levels - 1
            _check(self._lib.hsd_set_iid_acceptance(self._ctx, (ctypes.c_double * max(1, len(alphas)))(*alphas)))

    def set_trace(self, path, logit_calls=0):
        _check(self._lib.hsd_set_trace(self._ctx, path.encode() if path else None, logit_calls))

    def generate(self, prompt_ids, n_new, seed):
        """prompt_ids: CUDA int32 [batch, prompt_len] -> (tokens CUDA int32 [batch, n_new], [per-level stats
        dicts], (prompt_ms, generate_ms))."""
        batch, plen = prompt_ids.shape
        out = torch.empty(batch, n_new, dtype=torch.int32, device=prompt_ids.device)
        stats = (LevelStats * self.n_levels)()
        timing = (ctypes.c_double * 2)()
        _check(self._lib.hsd_generate(self._ctx, _dev(prompt_ids), batch, plen, n_new, seed, _stream(), _dev(out),
                                      stats, timing))
        return out, [s.as_dict() for s in stats], (timing[0], timing[1])

    def layer_logits(self, token_ids, layers):
        """token_ids: CUDA int32 [n_tokens] (<= 128); layers: ascending exit layers -> logits CUDA tensor
        [len(layers), n_tokens, vocab] in the model's storage dtype (shared final norm + head after each layer)."""
        n = int(token_ids.numel())
        lay = (ctypes.c_int32 * len(layers))(*[int(x) for x in layers])
        dt = torch.float32 if self.cfg["dtype"] == "fp32" else torch.bfloat16
        out = torch.empty(len(layers), n, self.cfg["vocab"], dtype=dt, device=token_ids.device)
        _check(self._lib.hsd_layer_logits(self._ctx, _dev(token_ids), n, lay, len(layers), _dev(out), _stream()))
        return out

    def close(self):
        if getattr(self, "_ctx", None):
            self._lib.hsd_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        self.close()


def read_trace(path):
    """Parse a decision log written by hsd_set_trace into a list of dicts (numpy logits as float32)."""
    import numpy as np
    recs = []
    with open(path, "rb") as f:
        while True:
            hdr = f.read(48)
            if len(hdr) < 48:
                break
            h = np.frombuffer(hdr, dtype=np.int32)
            assert int(h[0]) == 0x48534454
            level, seq, serial, ctx_len, t, n, rows, lrows, has_logits, V, dtype = (int(v) for v in h[1:12])
            n_tok = (n if level == 0 else t + 1)
            toks = np.frombuffer(f.read(4 * n_tok), dtype=np.int32).copy()
            logits = None
            if has_logits:
                if dtype == HSD_BF16:
                    raw = np.frombuffer(f.read(2 * lrows * V), dtype=np.uint16)
                    logits = (raw.astype(np.uint32) << 16).view(np.float32).reshape(lrows, V)
                else:
                    logits = np.frombuffer(f.read(4 * lrows * V), dtype=np.float32).reshape(lrows, V).copy()
            recs.append(dict(level=level, seq=seq, serial=serial, ctx_len=ctx_len, t=t, n=n, rows=rows,
                             tokens=toks, logits=logits))
    return recs


def hsd_expected_latency(costs, alphas, T):
    """Theorem 3.2 for the chain with costs c_0..c_K, alphas[i] = rate level i -> i+1, parameters T."""
    lib = library()
    _declare_engine(lib)
    n = len(costs)
    out = ctypes.c_double()
    _check(lib.hsd_expected_latency((ctypes.c_double * n)(*costs), (ctypes.c_double * max(1, n - 1))(*(alphas or [0])), n,
                                    (ctypes.c_int32 * max(1, n - 1))(*(T or [1])), ctypes.byref(out)))
    return out.value


def hsd_expected_latency_literal(costs, alphas, T):
    """Expected cost per token of Algorithm 1 as printed (verifiers see everything the level below collected)."""
    lib = library()
    _declare_engine(lib)
    n = len(costs)
    out = ctypes.c_double()
    _check(lib.hsd_expected_latency_literal((ctypes.c_double * n)(*costs), (ctypes.c_double * max(1, n - 1))(*(alphas or [0])),
                                            n, (ctypes.c_int32 * max(1, n - 1))(*(T or [1])), ctypes.byref(out)))
    return out.value


def hsd_search_T(costs, alphas, T_max=15, monotone=True):
    """argmin over T in [1, T_max]^K of the expected latency -> (T tuple, latency)."""
    lib = library()
    _declare_engine(lib)
    n = len(costs)
    out_T = (ctypes.c_int32 * max(1, n - 1))()
    out = ctypes.c_double()
    _check(lib.hsd_search_T((ctypes.c_double * n)(*costs), (ctypes.c_double * max(1, n - 1))(*(alphas or [0])), n, T_max,
                            1 if monotone else 0, out_T, ctypes.byref(out)))
    return tuple(out_T[i] for i in range(n - 1)), out.value



def hsd_pairwise_alpha(logits):
    """logits: CUDA tensor [n_models, n_rows, vocab] (fp32 or bf16) -> float64 CUDA tensor [n_models, n_models] of the
    acceptance rates alpha[i][j] = mean over rows of sum_x min(p_i(x), p_j(x))."""
    lib = library()
    _declare_engine(lib)
    L, R, V = logits.shape
    logits = logits.contiguous()
    need = lib.hsd_pairwise_alpha_workspace_bytes(L, R, V)
    if need == 0:
        raise HsdError("hsd_pairwise_alpha: unsupported sizes %s" % (tuple(logits.shape),))
    ws = torch.empty(need + 256, dtype=torch.uint8, device=logits.device)
    base = (ws.data_ptr() + 255) // 256 * 256
    out = torch.empty(L, L, dtype=torch.float64, device=logits.device)
    dtype = 1 if logits.dtype == torch.bfloat16 else 0
    if logits.dtype not in (torch.bfloat16, torch.float32):
        raise HsdError("hsd_pairwise_alpha: logits must be fp32 or bf16")
    _check(lib.hsd_pairwise_alpha(_dev(logits), dtype, L, R, V, R * V, ctypes.c_void_p(base),
                                  ws.numel() - (base - ws.data_ptr()), _dev(out), _stream()))
    return out


def hsd_search_hierarchy(costs, alpha, T_max=15):
    """Latency-optimal (sigma, T) over ordered subsets of the models ending in the target.
    costs: c_0..c_K; alpha[i][j]: acceptance rate of drafter i under verifier j (i < j).
    -> (latency, sigma tuple, T tuple)."""
    lib = library()
    _declare_engine(lib)
    n = len(costs)
    flat = [0.0] * (n * n)
    for i in range(n):
        for j in range(i + 1, n):
            flat[i * n + j] = float(alpha[i][j])
    sigma = (ctypes.c_int32 * n)()
    n_lev = ctypes.c_int32()
    out_T = (ctypes.c_int32 * max(1, n - 1))()
    out = ctypes.c_double()
    _check(lib.hsd_search_hierarchy((ctypes.c_double * n)(*costs), (ctypes.c_double * (n * n))(*flat), n, T_max, sigma,
                                    ctypes.byref(n_lev), out_T, ctypes.byref(out)))
    k = n_lev.value
    return out.value, tuple(sigma[i] for i in range(k)), tuple(out_T[i] for i in range(k - 1))

def hsd_stream_read_gbs(n_bytes=4 << 30, repeats=5):
    """Read-only streaming rate of this GPU's HBM in GB/s (hsd_stream_read over a buffer far larger than L2, best of
    `repeats` after one warm-up, CUDA events on the current stream)."""
    lib = library()
    _declare_engine(lib)
    buf = torch.empty(n_bytes, dtype=torch.uint8, device="cuda")
    buf.zero_()
    best = 0.0
    for i in range(repeats + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        _check(lib.hsd_stream_read(_dev(buf), n_bytes, None, _stream()))
        e1.record()
        e1.synchronize()
        if i > 0:
            best = max(best, n_bytes / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    del buf
    return best


def hsd_kernel_launches():
    lib = library()
    _declare_engine(lib)
    return int(lib.hsd_kernel_launches())


def hsd_gemm_workspace_bytes(R, N, K):
    lib = library()
    _declare_engine(lib)
    return int(lib.hsd_gemm_workspace_bytes(R, N, K))


def hsd_gemm_bf16(A, W, out=None, workspace=None, check=True):
    """A bf16 [R, K], W bf16 [N, K] (CUDA) -> fp32 [R, N] = A @ W^T on the tensor cores."""
    lib = library()
    _declare_engine(lib)
    R, K = A.shape
    N = W.shape[0]
    need = hsd_gemm_workspace_bytes(R, N, K)
    if need == 0:
        raise HsdError("hsd_gemm_bf16: unsupported shape R=%d N=%d K=%d" % (R, N, K))
    if workspace is None:
        workspace = torch.empty(need + 256, dtype=torch.uint8, device=A.device)
    base = (workspace.data_ptr() + 255) // 256 * 256
    if out is None:
        out = torch.empty(R, N, dtype=torch.float32, device=A.device)
    _check(lib.hsd_gemm_bf16(_dev(A), R, K, _dev(W), N, _dev(out), ctypes.c_void_p(base),
                             workspace.numel() - (base - workspace.data_ptr()), _stream()))
    if check:
        _check(lib.hsd_gemm_status(ctypes.c_void_p(base), _stream()))
    return out
