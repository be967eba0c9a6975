"""The model abstraction M_i(context) -> next-token distribution (Section 3.1), for the
early-exit family of Section 5.1: M_i is the first e_i layers of one decoder-only
transformer followed by the shared final norm and the shared output head (the
LayerSkip setting, where "the same LM head" serves every layer).  The other setting of
Section 5.1 (one trained output head per exit layer, a linear map from the embedding
dimension to the vocabulary; memory grows with the number of levels) is the optional
`exit_heads` entry of the weights: level i then uses its own head matrix, and its own
norm gain if one is given, in place of the shared ones.

The paper uses pretrained checkpoints and does not describe the network; the
architecture below is the benchmark contract's Llama-style decoder:
pre-norm residual blocks  x += Attn(RMSNorm(x));  x += MLP(RMSNorm(x)),
RMSNorm x * rsqrt(mean(x^2) + eps) * g, rotary embedding with half-split pairing
(k, k + hd/2) and angles pos * theta^(-2k/hd) (tables rounded to fp32), causal
attention with scale 1/sqrt(hd) and grouped KV heads, SwiGLU MLP
down(silu(gate(h)) * up(h)), untied output head, softmax at temperature 1.

Arithmetic: fp64 everywhere.  For bf16 models the stored-precision rounding points
are applied on top (weights are bf16; the normalised activations, q/k/v after
the rotary step, the attention output and the MLP activation are rounded to
bf16 where the CUDA path hands them to a matrix product or to the KV cache;
logits are rounded to bf16 when stored).  fp64 -> bf16 goes through fp32.

M_i(prefix) is a pure function of the prefix.  K/V per (layer, position) are
memoised and dropped past the first position where the prefix changed; the test
suite checks the memoised result equals a from-scratch evaluation.
"""
import numpy as np


def bf16_round(x):
    """Round to nearest-even bf16, returned as float64 values."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    r = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000))
    return r.view(np.float32).astype(np.float64)


def bf16_bits_to_f64(bits):
    """bf16 bit patterns (uint16) widened to float64: exact (a bf16 value is an fp32 value with a zero low half).
    Large matrices go through torch's conversion, which uses every host core; same values."""
    bits = np.ascontiguousarray(bits)
    if bits.size >= (1 << 20):
        import torch
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


class Transformer:
    """cfg: dict(n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab, dtype,
    rms_eps, rope_theta); weights: dict(embed, final_norm, lm_head, layers=[dict(attn_norm, wq,
    wk, wv, wo, mlp_norm, wg, wu, wd)]) of fp32 arrays (dtype 'fp32') or uint16 bf16 bit
    patterns (dtype 'bf16'), matrices stored [out_features, in_features].  Optional
    weights['exit_heads']: list over levels of None (shared head) or dict(lm_head[, final_norm])."""

    def __init__(self, cfg, weights, exits, cache_bytes=8 << 30, share_weights_with=None):
        """share_weights_with: another Transformer over the same weights whose widened (float64) copies of the
        matrices are reused instead of being made again (a cache only; no effect on any value)."""
        self.cfg, self.w, self.exits = dict(cfg), weights, list(exits)
        assert self.exits == sorted(self.exits) and self.exits[-1] == cfg["n_layers"]
        self.n_levels = len(self.exits)
        self.bf16 = cfg["dtype"] == "bf16"
        if share_weights_with is not None:
            assert share_weights_with.w is weights
            self._wide, self._acct = share_weights_with._wide, share_weights_with._acct
        else:
            self._wide, self._acct = {}, {"bytes": 0, "budget": cache_bytes}
        self.reset()

    # ------------------------------------------------------------------ weights
    def _mat(self, layer, name):
        key = (layer, name)
        hit = self._wide.get(key)
        if hit is not None:
            return hit
        raw = self.w[name] if layer is None else self.w["layers"][layer][name]
        wide = bf16_bits_to_f64(raw) if self.bf16 else raw.astype(np.float64)
        if self._acct["bytes"] + wide.nbytes <= self._acct["budget"]:
            self._wide[key] = wide
            self._acct["bytes"] += wide.nbytes
        return wide

    def _head(self, level, name):
        """The level's own output head / norm gain if it has one (Section 5.1, per-exit heads), else the shared one."""
        heads = self.w.get("exit_heads")
        own = heads[level] if heads is not None else None
        if own is None or own.get(name) is None:
            return self._mat(None, name)
        key = (("head", level), name)
        hit = self._wide.get(key)
        if hit is None:
            raw = own[name]
            hit = bf16_bits_to_f64(raw) if self.bf16 else raw.astype(np.float64)
            self._wide[key] = hit
        return hit

    def _rnd(self, x):
        return bf16_round(x) if self.bf16 else x

    # ------------------------------------------------------------------ state
    def reset(self):
        c = self.cfg
        self.tokens = []
        self.K = [np.zeros((0, c["n_kv_heads"], c["head_dim"])) for _ in range(c["n_layers"])]
        self.V = [np.zeros((0, c["n_kv_heads"], c["head_dim"])) for _ in range(c["n_layers"])]
        self.valid = [0] * c["n_layers"]
        self.last_logits64 = None

    def _rope(self, x, positions):
        hd = self.cfg["head_dim"]
        half = hd // 2
        k = np.arange(half, dtype=np.float64)
        inv = self.cfg["rope_theta"] ** (-2.0 * k / hd)
        ang = np.asarray(positions, dtype=np.float64)[:, None] * inv[None, :]
        cos = np.cos(ang).astype(np.float32).astype(np.float64)[:, None, :]
        sin = np.sin(ang).astype(np.float32).astype(np.float64)[:, None, :]
        a, b = x[..., :half], x[..., half:]
        return np.concatenate([a * cos - b * sin, b * cos + a * sin], axis=-1)

    def _rmsnorm(self, x, gain):
        ms = (x * x).mean(axis=-1, keepdims=True)
        return x / np.sqrt(ms + self.cfg["rms_eps"]) * gain

    # ------------------------------------------------------------------ forward
    def rows(self, level, context, draft_tokens):
        """Rows M_level(context + x_1..x_j), j = 0..t, as stored-precision logits (fp32 arrays)."""
        c = self.cfg
        seq = list(context) + list(draft_tokens)
        assert len(context) >= 1
        cp = 0
        while cp < min(len(seq), len(self.tokens)) and seq[cp] == self.tokens[cp]:
            cp += 1
        self.valid = [min(v, cp) for v in self.valid]
        self.tokens = seq
        e = self.exits[level]
        first_out = len(context) - 1
        start = min(min(self.valid[:e]), first_out)
        pos = np.arange(start, len(seq))
        R = len(pos)
        nq, nkv, hd = c["n_q_heads"], c["n_kv_heads"], c["head_dim"]
        group = nq // nkv
        x = self._mat(None, "embed")[np.asarray(seq[start:], dtype=np.int64)].copy()
        for l in range(e):
            h = self._rnd(self._rmsnorm(x, self._mat(l, "attn_norm")))
            q = (h @ self._mat(l, "wq").T).reshape(R, nq, hd)
            k = (h @ self._mat(l, "wk").T).reshape(R, nkv, hd)
            v = (h @ self._mat(l, "wv").T).reshape(R, nkv, hd)
            q = self._rnd(self._rope(q, pos))
            k = self._rnd(self._rope(k, pos))
            v = self._rnd(v)
            self.K[l] = np.concatenate([self.K[l][:start], k], axis=0)
            self.V[l] = np.concatenate([self.V[l][:start], v], axis=0)
            self.valid[l] = len(seq)
            att = np.empty((R, nq, hd))
            scale = 1.0 / np.sqrt(hd)
            for r in range(R):
                n_keys = start + r + 1                      # causal: keys at positions <= own
                Kc, Vc = self.K[l][:n_keys], self.V[l][:n_keys]
                for g in range(nkv):                      # the query heads that share KV head g, together
                    qg = q[r, g * group:(g + 1) * group]                 # [group, hd]
                    s = (Kc[:, g, :] @ qg.T) * scale                     # [n_keys, group]
                    p = np.exp(s - s.max(axis=0, keepdims=True))
                    p /= p.sum(axis=0, keepdims=True)
                    att[r, g * group:(g + 1) * group] = p.T @ Vc[:, g, :]
            att = self._rnd(att.reshape(R, nq * hd))
            x = x + att @ self._mat(l, "wo").T
            h = self._rnd(self._rmsnorm(x, self._mat(l, "mlp_norm")))
            gte = h @ self._mat(l, "wg").T
            up = h @ self._mat(l, "wu").T
            act = self._rnd(gte / (1.0 + np.exp(-gte)) * up)
            x = x + act @ self._mat(l, "wd").T
        xo = x[first_out - start:]
        hf = self._rnd(self._rmsnorm(xo, self._head(level, "final_norm")))
        logits = hf @ self._head(level, "lm_head").T
        self.last_logits64 = logits
        stored = self._rnd(logits) if self.bf16 else logits.astype(np.float32).astype(np.float64)
        return [stored[j].astype(np.float32) for j in range(stored.shape[0])]

    def rows_from_scratch(self, level, context, draft_tokens):
        """Same rows with every cache dropped first (the definition)."""
        self.reset()
        return self.rows(level, context, draft_tokens)


class ModelStack:
    """M_0..M_K as separate models over one vocabulary (Section 3.1: the hierarchy is any list of models with
    costs c_i; early exits of one decoder, as in Section 5.1, are one way to get such a list).  Level i is the
    whole of models[i] (a Transformer whose last exit is its full depth), with its own memoised keys / values.
    Same interface as Transformer towards Algorithm 1 / Algorithm 2: n_levels, rows(level, context, drafts)."""

    def __init__(self, models):
        self.models = list(models)
        self.n_levels = len(self.models)
        self.last_logits64 = None

    def reset(self):
        for m in self.models:
            m.reset()
        self.last_logits64 = None

    def rows(self, level, context, draft_tokens):
        m = self.models[level]
        out = m.rows(m.n_levels - 1, context, draft_tokens)
        self.last_logits64 = m.last_logits64
        return out
