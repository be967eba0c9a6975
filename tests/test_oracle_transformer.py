"""The oracle's model forward pinned to library routines (torch rms_norm, scaled_dot_product_attention,
silu, linear) on the same weights, and its memoisation pinned to the from-scratch definition."""
import numpy as np
import torch
import torch.nn.functional as F

from oracle.transformer import Transformer, bf16_round
from paper_2510_19705_b200 import inputs

CFG32 = inputs.model_cfg(3, 64, 4, 2, 160, 96, "fp32", head_dim=16)
CFG16 = inputs.model_cfg(3, 64, 4, 2, 160, 96, "bf16", head_dim=16)


def library_forward(cfg, w, n_layers, tokens, bf16):
    """Independent restatement with torch library ops in fp64; returns logits [len(tokens), V]."""
    rnd = (lambda x: x.to(torch.bfloat16).to(torch.float64)) if bf16 else (lambda x: x)
    W = lambda t: t.to(torch.float64)
    nq, nkv, hd, d = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["d_model"]
    L = len(tokens)
    x = W(w["embed"])[torch.tensor(tokens)]
    pos = torch.arange(L, dtype=torch.float64)
    inv = cfg["rope_theta"] ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd)
    ang = torch.outer(pos, inv)
    rot = torch.polar(torch.ones_like(ang), ang.to(torch.float32).to(torch.float64))
    # the oracle rounds cos / sin (not the angle) to fp32; the difference is far below tolerance

    def rope(t):                                   # [L, heads, hd], half-split pairing as complex numbers
        c = torch.complex(t[..., : hd // 2], t[..., hd // 2:]) * rot[:, None, :]
        return torch.cat([c.real, c.imag], dim=-1)

    for l in range(n_layers):
        lw = w["layers"][l]
        h = rnd(F.rms_norm(x, (d,), W(lw["attn_norm"]), cfg["rms_eps"]))
        q = rnd(rope(F.linear(h, W(lw["wq"])).view(L, nq, hd)))
        k = rnd(rope(F.linear(h, W(lw["wk"])).view(L, nkv, hd)))
        v = rnd(F.linear(h, W(lw["wv"])).view(L, nkv, hd))
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                           v.transpose(0, 1)[None], is_causal=True, enable_gqa=True)
        o = rnd(o[0].transpose(0, 1).reshape(L, nq * hd))
        x = x + F.linear(o, W(lw["wo"]))
        h = rnd(F.rms_norm(x, (d,), W(lw["mlp_norm"]), cfg["rms_eps"]))
        a = rnd(F.silu(F.linear(h, W(lw["wg"]))) * F.linear(h, W(lw["wu"])))
        x = x + F.linear(a, W(lw["wd"]))
    hf = rnd(F.rms_norm(x, (d,), W(w["final_norm"]), cfg["rms_eps"]))
    return F.linear(hf, W(w["lm_head"])).numpy()


def _setup(cfg, std=0.2):
    w = inputs.make_weights(cfg, seed=11, std=std)
    # non-trivial norm gains so that a dropped gain would show
    g = torch.Generator().manual_seed(5)
    for t in [w["final_norm"]] + [l[k] for l in w["layers"] for k in ("attn_norm", "mlp_norm")]:
        t.copy_((1.0 + 0.3 * torch.randn(t.shape, generator=g)).to(t.dtype))
    return w, Transformer(cfg, inputs.weights_to_numpy(w), exits=(1, 2, 3))


def test_fp32_model_matches_library_ops():
    w, m = _setup(CFG32)
    toks = inputs.make_prompts(CFG32["vocab"], 1, 12, seed=3)[0].tolist()
    for level, e in enumerate((1, 2, 3)):
        ref = library_forward(CFG32, w, e, toks, bf16=False)
        m.rows_from_scratch(level, toks[:8], toks[8:])
        got = m.last_logits64
        assert got.shape == (5, CFG32["vocab"])
        assert np.abs(got - ref[7:]).max() < 1e-6 * max(1.0, np.abs(ref).max())
        assert np.abs(ref).max() > 0.05               # the comparison is not vacuous


def test_bf16_model_matches_library_ops_with_the_same_rounding_points():
    w, m = _setup(CFG16)
    toks = inputs.make_prompts(CFG16["vocab"], 1, 10, seed=4)[0].tolist()
    ref = library_forward(CFG16, w, 3, toks, bf16=True)
    rows = m.rows_from_scratch(2, toks[:6], toks[6:])
    got = m.last_logits64
    # identical rounding points; an occasional 1-ulp bf16 flip of an activation moves logits slightly
    assert np.abs(got - ref[5:]).max() < 5e-3 * np.abs(ref).max()
    stored = np.stack(rows)
    assert np.array_equal(stored, bf16_round(got).astype(np.float32))


def test_per_exit_heads_replace_the_shared_head_at_their_level_only():
    """Section 5.1, one trained head per exit layer: level i's logits = own head x RMSNorm(hidden state at e_i, own
    gain); a level without an own head (here the target) and a head without an own gain use the shared ones."""
    w, _ = _setup(CFG32)
    heads = inputs.make_exit_heads(CFG32, 3, seed=21, std=0.2)
    del heads[1]["final_norm"]                        # level 1: own matrix, shared norm gain
    w["exit_heads"] = heads
    m = Transformer(CFG32, inputs.weights_to_numpy(w), exits=(1, 2, 3))
    toks = inputs.make_prompts(CFG32["vocab"], 1, 12, seed=3)[0].tolist()
    for level, e in enumerate((1, 2, 3)):
        own = heads[level] or {}
        w_level = dict(w, lm_head=own.get("lm_head", w["lm_head"]), final_norm=own.get("final_norm", w["final_norm"]))
        ref = library_forward(CFG32, w_level, e, toks, bf16=False)
        shared = library_forward(CFG32, w, e, toks, bf16=False)
        m.rows_from_scratch(level, toks[:8], toks[8:])
        got = m.last_logits64
        assert np.abs(got - ref[7:]).max() < 1e-6 * max(1.0, np.abs(ref).max())
        if level < 2:
            assert np.abs(ref - shared).max() > 0.05   # the own head matters
    # heads equal to the shared one change nothing
    w["exit_heads"] = [dict(lm_head=w["lm_head"], final_norm=w["final_norm"]), None, None]
    m2 = Transformer(CFG32, inputs.weights_to_numpy(w), exits=(1, 2, 3))
    m2.rows_from_scratch(0, toks[:8], toks[8:])
    assert np.abs(m2.last_logits64 - library_forward(CFG32, w, 1, toks, bf16=False)[7:]).max() < 1e-6


def test_bf16_round_is_nearest_even():
    x = torch.randn(4096, dtype=torch.float32) * 3
    x[:4] = torch.tensor([1.00390625, 1.01171875, -1.00390625, 0.0])     # exact ties
    assert np.array_equal(bf16_round(x.numpy()), x.to(torch.bfloat16).to(torch.float64).numpy())


def test_memoised_rows_equal_from_scratch_and_levels_share_the_cache():
    w, m = _setup(CFG32)
    toks = inputs.make_prompts(CFG32["vocab"], 1, 14, seed=9)[0].tolist()
    # a sequence of calls like Algorithm 1 makes them: level-0 steps, a level-1 verify, a rollback
    calls = [(0, toks[:6], []), (0, toks[:7], []), (1, toks[:6], toks[6:8]), (0, toks[:7] + [5], []),
             (2, toks[:6], [toks[6], 5, 9]), (1, toks[:9], toks[9:11]), (2, toks[:9], toks[9:12])]
    got = [np.stack(m.rows(*c)) for c in calls]
    fresh = Transformer(CFG32, m.w, exits=(1, 2, 3))
    for c, g in zip(calls, got):
        ref = np.stack(fresh.rows_from_scratch(*c))
        assert g.shape == (len(c[2]) + 1, CFG32["vocab"])
        assert np.abs(g - ref).max() < 1e-6


def test_rows_are_prefix_consistent():
    # row j of a verify call is the model's distribution after context + x_1..x_j
    w, m = _setup(CFG32)
    toks = inputs.make_prompts(CFG32["vocab"], 1, 9, seed=2)[0].tolist()
    rows = np.stack(m.rows(2, toks[:5], toks[5:8]))
    for j in range(4):
        one = m.rows_from_scratch(2, toks[:5 + j], [])[0]
        assert np.abs(rows[j] - one).max() < 1e-6


def test_bf16_forward_is_sensitive_to_fp32_level_noise():
    """Why the bf16 logits tolerance is statistical: nudging every value by 2e-6 (the size of fp32 accumulation
    error) before each bf16 rounding point moves the oracle's own logits by far more than 2e-6, because a
    value near a rounding boundary flips by a whole bf16 step and the flips compound through the layers."""
    from oracle import transformer as T
    cfg = inputs.model_cfg(3, 256, 8, 2, 704, 512, "bf16", head_dim=32)
    w = inputs.weights_to_numpy(inputs.make_weights(cfg, 3, std=0.05))
    prompt = inputs.make_prompts(cfg["vocab"], 1, 24, 3)[0].tolist()
    a = T.Transformer(cfg, w, (2, 3))
    a.rows(0, prompt, [])
    ref = a.last_logits64[0].copy()
    orig = T.bf16_round
    rng = np.random.default_rng(0)
    T.bf16_round = lambda x: orig(np.asarray(x, dtype=np.float64) * (1.0 + 2e-6 * rng.standard_normal(np.shape(x))))
    try:
        b = T.Transformer(cfg, w, (2, 3))
        b.rows(0, prompt, [])
        got = b.last_logits64[0]
    finally:
        T.bf16_round = orig
    rel = float(np.sqrt(((got - ref) ** 2).mean()) / ref.std())
    assert 2e-4 < rel < 5e-2, rel          # orders of magnitude above the 2e-6 that went in, still small


def test_stack_of_truncated_copies_is_the_early_exit_model():
    """Section 3.1's list of models, pinned to the early-exit family: the first e_i layers of one decoder written
    as separate models (own key / value memo each) give the rows, and Algorithm 1 the token stream and counters,
    of the early-exit model, exactly."""
    from oracle.hsd import HSD, SpecDecisions
    from oracle.transformer import ModelStack
    w, m = _setup(CFG32)
    w_np = inputs.weights_to_numpy(w)
    exits = (1, 2, 3)
    parts = []
    for e in exits:
        c, wt = inputs.truncated_model(CFG32, w_np, e)
        parts.append(Transformer(c, wt, (e,)))
    stack = ModelStack(parts)
    toks = inputs.make_prompts(CFG32["vocab"], 1, 9, seed=4)[0].tolist()
    for level in range(3):
        a = m.rows(level, toks, [3, 1, 4])
        b = stack.rows(level, toks, [3, 1, 4])
        assert all(np.array_equal(x, y) for x, y in zip(a, b))
    m.reset()
    stack.reset()
    r1, r2 = HSD(m, (2, 2), SpecDecisions(5)), HSD(stack, (2, 2), SpecDecisions(5))
    assert r1.generate(toks, 24) == r2.generate(toks, 24)
    assert [s.as_tuple() for s in r1.stats] == [s.as_tuple() for s in r2.stats]
