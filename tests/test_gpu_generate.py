"""End-to-end parity of hsd_generate with the oracle: token streams, per-level counters, logits."""
import os

import numpy as np
import pytest
import torch

from oracle import philox, sampling
from oracle.hsd import HSD, CoinDecisions, SpecDecisions
from oracle.transformer import Transformer
from paper_2510_19705_b200 import inputs

pytestmark = pytest.mark.gpu

STAT_KEYS = ("calls", "drafted", "tested", "accepted", "emitted")


def _setup(name, lib, max_batch=1, T=None, exits=None):
    wl = inputs.WORKLOADS[name]
    cfg = wl["model"]
    w_cpu = inputs.make_weights(cfg, wl["weight_seed"])
    w_gpu = {k: (v.cuda() if k != "layers" else [{n: t.cuda() for n, t in l.items()} for l in v]) for k, v in w_cpu.items()}
    exits = exits or wl["exits"]
    T = wl["T"] if T is None else T
    max_seq = wl["prompt"] + wl["n_new"] + sum(T) + len(exits) + 8
    eng = lib.Hsd(cfg, w_gpu, exits, T, max_batch=max_batch, max_seq=max_seq, page_size=wl["page"])
    oracle_model = Transformer(cfg, inputs.weights_to_numpy(w_cpu), exits)
    prompts = inputs.make_prompts(cfg["vocab"], max_batch, wl["prompt"], wl["prompt_seed"])
    return wl, cfg, eng, oracle_model, prompts, T


def _oracle_run(model, T, prompt, n_new, seed, seq=0):
    model.reset()
    run = HSD(model, T, SpecDecisions(seed, seq))
    toks = run.generate(prompt, n_new)
    return np.asarray(toks, dtype=np.int32), run


def _check_stats(gpu_stats, run):
    for lvl, st in enumerate(run.stats):
        for k in STAT_KEYS:
            assert gpu_stats[lvl][k] == getattr(st, k), (lvl, k, gpu_stats[lvl], st.as_tuple())


def test_tiny_fp32_streams_match_oracle_bit_exact(lib):
    wl, cfg, eng, om, prompts, T = _setup("tiny3", lib)
    p_gpu = prompts.cuda()
    for seed in range(4):
        toks, stats, _ = eng.generate(p_gpu, wl["n_new"], seed)
        want, run = _oracle_run(om, T, prompts[0].tolist(), wl["n_new"], seed)
        assert np.array_equal(toks[0].cpu().numpy(), want), seed
        _check_stats(stats, run)
        for s in stats[1:]:
            assert s["calls"] <= s["emitted"] <= s["drafted"] + s["calls"]      # 1 .. t+1 tokens per round


def test_tiny_fp32_logits_within_tolerance_and_trace_matches(lib, tmp_path):
    wl, cfg, eng, om, prompts, T = _setup("tiny3", lib)
    path = str(tmp_path / "trace.bin")
    eng.set_trace(path, logit_calls=10 ** 6)
    toks, stats, _ = eng.generate(prompts.cuda(), 24, 3)
    eng.set_trace(None)
    recs = lib.read_trace(path)
    want, run = _oracle_run(om, T, prompts[0].tolist(), 24, 3)
    assert np.array_equal(toks[0].cpu().numpy(), want)
    assert len(recs) == len(run.trace)
    for rec, orc in zip(recs, run.trace):
        lvl, serial, ctx_len, t, n, otoks = orc
        assert (rec["level"], rec["serial"], rec["ctx_len"]) == (lvl, serial, ctx_len)
        if lvl == 0:
            assert rec["tokens"].tolist() == list(otoks)
        else:
            assert (rec["t"], rec["n"]) == (t, n) and rec["tokens"][-1] == otoks[-1]
    # logits of every verification against the oracle's own forward (fp32: 1e-5 absolute)
    om.reset()
    full = prompts[0].tolist() + want.tolist()
    worst = 0.0
    for rec in recs:
        if rec["level"] == 0:
            continue
        drafts = rec["tokens"][:-1].tolist()
        context = _context_of(recs, rec, prompts[0].tolist())
        om.rows(rec["level"], context, drafts)
        worst = max(worst, float(np.abs(om.last_logits64 - rec["logits"]).max()))
    assert worst < 1e-5, worst


def _context_of(recs, rec, prompt):
    """Rebuild the token buffer at the time of `rec` by replaying the log up to it."""
    buf = list(prompt)
    for r in recs:
        if r is rec:
            break
        if r["level"] == 0:
            buf = buf[:r["ctx_len"]] + r["tokens"].tolist()
        else:
            buf = buf[:r["ctx_len"] + r["n"]] + [int(r["tokens"][-1])]
    return buf if rec is None else buf[:rec["ctx_len"]]


def test_degenerate_hierarchies(lib):
    # one level = ancestral sampling from the target; two levels = single-draft speculative decoding
    wl, cfg, eng, om, prompts, _ = _setup("tiny3", lib, T=(), exits=(4,))
    toks, stats, _ = eng.generate(prompts.cuda(), 20, 9)
    ctx = prompts[0].tolist()
    om.reset()
    for i in range(20):
        row = om.rows(0, ctx, [])[0]
        tok = sampling.categorical(row, philox.uniform24(9, 0, i, 0, philox.PURPOSE_DRAFT, 0))
        assert tok == int(toks[0, i])
        ctx.append(tok)
    assert stats[0]["emitted"] == 20
    wl, cfg, eng2, om2, prompts, T2 = _setup("tiny3", lib, T=(4,), exits=(2, 4))
    toks, stats, _ = eng2.generate(prompts.cuda(), 40, 1)
    want, run = _oracle_run(om2, T2, prompts[0].tolist(), 40, 1)
    assert np.array_equal(toks[0].cpu().numpy(), want)
    _check_stats(stats, run)


def test_shortest_inputs_engine_reuse_and_rejected_calls(lib):
    # a one-token prompt, a request that ends inside the first round (only its first token is returned), the same
    # engine used again with fewer sequences and another seed; every stream equals the oracle's
    wl, cfg, eng, om, prompts, T = _setup("tiny3", lib, max_batch=3)
    for batch, P, n_new, seed in ((3, 1, 1, 4), (1, 1, 7, 5), (2, 3, 30, 6), (3, wl["prompt"], wl["n_new"], 7)):
        pr = prompts[:batch, :P].contiguous()
        toks, stats, _ = eng.generate(pr.cuda(), n_new, seed)
        assert tuple(toks.shape) == (batch, n_new)
        for b in range(batch):
            want, _ = _oracle_run(om, T, pr[b].tolist(), n_new, seed, seq=b)
            assert np.array_equal(toks[b].cpu().numpy(), want), (batch, P, n_new, b)
    # calls that cannot run are refused with an error code before anything is launched
    for batch, P, n_new in ((4, 4, 4), (1, wl["prompt"], 10 ** 6), (1, 0, 4), (1, 4, 0)):
        pr = torch.zeros((batch, max(P, 1)), dtype=torch.int32).cuda()
        with pytest.raises(lib.HsdError, match="invalid argument"):
            eng.generate(pr[:, :P] if P else pr[:, :0], n_new, 1)
    toks, _, _ = eng.generate(prompts[:1].cuda(), 5, 7)          # the engine is still usable afterwards
    want, _ = _oracle_run(om, T, prompts[0].tolist(), 5, 7)
    assert np.array_equal(toks[0].cpu().numpy(), want)


def test_batch_sequences_equal_their_single_runs(lib):
    # sequences are independent: sequence b of a batch = the same prompt run alone with the same seed
    wl, cfg, eng, om, prompts, T = _setup("tiny3", lib, max_batch=3)
    toks, stats, _ = eng.generate(prompts.cuda(), 32, 5)
    for b in range(3):
        want, _ = _oracle_run(om, T, prompts[b].tolist(), 32, 5, seq=b)
        assert np.array_equal(toks[b].cpu().numpy(), want), b


def test_page_size_does_not_change_the_stream(lib):
    wl = inputs.WORKLOADS["tiny3"]
    cfg = wl["model"]
    w = inputs.make_weights(cfg, wl["weight_seed"], device="cuda")
    prompts = inputs.make_prompts(cfg["vocab"], 1, wl["prompt"], wl["prompt_seed"]).cuda()
    outs = []
    for page in (4, 16, 64):
        eng = lib.Hsd(cfg, w, wl["exits"], wl["T"], max_batch=1, max_seq=128, page_size=page)
        outs.append(eng.generate(prompts, 40, 2)[0].cpu())
        eng.close()
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[1], outs[2])


@pytest.mark.parametrize("name", ["mini3", "mini4long"])
def test_folded_finish_phases_give_the_stream_of_the_separate_phases(lib, name):
    """Decode passes fold the QKV finish (piece sum, rotary embedding, cache write) into the attention phase and,
    with at most four rows, the gate / up finish (piece sum, SwiGLU) into the down projection, whose CTAs build
    their activation tiles in shared memory; the norm after a residual projection starts on idle CTAs without a
    grid barrier in between.  hsd_set_phase_folding keeps the separate phases / the barrier.  Same sums in the same
    order: every combination gives the same token stream."""
    wl = inputs.WORKLOADS[name]
    cfg = wl["model"]
    w = inputs.make_weights(cfg, wl["weight_seed"], device="cuda")
    batch = wl.get("batch", 1)
    prompts = inputs.make_prompts(cfg["vocab"], batch, wl["prompt"], wl["prompt_seed"]).cuda()
    max_seq = wl["prompt"] + wl["n_new"] + sum(wl["T"]) + len(wl["exits"]) + 8
    outs = []
    for fold_qkv, fold_gu, early in ((True, True, True), (False, True, True), (True, False, False), (False, False, False),
                                     (True, True, False)):
        eng = lib.Hsd(cfg, w, wl["exits"], wl["T"], max_batch=batch, max_seq=max_seq, page_size=wl["page"])
        eng.set_phase_folding(fold_qkv, fold_gu, early)
        outs.append(eng.generate(prompts, wl["n_new"], 1)[0].cpu())
        eng.close()
    for o in outs[1:]:
        assert torch.equal(outs[0], o)


def test_mini_bf16_decisions_follow_the_oracle_on_the_same_logits(lib, tmp_path):
    """bf16: the two forwards differ by rounding, so the stream is checked call by call: given the
    library's own stored logits, the oracle's decision arithmetic must reproduce every token and accept
    count; the logits themselves must match the oracle's forward within 2e-2."""
    wl, cfg, eng, om, prompts, T = _setup("mini3", lib)
    _bf16_trace_check(lib, wl, eng, om, prompts, tmp_path)


def _bf16_trace_check(lib, wl, eng, om, prompts, tmp_path):
    path = str(tmp_path / "trace.bin")
    eng.set_trace(path, logit_calls=10 ** 6)
    toks, stats, _ = eng.generate(prompts.cuda(), wl["n_new"], 0)
    eng.set_trace(None)
    recs = lib.read_trace(path)
    prompt = prompts[0].tolist()
    rows_of = {}                   # level -> logits rows of the level's current frame, by buffer position
    worst = 0.0
    n_checked = 0
    for rec in recs:
        lvl, ctx, serial = rec["level"], rec["ctx_len"], rec["serial"]
        context = _context_of(recs, rec, prompt)
        if lvl == 0:
            buf = list(context)
            for j, tok in enumerate(rec["tokens"].tolist()):
                U = philox.uniform24(0, j, serial, 0, philox.PURPOSE_DRAFT, 0)
                assert sampling.categorical(rec["logits"][j], U) == tok
                rows_of[(0, len(buf))] = rec["logits"][j]
                buf.append(tok)
        else:
            drafts = rec["tokens"][:-1].tolist()
            dec = SpecDecisions(0, 0)
            n = len(drafts)
            for j, x in enumerate(drafts):
                if not dec.accept(rec["logits"][j], rows_of[(lvl - 1, ctx + j)], x, j, serial, lvl):
                    n = j
                    break
            assert n == rec["n"]
            q = rows_of[(lvl - 1, ctx + n)] if n < len(drafts) else None
            assert dec.final_sample(rec["logits"][n], q, serial, lvl) == int(rec["tokens"][-1])
            for j in range(n + 1):
                rows_of[(lvl, ctx + j)] = rec["logits"][j]
        if n_checked < 40:           # forward parity on the first calls (the oracle is slow)
            if lvl == 0:
                for j in range(len(rec["tokens"])):
                    om.rows(0, context + rec["tokens"][:j].tolist(), [])
                    worst = max(worst, float(np.abs(om.last_logits64[0] - rec["logits"][j]).max()))
            else:
                om.rows(lvl, context, drafts)
                worst = max(worst, float(np.abs(om.last_logits64 - rec["logits"]).max()))
            n_checked += 1
    assert n_checked >= 10 and worst < 2e-2, worst
    # the emitted stream is what the log says
    final = _context_of(recs, None, prompt)
    assert final[len(prompt):len(prompt) + wl["n_new"]] == toks[0].cpu().tolist()


def _with_exit_heads(name, lib, with_norm=True):
    wl, cfg, eng, om, prompts, T = _setup(name, lib)
    heads = inputs.make_exit_heads(cfg, len(wl["exits"]), seed=77, with_norm=with_norm)
    eng.set_exit_heads([None if h is None else {k: v.cuda() for k, v in h.items()} for h in heads])
    w_cpu = inputs.make_weights(cfg, wl["weight_seed"])
    w_cpu["exit_heads"] = heads
    om = Transformer(cfg, inputs.weights_to_numpy(w_cpu), wl["exits"])
    return wl, cfg, eng, om, prompts, T


def test_per_exit_heads_fp32_streams_match_oracle_bit_exact(lib):
    """Section 5.1, one head per exit layer (hsd_set_exit_heads): every drafting level has its own head matrix and
    norm gain; the stream still equals the oracle's, and it differs from the shared-head stream."""
    wl, cfg, eng, om, prompts, T = _with_exit_heads("tiny3", lib)
    p_gpu = prompts.cuda()
    for seed in range(3):
        toks, stats, _ = eng.generate(p_gpu, wl["n_new"], seed)
        want, run = _oracle_run(om, T, prompts[0].tolist(), wl["n_new"], seed)
        assert np.array_equal(toks[0].cpu().numpy(), want), seed
        _check_stats(stats, run)
    with_heads = [dict(s) for s in stats]
    eng.set_exit_heads(None)                       # back to the shared head: the plain model's stream and counters
    wl2, _, _, om2, _, _ = _setup("tiny3", lib)
    toks, stats, _ = eng.generate(p_gpu, wl["n_new"], 2)
    want, run = _oracle_run(om2, T, prompts[0].tolist(), wl["n_new"], 2)
    assert np.array_equal(toks[0].cpu().numpy(), want)
    assert [s["accepted"] for s in stats] != [s["accepted"] for s in with_heads]


def test_per_exit_heads_bf16_decisions_and_logits(lib, tmp_path):
    """The same on the tensor-core path (persistent forward: the level's own head map and norm gain)."""
    wl, cfg, eng, om, prompts, T = _with_exit_heads("mini3", lib)
    _bf16_trace_check(lib, wl, eng, om, prompts, tmp_path)


def test_iid_coin_acceptance_streams_match_oracle(lib):
    """Ablation mode (hsd_set_iid_acceptance): accept tests are biased coins; stream and counters equal the
    oracle's run with the same coins, the observed rates are the coins' and not the model's."""
    wl, cfg, eng, om, prompts, T = _setup("tiny3", lib)
    alphas = (0.35, 0.8)
    eng.set_iid_acceptance(list(alphas))
    p_gpu = prompts.cuda()
    for seed in range(3):
        toks, stats, _ = eng.generate(p_gpu, wl["n_new"], seed)
        om.reset()
        run = HSD(om, T, CoinDecisions(seed, alphas))
        want = np.asarray(run.generate(prompts[0].tolist(), wl["n_new"]), dtype=np.int32)
        assert np.array_equal(toks[0].cpu().numpy(), want), seed
        _check_stats(stats, run)
    eng.set_iid_acceptance([1.0, 1.0])
    toks, stats, _ = eng.generate(p_gpu, wl["n_new"], 0)
    assert all(s["accepted"] == s["drafted"] for s in stats[1:])      # every draft accepted
    eng.set_iid_acceptance(None)                                      # back to Algorithm 2's rule
    toks, stats, _ = eng.generate(p_gpu, wl["n_new"], 0)
    want, run = _oracle_run(om, T, prompts[0].tolist(), wl["n_new"], 0)
    assert np.array_equal(toks[0].cpu().numpy(), want)


# ----------------------------------------------------------------------------- separate models (one decoder per level)
def _to_cuda(w):
    return {k: (v.cuda() if k != "layers" else [{n: t.cuda() for n, t in l.items()} for l in v]) for k, v in w.items()}


def _setup_stack(name, lib, max_batch=1):
    from oracle.transformer import ModelStack
    st = inputs.STACKS[name]
    cfgs = st["models"]
    w_cpu = [inputs.make_weights(c, s) for c, s in zip(cfgs, st["weight_seeds"])]
    T = list(st["T"])
    max_seq = st["prompt"] + st["n_new"] + sum(T) + len(cfgs) + 8
    eng = lib.Hsd(cfgs, [_to_cuda(w) for w in w_cpu], None, T, max_batch=max_batch, max_seq=max_seq, page_size=st["page"])
    om = ModelStack([Transformer(c, inputs.weights_to_numpy(w), (c["n_layers"],)) for c, w in zip(cfgs, w_cpu)])
    prompts = inputs.make_prompts(cfgs[0]["vocab"], max_batch, st["prompt"], st["prompt_seed"])
    return st, eng, om, prompts, T


def test_separate_models_fp32_streams_match_oracle_bit_exact(lib):
    """Section 3.1's general hierarchy (hsd_create_models): three decoders of different depth, width and head
    layout over one vocabulary, each with a KV cache of its own.  Streams and per-level counters equal the
    oracle's run of Algorithm 1 over the same three models; a batch gives each sequence its single-run stream."""
    st, eng, om, prompts, T = _setup_stack("tiny_stack", lib, max_batch=3)
    for seed in range(3):
        toks, stats, _ = eng.generate(prompts[:1].cuda(), st["n_new"], seed)
        want, run = _oracle_run(om, T, prompts[0].tolist(), st["n_new"], seed)
        assert np.array_equal(toks[0].cpu().numpy(), want), seed
        _check_stats(stats, run)
    toks, _, _ = eng.generate(prompts.cuda(), st["n_new"], 1)
    for b in range(3):
        want, _ = _oracle_run(om, T, prompts[b].tolist(), st["n_new"], 1, seq=b)
        assert np.array_equal(toks[b].cpu().numpy(), want), b


def test_separate_models_equal_early_exits_when_they_are_truncated_copies(lib):
    """The first e_i layers of one decoder handed over as separate models (own caches, own prompt passes) compute
    the same functions M_i as the early-exit hierarchy: identical streams and counters (fp32, and bf16 on the
    tensor-core path)."""
    for name in ("tiny3", "mini3"):
        wl = inputs.WORKLOADS[name]
        cfg, exits, T = wl["model"], wl["exits"], list(wl["T"])
        w = _to_cuda(inputs.make_weights(cfg, wl["weight_seed"]))
        prompts = inputs.make_prompts(cfg["vocab"], 1, wl["prompt"], wl["prompt_seed"]).cuda()
        max_seq = wl["prompt"] + wl["n_new"] + sum(T) + len(exits) + 8
        a = lib.Hsd(cfg, w, exits, T, max_batch=1, max_seq=max_seq, page_size=wl["page"])
        parts = [inputs.truncated_model(cfg, w, e) for e in exits]
        b = lib.Hsd([p[0] for p in parts], [p[1] for p in parts], None, T, max_batch=1, max_seq=max_seq, page_size=wl["page"])
        ta, sa, _ = a.generate(prompts, wl["n_new"], 3)
        tb, sb, _ = b.generate(prompts, wl["n_new"], 3)
        assert torch.equal(ta, tb), name
        for x, y in zip(sa, sb):
            assert all(x[k] == y[k] for k in STAT_KEYS), name
        a.close()
        b.close()


def test_separate_models_bf16_decisions_and_logits(lib, tmp_path):
    """Separate bf16 decoders on the tensor-core path (the persistent forward per model): every decision follows
    the oracle on the logged logits, the logits match the oracle's forward of the level's own model within 2e-2."""
    st, eng, om, prompts, T = _setup_stack("mini_stack", lib)
    _bf16_trace_check(lib, st, eng, om, prompts, tmp_path)
