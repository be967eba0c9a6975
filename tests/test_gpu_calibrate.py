"""The calibration kernels (pairwise acceptance rates between exit layers) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import sampling as S
from paper_2510_19705_b200 import binding

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("L,R,V,dtype", [(3, 5, 777, torch.float32), (4, 9, 2048, torch.bfloat16), (2, 3, 5000, torch.bfloat16),
                                         (8, 4, 1500, torch.float32), (1, 2, 100, torch.float32)])
def test_pairwise_alpha_matches_oracle(lib, L, R, V, dtype):
    g = torch.Generator().manual_seed(L * 1000 + R)
    base = torch.randn(R, V, generator=g) * 2.5
    logits = torch.stack([base + 0.8 * (m + 1) * torch.randn(R, V, generator=g) for m in range(L)]).to(dtype)
    got = lib.hsd_pairwise_alpha(logits.cuda())
    torch.cuda.synchronize()
    want = S.pairwise_acceptance(logits.float().numpy().astype(np.float64))
    got = got.cpu().numpy()
    assert got.shape == (L, L) and np.array_equal(got, got.T) and np.array_equal(np.diag(got), np.ones(L))
    assert np.abs(got - want).max() < 2e-5, np.abs(got - want).max()
    again = lib.hsd_pairwise_alpha(logits.cuda()).cpu().numpy()          # no atomics: repeatable bit for bit
    assert np.array_equal(got, again)


def test_pairwise_alpha_of_a_model_stack(lib):
    """The rates between the exits of one random-init model on its own drafted positions feed the hierarchy
    search: nearer exits accept each other more often, and the search returns a valid chain."""
    from paper_2510_19705_b200 import inputs
    torch.manual_seed(0)
    R, V = 16, 2048
    h = torch.randn(R, V)
    logits = torch.stack([h + s * torch.randn(R, V) for s in (1.5, 1.0, 0.5, 0.0)]).bfloat16().cuda()
    alpha = lib.hsd_pairwise_alpha(logits).cpu().numpy()
    assert alpha[2, 3] > alpha[1, 3] > alpha[0, 3]
    lat, sigma, T = binding.hsd_search_hierarchy([0.1, 0.3, 1.0, 3.0], alpha.tolist(), 8)
    assert sigma[-1] == 3 and len(T) == len(sigma) - 1 and lat <= 3.0


def _engine(lib, name):
    from paper_2510_19705_b200 import inputs
    wl = inputs.WORKLOADS[name]
    cfg = wl["model"]
    w_cpu = inputs.make_weights(cfg, wl["weight_seed"])
    w = {k: (v.cuda() if k != "layers" else [{n: t.cuda() for n, t in l.items()} for l in v]) for k, v in w_cpu.items()}
    eng = lib.Hsd(cfg, w, wl["exits"], wl["T"], max_batch=1, max_seq=160, page_size=wl["page"])
    return wl, cfg, w_cpu, eng


def test_layer_logits_match_the_oracle_fp32(lib):
    """Logits of every exit layer at every position (shared final norm + head): fp32 model, 1e-5 bound."""
    from oracle.transformer import Transformer
    from paper_2510_19705_b200 import inputs
    wl, cfg, w_cpu, eng = _engine(lib, "tiny3")
    toks = inputs.make_prompts(cfg["vocab"], 1, 40, 21)[0]
    layers = [1, 2, 3, 4]
    got = eng.layer_logits(toks.cuda(), layers).cpu().numpy()
    om = Transformer(cfg, inputs.weights_to_numpy(w_cpu), layers)
    for i in range(len(layers)):
        om.reset()
        om.rows(i, toks[:1].tolist(), toks[1:].tolist())              # rows of positions 0 .. n-1
        want = np.asarray(om.last_logits64)
        assert got[i].shape == want.shape
        assert np.abs(got[i] - want).max() < 1e-5, (layers[i], np.abs(got[i] - want).max())
    # a generation afterwards still works on the same context
    out, stats, _ = eng.generate(inputs.make_prompts(cfg["vocab"], 1, wl["prompt"], wl["prompt_seed"]).cuda(), 8, 1)
    assert out.shape == (1, 8)
    eng.close()


def test_calibrate_then_search_end_to_end(lib):
    """bf16 stand-in model: exit-layer logits -> pairwise acceptance rates -> latency-optimal hierarchy."""
    from oracle.transformer import Transformer
    from paper_2510_19705_b200 import inputs
    wl, cfg, w_cpu, eng = _engine(lib, "mini3")
    toks = inputs.make_prompts(cfg["vocab"], 1, 96, 22)[0]
    layers = [1, 2, 3, 4, 5, 6]
    logits = eng.layer_logits(toks.cuda(), layers)
    eng.close()
    alpha = lib.hsd_pairwise_alpha(logits).cpu().numpy()
    # the rates of the library's own logits equal the oracle's formula on those logits
    want = S.pairwise_acceptance(logits.float().cpu().numpy().astype(np.float64))
    assert np.abs(alpha - want).max() < 2e-5
    # and the logits are the oracle's forward (first and last exit; bf16: a few 1e-2 at most on this depth)
    om = Transformer(cfg, inputs.weights_to_numpy(w_cpu), layers)
    for i in (0, len(layers) - 1):
        om.reset()
        om.rows(i, toks[:1].tolist(), toks[1:].tolist())
        ref = np.asarray(om.last_logits64)
        d = np.abs(logits[i].float().cpu().numpy() - ref)
        assert np.sqrt((d ** 2).mean()) < 2e-2 * max(1.0, float(np.std(ref))), (layers[i], float(d.max()))
    costs = [float(l) for l in layers]                              # cost of an exit ~ its depth
    lat, sigma, T = binding.hsd_search_hierarchy(costs, alpha.tolist(), 8)
    assert sigma[-1] == len(layers) - 1 and lat <= costs[-1] and len(T) == len(sigma) - 1
    assert abs(lat - __import__("oracle.latency", fromlist=["x"]).search_hierarchy(costs, alpha.tolist(), 8)[0]) <= 1e-12 * lat
