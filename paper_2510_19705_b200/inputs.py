"""Seeded synthetic inputs and the benchmark shapes.

Holds no arithmetic of the method: only shapes, random weights / prompts / logits and
dtype plumbing.  Both the CUDA library's harness and the CPU oracle's tests take their
inputs from here so that they see identical buffers.

The paper measured on CNN-DM / XSUM prompts with pretrained LayerSkip and Gemma2
checkpoints; neither is available offline, so random-init models of the configured shapes
and uniform-random prompts stand in for them.
"""
import numpy as np
import torch

LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "wg", "wu", "wd")


def model_cfg(n_layers, d_model, n_q_heads, n_kv_heads, d_ff, vocab, dtype, head_dim=None):
    return dict(n_layers=n_layers, d_model=d_model, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                head_dim=head_dim or d_model // n_q_heads, d_ff=d_ff, vocab=vocab, dtype=dtype,
                rms_eps=1e-5, rope_theta=10000.0)


# The five workloads of the benchmark contract (model, exits, T, batch, prompt, n_new, page).
WORKLOADS = {
    "tiny3": dict(model=model_cfg(4, 128, 4, 4, 512, 512, "fp32"), exits=(1, 2, 4), T=(3, 2),
                  batch=1, prompt=16, n_new=64, page=16, weight_seed=1, prompt_seed=1),
    "accept": dict(batch=64, t=8, vocab=32000, dtype="bf16", target_std=3.0, noise_std=1.0),
    "1b3": dict(model=model_cfg(16, 2048, 32, 8, 5632, 32000, "bf16"), exits=(4, 8, 16), T=(4, 2),
                batch=1, prompt=512, n_new=256, page=16, weight_seed=3, prompt_seed=3),
    "8b3": dict(model=model_cfg(32, 4096, 32, 8, 14336, 32000, "bf16"), exits=(4, 12, 32), T=None,
                batch=1, prompt=1024, n_new=256, page=16, weight_seed=4, prompt_seed=4),
    "8b4long": dict(model=model_cfg(32, 4096, 32, 8, 14336, 32000, "bf16"), exits=(2, 6, 16, 32),
                    T=(2, 2, 3), batch=16, prompt=8192, n_new=512, page=16, weight_seed=4,
                    prompt_seed=5),
    # small bf16 stand-in with the 8B-shape's structure (GQA, SwiGLU, 3 levels) that the
    # CPU oracle finishes in seconds; spans several GEMM tiles and ragged tails.
    "mini3": dict(model=model_cfg(6, 256, 8, 2, 704, 2048, "bf16", head_dim=32), exits=(1, 3, 6),
                  T=(3, 2), batch=1, prompt=24, n_new=48, page=16, weight_seed=7, prompt_seed=7),
    # small stand-in with the long-context config's structure: 4 levels, draft lengths (2, 2, 3), a batch,
    # 16-token pages, head size 128, and prompts long enough that every attention key split spans
    # several key tiles and many pages.
    "mini4long": dict(model=model_cfg(6, 256, 4, 1, 704, 2048, "bf16", head_dim=128), exits=(1, 2, 4, 6),
                      T=(2, 2, 3), batch=2, prompt=2100, n_new=24, page=16, weight_seed=9, prompt_seed=9),
}


# Hierarchies of separate models (one decoder per level, shared vocabulary): list of model configs, weight seeds.
STACKS = {
    # fp32, three decoders of different depth / width / head layout (vocabulary 512)
    "tiny_stack": dict(models=[model_cfg(1, 64, 2, 2, 192, 512, "fp32"), model_cfg(2, 96, 4, 2, 256, 512, "fp32", head_dim=32),
                               model_cfg(3, 128, 4, 4, 512, 512, "fp32")],
                       weight_seeds=(21, 22, 23), T=(3, 2), prompt=16, n_new=48, page=16, prompt_seed=2),
    # bf16 on the tensor-core path: two drafters of their own shape below the mini3 target
    "mini_stack": dict(models=[model_cfg(1, 256, 4, 1, 512, 2048, "bf16", head_dim=64), model_cfg(2, 512, 8, 2, 704, 2048, "bf16", head_dim=64),
                               model_cfg(6, 256, 8, 2, 704, 2048, "bf16", head_dim=32)],
                       weight_seeds=(31, 32, 7), T=(3, 2), prompt=24, n_new=40, page=16, prompt_seed=7),
}


def truncated_model(cfg, weights, n_layers):
    """The first n_layers layers of a decoder as a model of its own (same tensors, no copies): with the shared final
    norm and head this is early-exit level e = n_layers written as a separate model."""
    c = dict(cfg, n_layers=n_layers)
    w = dict(weights, layers=list(weights["layers"][:n_layers]))
    return c, w


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_weights(cfg, seed, device="cpu", std=0.02):
    """Matrices N(0, std^2) stored [out_features, in_features]; norm gains 1.  torch tensors in
    the model's storage dtype on ``device``."""
    dt = torch.float32 if cfg["dtype"] == "fp32" else torch.bfloat16
    g = _gen(seed, device)
    d, hd, ff, V = cfg["d_model"], cfg["head_dim"], cfg["d_ff"], cfg["vocab"]
    nq, nkv = cfg["n_q_heads"], cfg["n_kv_heads"]

    def mat(rows, cols):
        return (torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * std).to(dt)

    def ones(n):
        return torch.ones(n, device=device, dtype=dt)

    w = dict(embed=mat(V, d), final_norm=ones(d), lm_head=mat(V, d), layers=[])
    for _ in range(cfg["n_layers"]):
        w["layers"].append(dict(attn_norm=ones(d), wq=mat(nq * hd, d), wk=mat(nkv * hd, d),
                                wv=mat(nkv * hd, d), wo=mat(d, nq * hd), mlp_norm=ones(d),
                                wg=mat(ff, d), wu=mat(ff, d), wd=mat(d, ff)))
    return w


def make_exit_heads(cfg, n_levels, seed, device="cpu", std=0.02, with_norm=True):
    """One output head per drafting level (Section 5.1, the setting with a trained head per exit layer):
    list over levels of dict(lm_head [vocab, d] ~ N(0, std^2), final_norm [d] ~ 1 + 0.1 N(0, 1) if with_norm);
    the last level (the target) keeps the shared head (None).  Stand-in for trained heads: random-init."""
    dt = torch.float32 if cfg["dtype"] == "fp32" else torch.bfloat16
    g = _gen(seed, device)
    d, V = cfg["d_model"], cfg["vocab"]
    heads = []
    for _ in range(n_levels - 1):
        h = dict(lm_head=(torch.randn(V, d, generator=g, device=device, dtype=torch.float32) * std).to(dt))
        if with_norm:
            h["final_norm"] = (1.0 + 0.1 * torch.randn(d, generator=g, device=device, dtype=torch.float32)).to(dt)
        heads.append(h)
    heads.append(None)
    return heads


def weights_to_numpy(w):
    """fp32 tensors -> float32 arrays; bf16 tensors -> uint16 bit patterns (host copies)."""
    def conv(t):
        t = t.detach().cpu().contiguous()
        return t.view(torch.uint16).numpy() if t.dtype == torch.bfloat16 else t.numpy()
    out = {k: conv(v) for k, v in w.items() if k not in ("layers", "exit_heads")}
    out["layers"] = [{k: conv(v) for k, v in layer.items()} for layer in w["layers"]]
    if w.get("exit_heads") is not None:
        out["exit_heads"] = [None if h is None else {k: conv(v) for k, v in h.items()} for h in w["exit_heads"]]
    return out


def make_prompts(vocab, batch, length, seed):
    """Uniform-random token ids, int32 [batch, length] on the CPU."""
    g = _gen(seed, "cpu")
    return torch.randint(0, vocab, (batch, length), generator=g, dtype=torch.int32)


def make_accept_logits(batch, t, vocab, seed, device="cpu", target_std=3.0, noise_std=1.0,
                       dtype="bf16"):
    """Target logits [batch, t+1, vocab] ~ N(0, target_std^2); draft logits [batch, t, vocab] =
    the first t target rows (before rounding) + N(0, noise_std^2); both rounded to ``dtype``."""
    g = _gen(seed, device)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    tgt = torch.randn(batch, t + 1, vocab, generator=g, device=device, dtype=torch.float32) * target_std
    drf = tgt[:, :t, :] + torch.randn(batch, t, vocab, generator=g, device=device,
                                      dtype=torch.float32) * noise_std
    return tgt.to(dt).contiguous(), drf.to(dt).contiguous()


def logits_to_numpy(x):
    """Stored logits -> float32 numpy (bf16 widens exactly)."""
    return x.detach().cpu().to(torch.float32).numpy()
