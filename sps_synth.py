"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests and bench.

Holds only input recipes (model shapes, random-init weights, prompts, logit batches); none of the
method's arithmetic lives here.  Both sides receive the very same tensors.

Shapes follow the paper's workloads: batch 1, K = 4, a short prompt then a 128-token (summarisation-
like) or 512-context (code-like) generation, and the Hyperparams table's 70B target / 4B draft pair.
The datasets and trained weights the paper used are replaced by random-init models of those shapes.
"""
from __future__ import annotations

import numpy as np
import torch


def _cfg(n_layers, d_model, n_heads, d_head, d_ff, vocab, dtype):
    return dict(n_layers=n_layers, d_model=d_model, n_heads=n_heads, d_head=d_head, d_ff=d_ff, vocab=vocab,
                dtype=dtype, rms_eps=1e-5, rope_base=10000.0)


# dtype: 0 = fp32 weights and KV cache, 1 = bf16 weights and KV cache
CONFIGS = {
    # tiny fp32 pair: token-exact parity with the oracle
    "tiny": dict(target=_cfg(2, 256, 4, 64, 1024, 1024, 0), draft=_cfg(1, 128, 2, 64, 512, 1024, 0),
                 prompt_len=16, n_new=64, K=4, T=1.0),
    # same pair with a 16-token vocabulary: exact end-to-end distribution tests
    "tiny16": dict(target=_cfg(2, 256, 4, 64, 1024, 16, 0), draft=_cfg(1, 128, 2, 64, 512, 16, 0),
                   prompt_len=16, n_new=3, K=4, T=1.0),
    # tiny shapes with bf16 storage: exercises the bf16 kernels at oracle-friendly size
    "tiny_bf16": dict(target=_cfg(2, 256, 2, 128, 1024, 1024, 1), draft=_cfg(1, 128, 1, 128, 512, 1024, 1),
                      prompt_len=16, n_new=64, K=4, T=1.0),
    "mid": dict(target=_cfg(24, 2048, 16, 128, 8192, 32000, 1), draft=_cfg(6, 1024, 8, 128, 4096, 32000, 1),
                prompt_len=128, n_new=256, K=4, T=1.0),
    # Hyperparams table: target 8192 / 64 heads / 80 layers, draft 6144 / 48 heads / 8 layers
    "70b": dict(target=_cfg(80, 8192, 64, 128, 32768, 32000, 1), draft=_cfg(8, 6144, 48, 128, 24576, 32000, 1),
                prompt_len=128, n_new=128, K=4, T=1.0),
}

LAYER_MATS = ("wq", "wk", "wv", "wo", "w_up", "w_down")


def _shape(cfg, name):
    d, f, v = cfg["d_model"], cfg["d_ff"], cfg["vocab"]
    return {"tok_embed": (v, d), "unembed": (v, d), "wq": (d, d), "wk": (d, d), "wv": (d, d), "wo": (d, d),
            "w_up": (f, d), "w_down": (d, f)}[name]


def _tensor_seed(seed, tag, layer, name):
    names = ("tok_embed", "unembed") + LAYER_MATS
    return (seed * 1000003 + (0 if tag == "target" else 1) * 500009 + (layer + 1) * 1009 + names.index(name)) % (2 ** 31)


def _normal(shape, std, seed, device, dtype):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    t = torch.empty(shape, device=device, dtype=dtype)
    t.normal_(0.0, std, generator=g)
    return t


def make_weights(cfg, seed=0, tag="target", device="cpu", std=0.02, share_embed_from=None, body_gain=1.0):
    """Every matrix and embedding i.i.d. N(0, std^2); norm gains 1.  Returns torch tensors on `device`.

    share_embed_from: weights of a wider model whose first d_model columns of tok_embed / unembed are
    reused (the 70B-shaped pair shares its (un)embedding so that acceptance is non-zero).
    body_gain: scales wo and w_down (a documented deviation used only to reach higher acceptance).
    """
    tdt = torch.float32 if cfg["dtype"] == 0 else torch.bfloat16
    w = {}
    for name in ("tok_embed", "unembed"):
        if share_embed_from is not None:
            w[name] = share_embed_from[name][:, : cfg["d_model"]].contiguous()
        else:
            w[name] = _normal(_shape(cfg, name), std, _tensor_seed(seed, tag, -1, name), device, tdt)
    w["final_norm"] = torch.ones(cfg["d_model"], device=device, dtype=torch.float32)
    w["layers"] = []
    for l in range(cfg["n_layers"]):
        lw = {"attn_norm": torch.ones(cfg["d_model"], device=device, dtype=torch.float32),
              "ffn_norm": torch.ones(cfg["d_model"], device=device, dtype=torch.float32)}
        for name in LAYER_MATS:
            t = _normal(_shape(cfg, name), std, _tensor_seed(seed, tag, l, name), device, tdt)
            if body_gain != 1.0 and name in ("wo", "w_down"):
                t.mul_(body_gain)
            lw[name] = t
        w["layers"].append(lw)
    return w


def to_numpy(t: torch.Tensor) -> np.ndarray:
    """fp32 -> float32 array; bf16 -> uint16 bit patterns (what the oracle reads)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def weights_to_numpy(w):
    out = {k: to_numpy(w[k]) for k in ("tok_embed", "unembed", "final_norm")}
    out["layers"] = [{k: to_numpy(v) for k, v in lw.items()} for lw in w["layers"]]
    return out


def weights_to(w, device):
    out = {k: w[k].to(device) for k in ("tok_embed", "unembed", "final_norm")}
    out["layers"] = [{k: v.to(device) for k, v in lw.items()} for lw in w["layers"]]
    return out


def weight_bytes(cfg):
    """Bytes one forward pass must stream: all layer matrices + unembedding (+ gains, negligible)."""
    es = 4 if cfg["dtype"] == 0 else 2
    d, f, v = cfg["d_model"], cfg["d_ff"], cfg["vocab"]
    return cfg["n_layers"] * (4 * d * d + 2 * d * f) * es + v * d * es


def make_prompt(seed, length, vocab):
    g = torch.Generator()
    g.manual_seed(1234567 + seed)
    return torch.randint(0, vocab, (length,), generator=g, dtype=torch.int64).to(torch.int32).numpy()


def sampler_batch(B, K, V, sigma, seed=0, target_std=3.0):
    """Standalone-sampler inputs: target logits N(0, 3^2), draft = target + N(0, sigma^2),
    draft tokens drawn from softmax(draft logits).  Returns numpy (q [B,K+1,V], p [B,K,V], drafts [B,K])."""
    g = torch.Generator()
    g.manual_seed(777 + seed)
    q = torch.randn((B, K + 1, V), generator=g) * target_std
    p = q[:, :K, :] + torch.randn((B, K, V), generator=g) * sigma
    probs = torch.softmax(p.double().reshape(B * K, V), dim=-1) if K > 0 else None
    if K > 0:
        d = torch.multinomial(probs, 1, generator=g).reshape(B, K).to(torch.int32)
    else:
        d = torch.zeros((B, 0), dtype=torch.int32)
    return q.numpy().astype(np.float32), p.contiguous().numpy().astype(np.float32), d.numpy()
