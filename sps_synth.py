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


def _cfg(n_layers, d_model, n_heads, d_head, d_ff, vocab, dtype, n_kv_heads=0):
    """n_kv_heads: key / value heads (0 = n_heads); fewer than n_heads = grouped-query, 1 = multi-query attention."""
    return dict(n_layers=n_layers, d_model=d_model, n_heads=n_heads, d_head=d_head, d_ff=d_ff, vocab=vocab,
                dtype=dtype, rms_eps=1e-5, rope_base=10000.0, n_kv_heads=n_kv_heads or n_heads)


# dtype: 0 = fp32 weights and KV cache, 1 = bf16 weights and KV cache
CONFIGS = {
    # tiny fp32 pair: token-exact parity with the oracle
    "tiny": dict(target=_cfg(2, 256, 4, 64, 1024, 1024, 0), draft=_cfg(1, 128, 2, 64, 512, 1024, 0),
                 prompt_len=16, n_new=64, K=4, T=1.0),
    # same pair with a 16-token vocabulary: exact end-to-end distribution tests
    "tiny16": dict(target=_cfg(2, 256, 4, 64, 1024, 16, 0), draft=_cfg(1, 128, 2, 64, 512, 16, 0),
                   prompt_len=16, n_new=3, K=4, T=1.0),
    # the fp32 pair with a vocabulary of 8192: large enough for the samplers that spread a sequence over a thread-block
    # cluster, small enough for token-exact parity against the oracle
    "tiny_v8k": dict(target=_cfg(2, 256, 4, 64, 1024, 8192, 0), draft=_cfg(1, 128, 2, 64, 512, 8192, 0),
                     prompt_len=16, n_new=48, K=4, T=1.0),
    # tiny shapes with bf16 storage: exercises the bf16 kernels at oracle-friendly size
    "tiny_bf16": dict(target=_cfg(2, 256, 2, 128, 1024, 1024, 1), draft=_cfg(1, 128, 1, 128, 512, 1024, 1),
                      prompt_len=16, n_new=64, K=4, T=1.0),
    # the same shapes with int8 linear weights (dtype 2): bf16 matrices quantised per output row
    "tiny_q8": dict(target=_cfg(2, 256, 2, 128, 1024, 1024, 2), draft=_cfg(1, 128, 1, 128, 512, 1024, 2),
                    prompt_len=16, n_new=64, K=4, T=1.0),
    # one int8 layer wide enough (d_model = d_ff = 4096) for the 4096-long k-ranges the int8 kernel uses at one or two rows
    "q8_d4096": dict(target=_cfg(1, 4096, 32, 128, 4096, 512, 2), draft=_cfg(1, 4096, 32, 128, 4096, 512, 2),
                     prompt_len=4, n_new=8, K=1, T=1.0),
    "70b_q8": dict(target=_cfg(80, 8192, 64, 128, 32768, 32000, 2), draft=_cfg(8, 6144, 48, 128, 24576, 32000, 2),
                   prompt_len=128, n_new=128, K=4, T=1.0),
    # fewer key / value heads than query heads: grouped (4 -> 2) target, multi-query (2 -> 1) draft, fp32
    "tiny_gqa": dict(target=_cfg(2, 256, 4, 64, 1024, 1024, 0, 2), draft=_cfg(1, 128, 2, 64, 512, 1024, 0, 1),
                     prompt_len=16, n_new=64, K=4, T=1.0),
    # multi-query attention with bf16 storage (2 query heads share one key / value head)
    "tiny_mqa_bf16": dict(target=_cfg(2, 256, 2, 128, 1024, 1024, 1, 1), draft=_cfg(1, 128, 1, 128, 512, 1024, 1, 1),
                          prompt_len=16, n_new=64, K=4, T=1.0),
    # the 70B-shaped pair with 8 key / value heads (the KV cache shrinks 8x and 6x)
    "70b_gqa8": dict(target=_cfg(80, 8192, 64, 128, 32768, 32000, 1, 8), draft=_cfg(8, 6144, 48, 128, 24576, 32000, 1, 8),
                     prompt_len=128, n_new=128, K=4, T=1.0),
    "mid": dict(target=_cfg(24, 2048, 16, 128, 8192, 32000, 1), draft=_cfg(6, 1024, 8, 128, 4096, 32000, 1),
                prompt_len=128, n_new=256, K=4, T=1.0),
    # Hyperparams table: target 8192 / 64 heads / 80 layers, draft 6144 / 48 heads / 8 layers
    "70b": dict(target=_cfg(80, 8192, 64, 128, 32768, 32000, 1), draft=_cfg(8, 6144, 48, 128, 24576, 32000, 1),
                prompt_len=128, n_new=128, K=4, T=1.0),
}

LAYER_MATS = ("wq", "wk", "wv", "wo", "w_up", "w_down")


def _shape(cfg, name):
    d, f, v = cfg["d_model"], cfg["d_ff"], cfg["vocab"]
    dkv = cfg.get("n_kv_heads", cfg["n_heads"]) * cfg["d_head"]
    return {"tok_embed": (v, d), "unembed": (v, d), "wq": (d, d), "wk": (dkv, d), "wv": (dkv, d), "wo": (d, d),
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
    For dtype 2 the bf16 matrices are drawn the same way and then quantised (quantize_weights).

    share_embed_from: weights of a wider model whose first d_model columns of tok_embed / unembed are
    reused (the 70B-shaped pair shares its (un)embedding so that acceptance is non-zero).
    body_gain: scales wo and w_down (a documented deviation used only to reach higher acceptance).
    """
    tdt = torch.float32 if cfg["dtype"] == 0 else torch.bfloat16
    w = {}
    for name in ("tok_embed", "unembed"):
        if share_embed_from is not None:
            src = share_embed_from[name][:, : cfg["d_model"]]
            if src.dtype == torch.int8:      # an int8 source: back to bf16 first, quantised again below
                src = (src.float() * share_embed_from[name + "_scale"][:, None]).to(tdt)
            w[name] = src.contiguous()
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
    return quantize_weights(w) if cfg["dtype"] == 2 else w


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
    out = {k: v.to(device) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: v.to(device) for k, v in lw.items()} for lw in w["layers"]]
    return out


def quantize_rows(W):
    """Weight-only int8, one scale per output row: scale = max|w| / 127, byte = round(w / scale).  Returns
    (int8 [N, D], fp32 [N]).  Pure data preparation: what a matrix multiplied by these means is defined by the
    oracle on the dequantised matrix and by the library's kernels, each on its own."""
    Wf = W.float()
    scale = (Wf.abs().amax(dim=1).clamp_min(1e-12) / 127.0).float()
    q = torch.clamp(torch.round(Wf / scale[:, None]), -127, 127).to(torch.int8)
    return q, scale


def quantize_weights(w):
    """bf16 weights -> the dtype-2 layout: int8 linear matrices and unembedding with `<name>_scale`, bf16 token
    embedding, fp32 gains.  Matrices are converted one at a time (the 70B shape does not fit twice)."""
    out = {"tok_embed": w["tok_embed"], "final_norm": w["final_norm"]}
    out["unembed"], out["unembed_scale"] = quantize_rows(w["unembed"])
    out["layers"] = []
    for lw in w["layers"]:
        q = {"attn_norm": lw["attn_norm"], "ffn_norm": lw["ffn_norm"]}
        for k in LAYER_MATS:
            q[k], q[k + "_scale"] = quantize_rows(lw[k])
            lw[k] = None
        out["layers"].append(q)
    return out


def dequantized_numpy(wq):
    """What the oracle reads for a dtype-2 model: fp32 matrices scale * byte (exact in fp32), the bf16 token
    embedding widened to fp32.  Use with an fp32-weights oracle whose KV cache is bf16."""
    def deq(q, s):
        return (q.double().cpu() * s.double().cpu()[:, None]).float().numpy()
    out = {"tok_embed": wq["tok_embed"].float().cpu().numpy(), "final_norm": wq["final_norm"].cpu().numpy(),
           "unembed": deq(wq["unembed"], wq["unembed_scale"]), "layers": []}
    for lw in wq["layers"]:
        d = {"attn_norm": lw["attn_norm"].cpu().numpy(), "ffn_norm": lw["ffn_norm"].cpu().numpy()}
        for k in LAYER_MATS:
            d[k] = deq(lw[k], lw[k + "_scale"])
        out["layers"].append(d)
    return out


def weight_bytes(cfg):
    """Bytes one forward pass must stream: all layer matrices + unembedding (+ gains, negligible)."""
    es = {0: 4, 1: 2, 2: 1}[cfg["dtype"]]
    d, f, v = cfg["d_model"], cfg["d_ff"], cfg["vocab"]
    dkv = cfg.get("n_kv_heads", cfg["n_heads"]) * cfg["d_head"]
    return cfg["n_layers"] * (2 * d * d + 2 * dkv * d + 2 * d * f) * es + v * d * es


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
