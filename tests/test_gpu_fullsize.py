"""Parity at the bench's full layer shapes: the 70B-shaped target (d 8192, FFN 32768, 64 heads, V 32000) and
the 4B-shaped draft (d 6144, FFN 24576, 48 heads) with a reduced layer count, so that every kernel runs
in exactly the launch configuration `bench.py` times (same grids, k-splits and tile queues), and the
oracle -- fed the very weights read back from the device, one layer at a time -- finishes in seconds.
Tolerance: bf16 models, logits within 5e-2 abs (the benchmark spec); observed error is ~1e-3."""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2302_01318_b200 as sps
import sps_synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def oracle_logits(cfg, w_dev, tokens, positions_ctx, rows):
    """prefix tokens at positions 0..len-1 go through the oracle layer by layer together with `rows`; an int8 model is
    the fp32 model of its dequantised matrices with a bf16 cache"""
    seq = np.concatenate([tokens, rows]).astype(np.int32)
    pos = np.arange(len(seq), dtype=np.int32)
    q8 = cfg["dtype"] == 2
    emb_t = w_dev["tok_embed"][torch.from_numpy(seq.astype(np.int64)).to(DEV)]
    if q8:
        m = oracle.Transformer(dict(cfg, dtype=0), None, len(seq) + 1, cache_dtype=1)
        m.begin_rows(emb_t.float().cpu().numpy(), pos)
        for l, lw in enumerate(w_dev["layers"]):
            one = {k: lw[k].cpu().numpy() for k in ("attn_norm", "ffn_norm")}
            for k in sps_synth.LAYER_MATS:
                one[k] = (lw[k].float() * lw[k + "_scale"][:, None]).cpu().numpy()
            m.layer(l, one)
        un = (w_dev["unembed"].float() * w_dev["unembed_scale"][:, None]).cpu().numpy()
        out = m.end(sps_synth.to_numpy(w_dev["final_norm"]), un)
    else:
        m = oracle.Transformer(cfg, None, len(seq) + 1)
        m.begin_rows(sps_synth.to_numpy(emb_t), pos)
        for l, lw in enumerate(w_dev["layers"]):
            m.layer(l, {k: sps_synth.to_numpy(v) for k, v in lw.items()})
        out = m.end(sps_synth.to_numpy(w_dev["final_norm"]), sps_synth.to_numpy(w_dev["unembed"]))
    return out[len(tokens):]


@pytest.mark.parametrize("name", ["70b", "70b_q8", "70b_gqa8"])
def test_scoring_pass_at_70b_layer_shapes(name):
    c = sps_synth.CONFIGS[name]
    tc, dc = dict(c["target"], n_layers=2), dict(c["draft"], n_layers=1)
    wt = sps_synth.make_weights(tc, tag="target", device=DEV)
    wd = sps_synth.make_weights(dc, tag="draft", device=DEV, share_embed_from=wt)
    h = sps.Handle(tc, wt, dc, wd, max_seq=64, max_K=4)
    V = tc["vocab"]
    prompt = sps_synth.make_prompt(0, 20, V)
    rows = np.concatenate([prompt[-1:], sps_synth.make_prompt(1, 4, V)])
    h.sps_prefill(prompt)
    out = torch.zeros((5, V), device=DEV)
    worst = {}
    for which, cfg, w in ((0, tc, wt), (1, dc, wd)):
        h.sps_score(which, rows, out)
        got = out.cpu().numpy().astype(np.float64)
        want = oracle_logits(cfg, w, prompt[:-1], None, rows)
        worst[which] = float(np.abs(got - want).max())
        assert np.isfinite(got).all()
        assert worst[which] < 5e-2, worst
    print("worst logit error target / draft:", worst)
    # the whole loop runs at these shapes and keeps its invariants
    for K in (4, 1, 2):   # K = 1, 2: other shared-memory sizes of the cluster sampler at this vocabulary
        toks, st = h.sps_generate(prompt, 12, K, 1.0, 3)
        assert ((toks >= 0) & (toks < V)).all() and st["loops"] == sum(st["hist_emitted"]) and st["emitted"] - st["overshoot"] == 12
    h.close()


def test_scoring_pass_of_twelve_rows_at_70b_layer_shapes():
    """9..16 rows per pass (two or three sequences' K + 1 rows) stream the weights through the same tcgen05 kernel with
    a 32-column activation operand: twelve rows against the oracle, same tolerance."""
    c = sps_synth.CONFIGS["70b"]
    tc = dict(c["target"], n_layers=2)
    wt = sps_synth.make_weights(tc, tag="target", device=DEV)
    h = sps.Handle(tc, wt, None, None, max_seq=64, max_K=11)
    V = tc["vocab"]
    prompt = sps_synth.make_prompt(0, 9, V)
    rows = np.concatenate([prompt[-1:], sps_synth.make_prompt(1, 11, V)])
    h.sps_prefill(prompt)
    out = torch.zeros((12, V), device=DEV)
    h.sps_score(0, rows, out)
    got = out.cpu().numpy().astype(np.float64)
    want = oracle_logits(tc, wt, prompt[:-1], None, rows)
    err = float(np.abs(got - want).max())
    assert np.isfinite(got).all() and err < 5e-2, err
    h.close()


@pytest.mark.skipif(os.environ.get("SPS_SKIP_FULL_DEPTH") == "1",
                    reason="about a minute of CPU oracle time (80 layers of the 70B shape, one at a time); SPS_SKIP_FULL_DEPTH=1 was set")
def test_scoring_pass_at_full_depth():
    """All 80 layers of the 70B-shaped target: a 3-token prompt, then one scoring pass over five rows, against the
    oracle fed the same weights layer by layer (seven oracle rows in all: its cost is per row).  The bf16 tolerance
    (5e-2 abs) must hold at full depth too."""
    tc = sps_synth.CONFIGS["70b"]["target"]
    wt = sps_synth.make_weights(tc, tag="target", device=DEV)
    h = sps.Handle(tc, wt, None, None, max_seq=64, max_K=4)
    V = tc["vocab"]
    prompt = sps_synth.make_prompt(0, 3, V)
    rows = np.concatenate([prompt[-1:], sps_synth.make_prompt(1, 4, V)])
    h.sps_prefill(prompt)
    out = torch.zeros((5, V), device=DEV)
    h.sps_score(0, rows, out)
    got = out.cpu().numpy().astype(np.float64)
    want = oracle_logits(tc, wt, prompt[:-1], None, rows)
    err = float(np.abs(got - want).max())
    print(f"full depth (80 layers): worst logit error {err:.3e}, logits span [{want.min():.1f}, {want.max():.1f}]")
    assert np.isfinite(got).all() and err < 5e-2, err
    h.close()
