"""Helpers shared by the GPU parity tests: weights on both sides, oracle / library pairs."""
import numpy as np
import torch

import oracle
import paper_2302_01318_b200 as sps
import sps_synth


def have_gpu():
    return torch.cuda.is_available()


def oracle_model(cfg, w, max_seq):
    """The oracle over the same weights; an int8-weight model is the fp32 model of its dequantised matrices with
    the keys and values cached in bf16."""
    if cfg["dtype"] == 2:
        return oracle.Transformer(dict(cfg, dtype=0), sps_synth.dequantized_numpy(w), max_seq, cache_dtype=1)
    return oracle.Transformer(cfg, sps_synth.weights_to_numpy(w), max_seq)


def make_pair(name, max_seq=160, max_batch=1, max_K=4, flags=0, seed=0, draft_equals_target=False, std=0.02):
    """(library handle, oracle target, oracle draft, config) over the very same weights."""
    c = sps_synth.CONFIGS[name]
    wt = sps_synth.make_weights(c["target"], seed=seed, tag="target", std=std)
    if draft_equals_target:
        wd, dcfg = wt, c["target"]
    else:
        wd, dcfg = sps_synth.make_weights(c["draft"], seed=seed, tag="draft", std=std), c["draft"]
    ot, od = oracle_model(c["target"], wt, max_seq), oracle_model(dcfg, wd, max_seq)
    gt = sps_synth.weights_to(wt, "cuda")
    gd = gt if draft_equals_target else sps_synth.weights_to(wd, "cuda")
    h = sps.Handle(c["target"], gt, dcfg, gd, max_seq=max_seq, max_batch=max_batch, max_K=max_K, flags=flags)
    return h, ot, od, c


NEAR = oracle.FLAG_NEAR_ACCEPT | oracle.FLAG_NEAR_CDF
