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


def make_pair_multi(name, n, max_seq=160, max_K=4, flags=0, seed=0, std=0.02):
    """One library handle for n sequences and n oracle (target, draft) pairs over the same weights, each oracle pair
    with KV caches of its own (the oracle runs one sequence per model instance)."""
    c = sps_synth.CONFIGS[name]
    wt = sps_synth.make_weights(c["target"], seed=seed, tag="target", std=std)
    wd = sps_synth.make_weights(c["draft"], seed=seed, tag="draft", std=std)
    ots = [oracle_model(c["target"], wt, max_seq) for _ in range(n)]
    ods = [oracle_model(c["draft"], wd, max_seq) for _ in range(n)]
    h = sps.Handle(c["target"], sps_synth.weights_to(wt, "cuda"), c["draft"], sps_synth.weights_to(wd, "cuda"),
                   max_seq=max_seq, max_batch=n, max_K=max_K, flags=flags)
    return h, ots, ods, c


NEAR = oracle.FLAG_NEAR_ACCEPT | oracle.FLAG_NEAR_CDF


def oracle_generate(osps, prompt, n_new, K, T, seed, b=0, near=NEAR, K_min=None):
    """The oracle's generation taken loop by loop.  Besides the tokens it returns `first_flag`: the index of the first
    token that an oracle-flagged near tie could have changed (every token from the first flagged loop on), or None.
    A correct implementation may differ from the oracle at or after that index, never before it."""
    osps.reset(prompt)
    toks, s, first, drafts = [], 0, None, 0
    hist = np.zeros(K + 2, dtype=np.int64)
    K_max = K
    if K_min is not None:          # adaptive lookahead: the rule of sps_generate_adaptive, restated
        K = (K_min + K_max) // 2
    while len(toks) < n_new:
        r = osps.loop(K, T, seed, b, s)
        drafts += K
        if K_min is not None:
            K = min(K + 1, K_max) if r["n_accepted"] == K else (max(K - 1, K_min) if r["n_accepted"] == 0 else K)
        if first is None and ((r["flags"] & near) or r["draft_near_tie"]):
            first = len(toks)
        toks += [int(t) for t in r["tokens"][:r["n_emitted"]]]
        hist[r["n_emitted"]] += 1
        s += 1
    return {"tokens": np.array(toks[:n_new], dtype=np.int32), "loops": s, "first_flag": first, "hist_emitted": hist,
            "draft_calls": drafts}


def same_or_flagged(got, want):
    """True when `got` equals the oracle's tokens.  Otherwise the first difference must lie at or after the first
    token of the first flagged loop (asserted), and False is returned."""
    got = np.asarray(got)
    if np.array_equal(got, want["tokens"]):
        return True
    first_diff = int(np.nonzero(got != want["tokens"])[0][0])
    assert want["first_flag"] is not None and first_diff >= want["first_flag"], \
        (first_diff, want["first_flag"], got, want["tokens"])
    return False
