"""Tensor-parallel sharding on the CPU: the slicing recipe and the schedule of exchanges.

Sharding must not change the function a model computes (section Conditional Scoring: the sharded blocks are each
followed by an all-reduce).  Checked here, without a GPU, on a matrix-form restatement written for this test: (1) the
shards tile the original matrices; (2) the per-rank partial updates, summed after each block, reproduce the unsharded
forward pass (which another test ties to the oracle) to 1e-12, for multi-head, grouped-query and int8-dequantised
weights; (3) the same with two gloo ranks that each hold one shard and all-reduce (K + 1) x d_model numbers twice
per layer."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import sps_synth
from paper_2302_01318_b200 import tensor_parallel as tpar
from test_oracle_model import as_f64, gelu_tanh, matrix_forward, np_weights, round_storage


def block_partials(cfg, scfg, lw, x, which):
    """One rank's partial update of the residual stream x [n, d] from its shard `lw` of a layer: the attention block
    (which = 0) or the feed-forward block (which = 1).  Plain matrix form, float64."""
    d, dh, eps = cfg["d_model"], cfg["d_head"], cfg["rms_eps"]
    H, Hkv = scfg["n_heads"], scfg["n_kv_heads"]
    n = x.shape[0]

    def norm(v, g):
        return g.astype(np.float64) * v / np.sqrt((v ** 2).mean(-1, keepdims=True) + eps)
    if which == 1:
        return gelu_tanh(norm(x, lw["ffn_norm"]) @ as_f64(lw["w_up"]).T) @ as_f64(lw["w_down"]).T
    pos = np.arange(n)[:, None]
    freq = cfg["rope_base"] ** (-2.0 * np.arange(dh // 2) / dh)[None, :]
    cos, sin = np.cos(pos * freq), np.sin(pos * freq)

    def rope(a):
        a0, a1 = a[..., 0::2], a[..., 1::2]
        out = np.empty_like(a)
        out[..., 0::2] = a0 * cos[:, None, :] - a1 * sin[:, None, :]
        out[..., 1::2] = a0 * sin[:, None, :] + a1 * cos[:, None, :]
        return out
    h = norm(x, lw["attn_norm"])
    q = rope((h @ as_f64(lw["wq"]).T).reshape(n, H, dh))
    k = round_storage(rope((h @ as_f64(lw["wk"]).T).reshape(n, Hkv, dh)), cfg["dtype"])
    v = round_storage((h @ as_f64(lw["wv"]).T).reshape(n, Hkv, dh), cfg["dtype"])
    k, v = np.repeat(k, H // Hkv, axis=1), np.repeat(v, H // Hkv, axis=1)
    sc = np.einsum("ihd,jhd->hij", q, k) / np.sqrt(dh)
    sc = np.where(np.tril(np.ones((n, n), dtype=bool))[None], sc, -np.inf)
    pr = np.exp(sc - sc.max(-1, keepdims=True))
    pr /= pr.sum(-1, keepdims=True)
    o = np.einsum("hij,jhd->ihd", pr, v).reshape(n, H * dh)
    return o @ as_f64(lw["wo"]).T


def sharded_forward(cfg, shards, toks, reduce):
    """The tensor-parallel schedule: every block's partial updates are combined by `reduce` (the all-reduce) and added
    to the residual stream that all ranks share; shards[r] is rank r's weights (None for ranks held elsewhere)."""
    world = len(shards)
    scfg = tpar.shard_config(cfg, world)
    first = next(s for s in shards if s is not None)
    x = as_f64(first["tok_embed"])[toks]
    for l in range(cfg["n_layers"]):
        for which in (0, 1):
            x = x + reduce([block_partials(cfg, scfg, s["layers"][l], x, which) if s is not None else None for s in shards])
    g = first["final_norm"].astype(np.float64)
    return (g * x / np.sqrt((x ** 2).mean(-1, keepdims=True) + cfg["rms_eps"])) @ as_f64(first["unembed"]).T


@pytest.mark.parametrize("name,tag,world", [("tiny", "target", 2), ("tiny", "target", 4), ("tiny", "draft", 2),
                                            ("tiny_bf16", "target", 2), ("tiny_gqa", "target", 2)])
def test_sharded_partials_sum_to_the_unsharded_forward(name, tag, world):
    cfg = sps_synth.CONFIGS[name][tag]
    w = np_weights(cfg, seed=1, tag=tag, std=0.08)
    shards = [tpar.shard_weights(cfg, w, r, world) for r in range(world)]
    # (1) the shards tile the matrices
    for l, lw in enumerate(w["layers"]):
        for k in tpar.ROW_SHARDED:
            assert np.array_equal(np.concatenate([s["layers"][l][k] for s in shards], axis=0), lw[k])
        for k in tpar.COL_SHARDED:
            assert np.array_equal(np.concatenate([s["layers"][l][k] for s in shards], axis=1), lw[k])
        assert all(s["layers"][l][k].flags["C_CONTIGUOUS"] for s in shards for k in tpar.ROW_SHARDED + tpar.COL_SHARDED)
    sc = tpar.shard_config(cfg, world)
    assert sc["d_model"] == cfg["d_model"] and sc["n_heads"] * world == cfg["n_heads"] and sc["d_ff"] * world == cfg["d_ff"]
    # (2) summing the ranks' partial updates after every block reproduces the whole model
    toks = sps_synth.make_prompt(3, 9, cfg["vocab"])
    got = sharded_forward(cfg, shards, toks, lambda parts: sum(parts))
    want = matrix_forward(cfg, w, toks)
    assert np.abs(got - want).max() < 1e-12 * max(1.0, np.abs(want).max())


def test_int8_shards_dequantise_to_slices_of_the_dequantised_matrices():
    cfg = sps_synth.CONFIGS["tiny_q8"]["target"]
    wq = sps_synth.make_weights(cfg, seed=0, tag="target", std=0.08)
    full = sps_synth.dequantized_numpy(wq)
    for r in range(2):
        sh = sps_synth.dequantized_numpy(tpar.shard_weights(cfg, wq, r, 2))
        ref = tpar.shard_weights(dict(cfg, dtype=0), full, r, 2)
        for l in range(cfg["n_layers"]):
            for k in tpar.ROW_SHARDED + tpar.COL_SHARDED:
                assert np.array_equal(sh["layers"][l][k], ref["layers"][l][k]), (r, l, k)


def test_sharding_refuses_what_it_cannot_split():
    cfg = sps_synth.CONFIGS["tiny_gqa"]["draft"]          # one key / value head
    w = np_weights(cfg, tag="draft")
    with pytest.raises(ValueError):
        tpar.shard_weights(cfg, w, 0, 2)
    with pytest.raises(ValueError):
        tpar.shard_weights(sps_synth.CONFIGS["tiny"]["target"], np_weights(sps_synth.CONFIGS["tiny"]["target"]), 2, 2)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = sps_synth.CONFIGS["tiny"]["target"]
    w = np_weights(cfg, seed=1, tag="target", std=0.08)       # every rank draws the same weights and keeps its shard only
    shards = [tpar.shard_weights(cfg, w, r, world) if r == rank else None for r in range(world)]
    toks = sps_synth.make_prompt(3, 5, cfg["vocab"])            # K + 1 = 5 rows
    msgs = []

    def all_reduce(parts):
        t = torch.from_numpy(parts[rank].copy())
        msgs.append(tuple(t.shape))
        dist.all_reduce(t)
        return t.numpy()
    got = sharded_forward(cfg, shards, toks, all_reduce)
    out[rank] = (got, msgs)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_follow_the_exchange_schedule():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    cfg = sps_synth.CONFIGS["tiny"]["target"]
    w = np_weights(cfg, seed=1, tag="target", std=0.08)
    want = matrix_forward(cfg, w, sps_synth.make_prompt(3, 5, cfg["vocab"]))
    for r in range(2):
        got, msgs = out[r]
        assert np.abs(got - want).max() < 1e-12 * max(1.0, np.abs(want).max())
        # two exchanges per layer, each of (K + 1) x d_model numbers
        assert msgs == [(5, cfg["d_model"])] * (2 * cfg["n_layers"])
    assert np.array_equal(out[0][0], out[1][0])      # the ranks end with the same bits
