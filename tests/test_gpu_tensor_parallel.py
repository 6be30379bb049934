"""Tensor-parallel scoring on the GPU: a group of rank handles emulated on one GPU (the library's group calls step
the ranks through every pass phase by phase) against the oracle's UNSHARDED model and against an unsharded handle.
The real kernels run: every rank streams only its shard of the weights, and the two exchanges per layer go through
the push / reduce kernels and the inbox / flag buffers, with device pointers in place of peer mappings.
Tolerances: logits within 1e-3 (fp32) / 5e-2 (bf16, int8) of the oracle; every rank's logits bit-identical."""
import numpy as np
import pytest
import torch

import paper_2302_01318_b200 as sps
import sps_synth
from gpu_util import oracle_model
from paper_2302_01318_b200 import tensor_parallel as tpar

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL = {"tiny": 1e-3, "tiny_bf16": 5e-2, "tiny_q8": 5e-2, "tiny_gqa": 1e-3}


@pytest.mark.parametrize("name,world,with_draft", [("tiny", 2, True), ("tiny", 4, False), ("tiny_bf16", 2, False),
                                                   ("tiny_q8", 2, False), ("tiny_gqa", 2, False)])
def test_group_scoring_equals_the_unsharded_model(name, world, with_draft):
    c = sps_synth.CONFIGS[name]
    wt = sps_synth.make_weights(c["target"], tag="target")
    wd = sps_synth.make_weights(c["draft"], tag="draft") if with_draft else None
    gt = sps_synth.weights_to(wt, DEV)
    gd = sps_synth.weights_to(wd, DEV) if with_draft else None
    g = tpar.Group(world, c["target"], gt, c["draft"] if with_draft else None, gd, max_seq=96, max_K=4)
    V = c["target"]["vocab"]
    prompt = sps_synth.make_prompt(0, 40, V)                 # three prompt passes of up to 16 rows
    rows = np.concatenate([prompt[-1:], sps_synth.make_prompt(1, 4, V)])
    g.prefill(prompt)
    outs = [torch.zeros((5, V), device=DEV) for _ in range(world)]
    for which, cfg, w in ((0, c["target"], wt), (1, c["draft"], wd)):
        if w is None:
            continue
        g.score(which, rows, outs)
        torch.cuda.synchronize()
        om = oracle_model(cfg, w, 96)
        om.forward(prompt[:-1], np.arange(39), want_logits=False)
        want = om.forward64(rows, np.arange(39, 44))
        got = outs[0].cpu().numpy()
        err = np.abs(got - want).max()
        print(f"{name} x{world} model {which}: logit error vs the oracle {err:.2e}")
        assert err < TOL[name], err
        for r in range(1, world):
            assert torch.equal(outs[r], outs[0])             # same summation order on every rank
    # the unsharded handle on the same weights, same rows
    h = sps.Handle(c["target"], gt, None, None, max_seq=96, max_K=4)
    h.sps_prefill(prompt)
    ref = torch.zeros((5, V), device=DEV)
    g.score(0, rows, outs)
    h.sps_score(0, rows, ref)
    torch.cuda.synchronize()
    assert (outs[0] - ref).abs().max().item() < TOL[name] * 0.1
    # scoring again rewrites the same positions: same bits (exchange numbering carries on)
    again = [torch.zeros((5, V), device=DEV) for _ in range(world)]
    g.score(0, rows, again)
    torch.cuda.synchronize()
    assert torch.equal(again[0], outs[0])
    h.close()
    g.close()


@pytest.mark.parametrize("name,world", [("tiny", 2), ("tiny", 4)])
def test_group_generation_equals_the_oracle_loop(name, world):
    """The whole loop under tensor parallelism (both models sharded, every rank drafting, scoring and sampling on its
    own copy of the logits): rank 0's tokens equal the UNSHARDED oracle's outside flagged near ties, and the ranks never
    decide differently (the call itself checks that after every loop)."""
    import oracle
    from gpu_util import oracle_generate, same_or_flagged
    c = sps_synth.CONFIGS[name]
    # four ranks need a draft with four heads: one layer of the target's width stands in for the two-head draft
    dcfg = c["draft"] if c["draft"]["n_heads"] % world == 0 else dict(c["target"], n_layers=1, d_ff=512)
    wt = sps_synth.make_weights(c["target"], tag="target")
    wd = sps_synth.make_weights(dcfg, tag="draft")
    g = tpar.Group(world, c["target"], sps_synth.weights_to(wt, DEV), dcfg, sps_synth.weights_to(wd, DEV), max_seq=128, max_K=4)
    osps = oracle.Sps(oracle_model(c["target"], wt, 128), oracle_model(dcfg, wd, 128))
    V = c["target"]["vocab"]
    ok = 0
    for seed in range(4):
        prompt = sps_synth.make_prompt(seed, 16, V)
        got, st = g.generate(prompt, 32, 4, 1.0, seed)
        assert st["emitted"] - st["overshoot"] == 32 and st["loops"] == sum(st["hist_emitted"])
        ok += same_or_flagged(got, oracle_generate(osps, prompt, 32, 4, 1.0, seed))
    assert ok >= 3
    g.close()


def test_a_rank_whose_peer_never_arrives_gives_up_within_the_bound():
    """The per-process form of a pass on rank 0 alone: its peer never stores its partial update nor raises its flag,
    so the reduction's wait on that flag runs out (bound shortened to 3 ms), the kernel returns and the call reports
    SPS_ETIMEOUT -- nothing hangs, and the group works afterwards."""
    c = sps_synth.CONFIGS["tiny"]
    wt = sps_synth.make_weights(c["target"], tag="target")
    g = tpar.Group(2, c["target"], sps_synth.weights_to(wt, DEV), None, None, max_seq=64, max_K=4)
    V = c["target"]["vocab"]
    prompt = sps_synth.make_prompt(0, 8, V)
    sps.sps_debug_set_wait(3000, -1)
    try:
        with pytest.raises(sps.SpsError) as e:
            g.ranks[0].sps_prefill(prompt)          # a collective call made by one rank only
        assert e.value.code == sps.SPS_ETIMEOUT
    finally:
        sps.sps_debug_set_wait(0, -1)
    g.close()
    # a fresh group on the same device is unaffected
    g = tpar.Group(2, c["target"], sps_synth.weights_to(wt, DEV), None, None, max_seq=64, max_K=4)
    g.prefill(prompt)
    outs = [torch.zeros((1, V), device=DEV) for _ in range(2)]
    g.score(0, prompt[-1:], outs)
    torch.cuda.synchronize()
    om = oracle_model(c["target"], wt, 64)
    om.forward(prompt[:-1], np.arange(7), want_logits=False)
    assert np.abs(outs[0].cpu().numpy() - om.forward64(prompt[-1:], [7])).max() < 1e-3
    g.close()


def test_tensor_parallel_handles_state_their_requirements():
    c = sps_synth.CONFIGS["tiny"]
    gt = sps_synth.weights_to(sps_synth.make_weights(c["target"], tag="target"), DEV)
    sw = tpar.shard_weights(c["target"], gt, 0, 2)
    sc = tpar.shard_config(c["target"], 2)
    with pytest.raises(sps.SpsError):                         # a shard's shape without the flag
        sps.Handle(sc, sw, None, None, max_seq=64)
    h = sps.Handle(sc, sw, None, None, max_seq=64, flags=sps.CFG_TENSOR_PARALLEL)
    with pytest.raises(sps.SpsError) as e:                    # a pass before the peers are attached
        h.sps_prefill(sps_synth.make_prompt(0, 8, c["target"]["vocab"]))
    assert e.value.code == sps.SPS_ESTATE
    inbox, flags, nb, nf = h.tp_buffers()
    assert inbox and flags and nb > 0 and nf > 0
    with pytest.raises(sps.SpsError):                         # the own entry must be the own buffers
        h.tp_attach(0, 2, [flags, inbox], [flags, flags])
    h.close()
