"""Theorem 1 end to end through the library: the first three tokens that sps_generate_batch emits on the vocab-16
pair follow the target model's own law q(x1) q(x2 | x1) q(x3 | x1 x2) -- across loop boundaries, i.e. through the
extra token, the rollback, the draft's catch-up and the next loop's uniforms -- and every generation equals the
oracle's trial with the same sequence index outside oracle-flagged near ties.

Trial i runs as sequence index i (sps_set_sequence_index0 + position in the batch), so the oracle and the library
see the same uniforms.  The law is enumerated exactly from the oracle's target logits (4096 cells); chi-square with
small cells pooled, pass = p > 1e-3; unflagged mismatches with the oracle's trials <= 5e-5 of the trials."""
import numpy as np
import pytest

import oracle
import sps_synth
from gpu_util import NEAR, make_pair
from test_oracle_model import context_tables, target_law_3
from test_oracle_sampler import chi_square_p

pytestmark = pytest.mark.gpu

N_TRIALS = {1.0: 100_000, 0.25: 50_000}     # generations per (K, T); the oracle itself is pinned at 10^6 on the CPU


@pytest.fixture(scope="module")
def tiny16():
    c = sps_synth.CONFIGS["tiny16"]
    prompt = sps_synth.make_prompt(0, 6, 16)       # a short prompt: the prompt pass is repeated for every batch of trials
    wt = sps_synth.weights_to_numpy(sps_synth.make_weights(c["target"], tag="target"))
    wd = sps_synth.weights_to_numpy(sps_synth.make_weights(c["draft"], tag="draft"))
    tq = context_tables(c["target"], wt, prompt, 16, 2)
    tp = context_tables(c["draft"], wd, prompt, 16, 2)
    return prompt, tq, tp


@pytest.mark.parametrize("K,T", [(1, 1.0), (2, 1.0), (4, 1.0), (1, 0.25), (2, 0.25), (4, 0.25)])
def test_first_three_tokens_follow_the_target_law(tiny16, K, T):
    prompt, tq, tp = tiny16
    P = len(prompt)
    B = min(8, 16 // (K + 1))                     # fp32 pair: batch x (K + 1) <= 16 rows per pass
    h = make_pair("tiny16", max_seq=32, max_batch=B, max_K=K)[0]
    n = (N_TRIALS[T] + B - 1) // B * B
    got = np.zeros((n, 3), dtype=np.int32)
    prompts = np.tile(prompt, (B, 1))
    seed = 2024
    for i0 in range(0, n, B):
        h.sps_set_sequence_index0(i0)
        toks, _ = h.sps_generate_batch(prompts, 3, K, T, seed)
        got[i0:i0 + B] = toks
    h.close()
    assert ((got >= 0) & (got < 16)).all()
    # (1) the law, exactly enumerated from the oracle's target
    counts = np.bincount(got[:, 0] * 256 + got[:, 1] * 16 + got[:, 2], minlength=4096)
    law = target_law_3(tq, T)
    pval = chi_square_p(counts, law)
    # (2) generation by generation against the oracle's trials (table models of the same logits)
    mq, mp = oracle.TableModel(tq, 2, P), oracle.TableModel(tp, 2, P)
    r = oracle.trials_flagged(mq, mp, prompt, n_new=3, K=K, T=T, seed=seed, n_trials=n)
    differ = (got != r["tokens"]).any(axis=1)
    flagged = (r["flags"] & NEAR) != 0
    unflagged = int((differ & ~flagged).sum())
    print(f"K={K} T={T}: {n} generations, chi-square p = {pval:.3f}, {int(differ.sum())} differ from the oracle's "
          f"({int(flagged.sum())} flagged), {unflagged} of them unflagged")
    assert pval > 1e-3
    assert unflagged <= 5e-5 * n
    # the test has power: the draft's own law is rejected outright wherever it differs from the target's
    if T < 1.0:
        assert chi_square_p(counts, target_law_3(tp, T)) < 1e-6
