"""Pins for the oracle's adaptive lookahead: K follows its rule on sequences whose acceptance is known in
advance, and -- since K only depends on the past -- the generated tokens still follow the target's law
(Theorem 1 applies to every loop)."""
import numpy as np

import oracle
from test_oracle_sampler import PROMPT, chi_square_p, logit_of, sm, table_models


def test_identical_models_grow_the_lookahead_to_its_maximum():
    # p == q: every draft is accepted, a loop at lookahead K emits K + 1 tokens and K grows by one up to K_max.
    # K_min 1, K_max 5: K = 3, 4, 5, 5, ... -> tokens 4, 5, 6, 6, ...; 30 tokens need 4 + 5 + 6 + 6 + 6 + 6 = 33 >= 30: 6 loops
    rng = np.random.default_rng(0)
    rows = [(rng.normal(size=8) * 2).astype(np.float32) for _ in range(64)]
    tq, tp = table_models(rows, rows)
    r = oracle.Sps(tq, tp).generate_adaptive(PROMPT, 30, 1, 5, 1.0, 3)
    assert r["loops"] == 6 and r["draft_calls"] == 3 + 4 + 5 + 5 + 5 + 5


def test_disjoint_models_shrink_the_lookahead_to_its_minimum():
    # the draft only proposes tokens the target gives no mass: the first draft is always rejected, one token per loop,
    # K = 3, 2, 1, 1, ... with K_min 1, K_max 5
    q = logit_of([0.5, 0.5, 0.0, 0.0])
    p = logit_of([0.0, 0.0, 0.5, 0.5])
    tq, tp = table_models([q] * 32, [p] * 32)
    r = oracle.Sps(tq, tp).generate_adaptive(PROMPT, 10, 1, 5, 1.0, 9)
    assert r["loops"] == 10 and r["draft_calls"] == 3 + 2 + 1 * 8
    assert set(r["tokens"].tolist()) <= {0, 1}


def test_equal_bounds_reproduce_the_fixed_lookahead():
    rng = np.random.default_rng(2)
    q_rows = [(rng.normal(size=12) * 2).astype(np.float32) for _ in range(40)]
    p_rows = [(rng.normal(size=12) * 2).astype(np.float32) for _ in range(40)]
    tq, tp = table_models(q_rows, p_rows)
    s = oracle.Sps(tq, tp)
    a = s.generate_adaptive(PROMPT, 20, 3, 3, 0.8, 5)
    b = s.generate(PROMPT, 20, 3, 0.8, 5)
    assert (a["tokens"] == b["tokens"]).all() and a["loops"] == b["loops"]


def test_output_law_is_the_targets_under_adaptive_lookahead():
    """First three tokens of depth-2 table models against q(x1) q(x2 | x1) q(x3 | x1 x2), enumerated exactly."""
    V, n = 4, 300_000
    rng = np.random.default_rng(7)
    nctx = 1 + V + V * V
    tq = oracle.TableModel((rng.normal(size=(nctx, V)) * 1.5).astype(np.float32), depth=2, pos0=len(PROMPT) - 1)
    tp = oracle.TableModel((rng.normal(size=(nctx, V)) * 1.5).astype(np.float32), depth=2, pos0=len(PROMPT) - 1)
    r = oracle.trials_adaptive(tq, tp, PROMPT, 3, 1, 4, 1.0, 11, n)
    toks = r["tokens"]
    counts = np.zeros((V, V, V))
    np.add.at(counts, (toks[:, 0], toks[:, 1], toks[:, 2]), 1)
    # the target's law of three tokens from sequential scoring of every prefix
    want = np.zeros((V, V, V))

    def q_next(prefix):     # the target's next-token law after the prompt and `prefix`, from its own forward
        seq = np.concatenate([PROMPT, np.array(prefix, dtype=np.int32)])
        lg = tq.forward(seq[len(PROMPT) - 1:], np.arange(len(PROMPT) - 1, len(seq)))
        return sm(lg[-1].astype(np.float64))
    q1 = q_next([])
    for x1 in range(V):
        q2 = q_next([x1])
        for x2 in range(V):
            q3 = q_next([x1, x2])
            want[x1, x2] = q1[x1] * q2[x2] * q3
    assert abs(want.sum() - 1) < 1e-9
    assert chi_square_p(counts, want) > 1e-3
