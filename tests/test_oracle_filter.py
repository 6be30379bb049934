"""Pins for the oracle's top-k / nucleus / greedy filtering (section "Modified Rejection Sampling": standard
sampling methods modify the probabilities before the rejection scheme is applied): closed forms on geometric and
tied distributions, the identity settings, Theorem 1 with the filtered target as the law, and greedy decoding."""
import numpy as np
import pytest

import oracle
from test_oracle_sampler import PROMPT, chi_square_p, logit_of, sm, table_models


def geometric(V):
    # p_i proportional to 2^-i
    return (-np.arange(V) * np.log(2.0)).astype(np.float32)


def test_identity_settings_leave_softmax_untouched():
    rng = np.random.default_rng(0)
    for T in (0.7, 1.0, 1.3):
        lg = (rng.normal(size=50) * 3).astype(np.float32)
        want = oracle.softmax(lg, T)
        for k, p in ((0, 1.0), (50, 1.0), (77, 1.0)):
            got, near = oracle.filtered(lg, T, k, p)
            assert np.array_equal(got, want) and not near


def test_top_k_closed_form_on_a_geometric_law():
    lg = geometric(40)
    for k in (1, 2, 3, 7):
        got, _ = oracle.filtered(lg, 1.0, k, 1.0)
        w = 2.0 ** -np.arange(k)
        assert np.allclose(got[:k], w / w.sum(), rtol=1e-6, atol=0)
        assert (got[k:] == 0).all()
        assert abs(got.sum() - 1) < 1e-12


def test_nucleus_closed_form_on_a_geometric_law():
    # cumulative masses 1/2, 3/4, 7/8, 15/16, ...: the first to reach 0.8 is the third, 0.9 the fourth, 0.5 + eps the second
    lg = geometric(40)
    for top_p, n in ((0.8, 3), (0.9, 4), (0.4, 1), (0.6, 2), (0.76, 3)):
        got, near = oracle.filtered(lg, 1.0, 0, top_p)
        w = 2.0 ** -np.arange(n)
        assert np.allclose(got[:n], w / w.sum(), rtol=1e-6, atol=0), (top_p, got[:5])
        assert (got[n:] == 0).all()
        assert not near


def test_nucleus_with_temperature():
    # at T = 0.5 the law is proportional to 4^-i: masses 3/4, 15/16, 63/64
    lg = geometric(30)
    got, _ = oracle.filtered(lg, 0.5, 0, 0.9)
    w = 4.0 ** -np.arange(2)
    assert np.allclose(got[:2], w / w.sum(), rtol=1e-6) and (got[2:] == 0).all()


def test_top_k_then_nucleus():
    # top-3 of the geometric law is (4/7, 2/7, 1/7); 0.8 of that mass is reached at the second token
    lg = geometric(40)
    got, _ = oracle.filtered(lg, 1.0, 3, 0.8)
    assert np.allclose(got[:2], [2 / 3, 1 / 3], rtol=1e-6) and (got[2:] == 0).all()
    # a nucleus wider than the top-k set changes nothing
    a, _ = oracle.filtered(lg, 1.0, 3, 0.999)
    b, _ = oracle.filtered(lg, 1.0, 3, 1.0)
    assert np.array_equal(a, b)


def test_ties_at_the_cut_are_all_kept():
    got, _ = oracle.filtered(np.zeros(8, dtype=np.float32), 1.0, 3, 0.3)
    assert np.allclose(got, 1 / 8)
    lg = np.array([3, 2, 2, 1, 2, 0], dtype=np.float32)
    got, _ = oracle.filtered(lg, 1.0, 2, 1.0)
    assert (got > 0).tolist() == [True, True, True, False, True, False]
    assert np.allclose(got[[1, 2, 4]], got[1])
    # nucleus: exp(3) / Z = 0.53; reaching 0.6 needs the value 2, and all three of its tokens come along
    got, _ = oracle.filtered(lg, 1.0, 0, 0.6)
    assert (got > 0).tolist() == [True, True, True, False, True, False]


def test_exact_boundary_is_cut_there_and_flagged():
    lg = logit_of([0.5, 0.25, 0.25])
    got, near = oracle.filtered(lg, 1.0, 0, 0.5)
    assert got.tolist() == [1.0, 0.0, 0.0] and near
    got, near = oracle.filtered(lg, 1.0, 0, 0.3)
    assert got.tolist() == [1.0, 0.0, 0.0] and not near


def test_order_of_tokens_does_not_matter():
    rng = np.random.default_rng(3)
    lg = (rng.normal(size=64) * 2).astype(np.float32)
    perm = rng.permutation(64)
    for k, p in ((5, 1.0), (0, 0.7), (20, 0.9)):
        a, _ = oracle.filtered(lg, 0.9, k, p)
        b, _ = oracle.filtered(lg[perm], 0.9, k, p)
        assert np.allclose(a[perm], b, rtol=1e-12, atol=0)


@pytest.mark.parametrize("top_k,top_p", [(3, 1.0), (0, 0.7), (6, 0.85)])
def test_theorem_1_holds_for_the_filtered_target(top_k, top_p):
    """The emitted token follows the filtered target law whatever the (filtered) draft is; acceptance = sum min."""
    rng = np.random.default_rng(11)
    V, n = 16, 400_000
    ql, pl = (rng.normal(size=V) * 2).astype(np.float32), (rng.normal(size=V) * 2).astype(np.float32)
    tq, tp = table_models([ql] * 2, [pl] * 2)
    r = oracle.trials(tq, tp, PROMPT, n_new=1, K=1, T=0.9, seed=7, n_trials=n, top_k=top_k, top_p=top_p)
    qf, _ = oracle.filtered(ql, 0.9, top_k, top_p)
    pf, _ = oracle.filtered(pl, 0.9, top_k, top_p)
    tok = r["tokens"][:, 0]
    counts = np.bincount(tok, minlength=V)
    assert counts[qf == 0].sum() == 0
    assert chi_square_p(counts, qf) > 1e-3
    beta = np.minimum(pf, qf).sum()
    acc = (r["first_n_accepted"] == 1).mean()
    assert abs(acc - beta) <= 4 * np.sqrt(beta * (1 - beta) / n) + 1e-12
    # the test has power: the unfiltered target law is rejected
    q_plain = sm(ql.astype(np.float64), 0.9)
    big = q_plain * n >= 5
    stat = ((counts[big] - q_plain[big] * n) ** 2 / (q_plain[big] * n)).sum()
    assert stat > 10 * big.sum()


def test_greedy_is_top_k_1_and_follows_the_target_argmax():
    rng = np.random.default_rng(2)
    V, n_new = 12, 6
    q_rows = [(rng.normal(size=V) * 2).astype(np.float32) for _ in range(n_new + 4)]
    p_rows = [(rng.normal(size=V) * 2).astype(np.float32) for _ in range(n_new + 4)]
    tq, tp = table_models(q_rows, p_rows)
    want = [int(np.argmax(q_rows[i])) for i in range(n_new)]
    for K in (0, 1, 3):
        for seed in (1, 2):
            r = oracle.trials(tq, tp if K else None, PROMPT, n_new=n_new, K=K, T=1.0, seed=seed, n_trials=3, top_k=1)
            assert (r["tokens"] == np.array(want)).all()


def test_chain_with_filters_matches_its_definition_on_one_case():
    # K = 1, V = 4: draft token 2 is outside the target's top-2 set -> rejected whatever u is, resample from q' - p'
    ql = logit_of([0.5, 0.3, 0.15, 0.05])
    pl = logit_of([0.1, 0.2, 0.6, 0.1])
    q = np.stack([ql, ql])
    for seed in range(20):
        r = oracle.accept_chain(q, pl[None], [2], 1.0, seed, 0, 0, top_k=2)
        assert r["n_accepted"] == 0 and r["flags"] & oracle.FLAG_RESAMPLED
        # q' = (5/8, 3/8, 0, 0), p' = (0, 1/4, 3/4, 0): the residual lives on tokens 0 and 1
        assert r["tokens"][0] in (0, 1)
