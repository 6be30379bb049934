"""Pins for the oracle's modified rejection sampling against what the paper proves (Theorem 1 and
the notes after the acceptance rule): closed forms, exact enumeration, special cases."""
import itertools

import numpy as np
import pytest
from scipy.stats import chi2

import oracle

P = 4  # prompt length used with the table models
PROMPT = np.array([1, 0, 1, 0], dtype=np.int32)


def sm(l, T=1.0):
    l = np.asarray(l, dtype=np.float64) / T
    e = np.exp(l - l.max())
    return e / e.sum()


def logit_of(prob):
    # logits that softmax to `prob`; zero-probability entries get a logit so low that exp underflows to 0
    prob = np.asarray(prob, dtype=np.float64)
    with np.errstate(divide="ignore"):
        lg = np.where(prob > 0, np.log(np.maximum(prob, 1e-300)), -1e4)
    return lg.astype(np.float32)


def chi_square_p(counts, probs, min_expected=5.0):
    """one-sample chi-square p-value, pooling cells whose expected count is small"""
    counts = np.asarray(counts, dtype=np.float64).ravel()
    probs = np.asarray(probs, dtype=np.float64).ravel()
    n = counts.sum()
    exp = probs * n
    assert counts[exp == 0].sum() == 0, "mass observed in a zero-probability cell"
    big = exp >= min_expected
    c = list(counts[big])
    e = list(exp[big])
    if (~big).any() and exp[~big].sum() > 0:
        c.append(counts[~big].sum())
        e.append(exp[~big].sum())
    c, e = np.array(c), np.array(e)
    keep = e > 0
    stat = ((c[keep] - e[keep]) ** 2 / e[keep]).sum()
    return chi2.sf(stat, keep.sum() - 1)


def table_models(q_rows, p_rows):
    """context-free models: row i is the distribution of generated position i"""
    tq = oracle.TableModel(np.stack(q_rows), depth=0, pos0=P - 1)
    tp = oracle.TableModel(np.stack(p_rows), depth=0, pos0=P - 1)
    return tq, tp


CASES_1POS = {
    "v2": ([0.7, 0.3], [0.4, 0.6]),                    # p=(a,1-a), q=(b,1-b), b<a
    "v3_zero_in_q": ([0.5, 0.5, 0.0], [0.2, 0.3, 0.5]),
    "v3_zero_in_p": ([0.25, 0.0, 0.75], [0.1, 0.6, 0.3]),
    "v3_equal": ([0.2, 0.3, 0.5], [0.2, 0.3, 0.5]),
    "v3_near_disjoint": ([0.98, 0.01, 0.01], [0.01, 0.01, 0.98]),
    "v16": (None, None),
}


@pytest.mark.parametrize("name", list(CASES_1POS))
def test_single_position_joint_law(name):
    """Theorem 1: P(accepted, X=x) = min(p,q)(x); P(rejected, X=x) = max(0, q-p)(x); marginal q."""
    p, q = CASES_1POS[name]
    if p is None:
        rng = np.random.default_rng(5)
        p, q = sm(rng.normal(size=16) * 2), sm(rng.normal(size=16) * 2)
    p, q = np.array(p), np.array(q)
    V = len(p)
    n = 1_000_000
    tq, tp = table_models([logit_of(q)] * 2, [logit_of(p)] * 2)
    r = oracle.trials(tq, tp, PROMPT, n_new=1, K=1, T=1.0, seed=42, n_trials=n)
    tok = r["tokens"][:, 0]
    acc = r["first_n_accepted"] == 1
    cells = np.zeros((2, V))
    np.add.at(cells[0], tok[acc], 1)
    np.add.at(cells[1], tok[~acc], 1)
    want = np.stack([np.minimum(p, q), np.maximum(0.0, q - p)])
    assert abs(want.sum() - 1.0) < 1e-12
    assert chi_square_p(cells, want) > 1e-3
    # marginal law is q
    assert chi_square_p(cells.sum(0), q) > 1e-3
    # acceptance probability = sum min(p,q), 4 sigma
    beta = np.minimum(p, q).sum()
    sigma = np.sqrt(max(beta * (1 - beta), 1e-12) / n)
    assert abs(acc.mean() - beta) <= 4 * sigma + 1e-12
    if name == "v2":
        a, b = p[0], q[0]
        assert abs(beta - (1 - (a - b))) < 1e-12
        assert (tok[~acc] == 1).all()          # every resample is token 1
    if name == "v3_equal":
        assert acc.all()                        # p == q: never rejected
        assert (r["first_flags"] & oracle.FLAG_FALLBACK == 0).all()


def test_beta_reported_by_oracle_matches_definition():
    rng = np.random.default_rng(0)
    K, V = 3, 50
    ql = rng.normal(size=(K + 1, V)).astype(np.float32) * 3
    pl = (ql[:K] + rng.normal(size=(K, V))).astype(np.float32)
    for T in (1.0, 0.5):
        r = oracle.accept_chain(ql, pl, [0, 1, 2], T, 1, 0, 0, want_beta=True)
        for t in range(K):
            want = np.minimum(sm(ql[t], T), sm(pl[t], T)).sum()
            assert abs(r["beta"][t] - want) < 1e-12


def exact_chain_law(ps, qs):
    """Brute force over every draft sequence and accept pattern: exact law of (n_accepted, emitted tokens)."""
    K, V = len(ps), len(ps[0])
    law = {}
    for drafts in itertools.product(range(V), repeat=K):
        pd = np.prod([ps[t][drafts[t]] for t in range(K)])
        if pd == 0:
            continue
        reach = pd
        for t in range(K):
            d = drafts[t]
            ratio = min(1.0, qs[t][d] / ps[t][d])
            # rejected at t
            res = np.maximum(0.0, qs[t] - ps[t])
            if res.sum() > 0 and ratio < 1.0:
                res = res / res.sum()
                for x in range(V):
                    if res[x] > 0:
                        key = (t,) + drafts[:t] + (x,)
                        law[key] = law.get(key, 0.0) + reach * (1 - ratio) * res[x]
            reach *= ratio
        for x in range(V):
            key = (K,) + drafts + (x,)
            law[key] = law.get(key, 0.0) + reach * qs[K][x]
    return law


@pytest.mark.parametrize("V,K", [(2, 3), (3, 2), (4, 3)])
def test_chain_matches_exact_enumeration(V, K):
    rng = np.random.default_rng(100 + V * 10 + K)
    qs = [sm(rng.normal(size=V) * 1.5) for _ in range(K + 1)]
    ps = [sm(np.log(qs[t]) + rng.normal(size=V)) for t in range(K)]
    law = exact_chain_law(ps, qs)
    assert abs(sum(law.values()) - 1.0) < 1e-12
    # the exact law itself obeys the theorem: the token emitted at position t, given that position t
    # is reached, follows q_t, whatever happened before
    for t in range(K + 1):
        mass = np.zeros(V)
        for key, pr in law.items():
            a, toks = key[0], key[1:]
            if len(toks) > t:
                mass[toks[t]] += pr
        assert np.allclose(mass / mass.sum(), qs[t], atol=1e-12)
    n = 400_000
    tq, tp = table_models([logit_of(x) for x in qs], [logit_of(x) for x in ps] + [logit_of(ps[-1])])
    r = oracle.trials(tq, tp, PROMPT, n_new=K + 1, K=K, T=1.0, seed=7, n_trials=n)
    # only the first loop's outcome: n_accepted and the a+1 tokens it emitted
    keys = list(law)
    index = {k: i for i, k in enumerate(keys)}
    counts = np.zeros(len(keys))
    for a, row in zip(r["first_n_accepted"], r["tokens"]):
        counts[index[(int(a),) + tuple(int(x) for x in row[: a + 1])]] += 1
    assert chi_square_p(counts, [law[k] for k in keys]) > 1e-3


def test_stop_position_closed_form():
    """P(stop at j) = prod_{i<j} beta_i (1 - beta_j); P(all accepted) = prod beta_i;
    with equal beta the mean number emitted is (1 - beta^{K+1}) / (1 - beta)."""
    rng = np.random.default_rng(5)
    V, K, n = 16, 4, 500_000
    q = sm(rng.normal(size=V))
    p = sm(np.log(q) + rng.normal(size=V) * 0.8)
    beta = np.minimum(p, q).sum()
    assert 0.5 < beta < 0.9
    tq, tp = table_models([logit_of(q)] * (K + 1), [logit_of(p)] * (K + 1))
    r = oracle.trials(tq, tp, PROMPT, n_new=1, K=K, T=1.0, seed=99, n_trials=n)
    a = r["first_n_accepted"]
    want = np.array([beta ** j * (1 - beta) for j in range(K)] + [beta ** K])
    counts = np.bincount(a, minlength=K + 1)
    assert chi_square_p(counts, want) > 1e-3
    mean_emitted = (a + 1).mean()
    want_mean = (1 - beta ** (K + 1)) / (1 - beta)
    assert abs(mean_emitted - want_mean) < 4 * (a.std() / np.sqrt(n))
    # flags: bonus iff all accepted, resampled otherwise
    fl = r["first_flags"]
    assert ((fl & oracle.FLAG_BONUS != 0) == (a == K)).all()
    assert ((fl & oracle.FLAG_RESAMPLED != 0) == (a < K)).all()


def test_temperature_applies_to_both_models():
    rng = np.random.default_rng(8)
    V, n, T = 8, 300_000, 0.5
    ql, pl = rng.normal(size=V).astype(np.float32), rng.normal(size=V).astype(np.float32)
    q, p = sm(ql, T), sm(pl, T)
    tq = oracle.TableModel(np.stack([ql, ql]), depth=0, pos0=P - 1)
    tp = oracle.TableModel(np.stack([pl, pl]), depth=0, pos0=P - 1)
    r = oracle.trials(tq, tp, PROMPT, n_new=1, K=1, T=T, seed=5, n_trials=n)
    tok, acc = r["tokens"][:, 0], r["first_n_accepted"] == 1
    cells = np.zeros((2, V))
    np.add.at(cells[0], tok[acc], 1)
    np.add.at(cells[1], tok[~acc], 1)
    assert chi_square_p(cells, np.stack([np.minimum(p, q), np.maximum(0, q - p)])) > 1e-3


def test_wrong_resampling_rule_is_detected():
    """Negative control: drawing the replacement from q instead of the residual gives
    min(p,q) + (1-beta) q, and the same test must reject it."""
    p, q = np.array([0.7, 0.2, 0.1]), np.array([0.2, 0.3, 0.5])
    tq, tp = table_models([logit_of(q)] * 2, [logit_of(p)] * 2)
    r = oracle.trials(tq, tp, PROMPT, n_new=1, K=1, T=1.0, seed=42, n_trials=200_000, wrong_rule=True)
    counts = np.bincount(r["tokens"][:, 0], minlength=3)
    assert chi_square_p(counts, q) < 1e-6
    beta = np.minimum(p, q).sum()
    assert chi_square_p(counts, np.minimum(p, q) + (1 - beta) * q) > 1e-3


def plain_sampler(logits, T, u):
    """written independently of the oracle: inverse CDF of softmax(l/T) by cumulative sum"""
    w = sm(logits, T)
    c = np.cumsum(w)
    idx = np.nonzero(c > u * c[-1])[0]
    return int(idx[0]) if len(idx) else int(np.nonzero(w > 0)[0][-1])


def test_K0_is_autoregressive_sampling():
    """Algorithm 2 with an empty draft is Algorithm 1: token i is a plain draw from q(.|prefix)
    with u_res of (b, s=i, t=0)."""
    rng = np.random.default_rng(12)
    V, depth = 5, 3
    rows = sum(V ** l for l in range(depth + 1))
    table = (rng.normal(size=(rows, V)) * 2).astype(np.float32)
    tq = oracle.TableModel(table, depth=depth, pos0=P)
    sps = oracle.Sps(tq, None)
    for b in (0, 3):
        out = sps.generate(PROMPT, n_new=3, K=0, T=0.8, seed=17, b=b)
        assert out["loops"] == 3 and out["hist_emitted"][1] == 3
        ctx = []
        for i in range(3):
            off = sum(V ** l for l in range(len(ctx)))
            num = 0
            for tkn in ctx:
                num = num * V + tkn
            u = oracle.uniforms(17, b, i, 0)[2]
            want = plain_sampler(table[off + num], 0.8, u)
            assert out["tokens"][i] == want
            ctx.append(want)


def test_identical_models_accept_everything():
    """p == q: ratio is exactly 1, every draft accepted, K+1 tokens per loop, no fallback."""
    rng = np.random.default_rng(2)
    V, depth, K = 4, 3, 3
    rows = sum(V ** l for l in range(depth + 1))
    table = (rng.normal(size=(rows, V)) * 2).astype(np.float32)
    tq = oracle.TableModel(table, depth=depth, pos0=P)
    tp = oracle.TableModel(table, depth=depth, pos0=P)
    sps = oracle.Sps(tq, tp)
    for seed in range(20):
        sps.reset(PROMPT)
        r = sps.loop(K, 1.0, seed, 0, 0)
        assert r["n_accepted"] == K and r["n_emitted"] == K + 1
        assert r["flags"] & oracle.FLAG_BONUS and not r["flags"] & (oracle.FLAG_RESAMPLED | oracle.FLAG_FALLBACK)


def test_loop_invariants_and_truncation():
    rng = np.random.default_rng(21)
    V, depth = 3, 4
    rows = sum(V ** l for l in range(depth + 1))
    tq = oracle.TableModel((rng.normal(size=(rows, V)) * 2).astype(np.float32), depth=depth, pos0=P)
    tp = oracle.TableModel((rng.normal(size=(rows, V)) * 2).astype(np.float32), depth=depth, pos0=P)
    sps = oracle.Sps(tq, tp)
    for K in (1, 2, 5):
        for n_new in (1, 7, 20):
            out = sps.generate(PROMPT, n_new=n_new, K=K, T=1.0, seed=K * 100 + n_new)
            h = out["hist_emitted"]
            assert h[0] == 0 and h.sum() == out["loops"] <= n_new
            total = sum(j * h[j] for j in range(K + 2))
            assert n_new <= total <= n_new + K      # the last loop may overshoot by at most K
            assert len(out["tokens"]) == n_new and (out["tokens"] >= 0).all() and (out["tokens"] < V).all()


def test_accept_edge_conventions():
    V = 3
    # ratio >= 1 always accepts, whatever u is
    q, p = logit_of([0.6, 0.3, 0.1]), logit_of([0.2, 0.5, 0.3])
    for s in range(200):
        r = oracle.accept_chain(np.stack([q, q]), p[None], [0], 1.0, 3, 0, s)
        assert r["n_accepted"] == 1
    # q(d) == 0 never accepts, and the residual never returns a token with q == 0
    q0 = logit_of([0.0, 0.5, 0.5])
    for s in range(200):
        r = oracle.accept_chain(np.stack([q0, q0]), p[None], [0], 1.0, 3, 0, s)
        assert r["n_accepted"] == 0 and r["tokens"][0] in (1, 2) and r["flags"] & oracle.FLAG_RESAMPLED
    # strictness: u < ratio.  Find a trial whose u_acc is known and put the ratio exactly there
    u = oracle.uniforms(3, 0, 0, 0)[1]
    if 0 < u < 1:
        pp = np.array([0.5, 0.25, 0.25])
        qq = np.array([0.5 * u, 0.5, 0.5 - 0.5 * u])
        r = oracle.accept_chain(np.stack([logit_of(qq)] * 2), logit_of(pp)[None], [0], 1.0, 3, 0, 0)
        assert r["flags"] & oracle.FLAG_NEAR_ACCEPT   # sits on the boundary: flagged as a near tie


def test_sample_row_inverse_cdf_definition():
    rng = np.random.default_rng(4)
    for V in (2, 17, 1000):
        lg = (rng.normal(size=V) * 3).astype(np.float32)
        for T in (1.0, 0.3):
            for u in (0.0, 0.25, 0.5, 0.999999, 1 - 2.0 ** -24):
                tok, near = oracle.sample_row(lg, T, u)
                want = plain_sampler(lg, T, u)
                assert tok == want or near
    # adding a constant to every logit changes nothing
    lg = (rng.normal(size=64) * 3).astype(np.float32)
    for u in np.linspace(0.01, 0.99, 25):
        assert oracle.sample_row(lg, 1.0, u)[0] == oracle.sample_row(lg + 8.0, 1.0, u)[0]


def test_inverse_cdf_degenerate_exits():
    """The two exits of the inverse-CDF draw that rounding alone can reach, constructed on purpose: no running
    sum exceeds u * total (u = 1: beyond the generator's grid, which ends at 1 - 2^-24) -> the largest index of
    positive weight; weights that are all zero -> the last index.  Both are flagged as near ties."""
    # u = 1: the running sum never exceeds the total; trailing zero weights are skipped
    assert oracle.invcdf([0.2, 0.5, 0.3, 0.0, 0.0], 1.0) == (2, True)
    assert oracle.invcdf([0.0, 4.0, 0.0], 1.0) == (1, True)
    # through the public draw: a logit of -inf weighs exactly zero
    lg = np.array([0.3, 1.0, -np.inf], dtype=np.float32)
    assert oracle.sample_row(lg, 1.0, 1.0) == (1, True)
    # nothing has weight: the last index, flagged
    assert oracle.invcdf(np.zeros(6), 0.4) == (5, True)
    # the ordinary exit, on unnormalised weights, against a cumulative sum written here
    rng = np.random.default_rng(8)
    for V in (1, 2, 9, 300):
        w = rng.random(V) * rng.integers(0, 2, size=V)          # some exact zeros
        if w.sum() == 0:
            w[V // 2] = 1.0
        c = np.cumsum(w)
        for u in (0.0, 0.1, 0.5, 0.77, 1 - 2.0 ** -24):
            tok, near = oracle.invcdf(w, u)
            want = int(np.nonzero(c > u * c[-1])[0][0])
            assert (tok == want or near) and w[tok] > 0


def test_rejection_with_an_empty_residual_falls_back_to_the_target_law():
    """sum_x max(0, q(x) - p(x)) = 0 together with a rejection cannot happen in exact arithmetic (Theorem 1's
    proof: the rejection probability IS that sum).  Constructed here with p == q and a draft token of zero
    probability under both (0/0 rejects by convention): the token is then drawn from q_t with u_res, the
    fallback and resampled flags are set, and nothing of zero probability is returned."""
    lg = np.array([0.3, -np.inf, 1.2, -0.5], dtype=np.float32)
    q = sm(lg)
    c = np.cumsum(q)
    seen = set()
    for s in range(300):
        r = oracle.accept_chain(np.stack([lg, lg]), lg[None], [1], 1.0, 17, 2, s)
        assert r["n_accepted"] == 0
        assert r["flags"] & oracle.FLAG_FALLBACK and r["flags"] & oracle.FLAG_RESAMPLED
        assert not r["flags"] & oracle.FLAG_BONUS
        u_res = oracle.uniforms(17, 2, s, 0)[2]
        want = int(np.nonzero(c > u_res * c[-1])[0][0])
        assert r["tokens"][0] == want or r["flags"] & oracle.FLAG_NEAR_CDF
        assert r["tokens"][0] != 1 and r["tokens"][1] == -1
        seen.add(int(r["tokens"][0]))
    assert seen == {0, 2, 3}
    # an ordinary rejection (p != q) never takes the fallback
    p = np.array([2.0, 0.1, -1.0, 0.4], dtype=np.float32)
    for s in range(300):
        r = oracle.accept_chain(np.stack([lg, lg]), p[None], [0], 1.0, 17, 2, s)
        assert not r["flags"] & oracle.FLAG_FALLBACK
