"""Pins for the oracle's linear layer and for the row splitting every large mat-vec of the oracle goes through.

``oracle.linear`` is what every GPU linear-layer test is judged by, and ``parallel_rows`` only splits work over
threads from 2^22 multiply-adds on -- sizes no other CPU test reaches.  Both are checked here against an
independent float64 matrix product (numpy), on fp32 and on bf16-stored weights, ragged shapes included, and the
threaded runs must equal the one-thread run bit for bit."""
import numpy as np
import pytest

import oracle
import sps_synth
from test_oracle_model import as_f64, matrix_forward, np_weights


def _weights(rng, N, D, dtype):
    W = (rng.normal(size=(N, D)) * 0.05).astype(np.float32)
    # a deterministic, non-symmetric part so that a transposed or shifted index cannot cancel
    W += (np.arange(N, dtype=np.float32)[:, None] * 1e-3 - np.arange(D, dtype=np.float32)[None, :] * 7e-4)
    if dtype == 1:
        import torch
        return torch.from_numpy(W).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    return W


def _check(W, X):
    got = oracle.linear(W, X)
    want = X.astype(np.float64) @ as_f64(W).T
    assert got.shape == want.shape
    scale = np.abs(as_f64(W)).max() * np.abs(X).max() * W.shape[1]
    assert np.abs(got - want).max() <= 1e-13 * scale
    return got


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("M,N,D", [(1, 1, 1), (3, 37, 129), (5, 64, 256), (16, 33, 130), (2, 257, 31)])
def test_linear_is_the_matrix_product(dtype, M, N, D):
    """Y[m, n] = sum_k X[m, k] W[n, k] (section Conditional Scoring: the linear layers), small ragged shapes."""
    rng = np.random.default_rng(100 * M + N + D + dtype)
    X = rng.normal(size=(M, D)).astype(np.float32)
    _check(_weights(rng, N, D, dtype), X)


def test_linear_reads_bf16_bits_exactly():
    """a bf16 weight is its 16 bits followed by 16 zero bits of an fp32: one-hot activations read weights back"""
    import torch
    vals = torch.tensor([[1.0, -2.5, 3.0e-3, 0.0], [65280.0, -1.0e-20, 0.33203125, 7.0]]).to(torch.bfloat16)
    W = vals.view(torch.int16).numpy().view(np.uint16)
    got = oracle.linear(W, np.eye(4, dtype=np.float32))        # Y[m, n] = W[n, m]
    assert np.array_equal(got, vals.double().numpy().T)


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("M,N,D", [(1, 4096, 2048), (2, 4099, 1031), (3, 5, 1 << 19)])
def test_linear_threaded_rows_match_numpy_and_one_thread(dtype, M, N, D):
    """N * D * M >= 2^22: the rows are split over threads.  Ragged N (a short last range) and fewer rows than
    threads are both covered; every thread count gives the one-thread result bit for bit."""
    assert N * D * M >= 1 << 22
    rng = np.random.default_rng(N)
    X = rng.normal(size=(M, D)).astype(np.float32)
    W = _weights(rng, N, D, dtype)
    try:
        oracle.set_threads(1)
        one = _check(W, X)
        for t in (2, 3, 7, 8, 64):
            oracle.set_threads(t)
            assert oracle.num_threads() == t
            assert np.array_equal(_check(W, X), one), t
    finally:
        oracle.set_threads(0)


@pytest.mark.parametrize("dtype", [0, 1])
def test_transformer_with_threaded_matvecs_matches_the_matrix_restatement(dtype):
    """One layer at d_model = d_ff = 2048 (every mat-vec of the layer is 2^22 multiply-adds, the size from which
    rows are split): the forward pass equals the independent matrix-form restatement, and equals the
    one-thread run bit for bit."""
    cfg = sps_synth._cfg(1, 2048, 16, 128, 2048, 96, dtype)
    w = np_weights(cfg, seed=3, tag="target", std=0.04)
    toks = sps_synth.make_prompt(11, 5, cfg["vocab"])
    want = matrix_forward(cfg, w, toks)
    try:
        outs = []
        for t in (1, 4, 7):
            oracle.set_threads(t)
            outs.append(oracle.Transformer(cfg, w, max_seq=8).forward64(toks, np.arange(5)))
    finally:
        oracle.set_threads(0)
    assert np.abs(outs[0] - want).max() < 1e-9 * max(1.0, np.abs(want).max())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
