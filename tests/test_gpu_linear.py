"""GPU parity of the memory-bound linear layer (sps_linear) with its definition in the oracle.

Tolerance: fp32 accumulation of D products against a double sum.  With |w| ~ 0.02..1 and |x| ~ 1 the
result y has magnitude ~ sqrt(D)*|w|; the bound used is 2e-5 * sqrt(D) * max|w| * max|x| + 1e-6, far
inside the 1e-3 (fp32) / 5e-2 (bf16) logit tolerances; bf16 weights are exact inputs on both sides and
activations keep ~16 mantissa bits through the hi/lo split."""
import numpy as np
import pytest
import torch

import oracle
import paper_2302_01318_b200 as sps
import sps_synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run_linear(W, X):
    N, D = W.shape
    M = X.shape[0]
    dtype = 0 if W.dtype == torch.float32 else 1
    ws = torch.zeros(sps.sps_linear_workspace_bytes(dtype, M, N, D), dtype=torch.uint8, device=DEV)
    Y = torch.full((M, N), float("nan"), device=DEV)
    sps.sps_linear(W, X, Y, ws)
    # second call on the same workspace: the kernel must have left its counters ready
    Y2 = torch.full((M, N), float("nan"), device=DEV)
    sps.sps_linear(W, X, Y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(Y, Y2)       # and results are bit-reproducible
    return Y.cpu().numpy()


def tol(W, X, D):
    return 2e-5 * np.sqrt(D) * float(W.abs().max()) * float(X.abs().max()) + 1e-6


@pytest.mark.parametrize("M", [1, 2, 5, 8, 9, 16])
@pytest.mark.parametrize("N,D", [(1000, 256), (77, 128), (4099, 1024), (2048, 2048), (1536, 6144)])
def test_linear_bf16_small(M, N, D):
    g = torch.Generator().manual_seed(N + D + M)
    W = (torch.randn((N, D), generator=g) * 0.05).to(torch.bfloat16)
    X = torch.randn((M, D), generator=g)
    got = run_linear(W.to(DEV), X.to(DEV))
    want = oracle.linear(sps_synth.to_numpy(W), X.numpy())
    assert np.abs(got - want).max() <= tol(W.float(), X, D)


@pytest.mark.parametrize("M", [5, 7, 8, 9, 13, 16])
@pytest.mark.parametrize("N,D", [(8000, 4096), (9001, 4096), (2304, 8192), (4224, 3072), (1100, 6144), (16384, 16384)])
def test_linear_bf16_tensor_core_kernel_pieces(M, N, D):
    """Shapes the tcgen05 weight-streaming kernel takes (bf16, five rows or more, several k-splits): tiles of 128
    weight rows cut into equal pieces per CTA, so most tiles are shared by two CTAs and meet again in the epilogue
    kernel (partial sums + carry); N = 8000 and 1100 end in a ragged tile, N = 9001 also takes the epilogue's
    one-feature-at-a-time path, 4224 x 3072 has k-ranges of 24 k-blocks,
    1100 rows are fewer tiles than the grid has row ranges, 16384 x 16384 has eight k-splits; 9..16 rows use the
    32-column form of the operand."""
    g = torch.Generator().manual_seed(7 * N + D + M)
    W = (torch.randn((N, D), generator=g) * 0.05).to(torch.bfloat16)
    X = torch.randn((M, D), generator=g)
    got = run_linear(W.to(DEV), X.to(DEV))
    want = oracle.linear(sps_synth.to_numpy(W), X.numpy())
    assert np.abs(got - want).max() <= tol(W.float(), X, D)


@pytest.mark.parametrize("M", [1, 5, 16])
def test_linear_bf16_width_with_a_large_prime_factor(M):
    """D = 128 * 67 only splits into 67 ranges of 128: more than the TMA kernel's tile queues, so the
    register-streaming kernel takes it."""
    N, D = 300, 128 * 67
    g = torch.Generator().manual_seed(M)
    W = (torch.randn((N, D), generator=g) * 0.05).to(torch.bfloat16)
    X = torch.randn((M, D), generator=g)
    got = run_linear(W.to(DEV), X.to(DEV))
    want = oracle.linear(sps_synth.to_numpy(W), X.numpy())
    assert np.abs(got - want).max() <= tol(W.float(), X, D)


@pytest.mark.parametrize("M", [1, 2, 4, 5, 8, 9, 16])
@pytest.mark.parametrize("N,D", [(1000, 256), (77, 128), (4096, 2048), (1536, 6144), (300, 8192), (520, 1536), (200, 640), (90, 12288)])
def test_linear_int8_weights(M, N, D):
    """Weight-only int8: Y = scale[n] * X W^T against the oracle on the dequantised matrix (scale * q is exact in
    double; the kernel multiplies exact fp16 copies of the bytes and applies the scale to the sum)."""
    g = torch.Generator().manual_seed(N + D + M)
    q = torch.randint(-128, 128, (N, D), generator=g, dtype=torch.int32).to(torch.int8)
    q[0, :8] = torch.tensor([-128, 127, 0, -1, 1, 64, -64, 100], dtype=torch.int8)      # the corners of the range
    scale = (torch.rand(N, generator=g) * 0.01 + 0.001).float()
    X = torch.randn((M, D), generator=g)
    ws = torch.zeros(sps.sps_linear_workspace_bytes(2, M, N, D), dtype=torch.uint8, device=DEV)
    Y = torch.full((M, N), float("nan"), device=DEV)
    sps.sps_linear_scaled(q.to(DEV), scale.to(DEV), X.to(DEV), Y, ws)
    Y2 = torch.full((M, N), float("nan"), device=DEV)
    sps.sps_linear_scaled(q.to(DEV), scale.to(DEV), X.to(DEV), Y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(Y, Y2)
    Wd = (q.double() * scale.double()[:, None]).float()           # exact: 8-bit integer times an fp32 scale fits fp32
    want = oracle.linear(Wd.numpy(), X.numpy())
    assert np.abs(Y.cpu().numpy() - want).max() <= tol(Wd, X, D)


@pytest.mark.parametrize("M", [1, 5, 9])
@pytest.mark.parametrize("N,D", [(1024, 256), (130, 128), (515, 1024)])
def test_linear_fp32(M, N, D):
    g = torch.Generator().manual_seed(N + D + M)
    W = torch.randn((N, D), generator=g) * 0.05
    X = torch.randn((M, D), generator=g)
    got = run_linear(W.to(DEV), X.to(DEV))
    want = oracle.linear(W.numpy(), X.numpy())
    assert np.abs(got - want).max() <= tol(W, X, D)


@pytest.mark.parametrize("N,D", [(8192, 8192), (8192, 32768), (32000, 8192), (24576, 6144)])
def test_linear_full_size_sampled_rows(N, D):
    """the 70B-shaped layers at full size, M = 5 as in the bench: EVERY output feature of every row against the
    oracle's double dot products (the oracle splits the rows over the host's cores: a second or two per matrix)"""
    g = torch.Generator(device=DEV).manual_seed(N + D)
    W = torch.empty((N, D), device=DEV, dtype=torch.bfloat16).normal_(0, 0.02, generator=g)
    X = torch.randn((5, D), device=DEV, generator=g)
    got = run_linear(W, X)
    want = oracle.linear(sps_synth.to_numpy(W), X.cpu().numpy())
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= tol(W[:64].float(), X, D)


@pytest.mark.parametrize("N,D", [(32768, 8192), (8192, 32768)])
def test_linear_int8_full_size_sampled_rows(N, D):
    """the 70B-shaped feed-forward matrices as int8 at full size (268 MB each), M = 5 as in the bench: every
    output feature against the oracle's double dot products on the dequantised matrix"""
    g = torch.Generator(device=DEV).manual_seed(N + D)
    q = torch.randint(-127, 128, (N, D), device=DEV, generator=g, dtype=torch.int32).to(torch.int8)
    scale = (torch.rand(N, device=DEV, generator=g) * 1e-3 + 1e-4).float()
    X = torch.randn((5, D), device=DEV, generator=g)
    ws = torch.zeros(sps.sps_linear_workspace_bytes(2, 5, N, D), dtype=torch.uint8, device=DEV)
    Y = torch.full((5, N), float("nan"), device=DEV)
    sps.sps_linear_scaled(q, scale, X, Y, ws)
    torch.cuda.synchronize()
    got = Y.cpu().numpy()
    Wd = (q.double() * scale.double()[:, None]).float().cpu()     # the dequantised matrix the oracle's model is defined on
    want = oracle.linear(Wd.numpy(), X.cpu().numpy())
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= tol(Wd[:4096], X.cpu(), D)



def run_linear_wide(W, X):
    N, D = W.shape
    ws = torch.empty(sps.sps_linear_wide_workspace_bytes(N, D), dtype=torch.uint8, device=DEV)
    Y = torch.full((X.shape[0], N), float("nan"), device=DEV)
    sps.sps_linear_wide(W, X, Y, ws)
    torch.cuda.synchronize()
    return Y.cpu().numpy()


@pytest.mark.parametrize("M", [1, 5, 16, 17, 33, 48, 64, 65, 127, 128])
@pytest.mark.parametrize("N,D", [(256, 64), (300, 128), (1000, 256), (77, 1024), (4099, 2048), (513, 192), (8, 448), (257, 6144)])
def test_linear_wide_small(M, N, D):
    """The prompt-pass GEMM (up to 128 rows on the tcgen05 tensor cores) against the oracle: ragged N (tiles of
    256 weight rows), one to many k-blocks and k-splits, every row count class."""
    g = torch.Generator().manual_seed(N + D + M)
    W = (torch.randn((N, D), generator=g) * 0.05).to(torch.bfloat16)
    X = torch.randn((M, D), generator=g)
    got = run_linear_wide(W.to(DEV), X.to(DEV))
    want = oracle.linear(sps_synth.to_numpy(W), X.numpy())
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= tol(W.float(), X, D)
    # run to run the same bits (fixed k-split order)
    assert np.array_equal(got, run_linear_wide(W.to(DEV), X.to(DEV)))


@pytest.mark.parametrize("N,D", [(32768, 8192), (8192, 32768)])
def test_linear_wide_full_size_sampled_rows(N, D):
    """the 70B-shaped feed-forward matrices at full size with the prompt's 127 rows: every 16th output feature (one
    per 16-row group of every 256-row tile, plus the tiles' edges) of every row against the oracle's double dot
    products -- all of them would be 34 G multiply-adds of oracle time per matrix"""
    g = torch.Generator(device=DEV).manual_seed(N + D)
    W = torch.empty((N, D), device=DEV, dtype=torch.bfloat16).normal_(0, 0.02, generator=g)
    X = torch.randn((127, D), device=DEV, generator=g)
    got = run_linear_wide(W, X)
    rows = np.unique(np.concatenate([[0, 1, 255, 256, N - 1, N - 2], np.arange(0, N, 16) + (np.arange(0, N, 16) // 16) % 16]))
    rows = rows[rows < N]
    Wr = sps_synth.to_numpy(W[torch.from_numpy(rows).to(DEV)])
    want = oracle.linear(Wr, X.cpu().numpy())
    assert np.abs(got[:, rows] - want).max() <= tol(W[:64].float(), X.cpu(), D)
    assert np.isfinite(got).all()
