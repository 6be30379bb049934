"""sps_linear_static: the linear layer for hosts that cannot allocate device memory (code inside a
stream capture, a server with a frozen memory budget, a plugin that only receives buffers).  Its
scratch is a fixed array inside the library; the result must equal sps_linear's, call after call,
because every call reuses that array and finds the previous call's contents in it.

Collected last on purpose: a run that stops at the first failure has then run every other test."""
import pytest
import torch

import paper_2302_01318_b200 as sps

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("N,D,M,dt", [(4099, 2048, 5, torch.bfloat16), (8192, 8192, 3, torch.bfloat16),
                                      (1000, 256, 9, torch.bfloat16), (515, 1024, 2, torch.float32)])
def test_static_scratch_matches_workspace_version_twice(N, D, M, dt):
    g = torch.Generator(device=DEV).manual_seed(N + D + M)
    W = (torch.randn((N, D), device=DEV, generator=g) * 0.05).to(dt)
    dtype = 0 if dt == torch.float32 else 1
    ws = torch.zeros(sps.sps_linear_workspace_bytes(dtype, M, N, D), dtype=torch.uint8, device=DEV)
    for call in range(2):   # two calls in a row on the shared array, with different inputs
        X = torch.randn((M, D), device=DEV, generator=g)
        want = torch.full((M, N), float("nan"), device=DEV)
        got = torch.full((M, N), float("nan"), device=DEV)
        sps.sps_linear(W, X, want, ws)
        sps.sps_linear_static(W, X, got)
        torch.cuda.synchronize()
        # same kernel, same plan, same reduction order: the tolerance of the other linear tests
        # (2e-5 * sqrt(D) * max|w| * max|x| + 1e-6) is met with room to spare; in fact bit-equal
        tol = 2e-5 * (D ** 0.5) * float(W.float().abs().max()) * float(X.abs().max()) + 1e-6
        assert torch.isfinite(got).all()
        assert (got - want).abs().max().item() <= tol
        assert torch.equal(got, want)


def test_static_scratch_serves_alternating_shapes_without_allocating():
    """Two shapes with different numbers of k-splits and row ranges take turns on the one shared array: each call
    must find the counters and tile queues as it needs them, whatever the previous call's shape left behind.  Free
    device memory does not move across the calls (the entry point allocates nothing)."""
    g = torch.Generator(device=DEV).manual_seed(99)
    shapes = [(4099, 2048, 5), (1024, 8192, 3), (777, 1024, 12)]
    data = []
    for N, D, M in shapes:
        W = (torch.randn((N, D), device=DEV, generator=g) * 0.05).to(torch.bfloat16)
        X = torch.randn((M, D), device=DEV, generator=g)
        ws = torch.zeros(sps.sps_linear_workspace_bytes(1, M, N, D), dtype=torch.uint8, device=DEV)
        want = torch.empty((M, N), device=DEV)
        sps.sps_linear(W, X, want, ws)
        need = sps.sps_linear_static_floats_needed(1, M, N, D)
        assert 0 < need <= sps.sps_linear_static_max_floats() and need % (16 * N) == 0
        data.append((W, X, want, torch.empty((M, N), device=DEV)))
    sps.sps_linear_static(*data[0][:2], data[0][3])      # first call on the device: resolves the array's address
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for rnd in range(3):
        for W, X, want, got in data:
            got.fill_(float("nan"))
            sps.sps_linear_static(W, X, got)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()     # read before any torch op that might take memory for a temporary
        assert free1 == free0
        for W, X, want, got in data:
            assert torch.equal(got, want), rnd
        free0, _ = torch.cuda.mem_get_info()


def test_static_scratch_rejects_oversized_shapes():
    # the split-K scratch the shape needs must fit the array: 65536 rows with 16 splits do not
    assert sps.sps_linear_static_max_floats() == 4 << 20
    assert sps.sps_linear_static_floats_needed(1, 1, 65536, 32768) > sps.sps_linear_static_max_floats()
    assert sps.sps_linear_static_floats_needed(1, 1, 8, 100) == -1          # bf16 needs D % 128 == 0
    W = torch.zeros((8, 128), device=DEV, dtype=torch.bfloat16)
    X = torch.zeros((1, 128), device=DEV)
    Y = torch.zeros((1, 8), device=DEV)
    rc = sps.lib().sps_linear_static(W.data_ptr(), 1, X.data_ptr(), 1, 65536, 32768, Y.data_ptr(), None)
    assert rc == sps.SPS_EINVAL and b"static" in sps.lib().sps_last_error(None)
