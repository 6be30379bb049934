"""The give-up path of the kernels' bounded waits, run on purpose.

Every wait inside a kernel is bounded by the global timer; when the bound runs out the kernel records an error,
lets its copies in flight land, frees what it holds and returns, and the host reports SPS_ETIMEOUT.  Here the
bound is shortened to a few milliseconds and the copy producer of the first CTA leaves out one stage of its ring
(nothing is then in flight for it), so a consumer's wait runs out by construction.  Nothing hangs or faults: the
kernel ends by itself and the context stays usable, which the follow-up calls check."""
import numpy as np
import pytest
import torch

import oracle
import paper_2302_01318_b200 as sps
import sps_synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(autouse=True)
def restore_knobs():
    yield
    sps.sps_debug_set_wait(0, -1)


# five rows: the tcgen05 kernel (the MMA lane's wait on the missing stage runs out); two rows: the mma.sync kernel (a
# consumer warp's wait does).  Stages 1 and 3 are always among the first CTA's own.
@pytest.mark.parametrize("drop,M", [(1, 5), (3, 5), (1, 2), (3, 2)])
def test_linear_wait_runs_out_and_the_next_call_is_clean(drop, M):
    N, D = 4096, 4096
    g = torch.Generator().manual_seed(3)
    W = (torch.randn((N, D), generator=g) * 0.05).to(torch.bfloat16)
    X = torch.randn((M, D), generator=g)
    Wd, Xd = W.to(DEV), X.to(DEV)
    ws = torch.zeros(sps.sps_linear_workspace_bytes(1, M, N, D), dtype=torch.uint8, device=DEV)
    Y = torch.zeros((M, N), device=DEV)
    sps.sps_debug_set_wait(3000, drop)          # 3 ms bound; stage `drop` of CTA 0 is never asked for
    with pytest.raises(sps.SpsError) as e:
        sps.sps_linear(Wd, Xd, Y, ws, timed=True)
    assert e.value.code == sps.SPS_ETIMEOUT
    sps.sps_debug_set_wait(0, -1)
    want = oracle.linear(sps_synth.to_numpy(W), X.numpy())
    tol = 2e-5 * np.sqrt(D) * float(W.float().abs().max()) * float(X.abs().max()) + 1e-6
    # the same workspace recovers (the kernel re-armed its counters on the way out), and so does a fresh one
    for w in (ws, torch.zeros_like(ws)):
        Y.fill_(float("nan"))
        ms = sps.sps_linear(Wd, Xd, Y, w, timed=True)
        assert ms < 1.0
        assert np.abs(Y.cpu().numpy() - want).max() <= tol


def test_wide_gemm_wait_runs_out_and_the_next_call_is_clean():
    # 148 tiles of 256 weight rows: one k-split, eight k-blocks per CTA; k-block 4 of the first CTA is left out
    M, N, D = 100, 256 * 148, 512
    g = torch.Generator().manual_seed(4)
    W = (torch.randn((N, D), generator=g) * 0.05).to(torch.bfloat16)
    X = torch.randn((M, D), generator=g)
    Wd, Xd = W.to(DEV), X.to(DEV)
    ws = torch.zeros(sps.sps_linear_wide_workspace_bytes(N, D), dtype=torch.uint8, device=DEV)
    Y = torch.zeros((M, N), device=DEV)
    sps.sps_debug_set_wait(3000, 4)
    with pytest.raises(sps.SpsError) as e:
        sps.sps_linear_wide(Wd, Xd, Y, ws, timed=True)
    assert e.value.code == sps.SPS_ETIMEOUT
    sps.sps_debug_set_wait(0, -1)
    Y.fill_(float("nan"))
    ms = sps.sps_linear_wide(Wd, Xd, Y, ws, timed=True)
    assert ms < 2.0
    rows = np.arange(0, N, 997)                    # sampled weight rows, every activation row
    want = oracle.linear(sps_synth.to_numpy(W[rows]), X.numpy())
    tol = 2e-5 * np.sqrt(D) * float(W.float().abs().max()) * float(X.abs().max()) + 1e-6
    assert torch.isfinite(Y).all()
    assert np.abs(Y.cpu().numpy()[:, rows] - want).max() <= tol


def test_knob_limits():
    with pytest.raises(sps.SpsError):
        sps.sps_debug_set_wait(-1, -1)
    with pytest.raises(sps.SpsError):
        sps.sps_debug_set_wait(3_000_000, -1)      # never above the default bound
