"""The bounded waits of the two decoders that stage predictions with asynchronous copies.

In a correct run no such wait runs out, so the give-up path is reached on purpose, through the test hook of
approxifer_debug_decode: the work item that holds one chosen group is never announced to the threads that wait
for it, and the wait limit is shortened to 65,536 non-blocking probes (a few milliseconds; copies already
started have landed long before).  Nothing faults: the waiting threads give up, the CTA (or warp) that owned the
item stops and flags its unfinished groups with APPROXIFER_ST_TIMEOUT, the event is counted, every other group
is decoded as usual, and the next call works normally.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2109_09868_b200 as ap
from paper_2109_09868_b200 import binding

pytestmark = pytest.mark.gpu

DEC_TOL = 1e-4


def dev():
    return torch.device("cuda:0")


@pytest.mark.parametrize("kernel,K,W,C,G,withhold", [(3, 12, 20, 1000, 1500, 700),   # bulk-copy staged: ~10 items per CTA
                                                     (4, 8, 12, 10, 60000, 31234)])  # packed groups: ~2 items per warp
def test_a_wait_that_runs_out_is_reported_and_leaves_everything_else_intact(kernel, K, W, C, G, withhold):
    rng = np.random.default_rng(C)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(C))
    mask = np.full(G, 2**W - 1, dtype=np.uint32)
    mask[::3] &= ~np.uint32(2)
    want, n_ref, st_ref = oracle.decode(K, W, Yt.numpy(), mask)
    p = ap.make_params(K, W)
    dY, dm = Yt.to(dev()), ap.mask_tensor(mask)
    torch.cuda.synchronize()
    ap.reset_device_wait_timeouts()
    assert ap.device_wait_timeouts() == 0

    status = torch.zeros(G, dtype=torch.int32, device=dev())
    out = torch.full((G, K, C), float("nan"), device=dev())
    tuning = ap.decode_tuning(kernel=kernel, wait_limit=65536, withhold_group=withhold)
    ap.approxifer_decode(p, dY, dm, out, status=status, tuning=tuning)
    torch.cuda.synchronize()  # (i) the kernel ends by itself and the context is healthy

    st = status.cpu().numpy().view(np.uint32)
    timed_out = (st & binding.ST_TIMEOUT) != 0
    assert timed_out[withhold]                       # (ii) the withheld group is flagged ...
    assert 1 <= int(timed_out.sum()) <= G // 20      # ... together with at most the rest of its CTA's or warp's share
    got = out.cpu().numpy().astype(np.float64)
    ok = ~timed_out
    err = np.abs(got[ok] - want[ok]).reshape(int(ok.sum()), -1).max(axis=1)
    scale = np.abs(want[ok]).reshape(int(ok.sum()), -1).max(axis=1)
    assert np.all(err <= DEC_TOL * scale)            # every other group is decoded correctly
    np.testing.assert_array_equal(st[ok], st_ref[ok])
    assert ap.device_wait_timeouts() >= 1            # (iii) counted
    ap.reset_device_wait_timeouts()
    assert ap.device_wait_timeouts() == 0

    # (iv) the next ordinary call is correct everywhere
    status2 = torch.zeros(G, dtype=torch.int32, device=dev())
    out2 = ap.approxifer_decode(p, dY, dm, status=status2, tuning=ap.decode_tuning(kernel=kernel))
    got2 = out2.cpu().numpy().astype(np.float64)
    err2 = np.abs(got2 - want).reshape(G, -1).max(axis=1)
    assert np.all(err2 <= DEC_TOL * np.abs(want).reshape(G, -1).max(axis=1))
    np.testing.assert_array_equal(status2.cpu().numpy().view(np.uint32), st_ref)
    assert ap.device_wait_timeouts() == 0
