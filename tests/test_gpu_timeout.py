"""The bounded-wait abort path of the tcgen05 kernel, exercised without a fault.

NM_PLAN_DIAG_STALL makes CTA 0 arm the barrier of its first K step for 16 bytes more than it
requests: every copy lands, that barrier never completes, and the issuing warp's wait runs out
after a poll budget of about a millisecond.  The CTA must then report NM_ERR_TIMEOUT with the
site of the wait in the status word, free its tensor memory and return, so that the call ends
by itself and the next ordinary call on the same stream is correct."""
import numpy as np
import pytest
import torch

from paper_2607_12505_b200 import binding as nm
from paper_2607_12505_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

SITE_PRODUCER_WAITS_FOR_FREE_STAGE = 1
SITE_ISSUER_WAITS_FOR_STAGE = 2
SITE_EPILOGUE_WAITS_FOR_ACCUMULATOR = 3


@pytest.mark.parametrize("path,n,m", [(nm.NM_PATH_UMMA_SP24, 2, 4), (nm.NM_PATH_UMMA_DENSE, 4, 8)])
def test_stalled_wait_times_out_and_the_stream_stays_usable(path, n, m):
    T, O, K = 700, 512, 1024
    X = inputs.x_i8(T, K, "stall")
    W = inputs.w_i8(O, K, n, m, "stall")
    w = nm.nm_compress(W, n, m)
    Xd = torch.from_numpy(X).cuda()
    plan = gu.make_plan(T, w, nm.NM_OUT_I32, path=path, cta_group=1, split_k=1, tile_t=128, issuers=1)
    stalled = gu.make_plan(T, w, nm.NM_OUT_I32, path=path, cta_group=1, split_k=1, tile_t=128, issuers=1)
    stalled.reserved = nm.NM_PLAN_DIAG_STALL
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    Ybad = torch.zeros((T, O), dtype=torch.int32, device="cuda")
    nm.nm_spmm(Xd, w, plan=stalled, out=Ybad, out_dtype=nm.NM_OUT_I32, status=status)
    # the next ordinary call is enqueued right behind the stalled one, on the same stream
    status2 = torch.zeros(4, dtype=torch.int32, device="cuda")
    Y = nm.nm_spmm(Xd, w, plan=plan, out_dtype=nm.NM_OUT_I32, status=status2)
    torch.cuda.synchronize()                      # returns: the stalled launch ended by itself
    word = int(status[0].item()) & 0xFFFFFFFF
    assert word & 0xFF == nm.NM_ERR_TIMEOUT, hex(word)
    sites = word >> 8                     # one bit per wait site that ran out
    # the waits behind the stalled stage -- the issuing warp's for the stage itself, the epilogue's for the
    # accumulator, the producer's for the stage to be freed again when the ring is shorter than the K loop --
    # have the same budget: whichever runs out first raises the abort flag, the others then just leave
    allowed = (1 << SITE_PRODUCER_WAITS_FOR_FREE_STAGE) | (1 << SITE_ISSUER_WAITS_FOR_STAGE) | (1 << SITE_EPILOGUE_WAITS_FOR_ACCUMULATOR)
    assert sites != 0 and (sites & ~allowed) == 0, hex(word)
    assert int(status2[0].item()) == 0
    gu.check_against_oracle(X, W, n, m, Y.cpu().numpy())
    # only the tiles of CTA 0 are affected: every other CTA of the stalled launch ran normally
    tiles_o = O // 128
    grid = min(148, tiles_o * -(-T // 128))
    ref = Y.cpu().numpy()
    bad = Ybad.cpu().numpy()
    for item in range(tiles_o * -(-T // 128)):
        if item % grid == 0:
            continue
        tt, ot = divmod(item, tiles_o)
        sl = (slice(tt * 128, min(T, tt * 128 + 128)), slice(ot * 128, ot * 128 + 128))
        assert np.array_equal(bad[sl], ref[sl]), f"tile {item} of a CTA that did not stall is wrong"
