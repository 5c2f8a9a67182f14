"""The bounded device wait, made to run out.

Every wait inside the tensor-core kernels gives up after a time limit and makes its kernel report EP_ERR_TIMEOUT.
In the production kernels no wait ever runs out, so the library carries a one-block self-test kernel whose first warp
waits, with a short limit, on a barrier that by construction nothing completes.  No kernel is broken for this, nothing
faults, traps or spins without end: the wait simply expires, the status word says so, and the context stays usable."""
import numpy as np
import pytest
import torch

import oracle
import synth

pytestmark = pytest.mark.gpu


def test_an_expired_wait_is_reported_and_the_context_stays_usable():
    import paper_2604_01000_b200 as ep
    ctx = ep.Context(0)
    try:
        limit = 2_000_000                                      # about a millisecond
        w = ctx.selftest_wait_timeout(limit)
        torch.cuda.synchronize()
        waited0, waited1, claimed = (int(v) for v in w.tolist())
        assert claimed == 0                                    # neither wait may claim that the barrier completed
        assert limit < waited0 < 50 * limit                    # the first warp waited its limit, not for ever
        assert waited1 < 100 * limit                           # the second left with it: far below its own 4e9 clocks
        assert ctx.poll_status() == 5                          # EP_ERR_TIMEOUT
        assert ctx.poll_status() == 0                          # reported once
        # the next real call on the same context is clean and right
        wk = synth.scaled(synth.WORKLOADS["cfg4"], 9_001)
        emb = synth.embeddings(wk, device="cuda")
        init = emb[synth.init_centroid_rows(wk, device="cuda")].contiguous()
        got = ctx.kmeans(emb, wk.K, 2, init)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        ref = oracle.kmeans(emb.cpu().numpy(), wk.K, 2, init.cpu().numpy())
        diff = np.flatnonzero(got.assign.cpu().numpy() != ref.assign)
        assert np.all(ref.best2[diff] - ref.best1[diff] <= 1e-5 * ref.best2[diff])
        with pytest.raises(ep.EmbedPartError):
            ctx.selftest_wait_timeout(10 ** 10)                # a limit of seconds is refused on the host
    finally:
        ctx.close()
