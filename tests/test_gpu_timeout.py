"""A lost pipeline signal must end in SFB_DEV_TIMEOUT after the bounded wait, with the context still usable.

The tensor-core kernels hand shared-memory stages and accumulators between warps through mbarriers.
Every wait on one is bounded (about a second); when it runs out the CTA sets the status bit, all its
warps leave through the common exit (tensor memory released) and the launch completes.  The test hook
SFB_TEST_LOSE_SIGNAL=1 (read when the context is created, consumed by its first GEMM launch) makes the
first CTA, or CTA pair, skip ONE "stage free" signal: a flag that nothing sets.  Nothing traps, no
address is wrong, no loop is unbounded.
"""
import time

import pytest
import torch

from sfbgen import make_inputs, scaled
from tests.test_gpu_parity import _workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("path,over", [
    ("bf16", dict(J=512, D=4096, P=4, B=128, pool=1, labels="uniform")),       # single-CTA tiles, split reduction
    ("bf16", dict(J=4096, D=4096, P=8, B=256, pool=1, labels="uniform")),      # CTA pairs, fused softmax epilogue
    ("tf32x3", dict(J=512, D=2048, P=4, B=128, pool=1, labels="uniform")),     # compensated kernels (four operand tiles per stage)
])
def test_lost_signal_times_out_cleanly(path, over, monkeypatch):
    from paper_1511_08486_b200 import binding as B
    cfg = scaled("C4", **over)
    cfg["path"] = path
    inputs = make_inputs(cfg)
    monkeypatch.setenv("SFB_TEST_LOSE_SIGNAL", "1")
    wl = _workload(cfg, inputs, path)
    monkeypatch.delenv("SFB_TEST_LOSE_SIGNAL")
    fresh = _workload(cfg, inputs, path)
    try:
        t0 = time.perf_counter()
        wl.step(0, eta=1e-3)
        status = wl.ctx.status()                    # synchronises
        dt = time.perf_counter() - t0
        assert status & B.SFB_DEV_TIMEOUT
        assert dt < 30.0
        # the hook is spent and the context works: same result as a context that never lost a signal
        wl.reset()
        wl.sf_buf.zero_()
        wl.step(0, eta=1e-3)
        assert wl.ctx.status() == 0
        fresh.step(0, eta=1e-3)
        assert fresh.ctx.status() == 0
        assert torch.equal(wl.W, fresh.W) and torch.equal(wl.sf_buf, fresh.sf_buf)
    finally:
        wl.close()
        fresh.close()
