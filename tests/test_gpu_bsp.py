"""The sharded BSP step (factors per worker shard, exchange, apply of all pairs) on one GPU.

The processes of a multi-GPU run are played one after the other by a single context writing into one
SF buffer: the in-place all-gather leaves every process with exactly that buffer, so what follows the
exchange (header, apply) is the code a real run executes.  No kernel waits on another here.
"""
import numpy as np
import pytest
import torch

from oracle import sfb_oracle as orc
from sfbgen import get_config, make_inputs, scaled
from paper_1511_08486_b200.bsp import BspSfb, worker_range
from paper_1511_08486_b200.workload import shard_batch
from tests.test_gpu_parity import _workload
from tests.util import TOL, to_f64

pytestmark = pytest.mark.gpu

CASES = [
    ("C0", "f32", {}, 0.1),
    ("C0", "tf32", {}, 0.1),
    ("C1", "tf32", dict(J=200, D=1024, P=4, B=128), 1e-2),
    ("C1", "f32", dict(J=100, D=260, P=6, B=10), 1e-2),
    ("C1", "f32", dict(J=200, D=1024, P=4, B=128), 1e-2),          # large enough for the transposed-operand forward
    ("C2", "f32", dict(J=128, D=1024, P=4, B=64), 1e-3),
    ("C2", "f32", dict(J=40, D=300, P=4, B=6), 1e-3),
    ("C2", "tf32", dict(J=64, D=512, P=4, B=64), 1e-3),
    ("C3", "f32", dict(J=70, D=333, P=4, B=5, density=0.1), 1e-2),
    ("C3", "tf32", dict(J=512, D=2000, P=4, B=32), 1e-3),
    ("C4", "bf16", dict(J=512, D=1024, P=4, B=128, pool=1), 1e-4),
    # shard sizes that change the tile geometry (split reduction; width of the softmax partial tiles)
    ("C1", "tf32", {}, 1e-2),
    ("C4", "bf16", dict(J=4096, D=2048, P=8, B=256, pool=1), 1e-5),
]


@pytest.mark.parametrize("name,path,over,eta", CASES)
@pytest.mark.parametrize("world", [1, 2, 4])
def test_sharded_step_equals_single_step(name, path, over, eta, world):
    from paper_1511_08486_b200 import binding as B
    cfg = scaled(name, **over) if over else get_config(name)
    cfg["path"] = path
    if cfg["P"] % world:
        pytest.skip("workers do not split evenly")
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, path)
    try:
        wl.step(0, eta=eta)
        torch.cuda.synchronize()
        W_ref, buf_ref = wl.W.clone(), wl.sf_buf.clone()
        wl.reset()
        wl.sf_buf.zero_()
        t = wl.batches[0]
        for rank in range(world):                                   # the processes, one after the other
            first, n = worker_range(cfg["P"], world, rank)
            s = shard_batch(t, cfg["model"], first, n, cfg["B"])
            wl.ctx.factors_shard(wl.W, s["X"], s["aux"], wl.sf_buf, first, n)
        wl.ctx.commit_header(wl.sf_buf, 0)
        wl.ctx.apply(wl.W, wl.sf_buf, eta)
        assert wl.ctx.status() == 0
        # integer and copied parts of the buffer are bit-exact: header, directory, V or the CSR streams
        h_ref, U_ref, V_ref = orc.unpack(buf_ref.cpu().numpy())
        h, U, V = orc.unpack(wl.sf_buf.cpu().numpy())
        assert h == h_ref
        off, stride = B.sfb_sf_buffer_layout(wl.desc)
        assert torch.equal(wl.sf_buf[:off], buf_ref[:off])            # header and directory (nonzero counts too)
        if cfg["model"] == "sc":
            assert all(np.array_equal(a, b) for a, b in zip(V, V_ref))
        else:
            assert np.array_equal(V, V_ref)
        if world == 1:
            assert torch.equal(wl.sf_buf, buf_ref) and torch.equal(wl.W, W_ref)
        # a worker's factors may differ from the single-process ones only by the summation order of a split
        # reduction: far inside the path's tolerance
        assert orc.rel_fro(U, U_ref) <= 1e-6 if path == "f32" else orc.rel_fro(U, U_ref) <= 0.1 * TOL[path]
        dW, dW_ref = to_f64(wl.W) - to_f64(wl.W0), to_f64(W_ref) - to_f64(wl.W0)
        assert orc.rel_fro(dW, dW_ref) <= (1e-5 if path == "f32" else 0.1 * TOL[path])
    finally:
        wl.close()


def test_bsp_object_single_process():
    """BspSfb without a process group is the whole job on one GPU: same result as sfb_step."""
    cfg = scaled("C1", J=100, D=260, P=6, B=10)
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, "f32")
    try:
        wl.step(0, eta=0.01)
        torch.cuda.synchronize()
        W_ref, buf_ref = wl.W.clone(), wl.sf_buf.clone()
        wl.reset()
        wl.sf_buf.zero_()
        bsp = BspSfb(wl.ctx, wl.desc, wl.sf_buf)
        t = wl.batches[0]
        assert bsp.shard_rows() == slice(0, cfg["P"] * cfg["B"])
        bsp.step(wl.W, t["X"], t["aux"], 0.01, clock=0)
        assert wl.ctx.status() == 0
        assert torch.equal(wl.W, W_ref) and torch.equal(wl.sf_buf, buf_ref)
    finally:
        wl.close()


def test_shard_range_errors():
    from paper_1511_08486_b200 import binding as B
    cfg = scaled("C0", J=10, D=64, P=4, B=8)
    wl = _workload(cfg, make_inputs(cfg), "f32")
    try:
        t = wl.batches[0]
        for first, n in [(-1, 2), (3, 2), (0, 0), (0, 5)]:
            with pytest.raises(B.SfbError):
                wl.ctx.factors_shard(wl.W, t["X"], t["aux"], wl.sf_buf, first, n)
    finally:
        wl.close()


def test_bsp_bench_under_a_launcher_runs_the_nccl_exchange():
    """One rank under torch.distributed.run: the in-place NCCL all-gather of the stream region really runs
    (a group of one), and the bench line reports the job as one sharded job."""
    import json
    import os
    import subprocess
    import sys
    import socket
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with socket.socket() as sock:                      # a port nobody holds right now
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "1", "--master-addr",
           "127.0.0.1", "--master-port", str(port), "bench.py", "--gpus", "1", "--mode", "bsp", "--config", "C1", "--path",
           "tf32", "--J", "200", "--D", "1024", "--P", "4", "--B", "128", "--steps", "3", "--warmup", "3",
           "--no-cpu-baseline"]
    res = subprocess.run(cmd, cwd=root, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["scaling"] == "strong" and out["device_status"] == 0 and out["gpu_launches"] > 0
    assert out["config"]["parallelism"].startswith("bsp sfb")
    assert set(out["stages_ms"]) >= {"factors", "exchange", "apply"}


@pytest.mark.parametrize("path,over", [("f32", dict(J=40, D=300, P=4, B=6)), ("f32", dict(J=128, D=1024, P=4, B=64)),
                                       ("tf32", dict(J=64, D=512, P=4, B=64)), ("tf32x3", dict(J=260, D=1024, P=4, B=100))])
@pytest.mark.parametrize("world", [1, 2, 4])
def test_sharded_step_with_compaction(path, over, world):
    """compact = 1: every process compacts the streams of its own workers before the exchange, the directory's pair
    counts are rebuilt from the streams that arrived: same buffer (byte for byte: the kept pairs, their order and the
    counts do not depend on who computed them) and same update as the single-process compacted step."""
    cfg = scaled("C2", **over)
    cfg["path"] = path
    cfg["compact"] = 1
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, path)
    try:
        eta = 1e-3
        wl.step(0, eta=eta)
        torch.cuda.synchronize()
        W_ref, buf_ref = wl.W.clone(), wl.sf_buf.clone()
        h_ref, U_ref, V_ref = orc.unpack(buf_ref.cpu().numpy())
        assert h_ref["flags"] == orc.FLAG_COMPACT and 0 < sum(h_ref["n_sf"]) < cfg["K"]
        wl.reset()
        wl.sf_buf.zero_()
        t = wl.batches[0]
        for rank in range(world):
            first, n = worker_range(cfg["P"], world, rank)
            s = shard_batch(t, cfg["model"], first, n, cfg["B"])
            wl.ctx.factors_shard(wl.W, s["X"], s["aux"], wl.sf_buf, first, n)
        wl.ctx.commit_header(wl.sf_buf, 0)
        wl.ctx.apply(wl.W, wl.sf_buf, eta)
        assert wl.ctx.status() == 0
        h, U, V = orc.unpack(wl.sf_buf.cpu().numpy())
        assert h == h_ref and np.array_equal(V, V_ref)
        assert orc.rel_fro(U, U_ref) <= (1e-6 if path == "f32" else 0.1 * TOL[path])
        if world == 1:
            assert torch.equal(wl.sf_buf, buf_ref) and torch.equal(wl.W, W_ref)
        dW, dW_ref = to_f64(wl.W) - to_f64(wl.W0), to_f64(W_ref) - to_f64(wl.W0)
        assert orc.rel_fro(dW, dW_ref) <= (1e-5 if path == "f32" else 0.1 * TOL[path])
    finally:
        wl.close()
