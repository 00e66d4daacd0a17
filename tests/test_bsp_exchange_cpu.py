"""The exchange of the sharded BSP step on CPU: two gloo processes, each holding half of the workers.

Every process starts with only its own workers' streams in the SF buffer (what sfb_factors_shard leaves
there; here the bytes come from the oracle's packer), runs the library's all-gather over the stream
region, and must end with the complete buffer, from which every process makes the same update
(Section 4: under BSP all copies of W stay equal).
"""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _case(model):
    sys.path.insert(0, ROOT)
    from oracle import sfb_oracle as orc
    from sfbgen import make_inputs, scaled
    from tests.util import batch_of, oracle_factors
    if model == "mlr":
        cfg = scaled("C0", J=10, D=64, P=4, B=8)
    else:
        cfg = scaled("C3", J=24, D=90, P=4, B=3, density=0.1)
    inputs = make_inputs(cfg)
    batch = batch_of(inputs, cfg, 0)
    U, V, _ = oracle_factors(cfg, inputs["W"], batch)
    if model == "mlr":
        full = orc.pack(orc.MODEL_MLR, orc.DTYPE_F32, cfg["J"], cfg["D"], cfg["P"], cfg["B"], U, V, clock=3)
    else:
        full = orc.pack(orc.MODEL_SC, orc.DTYPE_F32, cfg["J"], cfg["D"], cfg["P"], cfg["B"], U,
                        csr=(batch["rowptr"], batch["idx"], batch["val"]), clock=3, nnz_capacity=inputs["nnz_capacity"])
    lay = orc.sf_layout(orc.MODEL_MLR if model == "mlr" else orc.MODEL_SC, orc.DTYPE_F32, cfg["J"], cfg["D"], cfg["P"],
                        cfg["B"], model != "mlr", inputs.get("nnz_capacity", 0))
    return cfg, inputs, batch, full, lay


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import sfb_oracle as orc
    from paper_1511_08486_b200.bsp import all_gather_streams, exchange_bytes, worker_range
    res = {}
    for model in ("mlr", "sc"):
        cfg, inputs, batch, full, lay = _case(model)
        off, stride, P = lay["streams_off"], lay["stream_stride"], cfg["P"]
        first, n = worker_range(P, world, rank)
        mine = np.zeros_like(full)
        mine[off + first * stride: off + (first + n) * stride] = full[off + first * stride: off + (first + n) * stride]
        buf = torch.from_numpy(mine)
        all_gather_streams(buf, off, stride, P)
        got = buf.numpy()
        got[:off] = full[:off]                       # header and directory: written locally by every process
        same = bool(np.array_equal(got, full))
        # every process applies all K pairs to its own copy of W
        h, U, V = orc.unpack(got)
        W0 = inputs["W"].astype(np.float64)
        if model == "mlr":
            W1 = orc.apply_dense(W0, U, V, 0.1)
        else:
            W1 = orc.apply_sparse(W0, U, V[0], V[1], V[2], 0.1)
        W_or, _, _ = orc.step(orc.MODEL_MLR if model == "mlr" else orc.MODEL_SC, inputs["W"], batch, 0.1)
        res[model] = (same, float(np.abs(W1 - W_or).max()), W1.tobytes(), exchange_bytes(P, world, stride))
    dist.barrier()
    out.put((rank, res))
    dist.destroy_process_group()


def test_two_processes_end_with_the_full_buffer_and_equal_updates():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for model in ("mlr", "sc"):
        for rank in (0, 1):
            same, err, _, nbytes = res[rank][model]
            assert same                                  # all-gather reproduced the packed message byte for byte
            assert err <= 1e-6                           # fp32 wire values: the update equals the oracle step to rounding
            assert nbytes["total"] == 2 * nbytes["shard_bytes"] and nbytes["sent_per_process"] == nbytes["shard_bytes"]
        assert res[0][model][2] == res[1][model][2]      # the two copies of W are bit-identical after the clock


def test_worker_range_and_byte_count():
    sys.path.insert(0, ROOT)
    import pytest
    from paper_1511_08486_b200.bsp import exchange_bytes, worker_range
    assert [worker_range(16, 4, r) for r in range(4)] == [(0, 4), (4, 4), (8, 4), (12, 4)]
    assert worker_range(6, 1, 0) == (0, 6)
    with pytest.raises(ValueError):
        worker_range(6, 4, 0)
    with pytest.raises(ValueError):
        worker_range(4, 2, 2)
    b = exchange_bytes(16, 8, 1024)
    assert b == {"shard_bytes": 2048, "sent_per_process": 2048 * 7, "total": 2048 * 8 * 7}
