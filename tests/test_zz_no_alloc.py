"""The allocation-free entry point `sfb_sc_factors_noalloc` against `sfb_compute_factors` and the fp64 oracle.

Some callers may not allocate device memory (graph capture in progress, latency-bound loops, a
fixed memory budget handed out by an outer framework), so they cannot create a context.  This
entry point keeps its scratch in a fixed array inside the library instead.  Because every call
shares that array and it keeps the previous call's contents, the check runs two different problems
back to back and compares each with the context-based entry point on the same inputs, and with the
oracle's definition u_i = W a_i - x_i directly.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

from oracle import sfb_oracle as orc
from sfbgen import make_inputs, scaled

pytestmark = pytest.mark.gpu


def _device_problem(cfg, dev):
    from paper_1511_08486_b200.workload import DeviceWorkload
    inputs = make_inputs(cfg)
    wl = DeviceWorkload(cfg, inputs, path="f32", device=dev)
    wl.compute_factors(0)                       # existing entry point (allocates its workspace in sfb_create)
    torch.cuda.synchronize()
    U_or = orc.sc_factors(inputs["W"], inputs["rowptr"][0], inputs["idx"][0], inputs["val"][0], inputs["Xdata"][0])
    return wl, wl.U.clone(), U_or


def test_noalloc_matches_context_entry_point_on_two_calls_in_a_row():
    from paper_1511_08486_b200 import binding as B
    dev = torch.device("cuda:0")
    # two problems of different shape, so that leftovers of the first call in the shared scratch
    # would corrupt the second if a call depended on them
    cfg_a = scaled("C3", J=512, D=2000, P=4, B=32)
    cfg_b = scaled("C3", J=70, D=333, P=3, B=5, density=0.1)
    wl_a, ref_a, or_a = _device_problem(cfg_a, dev)
    wl_b, ref_b, or_b = _device_problem(cfg_b, dev)
    try:
        outs = []
        status = torch.full((1,), 77, dtype=torch.int32, device=dev)
        for wl in (wl_a, wl_b):
            t = wl.batches[0]
            U = torch.full_like(wl.U, float("nan"))
            B.sfb_sc_factors_noalloc(wl.W, wl.cfg["J"], wl.cfg["D"], wl.K, t["rowptr"], t["idx"], t["val"], t["Xdata"],
                                     U, wl.ldu, dev_status=status)
            outs.append(U)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for got, ref, U_or, wl in zip(outs, (ref_a, ref_b), (or_a, or_b), (wl_a, wl_b)):
            g, r = got.cpu().numpy().astype(np.float64), ref.cpu().numpy().astype(np.float64)
            assert np.isfinite(g).all()
            err = np.linalg.norm(g - r) / np.linalg.norm(r)
            assert err <= 1e-5, f"relative error {err:.3e} against sfb_compute_factors"
            J = wl.cfg["J"]
            assert not g[:, J:].any(), "pad columns are written as zeros"
            e_or = orc.rel_fro(g[:, :J], U_or)
            assert e_or <= 1e-5, f"relative error {e_or:.3e} against the oracle's u = W a - x"
        # repeat the first problem: same answer again after the scratch held another problem
        t = wl_a.batches[0]
        U2 = torch.empty_like(wl_a.U)
        B.sfb_sc_factors_noalloc(wl_a.W, cfg_a["J"], cfg_a["D"], wl_a.K, t["rowptr"], t["idx"], t["val"], t["Xdata"],
                                 U2, wl_a.ldu)
        torch.cuda.synchronize()
        assert torch.equal(U2, outs[0])
    finally:
        wl_a.close()
        wl_b.close()


def test_noalloc_writes_every_pad_column_of_a_wider_output_row():
    """A caller may hand in rows wider than roundup(J, 4), even beyond the next 1024-column block: everything
    up to ldu is written (zeros beyond J), nothing of the caller's old bytes survives."""
    from paper_1511_08486_b200 import binding as B
    dev = torch.device("cuda:0")
    cfg = scaled("C3", J=1000, D=300, P=2, B=6, density=0.1)
    wl, _, U_or = _device_problem(cfg, dev)
    try:
        t = wl.batches[0]
        ldu = 2048
        U = torch.full((wl.K, ldu), float("nan"), dtype=torch.float32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        B.sfb_sc_factors_noalloc(wl.W, cfg["J"], cfg["D"], wl.K, t["rowptr"], t["idx"], t["val"], t["Xdata"], U, ldu,
                                 dev_status=status)
        torch.cuda.synchronize()
        g = U.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all() and not g[:, cfg["J"]:].any()
        assert orc.rel_fro(g[:, :cfg["J"]], U_or) <= 1e-5
        assert int(status.item()) == 0
    finally:
        wl.close()


def test_noalloc_rejects_problems_beyond_its_scratch():
    from paper_1511_08486_b200 import binding as B
    dev = torch.device("cuda:0")
    cap = B.sfb_noalloc_max_scratch_floats()
    assert cap == 4 << 20
    dummy = torch.zeros(64, dtype=torch.float32, device=dev)
    idummy = torch.zeros(64, dtype=torch.int32, device=dev)
    with pytest.raises(B.SfbError) as e:       # 4096 x 10000 needs 40.96 M values: over the 4 Mi limit, nothing launched
        B.sfb_sc_factors_noalloc(dummy, 4096, 10000, 4, idummy, idummy, dummy, dummy, dummy, 4096)
    assert e.value.code == -6 and "scratch" in str(e.value)
    with pytest.raises(B.SfbError) as e:
        B.sfb_sc_factors_noalloc(dummy, 8, 8, 4, idummy, idummy, dummy, dummy, dummy, 6)   # ldu < J
    assert e.value.code == -1
