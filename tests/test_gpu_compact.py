"""Inactive-pair compaction on the GPU (sfb_desc.compact = 1) against the oracle's compacted packer.

A pair whose u is all zeros is left out of the message: the committed buffer must equal, byte for byte, the
oracle's `pack(..., compact=True)` of the same factors; the update must be the one the full buffer gives
(bit-identical on the fp32 path, inside a tenth of the tolerance on the tensor-core paths, whose instructions
group the remaining pairs differently); the reported pair and byte counts must be the oracle's.
"""
import numpy as np
import pytest
import torch

from oracle import sfb_oracle as orc
from sfbgen import get_config, make_inputs, scaled
from tests.test_gpu_parity import _workload
from tests.util import MODEL_ID, TOL, assert_lines

pytestmark = pytest.mark.gpu


def _pair(cfg, inputs, path):
    full = _workload(cfg, inputs, path)
    ccfg = dict(cfg, compact=1)
    comp = _workload(ccfg, inputs, path)
    return full, comp


@pytest.mark.parametrize("path,over,eta", [
    ("f32", dict(J=40, D=300, P=3, B=7), 1e-3),
    ("f32", dict(J=300, D=8192, P=4, B=96), 1e-4),            # the pipelined large-tile apply walks the kept-pair list
    ("tf32", dict(J=72, D=1000, P=3, B=20), 1e-4),            # several workers share a reduction block: nothing skipped
    ("tf32", dict(J=260, D=1024, P=5, B=200), 1e-4),          # B >= one reduction block: whole blocks are skipped
    ("tf32x3", dict(J=260, D=1024, P=5, B=200), 1e-4),        # compensated path, blocks skipped
    ("tf32x3", dict(J=128, D=512, P=32, B=256), 1e-4),        # 8192 pairs: eight launches of the apply, directory offsets
    ("f32", {}, 1e-5),                                        # full size
    ("tf32", {}, 1e-5),
])
def test_dml_compacted_step(path, over, eta):
    cfg = scaled("C2", **over) if over else get_config("C2")
    cfg["path"] = path
    inputs = make_inputs(cfg)
    J, D, P, B, K = cfg["J"], cfg["D"], cfg["P"], cfg["B"], cfg["K"]
    full, comp = _pair(cfg, inputs, path)
    try:
        full.step(0, eta=eta)
        comp.step(0, eta=eta)
        torch.cuda.synchronize()
        assert full.ctx.status() == 0 and comp.ctx.status() == 0
        buf_f, buf_c = full.sf_buf.cpu().numpy(), comp.sf_buf.cpu().numpy()
        h_f, U_f, V_f = orc.unpack(buf_f)
        # the compacted buffer is the oracle's compaction of the very factors the full buffer carries
        ref_c = orc.pack(MODEL_ID["dml"], orc.DTYPE_F32, J, D, P, B, U_f, V_f, clock=0, compact=True)
        assert np.array_equal(buf_c, ref_c), f"compacted buffer differs at byte {np.nonzero(buf_c != ref_c)[0][:4]}"
        h_c, U_c, V_c = orc.unpack(buf_c)
        kept = int(np.any(U_f != 0, axis=1).sum())
        assert 0 < kept < K and sum(h_c["n_sf"]) == kept and h_c["flags"] == orc.FLAG_COMPACT
        assert comp.ctx.active_pairs() == kept
        assert comp.ctx.wire_bytes(comp.sf_buf) == orc.wire_bytes(buf_c) < full.ctx.wire_bytes(full.sf_buf) == orc.wire_bytes(buf_f)
        # same update as from the full buffer
        W_f, W_c = full.W.cpu().numpy(), comp.W.cpu().numpy()
        if path == "f32":
            assert np.array_equal(W_f, W_c), "fp32 path: the kept pairs are summed in the same order"
        W0 = inputs["W"].astype(np.float64)
        move_f, move_c = W_f.astype(np.float64) - W0, W_c.astype(np.float64) - W0
        # (the compensated path's error IS its accumulator's rounding, which depends on how many instructions a sum
        # takes: the two buffers may differ by a good part of that tolerance; both are held to it against the oracle)
        assert orc.rel_fro(move_c, move_f) <= (0.5 if path == "tf32x3" else 0.1) * TOL[path]
        # ... and the oracle's update from the compacted message (the GPU's own gate: the buffer's pairs)
        ref_move = -eta * orc.delta_w(U_c, V_c)
        storage = 2.0 ** -24 * np.linalg.norm(W0) / np.linalg.norm(ref_move)
        assert storage <= TOL[path]
        assert orc.rel_fro(move_c, ref_move) <= TOL[path] + storage
        assert_lines(move_c, ref_move, TOL[path], "W' - W from the compacted buffer",
                     extra_rows=2.0 ** -24 * np.linalg.norm(W0, axis=1), extra_cols=2.0 ** -24 * np.linalg.norm(W0, axis=0))
        # staged calls (factors, pack with compaction, apply) leave the same buffer and W as the step
        comp.reset()
        comp.sf_buf.zero_()
        comp.compute_factors(0)
        comp.pack(0, clock=0)
        comp.apply(eta)
        torch.cuda.synchronize()
        assert np.array_equal(comp.sf_buf.cpu().numpy(), buf_c) and np.array_equal(comp.W.cpu().numpy(), W_c)
        # partial apply: the first two workers' streams only
        if P > 2:
            comp.reset()
            comp.apply(eta, K=2 * B)
            torch.cuda.synchronize()
            ref2 = -eta * orc.delta_w(U_c[:2 * B], V_c[:2 * B])
            got2 = comp.W.cpu().numpy().astype(np.float64) - W0
            assert orc.rel_fro(got2, ref2) <= TOL[path] + 2.0 ** -24 * np.linalg.norm(W0) / np.linalg.norm(ref2)
        assert comp.ctx.status() == 0
    finally:
        full.close()
        comp.close()


@pytest.mark.parametrize("path", ["f32", "tf32"])
def test_no_active_pair_at_all_leaves_w_untouched(path):
    """Every pair dissimilar and far beyond the margin: the message is empty, the apply has no reduction block."""
    cfg = scaled("C2", J=130, D=512, P=3, B=64)
    cfg["path"] = path
    cfg["w_std"] = 1.0
    inputs = make_inputs(cfg)
    inputs["similar"] = np.zeros_like(inputs["similar"])
    comp = _workload(dict(cfg, compact=1), inputs, path)
    try:
        comp.step(0, eta=1e-3)
        torch.cuda.synchronize()
        assert comp.ctx.status() == 0
        assert torch.equal(comp.W, comp.W0)
        h, U, V = orc.unpack(comp.sf_buf.cpu().numpy())
        assert h["n_sf"] == [0, 0, 0] and not U.any() and not V.any()
        assert comp.ctx.active_pairs() == 0
        assert comp.ctx.wire_bytes(comp.sf_buf) == 128 + 3 * 32
    finally:
        comp.close()


def test_compaction_with_every_pair_active_changes_only_the_flag():
    cfg = scaled("C1", J=64, D=256, P=2, B=16, pool=1)
    cfg["path"] = "tf32"
    inputs = make_inputs(cfg)
    full, comp = _pair(cfg, inputs, "tf32")
    try:
        full.step(0, eta=0.5)
        comp.step(0, eta=0.5)
        torch.cuda.synchronize()
        a, b = full.sf_buf.cpu().numpy(), comp.sf_buf.cpu().numpy()
        assert np.nonzero(a != b)[0].tolist() == [8]
        assert torch.equal(full.W, comp.W)
        assert comp.ctx.active_pairs() == cfg["K"]
    finally:
        full.close()
        comp.close()


def test_compaction_is_refused_where_it_is_not_defined():
    from paper_1511_08486_b200 import binding as B
    with pytest.raises(B.SfbError) as e:
        B.Context(B.make_desc("sc", "f32", 8, 8, 2, 2, v_sparse=1, nnz_capacity=64, compact=1))
    assert e.value.code == -3
