"""GPU parity of the tensor-core (tcgen05 / TMEM / TMA) paths against the fp64 oracle.

bf16-in / fp32-accumulate: relative Frobenius error <= 1e-2; TF32: <= 2e-3.  Sizes start at a single
MMA tile and single pipeline stage (so a wrong descriptor or swizzle shows up in isolation), then
span several tiles, ragged edges handled by TMA zero fill, worker streams shorter than one
reduction block, and finally the full workload shapes.
"""
import pytest

from sfbgen import get_config, scaled
from tests.test_gpu_parity import check_config

pytestmark = pytest.mark.gpu


def _cfg(name, path, **kw):
    cfg = scaled(name, **kw)
    cfg["path"] = path
    return cfg


# ------------------------------------------------------------------------------------------------ bf16
def test_bf16_single_tile_single_stage():
    # one 128 x 128 output tile, one 64-deep reduction block in the apply
    check_config(_cfg("C4", "bf16", J=128, D=128, P=1, B=64, pool=1, labels="uniform"), "bf16", eta=0.5, steps=1)


def test_bf16_multi_stage_multi_tile():
    check_config(_cfg("C4", "bf16", J=256, D=512, P=2, B=128, pool=1, labels="uniform"), "bf16", eta=0.5, steps=2)
    check_config(_cfg("C4", "bf16", J=640, D=1024, P=4, B=64, pool=2, labels="uniform"), "bf16", eta=0.5, steps=2)


def test_bf16_ragged_and_short_streams():
    # J, D not multiples of the tile; B below one reduction block (several workers share a block);
    # B not a power of two (zero-filled slots); worker count not a multiple of the block's workers
    for J, D, P, B in ((100, 200, 3, 10), (300, 264, 5, 8), (130, 72, 7, 3), (1000, 520, 2, 100), (77, 1032, 3, 130)):
        check_config(_cfg("C4", "bf16", J=J, D=D, P=P, B=B, pool=1, labels="uniform"), "bf16", eta=0.5, steps=2)


def test_bf16_c4_reduced():
    check_config(_cfg("C4", "bf16", J=4096, D=8192, P=16, B=32, pool=2), "bf16", eta=1e-2, steps=3)


def test_bf16_c4_full():
    check_config(get_config("C4"), "bf16", eta=1e-3, steps=1)


# ------------------------------------------------------------------------------------------------ tf32
def test_tf32_single_tile_single_stage():
    check_config(_cfg("C1", "tf32", J=128, D=128, P=1, B=32, pool=1), "tf32", eta=0.5, steps=1)


def test_tf32_c0_and_ragged():
    check_config(_cfg("C0", "tf32"), "tf32", eta=1.0, steps=1)
    for J, D, P, B in ((100, 200, 3, 10), (300, 260, 5, 8), (257, 1000, 2, 100)):
        check_config(_cfg("C1", "tf32", J=J, D=D, P=P, B=B, pool=1), "tf32", eta=0.5, steps=2)


def test_tf32_c1_full():
    check_config(_cfg("C1", "tf32"), "tf32", eta=1.0, steps=2)


def test_tf32_dml():
    check_config(_cfg("C2", "tf32", J=72, D=1000, P=3, B=20), "tf32", eta=1e-4, steps=2)
    check_config(_cfg("C2", "tf32"), "tf32", eta=1e-5, steps=1)


def test_tf32_sparse_coding_dense_alternative():
    # the codes as dense tf32 rows through the tensor-core GEMMs; the wire buffer keeps them CSR
    check_config(_cfg("C3", "tf32", J=70, D=332, P=3, B=5, density=0.1), "tf32", eta=1e-2, steps=2)
    check_config(_cfg("C3", "tf32", J=512, D=2000, P=4, B=32), "tf32", eta=1e-3, steps=2)
    check_config(_cfg("C3", "tf32"), "tf32", eta=1e-4, steps=1)


def test_tf32_c1_hundred_steps():
    # the workload's own schedule: 100 steps over a pool of 8 minibatches, eta = 1e-2, free-running
    # against the oracle's trajectory (the oracle keeps W in fp64; the tolerance is on W_100 - W_0)
    check_config(_cfg("C1", "tf32"), "tf32", eta=1e-2, steps=100)


def test_bf16_c4_reduced_fifty_steps():
    # C4's 50-step schedule at a reduced shape the oracle finishes in seconds (J = 4096, K = 512)
    check_config(_cfg("C4", "bf16", J=4096, D=8192, P=16, B=32), "bf16", eta=1e-3, steps=50)


def test_pair_tiles_with_split_reduction_and_ragged_edges():
    """Forward GEMMs small enough to take CTA pairs with several reduction ranges: an odd number of 128-row
    units (the last pair is half empty), class counts that are no multiple of the tile, tf32 and bf16."""
    check_config(_cfg("C1", "tf32", J=1000, D=8192, P=3, B=128, pool=1), "tf32", eta=0.5, steps=2)
    check_config(_cfg("C2", "tf32", J=520, D=8192, P=5, B=100), "tf32", eta=1e-5, steps=1)
    check_config(_cfg("C4", "bf16", J=1000, D=16384, P=3, B=128, pool=1, labels="uniform"), "bf16", eta=0.5, steps=2)


def test_tf32_large_mlr_fused_softmax_epilogue():
    """A C4-shaped problem on the tf32 path: CTA pairs, folded loads and the fused exp / partial-sum epilogue
    with fp32 factors (the bf16 path's kernels instantiated for 4-byte values)."""
    check_config(_cfg("C4", "tf32", J=4096, D=4096, P=8, B=128, pool=1), "tf32", eta=1e-3, steps=2)


def test_many_workers_and_long_reductions():
    """K far beyond the benchmark shapes: 256 workers x 256 pairs on the bf16 path (65536 rank-one terms per
    update), and 256 workers x 64 pairs on the tf32 path (reduction blocks that span two workers)."""
    check_config(_cfg("C4", "bf16", J=256, D=256, P=256, B=256, pool=1, labels="uniform"), "bf16", eta=1e-3, steps=1)
    check_config(_cfg("C2", "tf32", J=128, D=256, P=256, B=64), "tf32", eta=1e-6, steps=1)


def test_bf16_c4_full_fifty_steps():
    """The workload's own schedule at full size: 50 steps over the pool of 4 minibatches (32768 x 8192, K = 4096,
    Zipf labels), free-running against the oracle's fp64 trajectory; the error is taken on W_50 - W_0, whole
    matrix, every row and every column.  (The oracle needs a few seconds per step.)"""
    cfg = get_config("C4")
    check_config(cfg, "bf16", eta=cfg["eta"], steps=cfg["steps"])
