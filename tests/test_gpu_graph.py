"""sfb_step recorded into a CUDA graph and replayed: the step allocates nothing, never synchronises and
orders all its work on the context's stream (the side-stream copy forks and joins by events), so it can
be captured once and replayed without per-launch host cost."""
import pytest
import torch

from sfbgen import make_inputs, scaled

pytestmark = pytest.mark.gpu

CASES = [
    ("C0", "f32", {}),
    ("C1", "f32", dict(J=100, D=260, P=3, B=10)),
    ("C1", "tf32", dict(J=200, D=1024, P=4, B=128)),
    ("C2", "tf32", dict(J=64, D=512, P=2, B=64)),
    ("C3", "f32", dict(J=70, D=333, P=3, B=5, density=0.1)),
    ("C4", "bf16", dict(J=512, D=1024, P=4, B=128, pool=1, labels="uniform")),
]


@pytest.mark.parametrize("name,path,over", CASES)
def test_captured_step_replays_to_the_same_weights(name, path, over):
    from paper_1511_08486_b200.workload import DeviceWorkload
    cfg = scaled(name, **over)
    cfg["path"] = path
    cfg["pool"] = 1
    inputs = make_inputs(cfg)
    eta = 1e-3
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        wl = DeviceWorkload(cfg, inputs, path=path, stream=side.cuda_stream)
        try:
            for _ in range(4):                                  # eager: 4 steps on the same minibatch
                wl.step(0, eta=eta)
            side.synchronize()
            assert wl.ctx.status() == 0
            W_eager = wl.W.clone()
            wl.reset()
            wl.step(0, eta=eta)                                 # step 1 eagerly (first-call set-up happens here)
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                wl.step(0, eta=eta)                             # recorded, not run
            for _ in range(3):
                graph.replay()                                  # steps 2..4
            torch.cuda.synchronize()
            assert wl.ctx.status() == 0
            assert torch.equal(wl.W, W_eager)
        finally:
            torch.cuda.synchronize()
            wl.close()


@pytest.mark.parametrize("name,path,over", [CASES[1], CASES[2], CASES[4]])
def test_captured_stage_calls_replay_to_the_same_weights(name, path, over):
    """The separate entry points in one graph: factors + pack + apply, and shard factors + header + apply."""
    from paper_1511_08486_b200.workload import DeviceWorkload
    cfg = scaled(name, **over)
    cfg["path"] = path
    cfg["pool"] = 1
    inputs = make_inputs(cfg)
    eta = 1e-3
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        wl = DeviceWorkload(cfg, inputs, path=path, stream=side.cuda_stream)
        try:
            t = wl.batches[0]

            def staged():
                wl.compute_factors(0)
                wl.pack(0, clock=0)
                wl.apply(eta)

            def sharded():
                wl.ctx.factors_shard(wl.W, t["X"], t["aux"], wl.sf_buf, 0, cfg["P"])
                wl.ctx.commit_header(wl.sf_buf, 0)
                wl.ctx.apply(wl.W, wl.sf_buf, eta)

            for fn in (staged, sharded):
                wl.reset()
                for _ in range(3):
                    fn()
                side.synchronize()
                W_eager = wl.W.clone()
                wl.reset()
                fn()
                side.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    fn()
                graph.replay()
                graph.replay()
                torch.cuda.synchronize()
                assert wl.ctx.status() == 0
                assert torch.equal(wl.W, W_eager)
        finally:
            torch.cuda.synchronize()
            wl.close()
