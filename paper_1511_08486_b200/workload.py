"""Places one synthetic workload (see `sfbgen`) on the device and drives the C ABI with it.

Only tensor allocation, host<->device copies and argument marshalling happen here.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def bf16_tensor(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> a torch.bfloat16 tensor holding exactly those bits."""
    return torch.from_numpy(bits.view(np.int16).copy()).to(device).view(torch.bfloat16)


def shard_batch(t: dict, model: str, first_worker: int, n_workers: int, Bsz: int) -> dict:
    """The part of a device minibatch `t` that belongs to workers [first_worker, first_worker + n_workers).

    Fresh contiguous tensors (so every pointer is aligned) plus the matching `aux`; sparse codes get
    row pointers that start at 0.  Copies only: what a process of a multi-process run would hold.
    """
    lo, hi = first_worker * Bsz, (first_worker + n_workers) * Bsz
    s = {}
    if model == "mlr":
        s["X"], s["labels"] = t["X"][lo:hi].clone(), t["labels"][lo:hi].clone()
        s["aux"] = B.make_aux(labels=s["labels"])
    elif model == "dml":
        s["X"], s["Xb"], s["similar"] = t["X"][lo:hi].clone(), t["Xb"][lo:hi].clone(), t["similar"][lo:hi].clone()
        s["aux"] = B.make_aux(Xb=s["Xb"], similar=s["similar"])
    else:
        rp = t["rowptr"][lo:hi + 1].clone()
        e0, e1 = int(rp[0].item()), int(rp[-1].item())
        s["X"] = None
        s["rowptr"] = rp - e0
        # keep at least one element so that the pointers are valid for a shard without nonzeros
        s["idx"] = t["idx"][e0:max(e1, e0 + 1)].clone() if t["idx"].numel() > e0 else torch.zeros_like(t["idx"][:1])
        s["val"] = t["val"][e0:max(e1, e0 + 1)].clone() if t["val"].numel() > e0 else torch.zeros_like(t["val"][:1])
        s["Xdata"] = t["Xdata"][lo:hi].clone()
        s["aux"] = B.make_aux(rowptr=s["rowptr"], idx=s["idx"], val=s["val"], Xdata=s["Xdata"])
    return s


GUARD_BYTES = 4096


class Guarded:
    """A device tensor placed between two guard bands of GUARD_BYTES bytes each, filled with 0xFF (a NaN pattern in
    fp32 and bf16).  `t` is the usable tensor (128-byte aligned); `intact()` tells whether both bands still hold
    their pattern.  A stray write lands in a band and is seen there; a stray read that feeds arithmetic turns the
    result into NaN."""

    def __init__(self, shape, dtype, device, fill=None):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.raw = torch.full((n + 2 * GUARD_BYTES,), 0xFF, dtype=torch.uint8, device=device)
        self.n = n
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(*shape)
        if fill is not None:
            self.t.copy_(fill)
        else:
            self.t.zero_()

    def intact(self) -> bool:
        lo, hi = self.raw[:GUARD_BYTES], self.raw[GUARD_BYTES + self.n:]
        return bool((lo == 0xFF).all().item()) and bool((hi == 0xFF).all().item())


class DeviceWorkload:
    """Device copies of the inputs of configuration `cfg`, a context, and the SF buffer.

    guard=True puts every tensor the library writes (W, the SF buffer, U, V) between guard bands
    (`guards_intact()` checks them) for tests that look for out-of-range accesses."""

    def __init__(self, cfg: dict, inputs: dict, path: str | None = None, device="cuda:0", stream=None, guard=False):
        self.cfg, self.device = cfg, torch.device(device)
        self._guards = []
        self.path = path or cfg["path"]
        model = cfg["model"]
        self.model = model
        J, D, P, Bsz = cfg["J"], cfg["D"], cfg["P"], cfg["B"]
        self.K = P * Bsz
        self.pool = cfg["pool"]
        sparse = model == "sc"
        self.desc = B.make_desc(model, self.path, J, D, P, Bsz, v_sparse=int(sparse), margin=cfg.get("margin", 1.0),
                                nnz_capacity=inputs.get("nnz_capacity", 0), compact=int(cfg.get("compact", 0)))
        self.ctx = B.Context(self.desc, stream)
        self.ldu, self.ldv = self.ctx.ldu, self.ctx.ldv
        dev = self.device
        self.W0 = torch.from_numpy(inputs["W"]).to(dev)
        self.W = self._alloc(self.W0.shape, torch.float32, guard, fill=self.W0)
        bf16 = self.path == "bf16"
        self.val_dtype = torch.bfloat16 if bf16 else torch.float32
        self.batches = []
        for b in range(self.pool):
            t = {}
            if model == "mlr":
                t["X"] = bf16_tensor(inputs["X_bits"][b], dev) if bf16 else torch.from_numpy(inputs["X"][b]).to(dev)
                t["labels"] = torch.from_numpy(inputs["labels"][b]).to(dev)
                t["aux"] = B.make_aux(labels=t["labels"])
            elif model == "dml":
                t["X"] = torch.from_numpy(inputs["Xa"][b]).to(dev)
                t["Xb"] = torch.from_numpy(inputs["Xb"][b]).to(dev)
                t["similar"] = torch.from_numpy(inputs["similar"]).to(dev)
                t["aux"] = B.make_aux(Xb=t["Xb"], similar=t["similar"])
            else:
                t["X"] = None
                t["rowptr"] = torch.from_numpy(inputs["rowptr"][b].view(np.int32).copy()).to(dev)
                t["idx"] = torch.from_numpy(inputs["idx"][b].view(np.int32).copy()).to(dev)
                t["val"] = torch.from_numpy(inputs["val"][b]).to(dev)
                t["Xdata"] = torch.from_numpy(inputs["Xdata"][b]).to(dev)
                t["aux"] = B.make_aux(rowptr=t["rowptr"], idx=t["idx"], val=t["val"], Xdata=t["Xdata"])
            self.batches.append(t)
        self.sf_buf = self._alloc((self.ctx.sf_buffer_bytes,), torch.uint8, guard)
        self.U = self._alloc((self.K, self.ldu), self.val_dtype, guard)
        self.V = None if sparse else self._alloc((self.K, self.ldv), self.val_dtype, guard)

    def _alloc(self, shape, dtype, guard, fill=None):
        if not guard:
            return fill.clone() if fill is not None else torch.zeros(*shape, dtype=dtype, device=self.device)
        g = Guarded(tuple(shape), dtype, self.device, fill)
        self._guards.append(g)
        return g.t

    def guards_intact(self) -> bool:
        return all(g.intact() for g in self._guards)

    def reset(self):
        self.W.copy_(self.W0)
        self.ctx.invalidate()

    def compute_factors(self, b: int = 0):
        t = self.batches[b % self.pool]
        self.ctx.compute_factors(self.W, t["X"], t["aux"], self.U, self.V)

    def pack(self, b: int = 0, clock: int = 0):
        t = self.batches[b % self.pool]
        self.ctx.pack(self.U, self.V, t["aux"], self.sf_buf, clock)

    def apply(self, eta: float, K: int | None = None):
        self.ctx.apply(self.W, self.sf_buf, eta, K)

    def step(self, t_idx: int, eta: float | None = None, K: int | None = None):
        t = self.batches[t_idx % self.pool]
        self.ctx.step(self.W, t["X"], t["aux"], self.sf_buf, self.cfg["eta"] if eta is None else eta, K, clock=t_idx)

    def loss(self, b: int = 0):
        """Minibatch objective of batch b at the current W: a one-element float64 device tensor (asynchronous)."""
        t = self.batches[b % self.pool]
        out = torch.zeros(1, dtype=torch.float64, device=self.W.device)
        self.ctx.loss(self.W, t["X"], t["aux"], out)
        return out

    def close(self):
        self.ctx.destroy()
