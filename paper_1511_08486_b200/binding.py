"""ctypes binding of the C ABI in include/sfb.h: same names, argument marshalling only.

Every step of the path runs inside libsfb.so's CUDA kernels.  If the library is missing or cannot
be loaded this module raises; there is no Python or CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

from .build import LIB_PATH

SFB_MLR, SFB_DML, SFB_SC = 0, 1, 2
SFB_PATH_F32, SFB_PATH_TF32, SFB_PATH_BF16, SFB_PATH_TF32X3 = 0, 1, 2, 3
SFB_OK = 0
SFB_DEV_BAD_LABEL, SFB_DEV_BAD_INDEX, SFB_DEV_BAD_HEADER, SFB_DEV_CAPACITY, SFB_DEV_TIMEOUT = 1, 2, 4, 8, 16

MODELS = {"mlr": SFB_MLR, "dml": SFB_DML, "sc": SFB_SC}
PATHS = {"f32": SFB_PATH_F32, "tf32": SFB_PATH_TF32, "bf16": SFB_PATH_BF16, "tf32x3": SFB_PATH_TF32X3}

# Every entry point include/sfb.h declares (checked by the CPU test-suite against the built library).
EXPORTS = (
    "sfb_create", "sfb_destroy", "sfb_sf_buffer_bytes", "sfb_ld", "sfb_compute_factors", "sfb_pack",
    "sfb_apply", "sfb_step", "sfb_invalidate", "sfb_status", "sfb_launch_count", "sfb_strerror",
    "sfb_profile", "sfb_stage_ms", "sfb_sc_factors_noalloc", "sfb_noalloc_max_scratch_floats",
    "sfb_halton_peers", "sfb_ssp_may_proceed", "sfb_prox", "sfb_step_host",
    "sfb_loss", "sfb_factors_shard", "sfb_commit_header", "sfb_sf_buffer_layout", "sfb_active_pairs",
    "sfb_wire_bytes",
)


class sfb_desc(C.Structure):
    _fields_ = [("model", C.c_int32), ("path", C.c_int32), ("J", C.c_int32), ("D", C.c_int32),
                ("P", C.c_int32), ("B", C.c_int32), ("v_sparse", C.c_int32), ("margin", C.c_float),
                ("nnz_capacity", C.c_uint64), ("compact", C.c_int32)]


class sfb_aux(C.Structure):
    _fields_ = [("labels", C.c_void_p), ("Xb", C.c_void_p), ("similar", C.c_void_p), ("rowptr", C.c_void_p),
                ("idx", C.c_void_p), ("val", C.c_void_p), ("Xdata", C.c_void_p), ("dual", C.c_void_p),
                ("sdca_step", C.c_float)]


class SfbError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None


def load_library(path: str | None = None) -> C.CDLL:
    """Loads libsfb.so (built in-tree by `build.build_library`) and declares the signatures."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} not found: build it first (python -m paper_1511_08486_b200.build)")
    lib = C.CDLL(path)
    vp = C.c_void_p
    lib.sfb_create.argtypes = [C.POINTER(sfb_desc), vp, C.POINTER(vp)]
    lib.sfb_create.restype = C.c_int
    lib.sfb_destroy.argtypes = [vp]
    lib.sfb_destroy.restype = C.c_int
    lib.sfb_sf_buffer_bytes.argtypes = [C.POINTER(sfb_desc)]
    lib.sfb_sf_buffer_bytes.restype = C.c_size_t
    lib.sfb_ld.argtypes = [C.POINTER(sfb_desc), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.sfb_ld.restype = C.c_int
    lib.sfb_compute_factors.argtypes = [vp, vp, vp, C.POINTER(sfb_aux), vp, vp]
    lib.sfb_compute_factors.restype = C.c_int
    lib.sfb_pack.argtypes = [vp, vp, vp, C.POINTER(sfb_aux), vp, C.c_uint32]
    lib.sfb_pack.restype = C.c_int
    lib.sfb_apply.argtypes = [vp, vp, vp, C.c_float, C.c_int32]
    lib.sfb_apply.restype = C.c_int
    lib.sfb_step.argtypes = [vp, vp, vp, C.POINTER(sfb_aux), vp, C.c_float, C.c_int32, C.c_uint32]
    lib.sfb_step.restype = C.c_int
    lib.sfb_step_host.argtypes = [vp, vp, vp, C.POINTER(sfb_aux), vp, C.c_float, C.c_int32, C.c_uint32, vp]
    lib.sfb_step_host.restype = C.c_int
    lib.sfb_prox.argtypes = [vp, vp]
    lib.sfb_prox.restype = C.c_int
    lib.sfb_active_pairs.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.sfb_active_pairs.restype = C.c_int
    lib.sfb_loss.argtypes = [vp, vp, vp, C.POINTER(sfb_aux), vp]
    lib.sfb_loss.restype = C.c_int
    lib.sfb_factors_shard.argtypes = [vp, vp, vp, C.POINTER(sfb_aux), vp, C.c_int32, C.c_int32]
    lib.sfb_factors_shard.restype = C.c_int
    lib.sfb_commit_header.argtypes = [vp, vp, C.c_uint32]
    lib.sfb_commit_header.restype = C.c_int
    lib.sfb_sf_buffer_layout.argtypes = [C.POINTER(sfb_desc), C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    lib.sfb_sf_buffer_layout.restype = C.c_int
    lib.sfb_wire_bytes.argtypes = [vp, vp, C.POINTER(C.c_uint64)]
    lib.sfb_wire_bytes.restype = C.c_int
    lib.sfb_invalidate.argtypes = [vp]
    lib.sfb_invalidate.restype = C.c_int
    lib.sfb_status.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.sfb_status.restype = C.c_int
    lib.sfb_launch_count.argtypes = [vp]
    lib.sfb_launch_count.restype = C.c_int64
    lib.sfb_profile.argtypes = [vp, C.c_int]
    lib.sfb_profile.restype = C.c_int
    lib.sfb_stage_ms.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.sfb_stage_ms.restype = C.c_int
    lib.sfb_sc_factors_noalloc.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, vp, vp, vp, vp, vp, C.c_int32, vp, vp]
    lib.sfb_sc_factors_noalloc.restype = C.c_int
    lib.sfb_noalloc_max_scratch_floats.argtypes = []
    lib.sfb_noalloc_max_scratch_floats.restype = C.c_int64
    lib.sfb_halton_peers.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_int32)]
    lib.sfb_halton_peers.restype = C.c_int
    lib.sfb_ssp_may_proceed.argtypes = [C.c_int64, C.POINTER(C.c_int64), C.c_int32, C.c_int64]
    lib.sfb_ssp_may_proceed.restype = C.c_int
    lib.sfb_strerror.argtypes = [C.c_int]
    lib.sfb_strerror.restype = C.c_char_p
    if path == LIB_PATH:
        _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().sfb_strerror(code).decode()


def make_desc(model, path, J, D, P, B, v_sparse=0, margin=1.0, nnz_capacity=0, compact=0) -> sfb_desc:
    return sfb_desc(MODELS.get(model, model), PATHS.get(path, path), J, D, P, B, int(v_sparse), float(margin),
                    int(nnz_capacity), int(compact))


def _ptr(t) -> int | None:
    """Device pointer of a torch tensor (or None)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def make_aux(labels=None, Xb=None, similar=None, rowptr=None, idx=None, val=None, Xdata=None, dual=None,
             sdca_step=0.0) -> sfb_aux:
    return sfb_aux(_ptr(labels), _ptr(Xb), _ptr(similar), _ptr(rowptr), _ptr(idx), _ptr(val), _ptr(Xdata), _ptr(dual),
                   float(sdca_step))


def sfb_sf_buffer_bytes(desc: sfb_desc) -> int:
    return int(load_library().sfb_sf_buffer_bytes(C.byref(desc)))


def sfb_sf_buffer_layout(desc: sfb_desc) -> tuple[int, int]:
    """(streams_off, stream_stride) in bytes: where the worker streams sit inside the SF buffer."""
    off, stride = C.c_uint64(0), C.c_uint64(0)
    r = load_library().sfb_sf_buffer_layout(C.byref(desc), C.byref(off), C.byref(stride))
    if r != SFB_OK:
        raise SfbError(r, "sfb_sf_buffer_layout")
    return int(off.value), int(stride.value)


def sfb_ld(desc: sfb_desc) -> tuple[int, int]:
    ldu, ldv = C.c_int32(0), C.c_int32(0)
    r = load_library().sfb_ld(C.byref(desc), C.byref(ldu), C.byref(ldv))
    if r != SFB_OK:
        raise SfbError(r, "sfb_ld")
    return ldu.value, ldv.value


def sfb_sc_factors_noalloc(W, J, D, K, rowptr, idx, val, Xdata, U, ldu, dev_status=None, stream=None) -> None:
    """Sparse-coding factors without any device allocation (see include/sfb.h); raises SfbError on a negative code.

    For callers that cannot allocate: no context is created, the scratch is a fixed array inside the
    library.  Calls share that array, so keep them on one stream.
    """
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    r = load_library().sfb_sc_factors_noalloc(_ptr(W), J, D, K, _ptr(rowptr), _ptr(idx), _ptr(val), _ptr(Xdata),
                                              _ptr(U), ldu, _ptr(dev_status), C.c_void_p(stream))
    if r != SFB_OK:
        raise SfbError(r, "sfb_sc_factors_noalloc")


def sfb_halton_peers(P: int, Q: int, p: int) -> list[int]:
    out = (C.c_int32 * max(Q, 1))()
    r = load_library().sfb_halton_peers(P, Q, p, out)
    if r != SFB_OK:
        raise SfbError(r, "sfb_halton_peers")
    return [int(out[i]) for i in range(Q)]


def sfb_ssp_may_proceed(t_p: int, tau, staleness: int) -> bool:
    arr = (C.c_int64 * len(tau))(*[int(t) for t in tau])
    r = load_library().sfb_ssp_may_proceed(int(t_p), arr, len(tau), int(staleness))
    if r < 0:
        raise SfbError(r, "sfb_ssp_may_proceed")
    return bool(r)


def sfb_noalloc_max_scratch_floats() -> int:
    return int(load_library().sfb_noalloc_max_scratch_floats())


class Context:
    """Owns one sfb_ctx.  Methods carry the C names without the prefix and raise SfbError on a negative code."""

    def __init__(self, desc: sfb_desc, stream: int | None = None):
        self._lib = load_library()
        self.desc = desc
        if stream is None:
            import torch
            stream = torch.cuda.current_stream().cuda_stream
        h = C.c_void_p(None)
        r = self._lib.sfb_create(C.byref(desc), C.c_void_p(stream), C.byref(h))
        if r != SFB_OK:
            raise SfbError(r, "sfb_create")
        self._h = h
        self.ldu, self.ldv = sfb_ld(desc)
        self.sf_buffer_bytes = sfb_sf_buffer_bytes(desc)
        self.K = desc.P * desc.B

    def _chk(self, r: int, what: str):
        if r != SFB_OK:
            raise SfbError(r, what)

    def compute_factors(self, W, X, aux: sfb_aux, U, V=None):
        self._chk(self._lib.sfb_compute_factors(self._h, _ptr(W), _ptr(X), C.byref(aux), _ptr(U), _ptr(V)),
                  "sfb_compute_factors")

    def pack(self, U, V, aux: sfb_aux | None, sf_buf, clock: int = 0):
        a = C.byref(aux) if aux is not None else None
        self._chk(self._lib.sfb_pack(self._h, _ptr(U), _ptr(V), a, _ptr(sf_buf), clock), "sfb_pack")

    def apply(self, W, sf_buf, eta: float, K: int | None = None):
        self._chk(self._lib.sfb_apply(self._h, _ptr(W), _ptr(sf_buf), eta, self.K if K is None else K), "sfb_apply")

    def step(self, W, X, aux: sfb_aux, sf_buf, eta: float, K: int | None = None, clock: int = 0):
        self._chk(self._lib.sfb_step(self._h, _ptr(W), _ptr(X), C.byref(aux), _ptr(sf_buf), eta,
                                     self.K if K is None else K, clock), "sfb_step")

    def step_host(self, W, X_host, aux_host: sfb_aux, sf_buf, eta: float, K: int | None = None, clock: int = 0,
                  header_host=None):
        """sfb_step with the minibatch in host memory (tensors on the CPU, ideally pinned)."""
        self._chk(self._lib.sfb_step_host(self._h, _ptr(W), _ptr(X_host), C.byref(aux_host), _ptr(sf_buf), eta,
                                          self.K if K is None else K, clock, _ptr(header_host)), "sfb_step_host")

    def prox(self, W):
        self._chk(self._lib.sfb_prox(self._h, _ptr(W)), "sfb_prox")

    def factors_shard(self, W, X, aux: sfb_aux, sf_buf, first_worker: int, n_workers: int):
        self._chk(self._lib.sfb_factors_shard(self._h, _ptr(W), _ptr(X), C.byref(aux), _ptr(sf_buf), first_worker,
                                              n_workers), "sfb_factors_shard")

    def commit_header(self, sf_buf, clock: int = 0):
        self._chk(self._lib.sfb_commit_header(self._h, _ptr(sf_buf), clock), "sfb_commit_header")

    def active_pairs(self) -> int:
        """Pairs the last step multiplied through (synchronises)."""
        n = C.c_int32(0)
        self._chk(self._lib.sfb_active_pairs(self._h, C.byref(n)), "sfb_active_pairs")
        return int(n.value)

    def loss(self, W, X, aux: sfb_aux, out):
        """Minibatch objective at W into `out` (one float64 on the device); asynchronous."""
        self._chk(self._lib.sfb_loss(self._h, _ptr(W), _ptr(X), C.byref(aux), _ptr(out)), "sfb_loss")

    def wire_bytes(self, sf_buf) -> int:
        """Bytes a broadcast of the committed buffer would carry (synchronises)."""
        n = C.c_uint64(0)
        self._chk(self._lib.sfb_wire_bytes(self._h, _ptr(sf_buf), C.byref(n)), "sfb_wire_bytes")
        return int(n.value)

    def invalidate(self):
        self._chk(self._lib.sfb_invalidate(self._h), "sfb_invalidate")

    def status(self) -> int:
        s = C.c_int32(0)
        self._chk(self._lib.sfb_status(self._h, C.byref(s)), "sfb_status")
        return s.value

    def profile(self, enable: bool):
        self._chk(self._lib.sfb_profile(self._h, int(enable)), "sfb_profile")

    def stage_ms(self) -> tuple[float, float, int]:
        f, a, n = C.c_float(0), C.c_float(0), C.c_int32(0)
        self._chk(self._lib.sfb_stage_ms(self._h, C.byref(f), C.byref(a), C.byref(n)), "sfb_stage_ms")
        return f.value, a.value, n.value

    def launch_count(self) -> int:
        return int(self._lib.sfb_launch_count(self._h))

    def destroy(self):
        if self._h is not None and self._h.value:
            self._lib.sfb_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
