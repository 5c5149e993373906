"""ctypes binding of libcompact.so: argument marshalling only.

Every step of the layer (projection generation, the three GEMMs, Adam and the
decompressed weight update) runs in the library's CUDA kernels.  torch is used
for device memory and streams.  There is no CPU fallback: if the library cannot
be loaded, `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional

import torch

from .build import LIB_PATH

OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_ALIGNMENT, ERR_DTYPE, ERR_EPOCH_MISMATCH, ERR_WORKSPACE, \
    ERR_UNSUPPORTED_ARCH, ERR_CUDA, ERR_DEVICE_TIMEOUT = range(1, 10)
ERR_SCRATCH_LIMIT = 10
ERR_TOO_MANY_LAYERS = 11
NOALLOC_SCRATCH_BYTES = 32 << 20
F32, BF16 = 0, 1

EXPORTS = [
    "compact_layer_create", "compact_layer_destroy", "compact_z_ld", "compact_workspace_bytes",
    "compact_fwd_workspace_bytes", "compact_group_fwd_workspace_bytes",
    "compact_saved_bytes", "compact_linear_fwd", "compact_linear_bwd", "compact_recompute_workspace_bytes",
    "compact_linear_bwd_recompute", "compact_group_workspace_bytes", "compact_group_fwd", "compact_group_bwd",
    "compact_adam_update", "compact_adam_update_noalloc",
    "compact_refresh_projection", "compact_layer_get_state", "compact_layer_set_state",
    "compact_layer_status", "compact_debug_wait_that_runs_out", "compact_debug_philox_u32", "compact_debug_philox_layer_u32", "compact_debug_sparse_terms", "compact_debug_projection",
    "compact_set_kernel_family", "compact_kernel_launch_count", "compact_status_string",
]


class LayerConfig(C.Structure):
    _fields_ = [("n", C.c_int32), ("m", C.c_int32), ("r", C.c_int32), ("dtype", C.c_int32),
                ("seed", C.c_uint64), ("layer_id", C.c_uint32), ("refresh_T", C.c_uint32),
                ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("alpha", C.c_float), ("sparse_s", C.c_int32)]


class LayerState(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("layer_id", C.c_uint32), ("epoch", C.c_uint32), ("step", C.c_uint64)]


_lib = None


def lib() -> C.CDLL:
    """Loads libcompact.so (built in-tree by `build.build_library`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2410_15352_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i64, u32p = C.c_void_p, C.c_int64, C.POINTER(C.c_uint32)
    L.compact_layer_create.argtypes = [C.POINTER(LayerConfig), C.POINTER(vp)]
    L.compact_layer_destroy.argtypes = [vp]
    L.compact_z_ld.argtypes = [vp]
    L.compact_z_ld.restype = i64
    L.compact_workspace_bytes.argtypes = [vp, i64]
    L.compact_workspace_bytes.restype = C.c_size_t
    L.compact_saved_bytes.argtypes = [vp, i64]
    L.compact_saved_bytes.restype = C.c_size_t
    L.compact_fwd_workspace_bytes.argtypes = [vp]
    L.compact_fwd_workspace_bytes.restype = C.c_size_t
    L.compact_linear_fwd.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, u32p, vp, C.c_size_t, vp]
    L.compact_linear_bwd.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, C.c_int, vp,
                                     C.c_size_t, vp]
    L.compact_recompute_workspace_bytes.argtypes = [vp, i64]
    L.compact_recompute_workspace_bytes.restype = C.c_size_t
    L.compact_linear_bwd_recompute.argtypes = [vp, i64, vp, i64, C.c_uint32, vp, i64, vp, i64, vp, i64, vp, i64, C.c_int,
                                               vp, C.c_size_t, vp]
    pp, ip = C.POINTER(C.c_void_p), C.POINTER(C.c_int64)
    L.compact_group_workspace_bytes.argtypes = [pp, C.c_int, i64]
    L.compact_group_workspace_bytes.restype = C.c_size_t
    L.compact_group_fwd_workspace_bytes.argtypes = [pp, C.c_int]
    L.compact_group_fwd_workspace_bytes.restype = C.c_size_t
    L.compact_group_fwd.argtypes = [pp, C.c_int, i64, vp, i64, pp, ip, pp, ip, pp, ip, u32p, vp, C.c_size_t, vp]
    L.compact_group_bwd.argtypes = [pp, C.c_int, i64, pp, ip, pp, ip, pp, ip, vp, i64, pp, ip, C.c_int, vp, C.c_size_t, vp]
    L.compact_adam_update.argtypes = [vp, vp, i64, vp, i64, vp, vp, C.c_uint32, C.c_float, vp, C.c_size_t, vp]
    L.compact_adam_update_noalloc.argtypes = [vp, vp, i64, vp, i64, vp, vp, C.c_uint32, C.c_float, vp]
    L.compact_refresh_projection.argtypes = [vp, C.c_int, u32p]
    L.compact_layer_get_state.argtypes = [vp, C.POINTER(LayerState)]
    L.compact_layer_set_state.argtypes = [vp, C.POINTER(LayerState)]
    L.compact_layer_status.argtypes = [vp]
    L.compact_debug_wait_that_runs_out.argtypes = [vp, vp]
    L.compact_debug_philox_u32.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_int32, C.c_int32, vp, vp]
    L.compact_debug_philox_layer_u32.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_int32, C.c_int32, vp, vp]
    L.compact_debug_sparse_terms.argtypes = [vp, C.c_uint32, vp, vp]
    L.compact_debug_projection.argtypes = [vp, C.c_uint32, vp, vp]
    L.compact_set_kernel_family.argtypes = [C.c_int]
    L.compact_kernel_launch_count.restype = C.c_uint64
    L.compact_status_string.argtypes = [C.c_int]
    L.compact_status_string.restype = C.c_char_p
    _lib = L
    return L


class CompactError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib().compact_status_string(code).decode()} (status {code})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise CompactError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def status_string(code: int) -> str:
    return lib().compact_status_string(code).decode()


def set_kernel_family(family: int) -> int:
    return lib().compact_set_kernel_family(family)


def kernel_launch_count() -> int:
    return int(lib().compact_kernel_launch_count())


def debug_philox_u32(seed: int, layer_id: int, epoch: int, n: int, r: int, stream=None, layer_form: bool = False) -> torch.Tensor:
    """Raw Philox words behind P; layer_form=True takes them from the function the GEMM kernels' generators call."""
    out = torch.empty((n, 4 * ((r + 7) // 8)), dtype=torch.int32, device="cuda")
    fn = lib().compact_debug_philox_layer_u32 if layer_form else lib().compact_debug_philox_u32
    _check(fn(seed, layer_id, epoch, n, r, _ptr(out), _stream(stream)), "debug_philox_u32")
    return out


class CompactLinear:
    """One compressed linear layer: thin handle over `compact_layer_t`."""

    def __init__(self, n: int, m: int, r: int, dtype: torch.dtype = torch.bfloat16, seed: int = 0,
                 layer_id: int = 0, refresh_T: int = 0, lr: float = 1e-3, beta1: float = 0.9,
                 beta2: float = 0.999, eps: float = 1e-8, alpha: float = 1.0, sparse_s: int = 0):
        """sparse_s > 0 selects the sparse Johnson-Lindenstrauss projection with that many terms per row of P."""
        self.n, self.m, self.r = n, m, r
        self.sparse_s = sparse_s
        self.dtype = dtype
        code = {torch.float32: F32, torch.bfloat16: BF16}.get(dtype)
        if code is None:
            raise CompactError(ERR_DTYPE, "CompactLinear")
        self.cfg = LayerConfig(n, m, r, code, seed, layer_id, refresh_T, lr, beta1, beta2, eps, alpha, sparse_s)
        self._h = C.c_void_p()
        _check(lib().compact_layer_create(C.byref(self.cfg), C.byref(self._h)), "compact_layer_create")
        self.ldz = int(lib().compact_z_ld(self._h))
        self._ws: Optional[torch.Tensor] = None

    def __del__(self):
        h = getattr(self, "_h", None)
        if h and _lib is not None:
            _lib.compact_layer_destroy(h)
            self._h = None

    # -- queries -------------------------------------------------------------------
    def workspace_bytes(self, tokens: int) -> int:
        return int(lib().compact_workspace_bytes(self._h, tokens))

    def saved_bytes(self, tokens: int) -> int:
        return int(lib().compact_saved_bytes(self._h, tokens))

    def state(self) -> LayerState:
        st = LayerState()
        _check(lib().compact_layer_get_state(self._h, C.byref(st)), "compact_layer_get_state")
        return st

    def set_state(self, seed: int, layer_id: int, epoch: int, step: int) -> None:
        st = LayerState(seed, layer_id, epoch, step)
        _check(lib().compact_layer_set_state(self._h, C.byref(st)), "compact_layer_set_state")

    @property
    def epoch(self) -> int:
        return int(self.state().epoch)

    @property
    def step(self) -> int:
        return int(self.state().step)

    def status(self) -> int:
        return int(lib().compact_layer_status(self._h))

    def debug_wait_that_runs_out(self, stream=None) -> None:
        """Launches the test kernel whose bounded wait gives up (sets this layer's status word)."""
        _check(lib().compact_debug_wait_that_runs_out(self._h, _stream(stream)), "compact_debug_wait_that_runs_out")

    def workspace(self, tokens: int) -> torch.Tensor:
        need = max(self.workspace_bytes(tokens), 256)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        return self._ws

    # -- Algorithm 1 ---------------------------------------------------------------
    def forward(self, X: torch.Tensor, W: torch.Tensor, Y: Optional[torch.Tensor] = None,
                Z: Optional[torch.Tensor] = None, keep_z: bool = True, stream=None, scratch: bool = True):
        """keep_z=False: nothing is kept for the backward (returns Z=None); use backward_recompute.
        scratch=False: the call gets no workspace, so P is generated inside the kernel (same Y and Z)."""
        tokens = X.shape[0]
        ws = self.workspace(tokens) if scratch else None
        if Y is None:
            Y = torch.empty((tokens, self.m), dtype=self.dtype, device=X.device)
        if Z is None and keep_z:
            Z = torch.empty((tokens, self.ldz), dtype=self.dtype, device=X.device)
        ep = C.c_uint32()
        _check(lib().compact_linear_fwd(self._h, tokens, _ptr(X), X.stride(0) if tokens else self.n, _ptr(W),
                                        W.stride(0), _ptr(Y), Y.stride(0) if tokens else self.m, _ptr(Z),
                                        (Z.stride(0) if tokens else self.ldz) if Z is not None else 0, C.byref(ep),
                                        _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream)),
               "compact_linear_fwd")
        return Y, Z, int(ep.value)

    # -- Algorithm 2 ---------------------------------------------------------------
    def backward(self, dY: torch.Tensor, Z: torch.Tensor, W: torch.Tensor, Gc: Optional[torch.Tensor] = None,
                 dX: Optional[torch.Tensor] = None, need_dX: bool = True, accumulate: bool = False, stream=None):
        tokens = dY.shape[0]
        if Gc is None:
            Gc = torch.empty((self.r, self.m), dtype=torch.float32, device=dY.device)
        if dX is None and need_dX:
            dX = torch.empty((tokens, self.n), dtype=self.dtype, device=dY.device)
        ws = self.workspace(tokens)
        _check(lib().compact_linear_bwd(self._h, tokens, _ptr(dY), dY.stride(0) if tokens else self.m, _ptr(Z),
                                        Z.stride(0) if tokens else self.ldz, _ptr(W), W.stride(0), _ptr(dX),
                                        (dX.stride(0) if tokens else self.n) if dX is not None else 0, _ptr(Gc),
                                        Gc.stride(0), int(accumulate), _ptr(ws), ws.numel(), _stream(stream)),
               "compact_linear_bwd")
        return dX, Gc

    def backward_recompute(self, X: torch.Tensor, epoch_of_fwd: int, dY: torch.Tensor, W: torch.Tensor,
                           Gc: Optional[torch.Tensor] = None, dX: Optional[torch.Tensor] = None, need_dX: bool = True,
                           accumulate: bool = False, stream=None):
        """Algorithm 2 for a forward that kept no Z: Z = X P is computed again into scratch."""
        tokens = dY.shape[0]
        if Gc is None:
            Gc = torch.empty((self.r, self.m), dtype=torch.float32, device=dY.device)
        if dX is None and need_dX:
            dX = torch.empty((tokens, self.n), dtype=self.dtype, device=dY.device)
        need = max(int(lib().compact_recompute_workspace_bytes(self._h, tokens)), 256)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        ws = self._ws
        _check(lib().compact_linear_bwd_recompute(self._h, tokens, _ptr(X), X.stride(0) if tokens else self.n,
                                                  epoch_of_fwd, _ptr(dY), dY.stride(0) if tokens else self.m, _ptr(W),
                                                  W.stride(0), _ptr(dX),
                                                  (dX.stride(0) if tokens else self.n) if dX is not None else 0,
                                                  _ptr(Gc), Gc.stride(0), int(accumulate), _ptr(ws), ws.numel(),
                                                  _stream(stream)),
               "compact_linear_bwd_recompute")
        return dX, Gc

    # -- Algorithm 3 ---------------------------------------------------------------
    def adam_update(self, W: torch.Tensor, Gc: torch.Tensor, M: torch.Tensor, V: torch.Tensor, epoch_of_Gc: int,
                    lr: float = math.nan, stream=None) -> None:
        ws = self.workspace(0)
        _check(lib().compact_adam_update(self._h, _ptr(W), W.stride(0), _ptr(Gc), Gc.stride(0), _ptr(M), _ptr(V),
                                         epoch_of_Gc, lr, _ptr(ws), ws.numel(), _stream(stream)),
               "compact_adam_update")

    def adam_update_noalloc(self, W: torch.Tensor, Gc: torch.Tensor, M: torch.Tensor, V: torch.Tensor,
                            epoch_of_Gc: int, lr: float = math.nan, stream=None) -> None:
        """Same update, for callers that cannot provide device memory: the scratch is a
        fixed array inside the library (NOALLOC_SCRATCH_BYTES per GPU).  Nothing is
        allocated here either: no workspace tensor is created.  Calls that may overlap
        on the GPU share that array and race; keep them on one stream."""
        _check(lib().compact_adam_update_noalloc(self._h, _ptr(W), W.stride(0), _ptr(Gc), Gc.stride(0), _ptr(M),
                                                 _ptr(V), epoch_of_Gc, lr, _stream(stream)),
               "compact_adam_update_noalloc")

    def refresh_projection(self, force: bool = False) -> int:
        ep = C.c_uint32()
        _check(lib().compact_refresh_projection(self._h, int(force), C.byref(ep)), "compact_refresh_projection")
        return int(ep.value)

    def debug_sparse_terms(self, epoch: Optional[int] = None, stream=None) -> torch.Tensor:
        """(n, sparse_s) int32: column in the low 31 bits, sign in bit 31, of every hashed term of P."""
        out = torch.empty((self.n, self.sparse_s), dtype=torch.int32, device="cuda")
        _check(lib().compact_debug_sparse_terms(self._h, self.epoch if epoch is None else epoch, _ptr(out),
                                                _stream(stream)), "compact_debug_sparse_terms")
        return out

    def debug_projection(self, epoch: Optional[int] = None, stream=None) -> torch.Tensor:
        P = torch.empty((self.n, self.r), dtype=self.dtype, device="cuda")
        _check(lib().compact_debug_projection(self._h, self.epoch if epoch is None else epoch, _ptr(P),
                                              _stream(stream)), "compact_debug_projection")
        return P


# -- groups of layers that share their input (q, k, v; gate, up) ----------------------------------
def _ptr_array(tensors):
    return (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


def _ld_array(tensors):
    return (C.c_int64 * len(tensors))(*[t.stride(0) for t in tensors])


class CompactGroup:
    """Layers with one input: Algorithm 1 and Algorithm 2 for all of them in one launch each."""

    def __init__(self, layers):
        self.layers = list(layers)
        self._h = (C.c_void_p * len(self.layers))(*[l._h for l in self.layers])
        self._ws = None

    def workspace(self, tokens: int) -> torch.Tensor:
        need = max(int(lib().compact_group_workspace_bytes(self._h, len(self.layers), tokens)), 256)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        return self._ws

    def forward(self, X: torch.Tensor, Ws, Ys=None, Zs=None, stream=None, scratch: bool = True):
        tokens = X.shape[0]
        ws = self.workspace(tokens) if scratch else None
        if Ys is None:
            Ys = [torch.empty((tokens, l.m), dtype=l.dtype, device=X.device) for l in self.layers]
        if Zs is None:
            Zs = [torch.empty((tokens, l.ldz), dtype=l.dtype, device=X.device) for l in self.layers]
        eps = (C.c_uint32 * len(self.layers))()
        _check(lib().compact_group_fwd(self._h, len(self.layers), tokens, _ptr(X), X.stride(0), _ptr_array(Ws), _ld_array(Ws),
                                       _ptr_array(Ys), _ld_array(Ys), _ptr_array(Zs), _ld_array(Zs), eps,
                                       _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream)),
               "compact_group_fwd")
        return Ys, Zs, [int(e) for e in eps]

    def backward(self, dYs, Zs, Ws, Gcs=None, dX=None, need_dX: bool = True, accumulate: bool = False, stream=None):
        tokens = dYs[0].shape[0]
        n = self.layers[0].n
        if Gcs is None:
            Gcs = [torch.empty((l.r, l.m), dtype=torch.float32, device=dYs[0].device) for l in self.layers]
        if dX is None and need_dX:
            dX = torch.empty((tokens, n), dtype=self.layers[0].dtype, device=dYs[0].device)
        self.workspace(tokens)
        _check(lib().compact_group_bwd(self._h, len(self.layers), tokens, _ptr_array(dYs), _ld_array(dYs), _ptr_array(Zs),
                                       _ld_array(Zs), _ptr_array(Ws), _ld_array(Ws), _ptr(dX), dX.stride(0) if dX is not None else 0,
                                       _ptr_array(Gcs), _ld_array(Gcs), int(accumulate), _ptr(self._ws), self._ws.numel(),
                                       _stream(stream)),
               "compact_group_bwd")
        return dX, Gcs
