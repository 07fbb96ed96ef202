"""ctypes binding of the C ABI in ``include/demo.h`` -- argument marshalling only.

``load_library()`` opens ``libdemo_b200.so`` (built in-tree by ``build.py``) and fails loudly if it
is missing: there is no CPU or eager fallback.  ``DemoTransform`` wraps one ``demo_ctx`` and turns
lists of torch tensors into the pointer arrays the ABI takes; method names follow the ABI
(``compress`` = ``demo_compress``, ``decode_apply`` = ``demo_decode_apply``, ...).
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libdemo_b200.so")

DEMO_F32, DEMO_BF16 = 0, 1
DEMO_PATH_AUTO, DEMO_PATH_GENERIC = 0, 1
DEMO_MOMENTUM_SPATIAL, DEMO_MOMENTUM_DCT = 0, 1
DEMO_AGG_SUM, DEMO_AGG_MEAN, DEMO_AGG_COUNT_MEAN = 0, 1, 2
DEMO_PHI_SIGN, DEMO_PHI_IDENTITY = 0, 1
RECORD_BYTES = 8

EXPORTS = [
    "demo_init", "demo_init_nd", "demo_payload_bytes", "demo_payload_layout", "demo_compress", "demo_decode_apply",
    "demo_decode_signs", "demo_apply_signs",
    "demo_step_host", "demo_decode_apply_static", "demo_set_lr", "demo_set_alpha", "demo_set_decode_mode", "demo_set_basis",
    "demo_set_basis_gaussian", "demo_get_basis", "demo_selftest_bounded_wait", "demo_set_path", "demo_set_momentum_domain", "demo_launch_count", "demo_device_status",
    "demo_status_string", "demo_free",
]


class DemoTensorDesc(ctypes.Structure):
    _fields_ = [("ndim", ctypes.c_int32), ("shape", ctypes.c_int64 * 2)]


ND_MAX_DIMS = 4


class DemoNdTensorDesc(ctypes.Structure):
    _fields_ = [("ndim", ctypes.c_int32), ("shape", ctypes.c_int64 * ND_MAX_DIMS), ("chunk", ctypes.c_int32 * ND_MAX_DIMS)]


class DemoConfig(ctypes.Structure):
    _fields_ = [
        ("beta", ctypes.c_float), ("chunk", ctypes.c_int32), ("topk", ctypes.c_int32), ("lr", ctypes.c_float),
        ("weight_decay", ctypes.c_float), ("num_workers", ctypes.c_int32), ("grad_dtype", ctypes.c_int32),
    ]


class DemoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s failed: status %d (%s)" % (where, status, demo_status_string(status)))


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Open the CUDA library and declare the ABI's signatures.  Raises if the library is absent."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(
            "CUDA library %s is missing: build it with `python -m paper_2411_19870_b200.build` "
            "(there is no CPU fallback)" % p)
    lib = ctypes.CDLL(p)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    pvp = ctypes.POINTER(ctypes.c_void_p)
    lib.demo_init.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(DemoConfig), ctypes.POINTER(DemoTensorDesc), i32, i32]
    lib.demo_init.restype = i32
    lib.demo_init_nd.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(DemoConfig), ctypes.POINTER(DemoNdTensorDesc), i32, i32]
    lib.demo_init_nd.restype = i32
    lib.demo_payload_bytes.argtypes = [vp]
    lib.demo_payload_bytes.restype = ctypes.c_size_t
    lib.demo_payload_layout.argtypes = [vp, i32, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(i32)]
    lib.demo_payload_layout.restype = i32
    lib.demo_compress.argtypes = [vp, i32, pvp, pvp, vp, vp]
    lib.demo_compress.restype = i32
    lib.demo_decode_apply.argtypes = [vp, pvp, i32, pvp, vp]
    lib.demo_decode_apply.restype = i32
    lib.demo_decode_signs.argtypes = [vp, pvp, i32, pvp, vp]
    lib.demo_decode_signs.restype = i32
    lib.demo_apply_signs.argtypes = [vp, pvp, pvp, vp]
    lib.demo_apply_signs.restype = i32
    lib.demo_step_host.argtypes = [vp, pvp, pvp, pvp, pvp, pvp, vp, vp]
    lib.demo_step_host.restype = i32
    lib.demo_decode_apply_static.argtypes = [ctypes.POINTER(DemoConfig), ctypes.POINTER(DemoTensorDesc), i32, pvp, i32,
                                             pvp, i32, vp]
    lib.demo_decode_apply_static.restype = i32
    lib.demo_set_lr.argtypes = [vp, ctypes.c_float]
    lib.demo_set_lr.restype = i32
    lib.demo_set_alpha.argtypes = [vp, ctypes.c_float]
    lib.demo_set_alpha.restype = i32
    lib.demo_set_decode_mode.argtypes = [vp, i32, i32]
    lib.demo_set_decode_mode.restype = i32
    lib.demo_set_basis.argtypes = [vp, vp, vp]
    lib.demo_set_basis.restype = i32
    lib.demo_set_basis_gaussian.argtypes = [vp, vp, vp]
    lib.demo_set_basis_gaussian.restype = i32
    lib.demo_get_basis.argtypes = [vp, vp, vp]
    lib.demo_get_basis.restype = i32
    lib.demo_selftest_bounded_wait.argtypes = [vp, i64, vp]
    lib.demo_selftest_bounded_wait.restype = i32
    lib.demo_set_path.argtypes = [vp, i32]
    lib.demo_set_path.restype = i32
    lib.demo_set_momentum_domain.argtypes = [vp, i32]
    lib.demo_set_momentum_domain.restype = i32
    lib.demo_launch_count.argtypes = [vp]
    lib.demo_launch_count.restype = i64
    lib.demo_device_status.argtypes = [vp, vp]
    lib.demo_device_status.restype = i32
    lib.demo_status_string.argtypes = [i32]
    lib.demo_status_string.restype = ctypes.c_char_p
    lib.demo_free.argtypes = [vp]
    lib.demo_free.restype = None
    if path is None:
        _lib = lib
    return lib


def demo_status_string(status: int) -> str:
    return load_library().demo_status_string(int(status)).decode()


def _ptr_array(ptrs: Sequence[int]):
    return (ctypes.c_void_p * len(ptrs))(*ptrs)


def _tensor_ptrs(tensors) -> List[int]:
    return [int(t.data_ptr()) for t in tensors]


def validate_tensors(tensors, shapes, dtype, device_index: Optional[int], what: str) -> None:
    """The C ABI takes bare pointers, so the layout it assumes is checked here: one contiguous tensor per
    shape, of the given dtype, on CUDA device ``device_index`` (``None``: any device; used by CPU tests)."""
    if len(tensors) != len(shapes):
        raise ValueError("%s: expected %d tensors, got %d" % (what, len(shapes), len(tensors)))
    for i, (t, shp) in enumerate(zip(tensors, shapes)):
        if tuple(t.shape) != tuple(shp):
            raise ValueError("%s[%d]: shape %s, expected %s" % (what, i, tuple(t.shape), tuple(shp)))
        if t.dtype != dtype:
            raise ValueError("%s[%d]: dtype %s, expected %s" % (what, i, t.dtype, dtype))
        if not t.is_contiguous():
            raise ValueError("%s[%d]: not contiguous" % (what, i))
        if device_index is not None and (not t.is_cuda or t.device.index != device_index):
            raise ValueError("%s[%d]: on %s, expected cuda:%d" % (what, i, t.device, device_index))


def decode_apply_static(shapes, payloads, params, *, chunk: int, topk: int, lr: float, weight_decay: float,
                        device: int = 0, stream=None) -> None:
    """``demo_decode_apply_static``: decode + update without a context and without any allocation by
    the library (its tables live in a fixed device array; see include/demo.h for the limits).
    ``payloads`` / ``params`` are lists of device tensors."""
    lib = load_library()
    descs = (DemoTensorDesc * len(shapes))()
    for d, s in zip(descs, shapes):
        d.ndim = len(s)
        for a in range(min(len(s), 2)):
            d.shape[a] = int(s[a])
    cfg = DemoConfig(0.0, chunk, topk, lr, weight_decay, len(payloads), DEMO_F32)
    st = lib.demo_decode_apply_static(ctypes.byref(cfg), descs, len(shapes), _ptr_array(_tensor_ptrs(payloads)),
                                      len(payloads), _ptr_array(_tensor_ptrs(params)), device,
                                      DemoTransform._stream(stream))
    if st != 0:
        raise DemoError(st, "demo_decode_apply_static")


class DemoTransform:
    """One ``demo_ctx``.  ``shapes`` is a list of 1-D / 2-D shapes in payload order (``demo_init``).
    With ``chunk_shapes`` (one tuple per tensor, same order as its shape) the context comes from
    ``demo_init_nd``: tensors of any order up to 4 with rectangular chunks; ``chunk`` is then unused."""

    def __init__(self, shapes, *, chunk: int = 0, topk: int, beta: float, lr: float, weight_decay: float,
                 num_workers: int, grad_dtype: int = DEMO_BF16, device: int = 0, chunk_shapes=None):
        self.lib = load_library()
        self.shapes = [tuple(int(d) for d in s) for s in shapes]
        self.chunk_shapes = None if chunk_shapes is None else [tuple(int(d) for d in s) for s in chunk_shapes]
        self.cfg = DemoConfig(beta, chunk, topk, lr, weight_decay, num_workers, grad_dtype)
        self.num_workers = num_workers
        self.device = device
        self._ctx = ctypes.c_void_p()
        if self.chunk_shapes is None:
            descs = (DemoTensorDesc * len(self.shapes))()
            for d, s in zip(descs, self.shapes):
                d.ndim = len(s)
                for a in range(min(len(s), 2)):
                    d.shape[a] = s[a]
            st = self.lib.demo_init(ctypes.byref(self._ctx), ctypes.byref(self.cfg), descs, len(self.shapes), device)
        else:
            if len(self.chunk_shapes) != len(self.shapes) or any(
                    len(c) != len(s) for c, s in zip(self.chunk_shapes, self.shapes)):
                raise ValueError("chunk_shapes: one chunk shape per tensor, of the tensor's order")
            nd = (DemoNdTensorDesc * len(self.shapes))()
            for d, s, c in zip(nd, self.shapes, self.chunk_shapes):
                d.ndim = len(s)
                for a in range(min(len(s), ND_MAX_DIMS)):
                    d.shape[a] = s[a]
                    d.chunk[a] = c[a]
            st = self.lib.demo_init_nd(ctypes.byref(self._ctx), ctypes.byref(self.cfg), nd, len(self.shapes), device)
        if st != 0:
            self._ctx = ctypes.c_void_p()
            raise DemoError(st, "demo_init" if self.chunk_shapes is None else "demo_init_nd")
        self._ptr_cache = {}
        self._payload_bytes = int(self.lib.demo_payload_bytes(self._ctx))
        self._payload_ok = set()   # (data pointer, size) of payload buffers already checked
        self._gdtype = torch.bfloat16 if grad_dtype == DEMO_BF16 else torch.float32

    # --- queries -------------------------------------------------------------------------------
    @property
    def payload_bytes(self) -> int:
        return self._payload_bytes

    def payload_layout(self, tensor: int):
        first, n_chunks, k_eff = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int32()
        st = self.lib.demo_payload_layout(self._ctx, tensor, ctypes.byref(first), ctypes.byref(n_chunks),
                                          ctypes.byref(k_eff))
        if st != 0:
            raise DemoError(st, "demo_payload_layout")
        return first.value, n_chunks.value, k_eff.value

    @property
    def launch_count(self) -> int:
        return int(self.lib.demo_launch_count(self._ctx))

    # --- marshalling helpers -------------------------------------------------------------------
    def _array(self, key, tensors, check=None):
        """Pointer array for a list of tensors, cached per key and data pointers.  ``check`` = (shapes,
        dtype, on_device) is verified whenever the pointers are new."""
        ptrs = tuple(_tensor_ptrs(tensors))
        hit = self._ptr_cache.get(key)
        if hit is None or hit[0] != ptrs:
            if check is not None:
                shapes, dtype, on_device = check
                validate_tensors(tensors, shapes, dtype, self.device if on_device else None, str(key))
            hit = (ptrs, _ptr_array(ptrs))
            self._ptr_cache[key] = hit
        return hit[1]

    def _check_payloads(self, payloads) -> None:
        for i, p in enumerate(payloads):  # (the library itself checks their number)
            self._check_payload(p, "payloads[%d]" % i)

    def _check_payload(self, p, what: str) -> None:
        ptr = (p.data_ptr(), p.numel())
        if ptr in self._payload_ok:
            return
        if p.dtype != torch.uint8 or not p.is_contiguous() or p.numel() < self.payload_bytes or not p.is_cuda \
                or p.device.index != self.device:
            raise ValueError("%s: need a contiguous uint8 tensor of at least %d bytes on cuda:%d"
                             % (what, self.payload_bytes, self.device))
        self._payload_ok.add(ptr)

    @staticmethod
    def _stream(stream) -> ctypes.c_void_p:
        if stream is None:
            import torch

            stream = torch.cuda.current_stream()
        return ctypes.c_void_p(int(getattr(stream, "cuda_stream", stream)))

    # --- the ABI calls -------------------------------------------------------------------------
    def compress(self, worker: int, grads, momentum, payload_out, stream=None) -> None:
        self._check_payload(payload_out, "payload_out")
        st = self.lib.demo_compress(self._ctx, worker, self._array(("g", worker), grads, (self.shapes, self._gdtype, True)),
                                    self._array(("m", worker), momentum, (self.shapes, torch.float32, True)),
                                    ctypes.c_void_p(payload_out.data_ptr()), self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_compress")

    def decode_apply(self, payloads, params, stream=None) -> None:
        self._check_payloads(payloads)
        st = self.lib.demo_decode_apply(self._ctx, self._array("p", payloads), len(payloads),
                                        self._array("x", params, (self.shapes, torch.float32, True)), self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_decode_apply")

    def decode_signs(self, payloads, signs_out, stream=None) -> None:
        """Parameter-server form: sign of the reconstructed momentum as int8 tensors shaped like the parameters."""
        self._check_payloads(payloads)
        st = self.lib.demo_decode_signs(self._ctx, self._array("p", payloads), len(payloads),
                                        self._array("s", signs_out, (self.shapes, torch.int8, True)), self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_decode_signs")

    def apply_signs(self, signs, params, stream=None) -> None:
        st = self.lib.demo_apply_signs(self._ctx, self._array("s", signs, (self.shapes, torch.int8, True)),
                                       self._array("x", params, (self.shapes, torch.float32, True)), self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_apply_signs")

    def step_host(self, host_grads, dev_grads, momentum, payloads, params, host_payloads_out=None, stream=None) -> None:
        """host_grads / dev_grads / momentum: lists over workers of lists of tensors."""
        flat = lambda ll: [t for l in ll for t in l]  # noqa: E731
        out = ctypes.c_void_p(host_payloads_out.data_ptr()) if host_payloads_out is not None else ctypes.c_void_p()
        st = self.lib.demo_step_host(self._ctx, self._array("hg", flat(host_grads)), self._array("dg", flat(dev_grads)),
                                     self._array("mm", flat(momentum)), self._array("p", payloads),
                                     self._array("x", params), out, self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_step_host")

    def set_lr(self, lr: float) -> None:
        st = self.lib.demo_set_lr(self._ctx, lr)
        if st != 0:
            raise DemoError(st, "demo_set_lr")

    def set_alpha(self, alpha: float) -> None:
        st = self.lib.demo_set_alpha(self._ctx, alpha)
        if st != 0:
            raise DemoError(st, "demo_set_alpha")

    def set_decode_mode(self, aggregation: int, phi: int) -> None:
        st = self.lib.demo_set_decode_mode(self._ctx, aggregation, phi)
        if st != 0:
            raise DemoError(st, "demo_set_decode_mode")

    def _host_matrix(self, a):
        a = a.detach().to("cpu", torch.float32).contiguous() if isinstance(a, torch.Tensor) else torch.tensor(a, dtype=torch.float32)
        s = self.basis_dim
        if a.dim() != 2 or a.shape[0] != a.shape[1] or (s and a.shape[0] != s):
            raise ValueError("expected an s x s matrix")
        return a

    @property
    def basis_dim(self) -> int:
        """The s of the s x s basis: the chunk size, also for a ``chunk_shapes`` context whose chunks are all s x s
        tiles / length-s segments behind leading extents of 1 (the library builds that one with ``demo_init``);
        0 for other ``chunk_shapes`` contexts, which have no caller-supplied basis."""
        if self.chunk_shapes is None:
            return self.cfg.chunk
        sizes = set()
        for c in self.chunk_shapes:
            lead = 0
            while lead < len(c) - 1 and c[lead] == 1:
                lead += 1
            if len(c) - lead > 2:
                return 0
            sizes.update(c[lead:])
        s = sizes.pop() if len(sizes) == 1 else 0
        return s if s in (8, 16, 32, 64, 128) else 0

    def set_basis(self, basis=None, stream=None) -> None:
        """s x s matrix whose rows are the basis vectors (host or device tensor); None restores the DCT."""
        keep = None if basis is None else self._host_matrix(basis)
        st = self.lib.demo_set_basis(self._ctx, None if keep is None else keep.data_ptr(), self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_set_basis")

    def set_basis_gaussian(self, gauss, stream=None) -> None:
        """Gram-Schmidt (on the device) of the rows of an s x s matrix of N(0,1) draws."""
        keep = self._host_matrix(gauss)
        st = self.lib.demo_set_basis_gaussian(self._ctx, keep.data_ptr(), self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_set_basis_gaussian")

    def get_basis(self, stream=None) -> torch.Tensor:
        s = self.basis_dim
        out = torch.empty((max(s, 1), max(s, 1)), dtype=torch.float32)
        st = self.lib.demo_get_basis(self._ctx, out.data_ptr(), self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_get_basis")
        return out

    def selftest_bounded_wait(self, limit_cycles: int, stream=None) -> None:
        st = self.lib.demo_selftest_bounded_wait(self._ctx, int(limit_cycles), self._stream(stream))
        if st != 0:
            raise DemoError(st, "demo_selftest_bounded_wait")

    def set_path(self, path: int) -> None:
        st = self.lib.demo_set_path(self._ctx, path)
        if st != 0:
            raise DemoError(st, "demo_set_path")

    def set_momentum_domain(self, domain: int) -> None:
        st = self.lib.demo_set_momentum_domain(self._ctx, domain)
        if st != 0:
            raise DemoError(st, "demo_set_momentum_domain")

    def device_status(self, stream=None) -> int:
        return int(self.lib.demo_device_status(self._ctx, self._stream(stream)))

    def close(self) -> None:
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self.lib.demo_free(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass
