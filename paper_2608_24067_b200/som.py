"""Thin Python binding over the C-ABI CUDA library (``include/som.h``).

Argument marshalling only: every step of the search runs in the library's kernels.
PyTorch supplies device memory and streams.  If ``libsom_b200.so`` is missing or cannot
be loaded this module raises; there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsom_b200.so")

SOM_OK = 0
STATUS_NAMES = {
    0: "SOM_OK", 1: "SOM_ERR_INVALID_ARG", 2: "SOM_ERR_NORMS_STALE", 3: "SOM_ERR_UNSUPPORTED",
    4: "SOM_ERR_CUDA", 5: "SOM_ERR_BAD_CSR", 6: "SOM_ERR_NO_DEVICE",
}

# every symbol include/som.h declares
EXPORTS = [
    "som_create", "som_norms", "som_bmu", "som_bmu_host", "som_validate_csr", "som_get_norms",
    "som_destroy", "som_status_string", "som_last_cuda_error", "som_set_timing", "som_get_timing",
    "som_launch_count", "som_set_option", "som_norms_noalloc", "som_bmu2", "som_create_f16", "som_update", "som_last_uncertain", "som_bmu_values",
    "som_bmu_host_async", "som_host_sync", "som_plan_create", "som_bmu_planned", "som_plan_destroy",
    "som_device_flags", "som_measure_fadd_peak", "som_measure_operand_paths", "som_tc_probe",
]

NOALLOC_MAX_M = 524288

_lib = None


class SomError(RuntimeError):
    def __init__(self, status: int, where: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        msg = "%s failed: %s" % (where, STATUS_NAMES.get(status, str(status)))
        if cuda_error:
            msg += " (cudaError %d)" % cuda_error
        super().__init__(msg)


def load_library():
    """Load the compiled CUDA library; raise if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "CUDA library %s not found: build it with `python -m paper_2608_24067_b200.build` "
            "(there is no CPU fallback)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    P, I32, I64, INT = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_int
    lib.som_create.argtypes = [ctypes.POINTER(P), I32, I64, P]
    lib.som_create_f16.argtypes = [ctypes.POINTER(P), I32, I64, P]
    lib.som_create_f16.restype = INT
    lib.som_norms.argtypes = [P, P]
    lib.som_bmu.argtypes = [P, P, P, I64, P, P, P]
    lib.som_bmu_host.argtypes = [P, P, P, I64, P, P, P]
    lib.som_bmu_host_async.argtypes = [P, P, P, I64, P, P, P]
    lib.som_bmu_host_async.restype = INT
    lib.som_host_sync.argtypes = [P]
    lib.som_host_sync.restype = INT
    lib.som_plan_create.argtypes = [P, P, P, I64, ctypes.POINTER(P), P]
    lib.som_plan_create.restype = INT
    lib.som_bmu_planned.argtypes = [P, P, P, P, P]
    lib.som_bmu_planned.restype = INT
    lib.som_plan_destroy.argtypes = [P]
    lib.som_plan_destroy.restype = INT
    lib.som_bmu2.argtypes = [P, P, P, I64, P, P, P, P, P]
    lib.som_bmu2.restype = INT
    lib.som_bmu_values.argtypes = [P, P, P, P, I64, P, P, P]
    lib.som_bmu_values.restype = INT
    lib.som_update.argtypes = [P, I32, I32, P, P, I64, P, I32, P]
    lib.som_update.restype = INT
    lib.som_validate_csr.argtypes = [P, P, P, I64, P]
    lib.som_get_norms.argtypes = [P, P, P]
    lib.som_destroy.argtypes = [P]
    lib.som_status_string.argtypes = [INT]
    lib.som_status_string.restype = ctypes.c_char_p
    lib.som_last_cuda_error.argtypes = [P]
    lib.som_set_timing.argtypes = [P, INT]
    lib.som_get_timing.argtypes = [P, P, INT]
    lib.som_launch_count.argtypes = [P]
    lib.som_launch_count.restype = I64
    lib.som_last_uncertain.argtypes = [P]
    lib.som_last_uncertain.restype = I64
    lib.som_set_option.argtypes = [P, INT, I64]
    lib.som_measure_fadd_peak.argtypes = [ctypes.POINTER(ctypes.c_double), P, I64, P]
    lib.som_measure_fadd_peak.restype = INT
    lib.som_measure_operand_paths.argtypes = [ctypes.POINTER(ctypes.c_double), INT, P, I64, P, I64, P]
    lib.som_measure_operand_paths.restype = INT
    lib.som_tc_probe.argtypes = [P, P, P, I32, I32, I32, I32, I32, I32, P, P, P, P, P]
    lib.som_tc_probe.restype = INT
    lib.som_device_flags.argtypes = [P, P]
    lib.som_device_flags.restype = INT
    lib.som_norms_noalloc.argtypes = [I32, I64, P, P, P]
    lib.som_norms_noalloc.restype = INT
    for name in ("som_create", "som_norms", "som_bmu", "som_bmu_host", "som_validate_csr",
                 "som_get_norms", "som_destroy", "som_last_cuda_error", "som_set_timing",
                 "som_get_timing", "som_set_option"):
        getattr(lib, name).restype = INT
    _lib = lib
    return lib


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev_ptr(t: torch.Tensor, dtype, name: str) -> int:
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CUDA tensor of %s" % (name, dtype))
    return t.data_ptr()


def _host_ptr(t: torch.Tensor, dtype, name: str) -> int:
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError("%s must be a contiguous CPU tensor of %s" % (name, dtype))
    return t.data_ptr()


def norms_noalloc(V: int, M: int, codebook: torch.Tensor, out: torch.Tensor, stream=None) -> torch.Tensor:
    """som_norms_noalloc: squared norms into a caller-provided fp32 CUDA tensor, for callers that
    must not allocate device memory (no handle, scratch lives inside the library; M is limited
    to NOALLOC_MAX_M).  ``out`` is written on ``stream``; nothing is allocated here either."""
    lib = load_library()
    if codebook.numel() != V * M or out.numel() != M:
        raise ValueError("codebook must hold V*M elements and out M elements")
    with torch.cuda.device(codebook.device):
        rc = lib.som_norms_noalloc(V, M, _dev_ptr(codebook, torch.float32, "codebook"),
                                   _dev_ptr(out, torch.float32, "out"), _stream_ptr(stream))
    if rc != SOM_OK:
        raise SomError(rc, "som_norms_noalloc")
    return out


def measure_operand_paths(device=None, stream=None, buffer_mb: int = 16) -> dict:
    """som_measure_operand_paths: bytes per clock and SM that reach registers from shared memory, from an
    L2-resident buffer (global loads), from both at once, and through a linear texture."""
    lib = load_library()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        rows = torch.zeros(buffer_mb << 18, dtype=torch.float32, device=dev)
        scratch = torch.empty(514 * sms + 2, dtype=torch.float32, device=dev)
        out = (ctypes.c_double * 4)()
        rc = lib.som_measure_operand_paths(out, 4, rows.data_ptr(), rows.numel() * 4, scratch.data_ptr(),
                                           scratch.numel(), _stream_ptr(stream))
    if rc != SOM_OK:
        raise SomError(rc, "som_measure_operand_paths")
    return {"shared": float(out[0]), "l2_global": float(out[1]), "shared_and_l2": float(out[2]), "l2_texture": float(out[3])}


def measure_fadd_peak(device=None, stream=None) -> float:
    """som_measure_fadd_peak: the FP32 add rate (adds/s) the current device delivers on independent
    add chains; the scratch tensor is allocated here, the measurement runs in the library."""
    lib = load_library()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        scratch = torch.empty(2048 * sms, dtype=torch.float32, device=dev)
        out = ctypes.c_double(0.0)
        rc = lib.som_measure_fadd_peak(ctypes.byref(out), scratch.data_ptr(), scratch.numel(), _stream_ptr(stream))
    if rc != SOM_OK:
        raise SomError(rc, "som_measure_fadd_peak")
    return float(out.value)


def tc_probe(rows: torch.Tensor, hnorm: torch.Tensor, bits: torch.Tensor, H: int, terms: int, n_tiles: int,
             mode: int = 7, repeats: int = 1, blocks: int = 1, stream=None) -> dict:
    """som_tc_probe: the densified hot-feature tile on tcgen05 (argument marshalling only).  Returns the
    first tile's partial scores [128, 64], the per-sample minima [blocks, 128], the cycles per block and
    the kernel's status word (tensors on the device; synchronise before reading)."""
    lib = load_library()
    dev = rows.device
    out = torch.zeros(128, 64, dtype=torch.float32, device=dev)
    mins = torch.zeros(blocks, 128, dtype=torch.float32, device=dev)
    cycles = torch.zeros(blocks, dtype=torch.int64, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if bits.dtype != torch.int32 or bits.numel() != n_tiles * 128 * (H // 32):
        raise ValueError("bits must be int32 [n_tiles * 128, H / 32]")
    with torch.cuda.device(dev):
        rc = lib.som_tc_probe(_dev_ptr(rows, torch.float32, "rows"), _dev_ptr(hnorm, torch.float32, "hnorm"),
                              bits.data_ptr(), H, terms, n_tiles, mode, repeats, blocks, out.data_ptr(),
                              mins.data_ptr(), cycles.data_ptr(), status.data_ptr(), _stream_ptr(stream))
    if rc != SOM_OK:
        raise SomError(rc, "som_tc_probe")
    return {"out": out, "mins": mins, "cycles": cycles, "status": status}


class Plan:
    """A batch plan (som_plan_create); search it with ``bmu()`` as often as the codebook changes."""

    def __init__(self, som_handle: "Som", indptr: torch.Tensor, indices: torch.Tensor, stream=None):
        self._som = som_handle
        self._lib = som_handle._lib
        self.indptr, self.indices = indptr, indices  # borrowed by the plan: keep them alive
        self.n = indptr.numel() - 1
        self._p = ctypes.c_void_p()
        rc = self._lib.som_plan_create(som_handle._h, _dev_ptr(indptr, torch.int32, "indptr"),
                                       _dev_ptr(indices, torch.int32, "indices"), self.n,
                                       ctypes.byref(self._p), _stream_ptr(stream))
        som_handle._check(rc, "som_plan_create")

    def bmu(self, out_bmu: torch.Tensor | None = None, out_dist: torch.Tensor | None = None, stream=None):
        dev = self._som.codebook.device
        if out_bmu is None:
            out_bmu = torch.empty(self.n, dtype=torch.int32, device=dev)
        if out_dist is None:
            out_dist = torch.empty(self.n, dtype=torch.float32, device=dev)
        rc = self._lib.som_bmu_planned(self._som._h, self._p, _dev_ptr(out_bmu, torch.int32, "out_bmu"),
                                       _dev_ptr(out_dist, torch.float32, "out_dist"), _stream_ptr(stream))
        self._som._check(rc, "som_bmu_planned")
        return out_bmu, out_dist

    def destroy(self):
        if self._p:
            self._lib.som_plan_destroy(self._p)
            self._p = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class Som:
    """Handle over a feature-major codebook resident on the GPU (borrowed, not copied): an fp32
    tensor (som_create) or an fp16 tensor (som_create_f16: fp16 storage, fp32 accumulation)."""

    def __init__(self, V: int, M: int, codebook: torch.Tensor):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        if codebook.numel() != V * M:
            raise ValueError("codebook must hold V*M elements")
        if codebook.dtype not in (torch.float32, torch.float16):
            raise TypeError("codebook must be a float32 or float16 CUDA tensor")
        ptr = _dev_ptr(codebook, codebook.dtype, "codebook")
        self.V, self.M = int(V), int(M)
        self.codebook = codebook  # keep the borrowed memory alive
        create = self._lib.som_create if codebook.dtype == torch.float32 else self._lib.som_create_f16
        with torch.cuda.device(codebook.device):
            rc = create(ctypes.byref(self._h), V, M, ptr)
        if rc != SOM_OK:
            self._h = ctypes.c_void_p()
            raise SomError(rc, "som_create")

    def _check(self, rc: int, where: str):
        if rc != SOM_OK:
            raise SomError(rc, where, self._lib.som_last_cuda_error(self._h))

    def norms(self, stream=None):
        """som_norms: recompute ||w_i||^2 (call after every codebook update)."""
        self._check(self._lib.som_norms(self._h, _stream_ptr(stream)), "som_norms")

    def bmu(self, indptr: torch.Tensor, indices: torch.Tensor, out_bmu: torch.Tensor | None = None,
            out_dist: torch.Tensor | None = None, stream=None):
        """som_bmu on device-resident CSR; returns (bmu int32 [n], min squared distance fp32 [n])."""
        n = indptr.numel() - 1
        dev = self.codebook.device
        if out_bmu is None:
            out_bmu = torch.empty(n, dtype=torch.int32, device=dev)
        if out_dist is None:
            out_dist = torch.empty(n, dtype=torch.float32, device=dev)
        rc = self._lib.som_bmu(self._h, _dev_ptr(indptr, torch.int32, "indptr"),
                               _dev_ptr(indices, torch.int32, "indices"), n,
                               _dev_ptr(out_bmu, torch.int32, "out_bmu"),
                               _dev_ptr(out_dist, torch.float32, "out_dist"), _stream_ptr(stream))
        self._check(rc, "som_bmu")
        return out_bmu, out_dist

    def bmu2(self, indptr: torch.Tensor, indices: torch.Tensor, stream=None):
        """som_bmu2: best and second-best unit per sample; returns (bmu, dist, bmu2, dist2)."""
        n = indptr.numel() - 1
        dev = self.codebook.device
        out = [torch.empty(n, dtype=dt, device=dev)
               for dt in (torch.int32, torch.float32, torch.int32, torch.float32)]
        rc = self._lib.som_bmu2(self._h, _dev_ptr(indptr, torch.int32, "indptr"),
                                _dev_ptr(indices, torch.int32, "indices"), n,
                                out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(), out[3].data_ptr(),
                                _stream_ptr(stream))
        self._check(rc, "som_bmu2")
        return tuple(out)

    def bmu_values(self, indptr: torch.Tensor, indices: torch.Tensor, values: torch.Tensor, stream=None):
        """som_bmu_values: sparse real-valued samples; returns (bmu int32 [n], squared distance fp32 [n])."""
        n = indptr.numel() - 1
        dev = self.codebook.device
        out_bmu = torch.empty(n, dtype=torch.int32, device=dev)
        out_dist = torch.empty(n, dtype=torch.float32, device=dev)
        rc = self._lib.som_bmu_values(self._h, _dev_ptr(indptr, torch.int32, "indptr"),
                                      _dev_ptr(indices, torch.int32, "indices"),
                                      _dev_ptr(values, torch.float32, "values"), n,
                                      out_bmu.data_ptr(), out_dist.data_ptr(), _stream_ptr(stream))
        self._check(rc, "som_bmu_values")
        return out_bmu, out_dist

    def update(self, rows: int, cols: int, indptr: torch.Tensor, indices: torch.Tensor, bmu: torch.Tensor,
               radius: int, stream=None):
        """som_update: batch update of the borrowed codebook in place (call norms() afterwards)."""
        n = indptr.numel() - 1
        rc = self._lib.som_update(self._h, rows, cols, _dev_ptr(indptr, torch.int32, "indptr"),
                                  _dev_ptr(indices, torch.int32, "indices"), n,
                                  _dev_ptr(bmu, torch.int32, "bmu"), radius, _stream_ptr(stream))
        self._check(rc, "som_update")

    def bmu_host(self, indptr: torch.Tensor, indices: torch.Tensor, out_bmu: torch.Tensor,
                 out_dist: torch.Tensor, stream=None):
        """som_bmu_host: CPU tensors in and out (pin them for speed); synchronises the stream."""
        n = indptr.numel() - 1
        rc = self._lib.som_bmu_host(self._h, _host_ptr(indptr, torch.int32, "indptr"),
                                    _host_ptr(indices, torch.int32, "indices"), n,
                                    _host_ptr(out_bmu, torch.int32, "out_bmu"),
                                    _host_ptr(out_dist, torch.float32, "out_dist"), _stream_ptr(stream))
        self._check(rc, "som_bmu_host")
        return out_bmu, out_dist

    def bmu_host_async(self, indptr: torch.Tensor, indices: torch.Tensor, out_bmu: torch.Tensor,
                       out_dist: torch.Tensor, stream=None):
        """som_bmu_host_async: pinned CPU tensors in and out; results are valid after host_sync()."""
        n = indptr.numel() - 1
        rc = self._lib.som_bmu_host_async(self._h, _host_ptr(indptr, torch.int32, "indptr"),
                                          _host_ptr(indices, torch.int32, "indices"), n,
                                          _host_ptr(out_bmu, torch.int32, "out_bmu"),
                                          _host_ptr(out_dist, torch.float32, "out_dist"), _stream_ptr(stream))
        self._check(rc, "som_bmu_host_async")

    def host_sync(self):
        self._check(self._lib.som_host_sync(self._h), "som_host_sync")

    def plan(self, indptr: torch.Tensor, indices: torch.Tensor, stream=None) -> "Plan":
        """som_plan_create: a reusable plan of this device-resident batch (keeps the tensors alive)."""
        return Plan(self, indptr, indices, stream)

    def validate_csr(self, indptr: torch.Tensor, indices: torch.Tensor, stream=None) -> bool:
        n = indptr.numel() - 1
        rc = self._lib.som_validate_csr(self._h, _dev_ptr(indptr, torch.int32, "indptr"),
                                        _dev_ptr(indices, torch.int32, "indices"), n,
                                        _stream_ptr(stream))
        if rc == 5:
            return False
        self._check(rc, "som_validate_csr")
        return True

    def device_flags(self, stream=None) -> int:
        """som_device_flags: status of what earlier calls skipped on the device (0 = nothing);
        synchronises the stream and clears the record."""
        return int(self._lib.som_device_flags(self._h, _stream_ptr(stream)))

    def get_norms(self, stream=None) -> torch.Tensor:
        out = torch.empty(self.M, dtype=torch.float32, device=self.codebook.device)
        self._check(self._lib.som_get_norms(self._h, out.data_ptr(), _stream_ptr(stream)), "som_get_norms")
        return out

    def set_timing(self, enable: bool):
        self._check(self._lib.som_set_timing(self._h, int(enable)), "som_set_timing")

    def get_timing(self) -> dict:
        buf = (ctypes.c_float * 5)()
        self._check(self._lib.som_get_timing(self._h, ctypes.cast(buf, ctypes.c_void_p), 5), "som_get_timing")
        return {"norms_ms": buf[0], "bmu_ms": buf[1], "plan_ms": buf[2], "search_ms": buf[3],
                "finalize_ms": buf[4]}

    def launch_count(self) -> int:
        return int(self._lib.som_launch_count(self._h))

    def last_uncertain(self) -> int:
        return int(self._lib.som_last_uncertain(self._h))

    def set_option(self, key: int, value: int):
        self._check(self._lib.som_set_option(self._h, key, value), "som_set_option")

    def destroy(self):
        if self._h:
            self._lib.som_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
