"""Thin ctypes binding of libzc's C ABI.

Argument marshalling only: every step of the codec runs in the library's CUDA kernels (or, for
the codebook and the statistics, in its host code).  The functions have the names of the C entry
points without the ``zc_`` prefix.  PyTorch supplies device memory and streams.

The library must be present (``paper_2508_19263_b200/libzc.so``, built by ``build.build_library``);
importing this module fails loudly when it is not — there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

FMT_BF16, FMT_FP8_E4M3, FMT_FP4_E2M1, FMT_SCALE_U8, FMT_FP8_E5M2 = 1, 2, 3, 4, 5
POLICY_AUTO, POLICY_HUFF_ALL, POLICY_RAW_ALL, POLICY_STATIC = 0, 1, 2, 3
MODE_RAW, MODE_HUFF = 0, 1
(OK, E_INVALID_ARG, E_UNSUPPORTED, E_BUFFER_TOO_SMALL, E_CORRUPT, E_CUDA, E_NOMEM, E_DEVICE_TIMEOUT, E_NO_CODE,
 E_TOO_LARGE) = range(10)
NOALLOC_MAX_CHUNKS = 65536


class ZcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_lib.zc_strerror(status).decode()} (status {status})")


class PlanInfo(C.Structure):
    _fields_ = [("format", C.c_uint32), ("group", C.c_uint32), ("chunk_bytes", C.c_uint32), ("n_chunks", C.c_uint32),
                ("n_elems", C.c_uint64), ("n_syms", C.c_uint64), ("input_bytes", C.c_uint64),
                ("syms_per_chunk", C.c_uint32), ("syms_per_subchunk", C.c_uint32)]


class StreamStats(C.Structure):
    _fields_ = [("n_syms", C.c_uint64), ("raw_bits", C.c_uint64), ("payload_bits", C.c_uint64),
                ("container_bytes", C.c_uint64), ("mode", C.c_uint32), ("n_active_symbols", C.c_uint32),
                ("max_len", C.c_uint32), ("reserved", C.c_uint32), ("avg_len", C.c_double),
                ("entropy_bits", C.c_double)]


class Stats(C.Structure):
    _fields_ = [("stream", StreamStats * 2), ("in_bytes", C.c_uint64), ("out_bytes", C.c_uint64),
                ("ratio_payload", C.c_double), ("ratio_container", C.c_double)]


class DictInfo(C.Structure):
    _fields_ = [("tolerance", C.c_double), ("baseline_ratio", C.c_double), ("last_ratio", C.c_double),
                ("n_observed", C.c_uint64), ("n_rebuilds", C.c_uint64), ("has_baseline", C.c_uint32), ("reserved", C.c_uint32)]


def _load():
    # ZC_LIBRARY: another build of the same library (the development build with in-kernel checks), for tests
    path = os.environ.get("ZC_LIBRARY") or _build.LIB
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run paper_2508_19263_b200.build.build_library() "
                          "(or __graft_entry__.build()) first; there is no fallback implementation")
    L = C.CDLL(path)
    vp, u64p = C.c_void_p, C.POINTER(C.c_uint64)
    L.zc_plan.restype = C.c_int
    L.zc_plan.argtypes = [C.c_int, C.c_uint64, C.c_uint32, C.POINTER(vp)]
    L.zc_plan_destroy.restype = None
    L.zc_plan_destroy.argtypes = [vp]
    L.zc_plan_get_info.restype = C.c_int
    L.zc_plan_get_info.argtypes = [vp, C.POINTER(PlanInfo)]
    L.zc_max_compressed_bytes.restype = C.c_size_t
    L.zc_max_compressed_bytes.argtypes = [vp]
    L.zc_workspace_bytes.restype = C.c_size_t
    L.zc_workspace_bytes.argtypes = [vp]
    L.zc_histogram.restype = C.c_int
    L.zc_histogram.argtypes = [vp, vp, vp, vp]
    L.zc_histogram_batch.restype = C.c_int
    L.zc_histogram_batch.argtypes = [C.c_uint32, C.POINTER(vp), C.POINTER(vp), vp, vp]
    L.zc_build_codebook.restype = C.c_int
    L.zc_build_codebook.argtypes = [vp, u64p, C.c_int, C.POINTER(vp)]
    L.zc_build_codebooks.restype = C.c_int
    L.zc_build_codebooks.argtypes = [C.c_uint32, C.POINTER(vp), u64p, C.c_int, C.c_uint32, C.POINTER(vp)]
    L.zc_codebook_destroy.restype = None
    L.zc_codebook_destroy.argtypes = [vp]
    L.zc_codebook_get.restype = C.c_int
    L.zc_codebook_get.argtypes = [vp, C.c_uint32, C.POINTER(C.c_uint32), C.POINTER(C.c_uint8), C.POINTER(C.c_uint32)]
    L.zc_compress.restype = C.c_int
    L.zc_compress.argtypes = [vp, vp, vp, vp, C.c_size_t, vp, u64p, vp]
    L.zc_compress_noalloc.restype = C.c_int
    L.zc_compress_noalloc.argtypes = [vp, vp, vp, vp, C.c_size_t, u64p, vp]
    L.zc_decompress.restype = C.c_int
    L.zc_decompress.argtypes = [vp, vp, C.c_size_t, vp, vp, vp]
    L.zc_compress_batch_workspace_bytes.restype = C.c_size_t
    L.zc_compress_batch_workspace_bytes.argtypes = [C.c_uint32, C.POINTER(vp)]
    L.zc_compress_batch.restype = C.c_int
    L.zc_compress_batch.argtypes = [C.c_uint32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(C.c_size_t),
                                    vp, C.c_size_t, u64p, vp]
    L.zc_decompress_batch.restype = C.c_int
    L.zc_decompress_batch.argtypes = [C.c_uint32, C.POINTER(vp), C.POINTER(vp), C.POINTER(C.c_size_t), C.POINTER(vp), vp, vp]
    L.zc_batch_status.restype = C.c_int
    L.zc_batch_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
    L.zc_histogram_xor.restype = C.c_int
    L.zc_histogram_xor.argtypes = [vp, vp, vp, vp, vp]
    L.zc_histogram_batch_xor.restype = C.c_int
    L.zc_histogram_batch_xor.argtypes = [C.c_uint32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp, vp]
    L.zc_compress_xor.restype = C.c_int
    L.zc_compress_xor.argtypes = [vp, vp, vp, vp, vp, C.c_size_t, vp, u64p, vp]
    L.zc_compress_batch_xor.restype = C.c_int
    L.zc_compress_batch_xor.argtypes = [C.c_uint32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                        C.POINTER(C.c_size_t), vp, C.c_size_t, u64p, vp]
    L.zc_decompress_xor.restype = C.c_int
    L.zc_decompress_xor.argtypes = [vp, vp, C.c_size_t, vp, vp, vp, vp]
    L.zc_decompress_batch_xor.restype = C.c_int
    L.zc_decompress_batch_xor.argtypes = [C.c_uint32, C.POINTER(vp), C.POINTER(vp), C.POINTER(C.c_size_t), C.POINTER(vp), C.POINTER(vp),
                                          vp, vp]
    L.zc_decompress_chunks.restype = C.c_int
    L.zc_decompress_chunks.argtypes = [vp, vp, C.c_size_t, C.c_uint32, C.c_uint32, vp, vp, vp]
    L.zc_device_status.restype = C.c_int
    L.zc_device_status.argtypes = [vp, vp, vp]
    L.zc_validate_container.restype = C.c_int
    L.zc_validate_container.argtypes = [vp, vp, C.c_size_t]
    L.zc_stats.restype = C.c_int
    L.zc_stats.argtypes = [vp, vp, u64p, vp, C.POINTER(Stats)]
    L.zc_dict_create.restype = C.c_int
    L.zc_dict_create.argtypes = [vp, u64p, C.c_double, C.POINTER(vp)]
    L.zc_dict_destroy.restype = None
    L.zc_dict_destroy.argtypes = [vp]
    L.zc_dict_codebook.restype = vp
    L.zc_dict_codebook.argtypes = [vp]
    L.zc_dict_observe.restype = C.c_int
    L.zc_dict_observe.argtypes = [vp, C.c_uint64, C.c_uint64, C.POINTER(C.c_int)]
    L.zc_dict_rebuild.restype = C.c_int
    L.zc_dict_rebuild.argtypes = [vp, vp, u64p]
    L.zc_dict_get_info.restype = C.c_int
    L.zc_dict_get_info.argtypes = [vp, C.POINTER(DictInfo)]
    L.zc_strerror.restype = C.c_char_p
    L.zc_strerror.argtypes = [C.c_int]
    L.zc_test_split16.restype = C.c_int
    L.zc_test_split16.argtypes = [C.c_int, vp, vp, vp]
    L.zc_test_merge16.restype = C.c_int
    L.zc_test_merge16.argtypes = [C.c_int, vp, vp, vp]
    L.zc_noalloc_status.restype = C.c_int
    L.zc_noalloc_status.argtypes = [vp]
    L.zc_test_encoder_workers.restype = C.c_uint32
    L.zc_test_encoder_workers.argtypes = [vp, C.c_uint32, C.c_uint32]
    L.zc_test_decoder_warps.restype = C.c_uint32
    L.zc_test_decoder_warps.argtypes = [vp, C.c_uint32]
    L.zc_test_debug_counts.restype = C.c_int
    L.zc_test_debug_counts.argtypes = [C.POINTER(C.c_uint32)]
    for name in ("zc_test_set_wait_limit", "zc_test_stall_encoder", "zc_test_stall_decoder"):
        getattr(L, name).restype = None
        getattr(L, name).argtypes = [C.c_uint32]
    return L


_lib = _load()


def _check(status: int, where: str):
    if status != OK:
        raise ZcError(status, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def strerror(status: int) -> str:
    return _lib.zc_strerror(status).decode()


class Plan:
    """zc_plan: the problem statement of one tensor (format, element count, chunk size)."""

    def __init__(self, fmt: int, n_elems: int, chunk_bytes: int):
        h = C.c_void_p()
        _check(_lib.zc_plan(fmt, n_elems, chunk_bytes, C.byref(h)), "zc_plan")
        self._h = h
        info = PlanInfo()
        _check(_lib.zc_plan_get_info(h, C.byref(info)), "zc_plan_get_info")
        self.info = info
        self.format, self.n_elems, self.chunk_bytes = fmt, n_elems, chunk_bytes
        self.n_syms, self.n_chunks, self.input_bytes = info.n_syms, info.n_chunks, info.input_bytes
        self.max_compressed_bytes = _lib.zc_max_compressed_bytes(h)
        self.workspace_bytes = _lib.zc_workspace_bytes(h)

    def __del__(self):
        h = getattr(self, "_h", None)
        if h and _lib is not None:
            _lib.zc_plan_destroy(h)
            self._h = None


def plan(fmt: int, n_elems: int, chunk_bytes: int) -> Plan:
    return Plan(fmt, n_elems, chunk_bytes)


class Codebook:
    """zc_build_codebook result: per stream a mode, 256 code lengths and 256 canonical code values."""

    def __init__(self, handle, owned: bool = True):
        self._h = handle
        self._owned = owned                      # a dictionary's codebook belongs to the dictionary

    def get(self, stream_idx: int):
        mode = C.c_uint32()
        lens = np.zeros(256, np.uint8)
        codes = np.zeros(256, np.uint32)
        _check(_lib.zc_codebook_get(self._h, stream_idx, C.byref(mode), lens.ctypes.data_as(C.POINTER(C.c_uint8)),
                                    codes.ctypes.data_as(C.POINTER(C.c_uint32))), "zc_codebook_get")
        return mode.value, lens, codes

    @property
    def modes(self):
        return [self.get(0)[0], self.get(1)[0]]

    def __del__(self):
        h = getattr(self, "_h", None)
        if h and _lib is not None and getattr(self, "_owned", True):
            _lib.zc_codebook_destroy(h)
            self._h = None


def histogram(p: Plan, d_in: torch.Tensor, d_hist: Optional[torch.Tensor] = None, stream=None,
              d_base: Optional[torch.Tensor] = None) -> torch.Tensor:
    """zc_histogram (zc_histogram_xor when d_base is given): returns a device tensor uint64-as-int64 [2, 256]."""
    assert d_in.is_cuda and d_in.is_contiguous()
    if d_hist is None:
        d_hist = torch.empty((2, 256), dtype=torch.int64, device=d_in.device)
    if d_base is None:
        _check(_lib.zc_histogram(p._h, d_in.data_ptr(), d_hist.data_ptr(), _stream_ptr(stream)), "zc_histogram")
    else:
        _check(_lib.zc_histogram_xor(p._h, d_in.data_ptr(), d_base.data_ptr(), d_hist.data_ptr(), _stream_ptr(stream)),
               "zc_histogram_xor")
    return d_hist


def _base_array(d_bases, n):
    """Host array of base-tensor pointers for the XOR-delta forms (None: no base at all, a None entry: none for that tensor)."""
    if d_bases is None:
        return None
    return (C.c_void_p * max(n, 1))(*[(t.data_ptr() if t is not None else None) for t in d_bases])


class HistogramBatch:
    """Argument arrays of zc_histogram_batch, marshalled once."""

    def __init__(self, plans, d_ins, d_bases=None):
        n = len(plans)
        assert len(d_ins) == n and (d_bases is None or len(d_bases) == n)
        self.n = n
        self._keep = (list(plans), list(d_ins), list(d_bases) if d_bases is not None else None)
        self.plans = (C.c_void_p * max(n, 1))(*[p._h.value for p in plans])
        self.ins = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in d_ins])
        self.bases = _base_array(d_bases, n)     # XOR-delta form when given


def histogram_batch(batch: HistogramBatch, d_hists: torch.Tensor, stream=None) -> torch.Tensor:
    """zc_histogram_batch: d_hists is a device tensor int64 [n, 2, 256] (uint64 counts)."""
    assert d_hists.is_cuda and d_hists.is_contiguous() and d_hists.numel() == 512 * batch.n and d_hists.element_size() == 8
    _check(_lib.zc_histogram_batch_xor(batch.n, batch.plans, batch.ins, batch.bases, d_hists.data_ptr(), _stream_ptr(stream)),
           "zc_histogram_batch")
    return d_hists


def build_codebook(p: Plan, h_hist, policy: int = POLICY_AUTO) -> Codebook:
    """zc_build_codebook: host only.  h_hist: array-like [2, 256] of counts."""
    h = np.asarray(h_hist)
    if h.dtype == np.int64 and h.flags.c_contiguous:
        h = h.view(np.uint64)                    # counts as produced by histogram(): no copy
    elif h.dtype != np.uint64 or not h.flags.c_contiguous:
        h = np.ascontiguousarray(h.astype(np.uint64))
    assert h.size == 512
    out = C.c_void_p()
    _check(_lib.zc_build_codebook(p._h, C.cast(h.ctypes.data, C.POINTER(C.c_uint64)), policy, C.byref(out)),
           "zc_build_codebook")
    return Codebook(out)


def _hist_ptr(h_hist):
    h = np.asarray(h_hist)
    if h.dtype == np.int64 and h.flags.c_contiguous:
        h = h.view(np.uint64)
    elif h.dtype != np.uint64 or not h.flags.c_contiguous:
        h = np.ascontiguousarray(h.astype(np.uint64))
    assert h.size == 512
    return h, C.cast(h.ctypes.data, C.POINTER(C.c_uint64))


class Dictionary:
    """zc_dict_*: a static codebook for K/V cache tensors plus the rule that says when to replace it."""

    def __init__(self, p: Plan, h_hist, tolerance: float):
        _keep, ptr = _hist_ptr(h_hist)
        self._h = C.c_void_p()
        _check(_lib.zc_dict_create(p._h, ptr, tolerance, C.byref(self._h)), "zc_dict_create")

    @property
    def codebook(self) -> Codebook:
        """The current codebook (not owned: valid until rebuild())."""
        return Codebook(C.c_void_p(_lib.zc_dict_codebook(self._h)), owned=False)

    def observe(self, input_bytes: int, container_bytes: int) -> bool:
        flag = C.c_int(0)
        _check(_lib.zc_dict_observe(self._h, input_bytes, container_bytes, C.byref(flag)), "zc_dict_observe")
        return bool(flag.value)

    def rebuild(self, p: Plan, h_hist) -> None:
        _keep, ptr = _hist_ptr(h_hist)
        _check(_lib.zc_dict_rebuild(self._h, p._h, ptr), "zc_dict_rebuild")

    @property
    def info(self) -> DictInfo:
        out = DictInfo()
        _check(_lib.zc_dict_get_info(self._h, C.byref(out)), "zc_dict_get_info")
        return out

    def __del__(self):
        h = getattr(self, "_h", None)
        if h and _lib is not None:
            _lib.zc_dict_destroy(h)
            self._h = None


def build_codebooks(plans, h_hists, policy: int = POLICY_AUTO, n_threads: int = 0):
    """zc_build_codebooks: the codebooks of many tensors, built on several host threads.
    h_hists: array-like [n, 2, 256] of counts."""
    n = len(plans)
    h = np.asarray(h_hists)
    if h.dtype == np.int64 and h.flags.c_contiguous:
        h = h.view(np.uint64)
    elif h.dtype != np.uint64 or not h.flags.c_contiguous:
        h = np.ascontiguousarray(h.astype(np.uint64))
    assert h.size == 512 * n
    handles = (C.c_void_p * max(n, 1))()
    plan_arr = (C.c_void_p * max(n, 1))(*[p._h.value for p in plans])
    _check(_lib.zc_build_codebooks(n, plan_arr, C.cast(h.ctypes.data, C.POINTER(C.c_uint64)), policy, n_threads, handles),
           "zc_build_codebooks")
    return [Codebook(C.c_void_p(handles[i])) for i in range(n)]


def compress(p: Plan, cb: Codebook, d_in: torch.Tensor, d_out: torch.Tensor, d_workspace: torch.Tensor,
             sync: bool = True, stream=None, d_base: Optional[torch.Tensor] = None) -> Optional[int]:
    """zc_compress (zc_compress_xor when d_base is given).  With sync=True returns the container size in bytes
    (and raises on a device-side error); with sync=False the call is asynchronous and returns None."""
    assert d_in.is_cuda and d_out.is_cuda and d_workspace.is_cuda
    assert d_workspace.numel() * d_workspace.element_size() >= p.workspace_bytes
    n = C.c_uint64(0)
    if d_base is None:
        st = _lib.zc_compress(p._h, cb._h, d_in.data_ptr(), d_out.data_ptr(), d_out.numel() * d_out.element_size(),
                              d_workspace.data_ptr(), C.byref(n) if sync else None, _stream_ptr(stream))
    else:
        st = _lib.zc_compress_xor(p._h, cb._h, d_in.data_ptr(), d_base.data_ptr(), d_out.data_ptr(),
                                  d_out.numel() * d_out.element_size(), d_workspace.data_ptr(), C.byref(n) if sync else None,
                                  _stream_ptr(stream))
    _check(st, "zc_compress")
    return n.value if sync else None


def compress_noalloc(p: Plan, cb: Codebook, d_in: torch.Tensor, d_out: torch.Tensor, sync: bool = True,
                     stream=None) -> Optional[int]:
    """zc_compress_noalloc: like compress() but without a workspace argument.  The scratch is a fixed array
    inside the library (at most NOALLOC_MAX_CHUNKS chunks; larger plans raise E_TOO_LARGE).  For callers that
    may not allocate device memory.  Calls that overlap on the GPU must not be issued: they share the scratch."""
    assert d_in.is_cuda and d_out.is_cuda
    n = C.c_uint64(0)
    st = _lib.zc_compress_noalloc(p._h, cb._h, d_in.data_ptr(), d_out.data_ptr(), d_out.numel() * d_out.element_size(),
                                  C.byref(n) if sync else None, _stream_ptr(stream))
    _check(st, "zc_compress_noalloc")
    return n.value if sync else None


def noalloc_status(stream=None) -> int:
    """zc_noalloc_status: device status of the last compress_noalloc call on the current device."""
    return int(_lib.zc_noalloc_status(_stream_ptr(stream)))


def decompress(p: Plan, d_comp: torch.Tensor, comp_bytes: int, d_out: torch.Tensor, d_workspace: torch.Tensor,
               stream=None, d_base: Optional[torch.Tensor] = None) -> None:
    """zc_decompress, or zc_decompress_xor when d_base is given (asynchronous; call device_status() to learn the
    outcome)."""
    assert d_comp.is_cuda and d_out.is_cuda and d_workspace.is_cuda
    assert d_out.numel() * d_out.element_size() >= p.input_bytes
    if d_base is None:
        _check(_lib.zc_decompress(p._h, d_comp.data_ptr(), comp_bytes, d_out.data_ptr(), d_workspace.data_ptr(),
                                  _stream_ptr(stream)), "zc_decompress")
    else:
        _check(_lib.zc_decompress_xor(p._h, d_comp.data_ptr(), comp_bytes, d_base.data_ptr(), d_out.data_ptr(),
                                      d_workspace.data_ptr(), _stream_ptr(stream)), "zc_decompress_xor")


def decompress_chunks(p: Plan, d_comp: torch.Tensor, comp_bytes: int, first_chunk: int, n_chunks: int, d_out: torch.Tensor,
                      d_workspace: torch.Tensor, stream=None) -> None:
    """zc_decompress_chunks: d_out receives the element bytes of chunks first_chunk .. first_chunk + n_chunks - 1."""
    assert d_comp.is_cuda and d_out.is_cuda and d_workspace.is_cuda
    _check(_lib.zc_decompress_chunks(p._h, d_comp.data_ptr(), comp_bytes, first_chunk, n_chunks, d_out.data_ptr(),
                                     d_workspace.data_ptr(), _stream_ptr(stream)), "zc_decompress_chunks")


def device_status(p: Plan, d_workspace: torch.Tensor, stream=None) -> int:
    return _lib.zc_device_status(p._h, d_workspace.data_ptr(), _stream_ptr(stream))


class CompressBatch:
    """Argument arrays of zc_compress_batch, marshalled once; set_codebooks() swaps in new codebooks."""

    def __init__(self, plans, d_ins, d_outs, d_bases=None):
        n = len(plans)
        assert len(d_ins) == n and len(d_outs) == n and (d_bases is None or len(d_bases) == n)
        self.n = n
        self._keep = (list(plans), list(d_ins), list(d_outs), list(d_bases) if d_bases is not None else None)
        self.bases = _base_array(d_bases, n)     # XOR-delta form when given
        self.plans = (C.c_void_p * n)(*[p._h.value for p in plans])
        self.ins = (C.c_void_p * n)(*[t.data_ptr() for t in d_ins])
        self.outs = (C.c_void_p * n)(*[t.data_ptr() for t in d_outs])
        self.caps = (C.c_size_t * n)(*[t.numel() for t in d_outs])
        self.cbs = (C.c_void_p * n)()
        self._cbs = None
        self.workspace_bytes = _lib.zc_compress_batch_workspace_bytes(n, self.plans)

    def set_codebooks(self, codebooks):
        assert len(codebooks) == self.n
        self._cbs = list(codebooks)
        for i, cb in enumerate(codebooks):
            self.cbs[i] = cb._h.value


def compress_batch(batch: CompressBatch, d_workspace: torch.Tensor, sync: bool = True, stream=None):
    """zc_compress_batch.  Returns the list of container sizes (sync=True) or None (asynchronous)."""
    sizes = (C.c_uint64 * max(batch.n, 1))()
    _check(_lib.zc_compress_batch_xor(batch.n, batch.plans, batch.cbs, batch.ins, batch.bases, batch.outs, batch.caps,
                                      d_workspace.data_ptr(), d_workspace.numel(), sizes if sync else None, _stream_ptr(stream)),
           "zc_compress_batch")
    return [int(v) for v in sizes[: batch.n]] if sync else None


class DecompressBatch:
    """Argument arrays of zc_decompress_batch, marshalled once and reusable for repeated calls."""

    def __init__(self, plans, d_comps, comp_bytes, d_outs, d_bases=None):
        n = len(plans)
        assert len(d_comps) == n and len(comp_bytes) == n and len(d_outs) == n and (d_bases is None or len(d_bases) == n)
        self.n = n
        self._keep = (list(plans), list(d_comps), list(d_outs), list(d_bases) if d_bases is not None else None)
        self.bases = _base_array(d_bases, n)     # XOR-delta form when given
        self.plans = (C.c_void_p * n)(*[p._h.value for p in plans])
        self.comps = (C.c_void_p * n)(*[t.data_ptr() for t in d_comps])
        self.sizes = (C.c_size_t * n)(*[int(b) for b in comp_bytes])
        self.outs = (C.c_void_p * n)(*[t.data_ptr() for t in d_outs])


def decompress_batch(batch: DecompressBatch, d_workspace: torch.Tensor, stream=None) -> None:
    """zc_decompress_batch (asynchronous; read the outcome with batch_status)."""
    _check(_lib.zc_decompress_batch_xor(batch.n, batch.plans, batch.comps, batch.sizes, batch.bases, batch.outs,
                                        d_workspace.data_ptr(), _stream_ptr(stream)), "zc_decompress_batch")


def batch_status(d_workspace: torch.Tensor, stream=None):
    """zc_batch_status: (status, index of the failing tensor or None)."""
    failed = C.c_uint32(0xFFFFFFFF)
    st = _lib.zc_batch_status(d_workspace.data_ptr(), C.byref(failed), _stream_ptr(stream))
    return st, (None if failed.value == 0xFFFFFFFF else failed.value)


def validate_container(p: Plan, h_container) -> int:
    c = np.ascontiguousarray(h_container, np.uint8)
    return _lib.zc_validate_container(p._h, c.ctypes.data, c.size)


def stats(p: Plan, cb: Codebook, h_hist, h_header=None) -> Stats:
    h = np.ascontiguousarray(np.asarray(h_hist).astype(np.uint64)).reshape(512)
    hd = None
    if h_header is not None:
        hd = np.ascontiguousarray(h_header, np.uint8)
        assert hd.size >= 128
    out = Stats()
    _check(_lib.zc_stats(p._h, cb._h, h.ctypes.data_as(C.POINTER(C.c_uint64)), hd.ctypes.data if hd is not None else None,
                         C.byref(out)), "zc_stats")
    return out


def test_split16(fmt: int, in16: np.ndarray):
    a = np.ascontiguousarray(in16, np.uint8)
    e, sm = np.zeros(8, np.uint8), np.zeros(8, np.uint8)
    _check(_lib.zc_test_split16(fmt, a.ctypes.data, e.ctypes.data, sm.ctypes.data), "zc_test_split16")
    return e, sm


def test_merge16(fmt: int, e8: np.ndarray, sm8: np.ndarray):
    e, sm = np.ascontiguousarray(e8, np.uint8), np.ascontiguousarray(sm8, np.uint8)
    out = np.zeros(16, np.uint8)
    _check(_lib.zc_test_merge16(fmt, e.ctypes.data, sm.ctypes.data, out.ctypes.data), "zc_test_merge16")
    return out


test_split16.__test__ = False
test_merge16.__test__ = False


def test_set_wait_limit(polls: int) -> None:
    """zc_test_set_wait_limit (0 restores the default)."""
    _lib.zc_test_set_wait_limit(polls)


def test_stall_encoder(first_ticket: int) -> None:
    """zc_test_stall_encoder (0 turns the stall off)."""
    _lib.zc_test_stall_encoder(first_ticket)


def test_stall_decoder(on: bool) -> None:
    """zc_test_stall_decoder."""
    _lib.zc_test_stall_decoder(1 if on else 0)


def test_debug_counts():
    """zc_test_debug_counts: (refused shared accesses, refused global accesses) of a development build, else None."""
    out = (C.c_uint32 * 2)()
    return (int(out[0]), int(out[1])) if _lib.zc_test_debug_counts(out) else None


def test_encoder_workers(p: Plan, n_coded: int, wide_slots: int) -> int:
    """zc_test_encoder_workers; wide_slots is the slot class 0, 1 or 2."""
    return int(_lib.zc_test_encoder_workers(p._h, n_coded, int(wide_slots)))


def test_decoder_warps(p: Plan, both_coded: bool) -> int:
    return int(_lib.zc_test_decoder_warps(p._h, 1 if both_coded else 0))
