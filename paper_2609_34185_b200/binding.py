"""ctypes binding of ``include/entropack.h`` (argument marshalling only).

Functions with the C names minus the ``ep_`` prefix call straight into the shared library.  The
``DeviceBlob`` / ``upload`` / ``decode`` helpers at the end move bytes with torch tensors and pass
their raw pointers; every step of the decode runs in the library's CUDA kernels.
"""
from __future__ import annotations

import ctypes as C
import os
import weakref

import numpy as np

BF16, FP16, FP8_E4M3, INT8, FP32, FP8_E5M2, UINT8, FIELDS_I32 = 0, 1, 2, 3, 4, 5, 6, 16
DTYPE_BYTES = {BF16: 2, FP16: 2, FP8_E4M3: 1, INT8: 1, FP32: 4, FP8_E5M2: 1, UINT8: 1}
NUM_TABLES = 17
MAX_BATCH = 16

_HERE = os.path.dirname(os.path.abspath(__file__))
# ENTROPACK_LIB selects another build of the same library (e.g. one compiled with different flags)
_LIB_PATH = os.environ.get("ENTROPACK_LIB") or os.path.join(_HERE, "libentropack_b200.so")


class EntroPackError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {strerror(status)} ({status})")
        self.status = status


class EncodeOpts(C.Structure):
    _fields_ = [("bracket_lo", C.c_double), ("bracket_hi", C.c_double), ("search_steps", C.c_int32),
                ("sample_vectors", C.c_uint32), ("tile_vectors", C.c_uint32), ("b_start", C.c_int32),
                ("b_max", C.c_int32), ("retained_bits", C.c_double), ("polish_steps", C.c_int32), ("polish_retained_bits", C.c_double),
                ("threads", C.c_int32), ("rdo_candidates", C.c_int32), ("rdo_sweeps", C.c_int32)]


class EncodeReport(C.Structure):
    _fields_ = [("s", C.c_double), ("stored_bpp", C.c_double), ("est_bpp_sample", C.c_double),
                ("cce_bits", C.c_double), ("bytes", C.c_uint64), ("sample_rows", C.c_uint32), ("b", C.c_int32)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class Info(C.Structure):
    _fields_ = [("R", C.c_uint32), ("C", C.c_uint32), ("V", C.c_uint32), ("n_tiles", C.c_uint32),
                ("b", C.c_uint32), ("J", C.c_uint32), ("coord_min", C.c_int32), ("coord_max", C.c_int32),
                ("s", C.c_float), ("off_tables", C.c_uint32), ("off_scales", C.c_uint32),
                ("off_tiles", C.c_uint32), ("off_payload", C.c_uint32), ("total_bytes", C.c_uint64),
                ("total_words", C.c_uint64), ("table_min", C.c_int32 * NUM_TABLES),
                ("table_K", C.c_uint32 * NUM_TABLES)]

    def as_dict(self):
        d = {k: getattr(self, k) for k, _ in self._fields_ if not k.startswith("table_")}
        d["table_min"] = list(self.table_min)
        d["table_K"] = list(self.table_K)
        return d


class DecodeJob(C.Structure):
    _fields_ = [("info", C.POINTER(Info)), ("d_stream", C.c_void_p), ("d_tile_index", C.c_void_p),
                ("d_row_scales", C.c_void_p), ("out_dtype", C.c_int32), ("d_out", C.c_void_p),
                ("d_scratch", C.c_void_p), ("scratch_bytes", C.c_size_t),
                ("tile_begin", C.c_uint32), ("tile_count", C.c_uint32), ("d_tables", C.c_void_p)]


_lib = None


def load():
    """Load the C-ABI library; there is no fallback when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with "
                          "`python -m paper_2609_34185_b200.build` (needs nvcc); there is no CPU fallback")
    L = C.CDLL(_LIB_PATH)
    L.ep_encode.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_double, C.POINTER(EncodeOpts), C.POINTER(C.c_void_p)]
    L.ep_pack_fields.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_int32, C.c_uint32, C.c_void_p, C.c_float,
                                 C.c_int32, C.POINTER(C.c_void_p)]
    L.ep_encode_device_workspace_bytes.restype = C.c_size_t
    L.ep_encode_device_workspace_bytes.argtypes = [C.c_uint32, C.c_uint32, C.c_double, C.POINTER(EncodeOpts)]
    L.ep_encode_device.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_double, C.POINTER(EncodeOpts), C.c_void_p,
                                   C.c_size_t, C.c_void_p, C.POINTER(C.c_void_p)]
    L.ep_blob_data.restype = C.c_void_p
    L.ep_blob_data.argtypes = [C.c_void_p]
    L.ep_blob_bytes.restype = C.c_size_t
    L.ep_blob_bytes.argtypes = [C.c_void_p]
    L.ep_blob_report.argtypes = [C.c_void_p, C.POINTER(EncodeReport)]
    L.ep_blob_free.argtypes = [C.c_void_p]
    L.ep_blob_free.restype = None
    L.ep_blob_info.argtypes = [C.c_void_p, C.c_size_t, C.POINTER(Info)]
    L.ep_validate.argtypes = [C.c_void_p, C.c_size_t]
    L.ep_decode_scratch_bytes.restype = C.c_size_t
    L.ep_decode_scratch_bytes.argtypes = [C.POINTER(Info)]
    L.ep_decode_tables_bytes.restype = C.c_size_t
    L.ep_decode_tables_bytes.argtypes = [C.POINTER(Info)]
    L.ep_prepare_tables.argtypes = [C.POINTER(Info), C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    L.ep_decode_tiles_per_sm.restype = C.c_uint32
    L.ep_decode_tiles_per_sm.argtypes = []
    L.ep_decode_tensor.argtypes = [C.POINTER(Info), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                   C.c_void_p, C.c_size_t, C.c_void_p]
    L.ep_decode_tiles.argtypes = [C.POINTER(Info), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                  C.c_void_p, C.c_size_t, C.c_uint32, C.c_uint32, C.c_void_p]
    L.ep_decode_tensor_static.argtypes = [C.POINTER(Info), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                          C.c_void_p]
    L.ep_decode_gemm.argtypes = [C.POINTER(Info), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32,
                                 C.c_void_p, C.c_void_p]
    L.ep_decode_batch.argtypes = [C.POINTER(DecodeJob), C.c_int32, C.c_void_p]
    L.ep_last_device_status.argtypes = [C.c_void_p]
    L.ep_strerror.restype = C.c_char_p
    L.ep_strerror.argtypes = [C.c_int]
    L.ep_default_tile_vectors.restype = C.c_uint32
    L.ep_default_tile_vectors.argtypes = [C.c_double]
    L.ep_suggest_tile_vectors_batch.restype = C.c_uint32
    L.ep_suggest_tile_vectors_batch.argtypes = [C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.c_uint32, C.c_double, C.c_uint32]
    L.ep_suggest_tile_vectors.restype = C.c_uint32
    L.ep_suggest_tile_vectors.argtypes = [C.c_uint32, C.c_uint32, C.c_double, C.c_uint32]
    L.ep_encode_opts_default.argtypes = [C.POINTER(EncodeOpts)]
    L.ep_encode_opts_default.restype = None
    _lib = L
    return L


def strerror(status: int) -> str:
    try:
        return load().ep_strerror(int(status)).decode()
    except ImportError:
        return "library not built"


def _check(rc: int, what: str):
    if rc != 0:
        raise EntroPackError(rc, what)


def default_tile_vectors(target_bpp: float) -> int:
    return load().ep_default_tile_vectors(float(target_bpp))


def decode_tiles_per_sm() -> int:
    """ep_decode_tiles_per_sm: tiles the decode kernel works on at a time per SM."""
    return int(load().ep_decode_tiles_per_sm())


def suggest_tile_vectors(R: int, Cc: int, target_bpp: float, decode_slots: int = 148 * 48) -> int:
    """ep_suggest_tile_vectors: tile size that fills whole rounds of `decode_slots` concurrent tiles."""
    return load().ep_suggest_tile_vectors(R, Cc, float(target_bpp), decode_slots)


def suggest_tile_vectors_batch(shapes, target_bpp: float, decode_ctas: int) -> int:
    """ep_suggest_tile_vectors_batch: one tile size for tensors decoded together by one batched launch."""
    n = len(shapes)
    Rs = (C.c_uint32 * n)(*[int(s[0]) for s in shapes])
    Cs = (C.c_uint32 * n)(*[int(s[1]) for s in shapes])
    return int(load().ep_suggest_tile_vectors_batch(Rs, Cs, n, float(target_bpp), int(decode_ctas)))


class Blob:
    """Host copy of a stored representation plus what the encoder reported."""

    def __init__(self, data: np.ndarray, report: dict | None = None):
        self.data = np.ascontiguousarray(data, np.uint8)
        self.report = report or {}
        self.info = blob_info(self.data)

    def __len__(self):
        return self.data.size

    @property
    def stored_bpp(self) -> float:
        return 8.0 * self.data.size / (self.info.R * self.info.C)


def _take(handle: C.c_void_p) -> Blob:
    L = load()
    n = L.ep_blob_bytes(handle)
    rep = EncodeReport()
    L.ep_blob_report(handle, C.byref(rep))
    # no copy: the array views the library's buffer, which is freed when the array (and every view of it) is gone
    data = np.ctypeslib.as_array(C.cast(L.ep_blob_data(handle), C.POINTER(C.c_uint8)), shape=(n,))
    weakref.finalize(data, L.ep_blob_free, handle)
    return Blob(data, rep.as_dict())


def encode_opts(**kw) -> EncodeOpts:
    o = EncodeOpts()
    load().ep_encode_opts_default(C.byref(o))
    for k, v in kw.items():
        setattr(o, k, v)
    return o


def encode(W: np.ndarray, target_bpp: float, **opts) -> Blob:
    """ep_encode: compress a host fp32 matrix to about target_bpp stored bits per weight."""
    W = np.ascontiguousarray(W, np.float32)
    if W.ndim != 2:
        raise ValueError("W must be a 2-D matrix")
    o = encode_opts(**opts)
    h = C.c_void_p()
    _check(load().ep_encode(W.ctypes.data, W.shape[0], W.shape[1], float(target_bpp), C.byref(o), C.byref(h)), "ep_encode")
    return _take(h)


def encode_device(W_dev, target_bpp: float, workspace=None, stream=None, **opts) -> Blob:
    """ep_encode_device: the encoder with its heavy steps on the GPU.  W_dev is a CUDA float32 tensor [R, C];
    the result is the same host blob ep_encode gives for the same matrix and options."""
    torch = _torch()
    assert W_dev.is_cuda and W_dev.dtype == torch.float32 and W_dev.dim() == 2 and W_dev.is_contiguous()
    R, Cc = W_dev.shape
    o = encode_opts(**opts)
    need = load().ep_encode_device_workspace_bytes(R, Cc, float(target_bpp), C.byref(o))
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(need, dtype=torch.uint8, device=W_dev.device)
    h = C.c_void_p()
    _check(load().ep_encode_device(W_dev.data_ptr(), R, Cc, float(target_bpp), C.byref(o), workspace.data_ptr(),
                                   workspace.numel(), _stream_handle(stream), C.byref(h)), "ep_encode_device")
    return _take(h)


def pack_fields(fields: np.ndarray, R: int, Cc: int, b: int, V: int, row_scales: np.ndarray, s_info: float = 0.0,
                threads: int = 0) -> Blob:
    """ep_pack_fields: final tables + tile coding of given (c, z1..z7, m) tuples."""
    fields = np.ascontiguousarray(fields, np.int32)
    row_scales = np.ascontiguousarray(row_scales, np.float32)
    assert fields.shape == (R * Cc // 8, 9) and row_scales.shape == (R,)
    h = C.c_void_p()
    _check(load().ep_pack_fields(fields.ctypes.data, R, Cc, b, V, row_scales.ctypes.data, float(s_info), threads,
                                 C.byref(h)), "ep_pack_fields")
    return _take(h)


def blob_info(data: np.ndarray) -> Info:
    data = np.ascontiguousarray(data, np.uint8)
    inf = Info()
    _check(load().ep_blob_info(data.ctypes.data, data.size, C.byref(inf)), "ep_blob_info")
    return inf


def validate(data: np.ndarray) -> int:
    """ep_validate: returns the status instead of raising, so that tests can inspect it."""
    data = np.ascontiguousarray(data, np.uint8)
    return load().ep_validate(data.ctypes.data, data.size)


def decode_scratch_bytes(info: Info) -> int:
    return load().ep_decode_scratch_bytes(C.byref(info))


def decode_tables_bytes(info: Info) -> int:
    return load().ep_decode_tables_bytes(C.byref(info))


def prepare_tables(info: Info, d_stream: int, d_tables: int, tables_bytes: int, stream: int = 0) -> None:
    """ep_prepare_tables with raw device addresses (ints)."""
    _check(load().ep_prepare_tables(C.byref(info), d_stream, d_tables, tables_bytes, stream or None), "ep_prepare_tables")


def decode_tensor(info: Info, d_stream: int, d_tile_index: int, d_row_scales: int, out_dtype: int, d_out: int,
                  d_scratch: int = 0, scratch_bytes: int = 0, stream: int = 0) -> None:
    """ep_decode_tensor with raw device addresses (ints)."""
    _check(load().ep_decode_tensor(C.byref(info), d_stream, d_tile_index, d_row_scales, out_dtype, d_out,
                                   d_scratch or None, scratch_bytes, stream or None), "ep_decode_tensor")


def decode_tiles(info: Info, d_stream: int, d_tile_index: int, d_row_scales: int, out_dtype: int, d_out: int,
                 tile_begin: int, tile_count: int, d_scratch: int = 0, scratch_bytes: int = 0, stream: int = 0) -> None:
    """ep_decode_tiles: decode tiles [tile_begin, tile_begin + tile_count) only; d_out is the address element
    (0, 0) of the full tensor has (or would have: a shard holder passes its base minus the shard's offset)."""
    _check(load().ep_decode_tiles(C.byref(info), d_stream, d_tile_index, d_row_scales, out_dtype, d_out,
                                  d_scratch or None, scratch_bytes, tile_begin, tile_count, stream or None),
           "ep_decode_tiles")


def decode_tensor_static(info: Info, d_stream: int, d_tile_index: int, d_row_scales: int, out_dtype: int, d_out: int,
                         stream: int = 0) -> None:
    """ep_decode_tensor_static: the same decode for callers that cannot allocate a scratch buffer; large lookup
    tables go to a fixed area inside the library (b <= 13).  Calls sharing a device must not overlap."""
    _check(load().ep_decode_tensor_static(C.byref(info), d_stream, d_tile_index, d_row_scales, out_dtype, d_out,
                                          stream or None), "ep_decode_tensor_static")


def decode_gemm(info: Info, d_stream: int, d_tile_index: int, d_row_scales: int, d_tables: int, d_x: int, T: int, d_y: int,
                stream: int = 0) -> None:
    """ep_decode_gemm with raw device addresses: y[T, R] (fp32) = x[T, C] (bf16) times the decoded weights, transposed."""
    _check(load().ep_decode_gemm(C.byref(info), d_stream, d_tile_index, d_row_scales, d_tables, d_x, T, d_y, stream or None),
           "ep_decode_gemm")


def decode_batch(jobs: list[DecodeJob], stream: int = 0) -> None:
    arr = (DecodeJob * len(jobs))(*jobs)
    _check(load().ep_decode_batch(arr, len(jobs), stream or None), "ep_decode_batch")


def last_device_status(stream: int = 0) -> int:
    return load().ep_last_device_status(stream or None)


# ---- torch plumbing: device memory and streams only ---------------------------------------------

def _torch():
    import torch
    return torch


def _out_torch_dtype(dt: int):
    torch = _torch()
    return {BF16: torch.bfloat16, FP16: torch.float16, FP8_E4M3: torch.float8_e4m3fn, INT8: torch.int8,
            FP32: torch.float32, FP8_E5M2: torch.float8_e5m2, UINT8: torch.uint8}[dt]


class DeviceBlob:
    """A blob resident in device memory: one uint8 tensor plus the host-side Info."""

    def __init__(self, dev, info: Info, prepare: bool = True):
        self.dev = dev
        self.info = info
        base = dev.data_ptr()
        self.d_stream = base
        self.d_tile_index = base + info.off_tiles
        self.d_row_scales = base + info.off_scales
        self.scratch = None
        self.tables = None
        torch = _torch()
        if prepare:
            # the lookup tables depend on the stream only: derive them once, here, not in every decode
            self.tables = torch.empty(decode_tables_bytes(info), dtype=torch.uint8, device=dev.device)
            with torch.cuda.device(dev.device):
                prepare_tables(info, self.d_stream, self.tables.data_ptr(), self.tables.numel(), _stream_handle(None))
        else:
            nb = decode_scratch_bytes(info)
            if nb:
                self.scratch = torch.empty(nb, dtype=torch.uint8, device=dev.device)

    def job(self, out_dtype: int, d_out: int, d_row_scales: int | None = None, tiles: range | None = None) -> DecodeJob:
        return DecodeJob(C.pointer(self.info), self.d_stream, self.d_tile_index,
                         self.d_row_scales if d_row_scales is None else d_row_scales, out_dtype, d_out,
                         self.scratch.data_ptr() if self.scratch is not None else None,
                         self.scratch.numel() if self.scratch is not None else 0,
                         tiles.start if tiles is not None else 0, len(tiles) if tiles is not None else 0,
                         self.tables.data_ptr() if self.tables is not None else None)


def upload(blob: Blob | np.ndarray, device="cuda", pinned=None, non_blocking=False, prepare: bool = True) -> DeviceBlob:
    """Copy a blob to the device.  prepare=True also derives the decoder's lookup tables there once
    (ep_prepare_tables); prepare=False leaves that to every decode call (scratch is allocated if the stream needs it)."""
    torch = _torch()
    data = blob.data if isinstance(blob, Blob) else np.ascontiguousarray(blob, np.uint8)
    info = blob.info if isinstance(blob, Blob) else blob_info(data)
    host = pinned if pinned is not None else torch.from_numpy(data)
    dev = host.to(device, non_blocking=non_blocking)
    return DeviceBlob(dev, info, prepare)


def _stream_handle(stream) -> int:
    torch = _torch()
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def decode(dblob: DeviceBlob, out_dtype: int = BF16, out=None, row_scales=None, stream=None):
    """Decode one device-resident blob into a [R, C] tensor of the requested type (or int32
    [R*C/8, 9] fields for FIELDS_I32).  Asynchronous on the given (or current) torch stream."""
    torch = _torch()
    I = dblob.info
    if out is None:
        if out_dtype == FIELDS_I32:
            out = torch.empty((I.R * I.C // 8, 9), dtype=torch.int32, device=dblob.dev.device)
        else:
            out = torch.empty((I.R, I.C), dtype=_out_torch_dtype(out_dtype), device=dblob.dev.device)
    sc = dblob.d_row_scales if row_scales is None else row_scales.data_ptr()
    if dblob.tables is not None:
        decode_batch([dblob.job(out_dtype, out.data_ptr(), sc)], _stream_handle(stream))
    else:
        decode_tensor(I, dblob.d_stream, dblob.d_tile_index, sc, out_dtype, out.data_ptr(),
                      dblob.scratch.data_ptr() if dblob.scratch is not None else 0,
                      dblob.scratch.numel() if dblob.scratch is not None else 0, _stream_handle(stream))
    return out


def decode_tile_range(dblob: DeviceBlob, tiles: range, out_dtype: int = BF16, out=None, stream=None):
    """Decode a contiguous range of tiles into a buffer that holds exactly their blocks: a flat tensor of
    (blocks of the range) * 8 elements, allocated here unless given.  The shard of a tensor-parallel rank."""
    torch = _torch()
    I = dblob.info
    nvec = I.R * (I.C // 8)
    first, last = tiles.start * I.V, min(tiles.stop * I.V, nvec)
    esize = DTYPE_BYTES[out_dtype]
    if out is None:
        out = torch.empty((last - first) * 8, dtype=_out_torch_dtype(out_dtype), device=dblob.dev.device)
    assert out.numel() >= (last - first) * 8 and out.data_ptr() % 16 == 0
    if dblob.tables is not None:
        decode_batch([dblob.job(out_dtype, out.data_ptr() - first * 8 * esize, tiles=tiles)], _stream_handle(stream))
    else:
        decode_tiles(I, dblob.d_stream, dblob.d_tile_index, dblob.d_row_scales, out_dtype,
                     out.data_ptr() - first * 8 * esize, tiles.start, len(tiles),
                     dblob.scratch.data_ptr() if dblob.scratch is not None else 0,
                     dblob.scratch.numel() if dblob.scratch is not None else 0, _stream_handle(stream))
    return out


def decode_matmul(dblob: DeviceBlob, x, out=None, stream=None):
    """x [T, C] bfloat16 times the blob's decoded BF16 weights [R, C], transposed: [T, R] float32, the weights going
    from the stream into the tensor cores without passing through global memory (ep_decode_gemm; at most 32 tokens per
    launch, more are taken 32 at a time; the stream needs one tile per row, see the header)."""
    torch = _torch()
    I = dblob.info
    assert x.dtype == torch.bfloat16 and x.dim() == 2 and x.shape[1] == I.C and x.is_contiguous()
    if dblob.tables is None:
        raise EntroPackError(-7, "decode_matmul needs prepared tables (upload(..., prepare=True))")
    T = x.shape[0]
    if out is None:
        out = torch.empty((T, I.R), dtype=torch.float32, device=x.device)
    assert out.dtype == torch.float32 and out.shape == (T, I.R) and out.is_contiguous()
    h = _stream_handle(stream)
    for t0 in range(0, T, 32):
        n = min(32, T - t0)
        decode_gemm(I, dblob.d_stream, dblob.d_tile_index, dblob.d_row_scales, dblob.tables.data_ptr(),
                    x[t0:t0 + n].data_ptr(), n, out[t0:t0 + n].data_ptr(), h)
    return out


def decode_many(dblobs: list[DeviceBlob], out_dtype: int, outs: list, stream=None) -> None:
    """One ep_decode_batch launch per MAX_BATCH tensors."""
    h = _stream_handle(stream)
    for i in range(0, len(dblobs), MAX_BATCH):
        jobs = [d.job(out_dtype, o.data_ptr()) for d, o in zip(dblobs[i:i + MAX_BATCH], outs[i:i + MAX_BATCH])]
        decode_batch(jobs, h)
