"""ctypes driver for the plain-C EntroPack oracle (test infrastructure only).

Only tests, the smoke check and the bench's CPU-baseline / reference arm may
import this package; the product path never does.  The C source is compiled
with gcc on first use (``-ffp-contract=off`` so that no multiply-add is fused).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "entropack_oracle.c")
_LIB = os.path.join(_HERE, "libentropack_oracle.so")

BF16, FP16, E4M3, INT8, FP32, E5M2, UINT8 = 0, 1, 2, 3, 4, 5, 6
DTYPE_SIZE = {BF16: 2, FP16: 2, E4M3: 1, INT8: 1, FP32: 4, E5M2: 1, UINT8: 1}
_NP_OUT = {BF16: np.uint16, FP16: np.uint16, E4M3: np.uint8, INT8: np.int8, FP32: np.float32, E5M2: np.uint8,
           UINT8: np.uint8}


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class Opts(C.Structure):
    _fields_ = [("bracket_lo", C.c_double), ("bracket_hi", C.c_double), ("search_steps", C.c_int32),
                ("sample_vectors", C.c_uint32), ("tile_vectors", C.c_uint32), ("b_start", C.c_int32),
                ("b_max", C.c_int32), ("retained_bits", C.c_double), ("polish_steps", C.c_int32),
                ("polish_retained_bits", C.c_double), ("rdo_candidates", C.c_int32), ("rdo_sweeps", C.c_int32)]


class Report(C.Structure):
    _fields_ = [("s", C.c_double), ("b", C.c_int32), ("V", C.c_uint32), ("n_tiles", C.c_uint32),
                ("total_words", C.c_uint64), ("bytes", C.c_uint64), ("stored_bpp", C.c_double),
                ("est_bpp_sample", C.c_double), ("cce_bits", C.c_double), ("est_bytes_full", C.c_double),
                ("sample_rows", C.c_uint32), ("coord_min", C.c_int32), ("coord_max", C.c_int32)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.epo_rel_l2.restype = C.c_double
        _lib.epo_row_rms.restype = C.c_float
        _lib.epo_default_tile_vectors.restype = C.c_uint32
        _lib.epo_default_tile_vectors.argtypes = [C.c_double]
        _lib.epo_sample_rows.restype = C.c_uint32
        _lib.epo_num_threads.restype = C.c_int
    return _lib


def _p(a, t=C.c_void_p):
    return a.ctypes.data_as(t)


def default_opts(**kw) -> Opts:
    o = Opts()
    lib().epo_default_opts(C.byref(o))
    for k, v in kw.items():
        setattr(o, k, v)
    return o


def num_threads() -> int:
    return lib().epo_num_threads()


def set_threads(n: int) -> None:
    lib().epo_set_threads(C.c_int(n))


def default_tile_vectors(target_bpp: float) -> int:
    return lib().epo_default_tile_vectors(float(target_bpp))


def row_rms(x: np.ndarray) -> float:
    x = np.ascontiguousarray(x, np.float32)
    return float(lib().epo_row_rms(_p(x), C.c_uint32(x.size)))


def e8_nearest(Y: np.ndarray):
    """Nearest E8 point of one 8-vector: returns (c, z[8]) with p = z + c/2."""
    Y = np.ascontiguousarray(Y, np.float32)
    assert Y.shape == (8,)
    c = C.c_int32()
    z = np.zeros(8, np.int32)
    lib().epo_e8_nearest(_p(Y), C.byref(c), _p(z))
    return c.value, z


def fields_from_point(c: int, z: np.ndarray) -> np.ndarray:
    z = np.ascontiguousarray(z, np.int32)
    f = np.zeros(9, np.int32)
    lib().epo_fields_from_point(C.c_int32(c), _p(z), _p(f))
    return f


def point2_from_fields(f: np.ndarray) -> np.ndarray:
    """Doubled lattice point q = 2p (integers) from a field tuple."""
    f = np.ascontiguousarray(f, np.int32)
    q = np.zeros(8, np.int32)
    lib().epo_point2_from_fields(_p(f), _p(q))
    return q


def rdo_ratios(K: int) -> np.ndarray:
    """The K nested candidate ratios of the per-row refinement."""
    out = np.zeros(max(K, 1), np.float64)
    lib().epo_rdo_ratios(C.c_int(K), _p(out))
    return out[:K]


def quantise(W: np.ndarray, s: float):
    """Fields [R*C/8, 9] and row RMS of W quantised at search scale s."""
    W = np.ascontiguousarray(W, np.float32)
    R, Cc = W.shape
    fields = np.zeros((R * Cc // 8, 9), np.int32)
    mu = np.zeros(R, np.float32)
    lib().epo_quantise(_p(W), C.c_uint32(R), C.c_uint32(Cc), C.c_float(s), _p(fields), _p(mu))
    return fields, mu


def normalise_freqs(n: np.ndarray, b: int) -> np.ndarray:
    n = np.ascontiguousarray(n, np.uint64)
    f = np.zeros(n.size, np.uint32)
    lib().epo_normalise_freqs(_p(n), C.c_uint32(n.size), C.c_int(b), _p(f))
    return f


def model_stats(fields: np.ndarray, rows: int, b: int, V: int, retained: float = 16.0):
    fields = np.ascontiguousarray(fields, np.int32)
    nvec = fields.shape[0]
    cce, est, hc, hp = C.c_double(), C.c_double(), C.c_double(), C.c_double()
    obs = np.zeros(17, np.uint32)
    lib().epo_model_stats(_p(fields), C.c_uint64(nvec), C.c_uint64(rows), C.c_int(b), C.c_uint32(V),
                          C.c_double(retained), C.byref(cce), C.byref(est), C.byref(hc), C.byref(hp), _p(obs))
    return {"cce": cce.value, "est_bits": est.value, "ideal_cond_bits": hc.value,
            "ideal_pooled_bits": hp.value, "observed": obs}


def sample_rows(R: int, Cc: int, budget: int = 1 << 18) -> np.ndarray:
    out = np.zeros(R, np.uint32)
    n = lib().epo_sample_rows(C.c_uint32(R), C.c_uint32(Cc), C.c_uint32(budget), _p(out))
    return out[:n].copy()


def refit(W: np.ndarray, fields: np.ndarray, s: float, mu: np.ndarray) -> np.ndarray:
    W = np.ascontiguousarray(W, np.float32)
    fields = np.ascontiguousarray(fields, np.int32)
    mu = np.ascontiguousarray(mu, np.float32)
    R, Cc = W.shape
    sig = np.zeros(R, np.float32)
    lib().epo_refit(_p(W), C.c_uint32(R), C.c_uint32(Cc), _p(fields), C.c_float(s), _p(mu), _p(sig))
    return sig


def _take_blob(ptr, n) -> np.ndarray:
    buf = np.ctypeslib.as_array(C.cast(ptr, C.POINTER(C.c_uint8)), shape=(n.value,)).copy()
    lib().epo_free(ptr)
    return buf


def pack(fields: np.ndarray, R: int, Cc: int, b: int, V: int, sigma: np.ndarray, s_info: float = 0.0):
    """Final tables + tile encode + stored representation of given fields."""
    fields = np.ascontiguousarray(fields, np.int32)
    sigma = np.ascontiguousarray(sigma, np.float32)
    ptr, n, cce = C.c_void_p(), C.c_size_t(), C.c_double()
    rc = lib().epo_pack(_p(fields), C.c_uint32(R), C.c_uint32(Cc), C.c_int(b), C.c_uint32(V), _p(sigma),
                        C.c_float(s_info), C.byref(ptr), C.byref(n), C.byref(cce))
    if rc:
        raise RuntimeError(f"epo_pack failed: {rc}")
    return _take_blob(ptr, n), cce.value


def encode(W: np.ndarray, target_bpp: float, opts: Opts | None = None):
    """Whole encoder (Algorithm 1, refit, tile encode). Returns (blob uint8[], report dict)."""
    W = np.ascontiguousarray(W, np.float32)
    R, Cc = W.shape
    ptr, n, rep = C.c_void_p(), C.c_size_t(), Report()
    rc = lib().epo_encode(_p(W), C.c_uint32(R), C.c_uint32(Cc), C.c_double(target_bpp),
                          C.byref(opts) if opts is not None else None, C.byref(ptr), C.byref(n), C.byref(rep))
    if rc:
        raise RuntimeError(f"epo_encode failed: {rc}")
    return _take_blob(ptr, n), rep.as_dict()


def info(blob: np.ndarray) -> dict:
    blob = np.ascontiguousarray(blob, np.uint8)
    out = np.zeros(16, np.uint64)
    rc = lib().epo_info(_p(blob), C.c_size_t(blob.size), _p(out))
    if rc:
        raise ValueError(f"not a valid stream: {rc}")
    keys = ["R", "C", "V", "n_tiles", "b", "coord_min", "coord_max", "off_tables", "off_scales",
            "off_tiles", "off_payload", "total_bytes", "total_words"]
    d = {k: int(np.int64(v)) for k, v in zip(keys, out)}
    d["s"] = float(np.frombuffer(out[13:14].tobytes()[:4], np.float32)[0])
    return d


def decode(blob: np.ndarray, dtype: int = BF16, scales: np.ndarray | None = None, want_fields: bool = False,
           tiles: tuple[int, int] | None = None):
    """Decode a stream (or a tile range of it). Returns (weights-as-bit-patterns [R, C], fields or None).

    With a tile range only that range of the returned arrays is written."""
    blob = np.ascontiguousarray(blob, np.uint8)
    inf = info(blob)
    R, Cc = inf["R"], inf["C"]
    out = np.zeros((R, Cc), _NP_OUT[dtype])
    fields = np.zeros((R * Cc // 8, 9), np.int32) if want_fields else None
    sc = None if scales is None else np.ascontiguousarray(scales, np.float32)
    t0, t1 = tiles if tiles is not None else (0, inf["n_tiles"])
    rc = lib().epo_decode_tiles(_p(blob), C.c_size_t(blob.size), C.c_uint32(t0), C.c_uint32(t1),
                                _p(sc) if sc is not None else None, C.c_int(dtype), _p(out),
                                _p(fields) if fields is not None else None)
    if rc:
        raise RuntimeError(f"oracle decode failed: {rc}")
    return out, fields


def snap(v: np.ndarray, dtype: int) -> np.ndarray:
    v = np.ascontiguousarray(v, np.float32)
    out = np.zeros(v.shape, _NP_OUT[dtype])
    lib().epo_snap(_p(v), C.c_size_t(v.size), C.c_int(dtype), _p(out))
    return out


def rel_l2(W: np.ndarray, What: np.ndarray) -> float:
    W = np.ascontiguousarray(W, np.float32)
    What = np.ascontiguousarray(What, np.float32)
    return float(lib().epo_rel_l2(_p(W), _p(What), C.c_size_t(W.size)))
