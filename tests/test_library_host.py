"""CPU-side checks of the library: exported C ABI, host encoder against the oracle (byte-identical
streams on the same inputs), library stream -> oracle decoder, structural validation."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2609_34185_b200 as ep
from paper_2609_34185_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "entropack.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(ep_[a-z0-9_]+)\s*\(", hdr))
    assert {"ep_encode", "ep_decode_tensor", "ep_decode_batch", "ep_blob_info", "ep_validate"} <= names
    lib = ep.load()
    for n in sorted(names):
        assert hasattr(lib, n), n
    assert lib.ep_version() == 1


@pytest.mark.parametrize("shape,bpp,V", [((512, 512), 4.0, 4096), ((96, 1024), 2.0, 0), ((64, 2048), 6.0, 455),
                                         ((33, 264), 3.0, 100), ((8, 8), 4.0, 0)])
def test_host_encoder_matches_oracle_byte_for_byte(shape, bpp, V):
    W = synth.gaussian_rows(shape[0], shape[1], 100 + shape[0])
    lib_blob = ep.encode(W, bpp, tile_vectors=V)
    ora_blob, rep = oracle.encode(W, bpp, oracle.default_opts(tile_vectors=V))
    assert np.array_equal(lib_blob.data, ora_blob)
    assert lib_blob.report["s"] == rep["s"] and lib_blob.report["b"] == rep["b"]
    assert ep.validate(lib_blob.data) == 0


def test_other_distributions_and_threads():
    for W, bpp in ((synth.student_t_rows(256, 1024, 3), 3.0), (synth.laplace_rows(128, 2048, 4), 5.0),
                   (synth.gaussian_rows(128, 1024, 5, outlier_p=0.001), 2.5)):
        a = ep.encode(W, bpp, threads=1)
        b = ep.encode(W, bpp, threads=5)
        o, _ = oracle.encode(W, bpp)
        assert np.array_equal(a.data, b.data) and np.array_equal(a.data, o)
        assert abs(a.stored_bpp - bpp) < 0.02 * bpp


@pytest.mark.timeout(120)
def test_search_survives_sample_alphabets_beyond_the_precision():
    # low starting precision at a high rate: the fine end of the scale search sees more than 2^b symbols per
    # table in the sample; such a scale counts as too fine (no b-bit table exists for it) and the search goes on
    W = synth.laplace_rows(256, 2048, 11)
    for b0, bpp in ((9, 8.0), (9, 7.0), (10, 8.0)):
        a = ep.encode(W, bpp, b_start=b0)
        o, rep = oracle.encode(W, bpp, oracle.default_opts(b_start=b0))
        assert np.array_equal(a.data, o)
        assert max(a.info.table_K) <= 1 << a.info.b
        assert abs(a.stored_bpp - bpp) < 0.01 * bpp
        back, _ = oracle.decode(a.data, oracle.FP32)
        assert oracle.rel_l2(W, back) < 0.02
    # frequency normalisation itself ends even when no valid table exists (more symbols than slots)
    f = oracle.normalise_freqs(np.ones(600, np.uint64), 9)
    assert f.min() == 1 and f.sum() == 600


def test_library_stream_decodes_with_the_oracle():
    W = synth.laplace_rows(64, 1024, 8)
    blob = ep.encode(W, 4.0, tile_vectors=77)
    out, fields = oracle.decode(blob.data, oracle.FP32, want_fields=True)
    qf, _ = oracle.quantise(W, blob.report["s"])
    assert np.array_equal(fields, qf)
    e = oracle.rel_l2(W, out)
    assert 0.03 < e < 0.2
    # pack_fields of the same fields and scales reproduces the stream
    I = blob.info
    sig = blob.data[I.off_scales:I.off_scales + 4 * I.R].view(np.float32)
    again = ep.pack_fields(fields, I.R, I.C, I.b, I.V, sig, s_info=I.s)
    assert np.array_equal(again.data, blob.data)


def test_zero_matrix_and_constant_rows():
    W = np.zeros((16, 64), np.float32)
    blob = ep.encode(W, 4.0)
    o, _ = oracle.encode(W, 4.0)
    assert np.array_equal(blob.data, o)
    out, _ = oracle.decode(blob.data, oracle.BF16)
    assert not out.any()
    W = np.tile(np.arange(1, 65, dtype=np.float32), (4, 1))
    blob = ep.encode(W, 6.0)
    assert np.array_equal(blob.data, oracle.encode(W, 6.0)[0])


def test_bad_arguments():
    lib = ep.load()
    h = ctypes.c_void_p()
    W = np.zeros((4, 12), np.float32)
    assert lib.ep_encode(W.ctypes.data, 4, 12, 4.0, None, ctypes.byref(h)) == -1      # C % 8 != 0
    assert lib.ep_encode(None, 4, 16, 4.0, None, ctypes.byref(h)) == -1
    assert lib.ep_encode(W.ctypes.data, 4, 8, -1.0, None, ctypes.byref(h)) == -1
    assert ep.strerror(-2).startswith("malformed")
    # the fused decode + matrix product refuses on the host, before any CUDA call, what it cannot serve
    blob = ep.encode(synth.gaussian_rows(32, 512, 7), 4.0, tile_vectors=64)
    I = blob.info
    fake = 4096                                                    # (never dereferenced: the checks come first)
    assert lib.ep_decode_gemm(None, fake, fake, fake, fake, fake, 4, fake, None) == -1
    assert lib.ep_decode_gemm(ctypes.byref(I), fake, fake, fake, fake, fake, 0, fake, None) == -1        # no tokens
    assert lib.ep_decode_gemm(ctypes.byref(I), fake, fake, fake, fake, fake + 2, 4, fake, None) == -1    # misaligned x
    assert lib.ep_decode_gemm(ctypes.byref(I), fake, fake, fake, fake + 16, fake, 4, fake, None) == -7   # misaligned tables
    assert lib.ep_decode_gemm(ctypes.byref(I), fake, fake, fake, fake, fake, 33, fake, None) == -3       # more than 32 tokens
    blob = ep.encode(synth.gaussian_rows(32, 512, 7), 4.0, tile_vectors=50)
    I = blob.info
    assert lib.ep_decode_gemm(ctypes.byref(I), fake, fake, fake, fake, fake, 4, fake, None) == -3        # not one tile per row


def test_validate_rejects_damaged_structure():
    W = synth.gaussian_rows(32, 512, 6)
    blob = ep.encode(W, 4.0, tile_vectors=64)
    good = blob.data
    I = blob.info
    assert ep.validate(good) == 0

    def broken(mut):
        b = good.copy()
        mut(b)
        return ep.validate(b)

    assert broken(lambda b: b.__setitem__(0, 0)) == -2                                  # magic
    assert broken(lambda b: b.__setitem__(6, 16)) == -2                                 # b out of range
    assert ep.validate(good[:-2]) == -2                                                 # truncated
    assert broken(lambda b: b.__setitem__(I.off_tables + 8 * 17, b[I.off_tables + 8 * 17] ^ 1)) == -2  # freq sum
    assert broken(lambda b: b[I.off_tiles:I.off_tiles + 4].fill(0)) == -2               # state below 2^15
    assert broken(lambda b: b[I.off_tiles + 128:I.off_tiles + 132].fill(0xFF)) == -2    # offset beyond payload
    def swap_offsets(b):
        o1 = I.off_tiles + 132 + 128
        o2 = I.off_tiles + 2 * 132 + 128
        t = b[o1:o1 + 4].copy(); b[o1:o1 + 4] = b[o2:o2 + 4]; b[o2:o2 + 4] = t
    assert broken(swap_offsets) == -2                                                   # offsets not monotone
    with pytest.raises(ep.EntroPackError):
        ep.blob_info(good[:40])


def test_suggested_tile_size_fills_whole_rounds_of_slots():
    slots = 148 * ep.decode_tiles_per_sm()
    for R, C, bpp in ((8192, 8192, 4.0), (8192, 8192, 2.0), (8192, 8192, 6.0), (10240, 3840, 4.0), (5120, 17408, 3.5)):
        V = ep.suggest_tile_vectors(R, C, bpp, slots)
        assert V <= ep.default_tile_vectors(bpp) and V % 32 == 0
        tiles = -(-(R * C // 8) // V)
        rounds = -(-tiles // slots)
        assert tiles > 0.93 * rounds * slots                      # the last round is nearly full
    assert ep.suggest_tile_vectors(512, 512, 4.0, slots) == ep.default_tile_vectors(4.0) // 4 // 32 * 32    # small tensor: floor
    assert ep.suggest_tile_vectors(4096, 4096, 3.0, 0) == ep.default_tile_vectors(3.0)


def test_suggested_tile_size_for_a_batch_minimises_the_number_of_group_steps():
    ctas = 148

    def steps(shapes, V):                     # rounds per CTA times groups per round (plus the fixed cost per round)
        rounds = sum(-(-(-(-(R * (C // 8)) // V)) // ep.decode_tiles_per_sm()) for R, C in shapes)
        return -(-rounds // ctas) * (V // 32 + 2)

    for shapes, bpp in ((synth.BLOCK_SHAPES, 3.5), (synth.BLOCK_SHAPES, 2.5), ([(8192, 8192)], 4.0),
                        ([(4096, 4096), (4096, 11008), (11008, 4096)], 4.0), ([(256, 256), (128, 1024)], 6.0)):
        V = ep.suggest_tile_vectors_batch(shapes, bpp, ctas)
        vmax = ep.default_tile_vectors(bpp)
        lo = max(32, vmax // 4 // 32 * 32)
        assert V % 32 == 0 and lo <= V <= vmax
        best = min(steps(shapes, v) for v in range(lo, vmax + 1, 32))
        assert steps(shapes, V) == best
        assert all(steps(shapes, v) > best for v in range(V + 32, vmax + 1, 32))      # the largest of the best
    assert ep.suggest_tile_vectors_batch([(8192, 8192)], 4.0, 0) == ep.default_tile_vectors(4.0)


def test_bench_tile_size_rules_mirror_the_library():
    # the CPU arm of bench.py must not load the CUDA library, so it carries the two tile-size rules in Python
    import bench
    assert bench.TILES_PER_SM == ep.decode_tiles_per_sm()
    for bpp in (2.0, 3.5, 4.0, 6.0, 8.0):
        vmax = ep.default_tile_vectors(bpp)
        assert oracle.default_tile_vectors(bpp) == vmax
        for R, C in ((8192, 8192), (512, 512), (4096, 4096), (10240, 3840), (5120, 17408), (64, 256)):
            for slots in (148 * 32, 132 * 32, 0):
                assert bench.suggest_v_py(R, C, vmax, slots) == ep.suggest_tile_vectors(R, C, bpp, slots), (R, C, bpp)
        for shapes in (synth.BLOCK_SHAPES, [(8192, 8192)], [(4096, 4096), (4096, 11008), (11008, 4096)]):
            for ctas in (148, 132, 0):
                assert bench.suggest_v_batch_py(shapes, vmax, ctas) == ep.suggest_tile_vectors_batch(shapes, bpp, ctas)
