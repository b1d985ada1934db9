"""GPU parity: the fused CUDA decoder against the oracle, element by element, through the C ABI.
Both directions (library stream -> oracle decoder is covered on CPU; here library stream and oracle
stream -> GPU decoder), all output types, ragged shapes, and the full-size benchmark configurations."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34185_b200 as ep
from paper_2609_34185_b200 import synth

pytestmark = pytest.mark.gpu

ORACLE_DT = {ep.BF16: oracle.BF16, ep.FP16: oracle.FP16, ep.FP8_E4M3: oracle.E4M3, ep.INT8: oracle.INT8,
             ep.FP32: oracle.FP32, ep.FP8_E5M2: oracle.E5M2, ep.UINT8: oracle.UINT8}


def _bits(t: torch.Tensor) -> np.ndarray:
    if t.dtype in (torch.bfloat16, torch.float16):
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    if t.dtype in (torch.float8_e4m3fn, torch.float8_e5m2):
        return t.view(torch.uint8).cpu().numpy()
    if t.dtype == torch.float32:
        return t.view(torch.int32).cpu().numpy().view(np.uint32)
    return t.cpu().numpy()


def _check_all_types(blob_bytes, scales=None):
    sc_dev = None if scales is None else torch.from_numpy(scales).cuda()
    ref = {odt: oracle.decode(blob_bytes, odt, scales=scales, want_fields=True) for odt in ORACLE_DT.values()}
    # lookup tables prepared once at upload (ep_prepare_tables), and derived inside every decode call
    for prepare in (True, False):
        d = ep.upload(blob_bytes, prepare=prepare)
        for dt, odt in ORACLE_DT.items():
            got = ep.decode(d, dt, row_scales=sc_dev)
            torch.cuda.synchronize()
            want = ref[odt][0].view(np.uint32) if dt == ep.FP32 else ref[odt][0]
            assert np.array_equal(_bits(got), want), f"dtype {dt}, prepared tables {prepare}"
        f = ep.decode(d, ep.FIELDS_I32)
        assert np.array_equal(f.cpu().numpy(), ref[oracle.BF16][1]), f"fields, prepared tables {prepare}"
        assert ep.last_device_status() == 0


def test_config1_all_types_both_directions():
    W = synth.config1()
    lib_blob = ep.encode(W, 4.0, tile_vectors=4096)          # one tile per 64 rows
    assert lib_blob.info.n_tiles == 8
    _check_all_types(lib_blob.data)
    ora_blob, rep = oracle.encode(W, 4.0, oracle.default_opts(tile_vectors=4096))
    _check_all_types(ora_blob)
    assert abs(rep["stored_bpp"] - 4.0) < 0.04
    # weight error against the original matches the oracle's (same points, same scales)
    got = ep.decode(ep.upload(lib_blob), ep.BF16).float().cpu().numpy()
    ref, _ = oracle.decode(ora_blob, oracle.BF16)
    ref = torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).float().numpy()
    e_gpu, e_ref = oracle.rel_l2(W, got), oracle.rel_l2(W, ref)
    assert abs(e_gpu - e_ref) <= 1e-6 * e_ref


@pytest.mark.parametrize("R,C,V,bpp", [
    (8, 8, 0, 4.0),          # a single vector per row, one tiny tile
    (3, 40, 32, 3.0),        # 5 vectors per row: groups straddle rows
    (33, 264, 100, 3.0),     # V not a multiple of 32, ragged last tile
    (64, 2048, 455, 6.0),    # the paper's 8 bpp tile size
    (96, 1024, 1820, 2.0),   # default 4 bpp tile size, low rate
    (5, 4096, 3640, 5.0),
    (256, 256, 33, 4.5),     # many tiny tiles
])
def test_ragged_shapes_all_types(R, C, V, bpp):
    W = synth.laplace_rows(R, C, 1000 + R + C)
    blob = ep.encode(W, bpp, tile_vectors=V)
    _check_all_types(blob.data)


def test_row_scale_edge_cases():
    W = synth.gaussian_rows(16, 512, 31)
    blob = ep.encode(W, 4.0, tile_vectors=100)
    sc = np.array([0.0, -0.0, 1.0, -1.0, 1e30, -1e30, 3e38, 1e-30, 1e-38, 1e-42, 65504.0 / 8, 448.0 / 4, 127.0, 0.5,
                   2.0 ** -20, 7.0], np.float32)
    _check_all_types(blob.data, scales=sc)


def test_single_symbol_tables_and_low_precision():
    # every coordinate zero in coset 1, wide alphabets in coset 0, b = 9
    rng = np.random.default_rng(5)
    n = 4 * 80
    fields = np.zeros((n, 9), np.int32)
    fields[:, 0] = rng.integers(0, 2, n)
    z = np.rint(rng.standard_normal((n, 8)) * 3).astype(np.int32)
    fields[:, 1:] = np.where(fields[:, :1] == 0, z, 0)
    blob = ep.pack_fields(fields, 4, 640, 9, 64, np.linspace(0.5, 2, 4).astype(np.float32))
    _check_all_types(blob.data)
    # only one coset ever used
    fields[:, 0] = 0
    fields[:, 1:] = z
    blob = ep.pack_fields(fields, 4, 640, 10, 50, np.ones(4, np.float32))
    _check_all_types(blob.data)


def test_batch_decode_matches_single():
    blobs = [ep.encode(synth.gaussian_rows(64 + 32 * i, 512 + 256 * i, 50 + i), 2.5 + 0.5 * i, tile_vectors=200 + 37 * i)
             for i in range(5)]
    devs = [ep.upload(b) for b in blobs]
    outs = [torch.empty((b.info.R, b.info.C), dtype=torch.bfloat16, device="cuda") for b in blobs]
    ep.decode_many(devs, ep.BF16, outs)
    torch.cuda.synchronize()
    for b, o in zip(blobs, outs):
        ref, _ = oracle.decode(b.data, oracle.BF16)
        assert np.array_equal(_bits(o), ref)
    assert ep.last_device_status() == 0


def test_streams_without_payload_words_and_many_jobs():
    # an all-zero matrix has one symbol per table: no payload word at all
    zero = ep.encode(np.zeros((32, 512), np.float32), 4.0, tile_vectors=64)
    assert zero.info.total_words == 0
    _check_all_types(zero.data)
    const = ep.encode(np.tile(np.arange(1, 257, dtype=np.float32), (8, 1)), 5.0, tile_vectors=32)
    _check_all_types(const.data)
    # more tensors than one launch takes (16): decode_many splits them
    blobs = [ep.encode(synth.gaussian_rows(32, 256 + 8 * i, 600 + i), 3.0 + 0.1 * i, tile_vectors=40 + i) for i in range(19)]
    devs = [ep.upload(b) for b in blobs]
    outs = [torch.empty((b.info.R, b.info.C), dtype=torch.float16, device="cuda") for b in blobs]
    ep.decode_many(devs, ep.FP16, outs)
    torch.cuda.synchronize()
    for b, o in zip(blobs, outs):
        assert np.array_equal(_bits(o), oracle.decode(b.data, oracle.FP16)[0])
    assert ep.last_device_status() == 0


def test_damaged_payload_is_flagged_not_fatal():
    W = synth.gaussian_rows(64, 1024, 9)
    blob = ep.encode(W, 4.0, tile_vectors=128)
    bad = blob.data.copy()
    I = blob.info
    bad[I.off_payload + 2 * (I.total_words // 2)] ^= 0x10       # structure still valid
    bad[I.off_payload + 2 * I.total_words - 1] ^= 0x01          # and the very last word
    assert ep.validate(bad) == 0
    out = ep.decode(ep.upload(bad), ep.BF16)
    assert ep.last_device_status() == -2
    assert ep.last_device_status() == 0                          # the word is cleared after reading
    # the context is still usable and a good stream decodes cleanly afterwards
    good = ep.decode(ep.upload(blob), ep.BF16)
    ref, _ = oracle.decode(blob.data, oracle.BF16)
    assert np.array_equal(_bits(good), ref) and ep.last_device_status() == 0


def test_decode_argument_checks():
    blob = ep.encode(synth.gaussian_rows(16, 64, 1), 4.0)
    d = ep.upload(blob)
    out = torch.empty((16, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ep.EntroPackError):
        ep.decode_tensor(d.info, d.d_stream, d.d_tile_index, d.d_row_scales, ep.BF16, out.data_ptr() + 2)
    with pytest.raises(ep.EntroPackError):
        ep.decode_tensor(d.info, d.d_stream, d.d_tile_index, d.d_row_scales, 7, out.data_ptr())
    with pytest.raises(ep.EntroPackError):
        ep.decode_tensor(d.info, 0, d.d_tile_index, d.d_row_scales, ep.BF16, out.data_ptr())


# ---- streams whose lookup tables do not fit shared memory (b >= 12 or coordinate range > 1024) -----

def test_large_table_path_high_precision_and_high_rate():
    W = synth.laplace_rows(96, 1024, 77)
    for kw, bpp in ((dict(b_start=12), 4.0), (dict(), 8.0), (dict(b_start=15, tile_vectors=100), 5.0),
                    (dict(b_start=13, tile_vectors=33), 3.0)):
        blob = ep.encode(W, bpp, **kw)
        flat = 17 * 4 << blob.info.b                  # seventeen tables of 2^b four-byte entries
        assert blob.info.b >= 12 and ep.decode_scratch_bytes(blob.info) >= flat
        if blob.info.b > 12:                          # (b = 12 adds the two-level tables of the hot loop)
            assert ep.decode_scratch_bytes(blob.info) == flat
        _check_all_types(blob.data)
        if "tile_vectors" not in kw:          # tiny tiles are metadata-bound: no rate claim there
            assert abs(blob.stored_bpp - bpp) < 0.02 * bpp
    # oracle stream, paper's 8 bpp defaults (b = 12, 4096-symbol tiles)
    ora, rep = oracle.encode(synth.gaussian_rows(64, 2048, 5), 8.0)
    assert rep["b"] == 12 and rep["V"] == 455
    _check_all_types(ora)


def test_large_table_path_wide_coordinate_range():
    # b = 11 but coordinates spread over more than 512 values: a few huge outliers
    rng = np.random.default_rng(3)
    n = 6 * 64
    fields = np.zeros((n, 9), np.int32)
    fields[:, 0] = rng.integers(0, 2, n)
    fields[:, 1:] = np.rint(rng.standard_normal((n, 8)) * 4).astype(np.int32)
    fields[5, 3] = 700
    fields[77, 8] = -400
    fields[100, 1] = -3000
    blob = ep.pack_fields(fields, 6, 512, 11, 50, np.linspace(0.01, 0.02, 6).astype(np.float32))
    assert ep.decode_scratch_bytes(blob.info) > 0
    _check_all_types(blob.data)


def test_coordinate_range_up_to_1024_stays_on_the_shared_memory_path():
    # the table entry's code field holds ten bits: coordinates spread over 513 .. 1024 values need no scratch
    rng = np.random.default_rng(4)
    n = 8 * 64
    fields = np.zeros((n, 9), np.int32)
    fields[:, 0] = rng.integers(0, 2, n)
    fields[:, 1:] = np.rint(rng.standard_normal((n, 8)) * 6).astype(np.int32)
    fields[3, 2] = 500
    fields[90, 7] = -520          # z range -520 .. 500: 1021 values, even base -520
    fields[200, 8] = 250          # m = 250 stands for z8 = 500 or 501
    fields[201, 8] = -260         # and z8 = -520 or -519
    blob = ep.pack_fields(fields, 8, 512, 11, 64, np.linspace(0.01, 0.03, 8).astype(np.float32))
    assert ep.decode_scratch_bytes(blob.info) == 0
    _check_all_types(blob.data)
    # one value more on either side no longer fits
    fields[4, 1] = 504
    blob = ep.pack_fields(fields, 8, 512, 11, 64, np.linspace(0.01, 0.03, 8).astype(np.float32))
    assert ep.decode_scratch_bytes(blob.info) > 0
    _check_all_types(blob.data)
    # Laplace rows at 7 bpp: b = 11 with coordinates beyond +-256
    blob = ep.encode(synth.laplace_rows(512, 4096, 4), 7.0)
    assert blob.info.b == 11 and blob.info.coord_max - blob.info.coord_min > 512
    assert ep.decode_scratch_bytes(blob.info) == 0
    _check_all_types(blob.data)


def test_two_level_tables_of_2_to_the_12_slot_streams():
    # b = 12 (the paper's setting for 8 bpp): slot -> coordinate code in shared memory, one entry per (table, code),
    # those of the 528 codes around zero in shared memory, all of them in global memory.  Heavy-tailed rows put many
    # coordinates outside the window; tensors wide enough for the hot loop, all output types, tile ranges, a batch.
    W = synth.student_t_rows(192, 4096, 61)
    blob = ep.encode(W, 8.0)
    I = blob.info
    flat = 17 * 4 << 12
    assert I.b == 12 and max(I.table_K) > 264 and ep.decode_scratch_bytes(I) > flat
    _check_all_types(blob.data)
    other = ep.encode(synth.gaussian_rows(64, 2048, 62), 4.0, b_start=12, tile_vectors=100)
    small = ep.encode(synth.gaussian_rows(64, 2048, 63), 4.0)
    outs = [torch.empty((b.info.R, b.info.C), dtype=torch.float16, device="cuda") for b in (blob, small, other)]
    ep.decode_many([ep.upload(blob), ep.upload(small), ep.upload(other, prepare=False)], ep.FP16, outs)
    torch.cuda.synchronize()
    for b, o in zip((blob, small, other), outs):
        assert np.array_equal(_bits(o), oracle.decode(b.data, oracle.FP16)[0])
    d = ep.upload(blob)
    part = ep.decode_tile_range(d, range(3, 11), ep.BF16)
    torch.cuda.synchronize()
    ref = oracle.decode(blob.data, oracle.BF16)[0].reshape(-1)
    assert np.array_equal(_bits(part), ref[3 * I.V * 8:11 * I.V * 8])
    rng = np.random.default_rng(64)
    n = 64 * 512 // 8
    two = 16 * 4096 * 2 + 16 * 528 * 4 + 16 * 4096 * 4
    fields = np.zeros((n, 9), np.int32)
    fields[:, 0] = rng.integers(0, 2, n)
    # nearly the widest coordinate range the two levels take (4096 values), uniformly filled: most lookups leave
    # the window
    fields[:, 1:8] = rng.integers(-2040, 2040, (n, 7))
    fields[:, 8] = rng.integers(-1000, 1000, n)
    full = ep.pack_fields(fields, 64, 512, 12, 64, np.full(64, 0.001, np.float32))
    assert ep.decode_scratch_bytes(full.info) == two + flat
    _check_all_types(full.data)
    # coordinates on one side of zero (the window cannot be centred), one field constant (a lone symbol: f = 2^12)
    fields[:, 1:8] = rng.integers(0, 1500, (n, 7))
    fields[:, 3] = 7
    fields[:, 8] = rng.integers(0, 40, n)
    onesided = ep.pack_fields(fields, 64, 512, 12, 64, np.full(64, 0.001, np.float32))
    assert onesided.info.table_K[3] == 1 and ep.decode_scratch_bytes(onesided.info) == two + flat
    _check_all_types(onesided.data)
    # a wider range than that: the flat tables in global memory serve the stream
    fields[:, 1:] = rng.integers(-2500, 2500, (n, 8))
    wide = ep.pack_fields(fields, 64, 512, 12, 64, np.full(64, 0.001, np.float32))
    assert ep.decode_scratch_bytes(wide.info) == flat
    _check_all_types(wide.data)
    assert ep.last_device_status() == 0


def test_single_symbol_tables_at_b11():
    rng = np.random.default_rng(5)
    n = 4 * 64
    fields = np.zeros((n, 9), np.int32)                      # coset always 0: the coset table has one symbol
    fields[:, 1:] = np.rint(rng.standard_normal((n, 8)) * 3).astype(np.int32)
    # the coset is decoded by comparing the slot with the frequency of coset 0: a lone coset (f = 2^11) needs no table
    blob = ep.pack_fields(fields, 4, 512, 11, 40, np.full(4, 0.02, np.float32))
    assert blob.info.table_K[0] == 1 and ep.decode_scratch_bytes(blob.info) == 0
    _check_all_types(blob.data)
    only1 = fields.copy()
    only1[:, 0] = 1                                          # coset always 1
    blob = ep.pack_fields(only1, 4, 512, 11, 40, np.full(4, 0.02, np.float32))
    assert blob.info.table_K[0] == 1 and blob.info.table_min[0] == 1 and ep.decode_scratch_bytes(blob.info) == 0
    _check_all_types(blob.data)
    # a lone coordinate symbol has frequency 2^11, one bit more than the shared-memory entry's frequency field
    lone = fields.copy()
    lone[:, 3] = 2
    blob = ep.pack_fields(lone, 4, 512, 11, 40, np.full(4, 0.02, np.float32))
    assert blob.info.table_K[3] == 1 and ep.decode_scratch_bytes(blob.info) > 0
    _check_all_types(blob.data)
    blob10 = ep.pack_fields(lone, 4, 512, 10, 40, np.full(4, 0.02, np.float32))
    assert ep.decode_scratch_bytes(blob10.info) == 0        # f = 2^10 fits
    _check_all_types(blob10.data)


def test_large_table_path_needs_scratch_and_mixes_in_a_batch():
    W = synth.gaussian_rows(64, 512, 8)
    big = ep.encode(W, 4.0, b_start=12)
    small = ep.encode(W, 4.0)
    d_big, d_small = ep.upload(big), ep.upload(small)
    out = torch.empty((64, 512), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ep.EntroPackError) as ei:
        ep.decode_tensor(d_big.info, d_big.d_stream, d_big.d_tile_index, d_big.d_row_scales, ep.BF16, out.data_ptr())
    assert ei.value.status == -7
    outs = [torch.empty((64, 512), dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    ep.decode_many([d_small, d_big, d_small], ep.BF16, outs)
    torch.cuda.synchronize()
    for b, o in zip((small, big, small), outs):
        ref, _ = oracle.decode(b.data, oracle.BF16)
        assert np.array_equal(_bits(o), ref)
    assert ep.last_device_status() == 0


# ---- full-size configurations, in the launch configuration the bench times -----------------------

def _full_compare(W, bpp, dt, V=0):
    blob = ep.encode(W, bpp, tile_vectors=V)
    assert abs(blob.stored_bpp - bpp) < 0.01 * bpp, blob.stored_bpp
    d = ep.upload(blob)
    got = ep.decode(d, dt)
    ref, _ = oracle.decode(blob.data, ORACLE_DT[dt])
    torch.cuda.synchronize()
    assert np.array_equal(_bits(got), ref)
    assert ep.last_device_status() == 0
    return blob


def test_config2_full_size():
    _full_compare(synth.config2(), 3.0, ep.BF16)


def test_config4_full_size_three_rates():
    W = synth.config4()
    _full_compare(W, 4.0, ep.FP16)
    _full_compare(W, 2.0, ep.FP16)
    _full_compare(W, 6.0, ep.FP16)


def test_config4_every_rate_of_the_sweep_at_the_tile_size_the_bench_uses():
    # the whole sweep 2.0, 2.5 .. 6.0 bpp as `bench.py` times it: streams from the GPU encoder, tile size from
    # ep_suggest_tile_vectors, FP16 output; every weight against the oracle and the stored rate within 1 %
    slots = ep.decode_tiles_per_sm() * torch.cuda.get_device_properties(0).multi_processor_count
    Wd = torch.from_numpy(synth.config4()).cuda()
    out = torch.empty((8192, 8192), dtype=torch.float16, device="cuda")
    for bpp in (2.0, 2.5, 3.0, 3.5, 4.0, 4.5, 5.0, 5.5, 6.0):
        blob = ep.encode_device(Wd, bpp, tile_vectors=ep.suggest_tile_vectors(8192, 8192, bpp, slots))
        assert abs(blob.stored_bpp - bpp) < 0.01 * bpp, (bpp, blob.stored_bpp)
        ep.decode(ep.upload(blob), ep.FP16, out=out)
        ref, _ = oracle.decode(blob.data, oracle.FP16)
        torch.cuda.synchronize()
        assert np.array_equal(_bits(out), ref), bpp
    assert ep.last_device_status() == 0


def _container(W, kind):
    """Row-scaled FP8 / INT8 container values of W as fp32 (the low-precision route compresses these)."""
    a, Wc = synth.to_container(W, kind)
    if kind == "fp8":
        return a, torch.from_numpy(Wc).to(torch.float8_e4m3fn).float().numpy()
    return a, np.clip(np.rint(Wc), -128, 127).astype(np.float32)


@pytest.mark.parametrize("kind,dt,odt", [("fp8", ep.FP8_E4M3, oracle.E4M3), ("int8", ep.INT8, oracle.INT8)])
def test_config3_whole_bundle_in_one_batched_launch(kind, dt, odt):
    # the seven tensors of the block bundle at full size (372 M weights), each first scaled row by row into the
    # FP8 / INT8 container, compressed at 2.5 bpp and decoded into that container by ONE ep_decode_batch launch:
    # every byte against the oracle; the per-row output scale a_r then brings the weights back (error vs the source)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    V = ep.suggest_tile_vectors_batch(synth.BLOCK_SHAPES, 2.5, sms)
    blobs, scales, sources = [], [], []
    for i in range(7):
        W = synth.config3_tensor(i)
        a, Wc = _container(W, kind)
        blobs.append(ep.encode_device(torch.from_numpy(Wc).cuda(), 2.5, tile_vectors=V))
        scales.append(a)
        if i in (0, 4):
            sources.append((i, W))
        del W, Wc
    total = sum(b.info.R * b.info.C for b in blobs)
    assert abs(8.0 * sum(len(b) for b in blobs) / total - 2.5) < 0.025
    tdt = torch.float8_e4m3fn if kind == "fp8" else torch.int8
    buf = torch.empty(total, dtype=tdt, device="cuda")
    outs, at = [], 0
    for b in blobs:
        n = b.info.R * b.info.C
        outs.append(buf[at:at + n].view(b.info.R, b.info.C))
        at += n
    ep.decode_many([ep.upload(b) for b in blobs], dt, outs)
    torch.cuda.synchronize()
    assert ep.last_device_status() == 0
    for b, o in zip(blobs, outs):
        ref, _ = oracle.decode(b.data, odt)
        assert np.array_equal(_bits(o).view(ref.dtype), ref), (kind, b.info.R, b.info.C)
    for i, W in sources:                                        # container value times its row's output scale
        back = outs[i].float().cpu().numpy() * scales[i][:, None]
        assert oracle.rel_l2(W, back) < 0.25                   # 2.5 bpp: about 20 % on these rows


def test_config3_one_wide_tensor_fp8_and_int8_containers():
    # MLP-shaped tensor of the block bundle, pre-scaled to the FP8 / INT8 container as in the paper's
    # low-precision route; decoded values must equal the oracle's in that container
    W = synth.config3_tensor(4, shape=(2048, 17408))
    for kind, dt, tdt in (("fp8", ep.FP8_E4M3, torch.float8_e4m3fn), ("int8", ep.INT8, None)):
        a, Wc = synth.to_container(W, kind)
        if tdt is not None:
            Wc = torch.from_numpy(Wc).to(tdt).float().numpy()
        else:
            Wc = np.clip(np.rint(Wc), -128, 127).astype(np.float32)
        _full_compare(Wc, 2.5, dt)


def test_config4_with_the_tile_size_the_bench_uses():
    V = ep.suggest_tile_vectors(8192, 8192, 4.0, ep.decode_tiles_per_sm() * torch.cuda.get_device_properties(0).multi_processor_count)
    blob = _full_compare(synth.config4(), 4.0, ep.FP16, V)
    assert blob.info.V == V


def test_config5_one_layer_batched_as_the_bench_times_it():
    # the seven tensors of one layer at full size (372 M parameters), one tile size from ep_suggest_tile_vectors_batch,
    # streams from the GPU encoder, one batched launch into one reused BF16 buffer: every weight against the oracle
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    V = ep.suggest_tile_vectors_batch(synth.BLOCK_SHAPES, 3.5, sms)
    blobs = []
    for i in range(7):
        W = synth.config5_tensor(0, i)
        blobs.append(ep.encode_device(torch.from_numpy(W).cuda(), 3.5, tile_vectors=V))
        del W
    total = sum(b.info.R * b.info.C for b in blobs)
    assert abs(8.0 * sum(len(b) for b in blobs) / total - 3.5) < 0.035
    buf = torch.empty(total, dtype=torch.bfloat16, device="cuda")
    outs, at = [], 0
    for b in blobs:
        n = b.info.R * b.info.C
        outs.append(buf[at:at + n].view(b.info.R, b.info.C))
        at += n
    ds = [ep.upload(b) for b in blobs]
    ep.decode_many(ds, ep.BF16, outs)
    torch.cuda.synchronize()
    assert ep.last_device_status() == 0
    for b, o in zip(blobs, outs):
        ref, _ = oracle.decode(b.data, oracle.BF16)
        assert np.array_equal(_bits(o), ref), (b.info.R, b.info.C)


# ---- tile ranges: the shard of a tensor-parallel rank ------------------------------------------------

def test_tile_ranges_tile_the_tensor_and_write_nothing_else():
    from paper_2609_34185_b200.sharding import shard_range
    for W, bpp, V, dt, odt in ((synth.gaussian_rows(96, 1024, 21), 4.0, 100, ep.BF16, oracle.BF16),
                               (synth.laplace_rows(40, 264, 22), 3.0, 33, ep.FP8_E4M3, oracle.E4M3),
                               (synth.laplace_rows(64, 2048, 23), 8.0, 0, ep.FP16, oracle.FP16)):      # b = 12 path
        blob = ep.encode(W, bpp, tile_vectors=V)
        d = ep.upload(blob)
        I = blob.info
        ref, _ = oracle.decode(blob.data, odt)
        ref = np.ascontiguousarray(ref).reshape(-1).view(np.uint8)
        es = ep.DTYPE_BYTES[dt]
        nvec = I.R * (I.C // 8)
        for world in (1, 2, 3, 5):
            pieces = []
            for rank in range(world):
                tiles = shard_range(I.n_tiles, world, rank)
                if len(tiles) == 0:
                    continue
                out = ep.decode_tile_range(d, tiles, dt)
                torch.cuda.synchronize()
                first, last = tiles.start * I.V, min(tiles.stop * I.V, nvec)
                got = out.view(torch.uint8).cpu().numpy().reshape(-1)
                assert got.size == (last - first) * 8 * es
                assert np.array_equal(got, ref[first * 8 * es:last * 8 * es]), (W.shape, world, rank)
                part, _ = oracle.decode(blob.data, odt, tiles=(tiles.start, tiles.stop))     # the oracle's own range decode
                part = np.ascontiguousarray(part).reshape(-1).view(np.uint8)
                assert np.array_equal(got, part[first * 8 * es:last * 8 * es])
                pieces.append(got)
            assert np.array_equal(np.concatenate(pieces), ref)
        # in place in a full-size buffer: bytes outside the range keep their fill value (the plain call: tables
        # derived inside the decode, caller scratch where the stream needs it)
        d = ep.upload(blob, prepare=False)
        full = torch.full((I.R * I.C * es,), 0xA5, dtype=torch.uint8, device="cuda")
        t0, cnt = I.n_tiles // 3, max(1, I.n_tiles // 3)
        ep.decode_tiles(I, d.d_stream, d.d_tile_index, d.d_row_scales, dt, full.data_ptr(), t0, cnt,
                        d.scratch.data_ptr() if d.scratch is not None else 0,
                        d.scratch.numel() if d.scratch is not None else 0)
        torch.cuda.synchronize()
        got = full.cpu().numpy()
        a, b = t0 * I.V * 8 * es, min((t0 + cnt) * I.V, nvec) * 8 * es
        assert np.array_equal(got[a:b], ref[a:b]) and np.all(got[:a] == 0xA5) and np.all(got[b:] == 0xA5)
        assert ep.last_device_status() == 0
        for bad in ((I.n_tiles, 1), (0, I.n_tiles + 1), (1, 0)):
            with pytest.raises(ep.EntroPackError):
                ep.decode_tiles(I, d.d_stream, d.d_tile_index, d.d_row_scales, dt, full.data_ptr(), bad[0], bad[1],
                                d.scratch.data_ptr() if d.scratch is not None else 0,
                                d.scratch.numel() if d.scratch is not None else 0)


def test_batch_shares_cross_jobs_with_different_tile_sizes():
    # the launch's rounds are split over the CTAs by cost (groups per round): tiny tensors make one CTA's share
    # span several jobs (tables rebuilt in between), a big one spreads over many CTAs, tile sizes differ per job
    rng = np.random.default_rng(12)
    specs = [(8, 256, 32), (16, 512, 33), (8, 264, 5), (2048, 2048, 455), (32, 256, 100), (64, 1024, 1792),
             (8, 8, 0), (512, 4096, 1820), (24, 512, 64), (1024, 1024, 96), (8, 512, 1), (40, 2048, 640),
             (16, 256, 0), (256, 256, 128), (8, 1024, 31), (128, 8192, 3640)]
    blobs, outs = [], []
    for i, (R, C, V) in enumerate(specs):
        W = synth.gaussian_rows(R, C, 500 + i) if i % 2 else synth.laplace_rows(R, C, 500 + i)
        blobs.append(ep.encode(W, float(rng.choice([2.0, 3.0, 4.0, 5.0])), tile_vectors=V))
        outs.append(torch.empty((R, C), dtype=torch.float16, device="cuda"))
    ds = [ep.upload(b) for b in blobs]
    ep.decode_many(ds, ep.FP16, outs)
    torch.cuda.synchronize()
    for b, o in zip(blobs, outs):
        ref, _ = oracle.decode(b.data, oracle.FP16)
        assert np.array_equal(_bits(o), ref), (b.info.R, b.info.C, b.info.V)
    assert ep.last_device_status() == 0
    # the same tensors in the opposite order (other shares, other job boundaries) and as fields
    outs2 = [torch.empty((b.info.R * b.info.C // 8, 9), dtype=torch.int32, device="cuda") for b in blobs]
    ep.decode_many(ds[::-1], ep.FIELDS_I32, outs2[::-1])
    torch.cuda.synchronize()
    for b, o in zip(blobs, outs2):
        _, f = oracle.decode(b.data, oracle.BF16, want_fields=True)
        assert np.array_equal(o.cpu().numpy(), f)


def test_decode_calls_can_be_captured_in_a_cuda_graph_and_replayed():
    # a decode call only enqueues kernels on the given stream (after the first call per output type has set the
    # kernel's shared-memory attribute), so a layer's launches can be recorded once and replayed
    Ws = [synth.gaussian_rows(128, 1024, 61), synth.laplace_rows(64, 2048, 62), synth.gaussian_rows(96, 512, 63)]
    blobs = [ep.encode(W, 4.0) for W in Ws] + [ep.encode(Ws[0], 4.0, b_start=12)]      # the last one needs scratch
    ds = [ep.upload(b) for b in blobs]
    outs = [torch.zeros((b.info.R, b.info.C), dtype=torch.bfloat16, device="cuda") for b in blobs]
    ep.decode_many(ds, ep.BF16, outs)                  # warm-up outside the capture
    torch.cuda.synchronize()
    for o in outs:
        o.zero_()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            ep.decode_many(ds[:3], ep.BF16, outs[:3], stream=side)
            ep.decode(ds[3], ep.BF16, out=outs[3], stream=side)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for rep in range(2):
        for o in outs:
            o.zero_()
        g.replay()
        torch.cuda.synchronize()
        for b, o in zip(blobs, outs):
            ref, _ = oracle.decode(b.data, oracle.BF16)
            assert np.array_equal(_bits(o), ref)
    assert ep.last_device_status() == 0


def test_largest_supported_tensor_byte_offsets_beyond_two_to_the_31():
    # 30000 x 32768 = 983 M weights: the FP32 output is 3.93 GB, so the kernels' 32-bit byte offsets run close to
    # their end; one more row would be refused.  Input drawn on the device (seeded), stream from the GPU encoder.
    R, C = 30000, 32768
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    Wd = torch.randn(R, C, generator=g, device="cuda", dtype=torch.float32) * 0.02
    blob = ep.encode_device(Wd, 3.0)
    del Wd
    assert abs(blob.stored_bpp - 3.0) < 0.03
    d = ep.upload(blob)
    for dt, odt in ((ep.FP32, oracle.FP32), (ep.INT8, oracle.INT8)):
        out = ep.decode(d, dt)
        torch.cuda.synchronize()
        ref, _ = oracle.decode(blob.data, odt)
        got = out.view(torch.uint8).cpu().numpy().reshape(-1)
        assert np.array_equal(got, np.ascontiguousarray(ref).reshape(-1).view(np.uint8))
        del out, got, ref
    assert ep.last_device_status() == 0
    tiles = range(blob.info.n_tiles - 1000, blob.info.n_tiles)          # a shard at the far end of the offsets
    sh = ep.decode_tile_range(d, tiles, ep.FP32)
    torch.cuda.synchronize()
    part, _ = oracle.decode(blob.data, oracle.FP32, tiles=(tiles.start, tiles.stop))
    first = tiles.start * blob.info.V * 8
    assert np.array_equal(sh.view(torch.int32).cpu().numpy(), part.reshape(-1)[first:].view(np.int32))
    # a tensor whose offsets would not fit is refused, not decoded wrongly
    import copy
    big = copy.copy(blob.info)
    big.R = 32768
    out = torch.empty(16, dtype=torch.float32, device="cuda")
    with pytest.raises(ep.EntroPackError) as ei:
        ep.decode_tensor(big, d.d_stream, d.d_tile_index, d.d_row_scales, ep.FP32, out.data_ptr())
    assert ei.value.status == -3
