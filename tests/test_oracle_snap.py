"""Pins for the oracle's snap_tau (Eq. 19): library casts on in-range values, every rounding
boundary of FP8-E4M3, saturation, INT8 half-way cases."""
import numpy as np
import torch

import oracle


def _vals():
    rng = np.random.default_rng(0)
    v = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(3.0),
        (rng.standard_normal(5000) * 1e-3).astype(np.float32),
        (rng.standard_normal(5000) * 100).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 0.5, 1.5, 2.5, -2.5, 1e-8, -1e-8, 6e-8, 3e-5, 448.0, -448.0], np.float32),
    ])
    return v


def test_bf16_matches_library_cast():
    v = np.concatenate([_vals(), np.array([3.3e38, -3.3e38, 3.4e38, 1e-40, -1e-41], np.float32)])
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.snap(v, oracle.BF16), ref)


def test_fp16_matches_library_cast_in_range_and_saturates():
    v = _vals()
    ref = torch.from_numpy(v).to(torch.float16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.snap(v, oracle.FP16), ref)
    # subnormal halves and the largest finite value
    t = np.array([5.9e-8, 2.9e-8, 3.1e-8, 6.1e-5, 65504.0, 65519.0, 65520.0, 1e9, -1e9, np.inf, -np.inf], np.float32)
    got = oracle.snap(t, oracle.FP16)
    ref = torch.from_numpy(t[:6]).to(torch.float16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got[:6], ref)
    assert list(got[6:]) == [0x7BFF, 0x7BFF, 0xFBFF, 0x7BFF, 0xFBFF]


def test_e4m3_matches_library_cast_in_range():
    v = _vals()
    v = v[np.abs(v) <= 448.0]
    ref = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(oracle.snap(v, oracle.E4M3), ref)


def test_e4m3_every_rounding_boundary():
    # all 127 non-negative finite codes, decoded by the format's definition
    codes = np.arange(0, 0x7F, dtype=np.uint8)
    e = (codes >> 3).astype(np.int64)
    m = (codes & 7).astype(np.float64)
    val = np.where(e == 0, m * 2.0 ** -9, (1 + m / 8) * 2.0 ** (e - 7))
    assert val[-1] == 448.0 and val[1] == 2.0 ** -9
    for sign in (1.0, -1.0):
        sb = 0 if sign > 0 else 0x80
        exact = (sign * val).astype(np.float32)
        assert np.array_equal(oracle.snap(exact, oracle.E4M3), codes | sb)
        mid = 0.5 * (val[:-1] + val[1:])
        midf = (sign * mid).astype(np.float32)
        assert np.array_equal(midf.astype(np.float64), sign * mid)      # midpoints are exact in fp32
        even = np.where(codes[:-1] % 2 == 0, codes[:-1], codes[1:])     # ties go to the even code
        assert np.array_equal(oracle.snap(midf, oracle.E4M3), even | sb)
        below = np.nextafter(midf, np.float32(0.0))
        above = np.nextafter(midf, np.float32(sign * np.inf))
        assert np.array_equal(oracle.snap(below, oracle.E4M3), codes[:-1] | sb)
        assert np.array_equal(oracle.snap(above, oracle.E4M3), codes[1:] | sb)
    # saturation, never NaN
    t = np.array([464.0, 465.0, 1e6, np.inf, -500.0, -np.inf], np.float32)
    assert list(oracle.snap(t, oracle.E4M3)) == [0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0xFE]


def test_e5m2_matches_library_cast_in_range_and_saturates():
    v = _vals()
    v = np.concatenate([v, np.array([1.5e-5, 7.6e-6, 2.3e-5, 3e-5, 6.1e-5, 57344.0, 50000.0], np.float32)])
    v = v[np.abs(v) <= 57344.0]
    ref = torch.from_numpy(v).to(torch.float8_e5m2).view(torch.uint8).numpy()
    assert np.array_equal(oracle.snap(v, oracle.E5M2), ref)
    t = np.array([61439.0, 61440.0, 1e9, np.inf, -1e9], np.float32)     # beyond the last rounding boundary: saturate
    assert list(oracle.snap(t, oracle.E5M2)) == [0x7B, 0x7B, 0x7B, 0x7B, 0xFB]


def test_uint8_round_half_even_and_saturation():
    t = np.array([0.5, 1.5, 2.5, -0.5, -3.0, 254.5, 255.5, 300.0, 127.49, 128.5], np.float32)
    assert list(oracle.snap(t, oracle.UINT8)) == [0, 2, 2, 0, 0, 254, 255, 255, 127, 128]


def test_int8_round_half_even_and_saturation():
    t = np.array([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 126.5, 127.5, 300.0, -128.5, -129.5, -1e9, 3.49, -3.51],
                 np.float32)
    assert list(oracle.snap(t, oracle.INT8)) == [0, 2, 2, 0, -2, -2, 126, 127, 127, -128, -128, -128, 3, -4]
    v = _vals()
    ref = np.clip(np.rint(v.astype(np.float64)), -128, 127).astype(np.int8)
    assert np.array_equal(oracle.snap(v, oracle.INT8), ref)


def test_decoded_weights_are_snapped_products():
    # Eq. 19 end to end on a tiny stream: weight = snap(fl32(sigma_r * p)) with p from Eq. 5
    from paper_2609_34185_b200 import synth
    W = synth.gaussian_rows(16, 256, 5)
    blob, rep = oracle.encode(W, 5.0, oracle.default_opts(tile_vectors=50))
    inf = oracle.info(blob)
    sig = blob[inf["off_scales"]:inf["off_scales"] + 4 * 16].view(np.float32)
    out, fields = oracle.decode(blob, oracle.BF16, want_fields=True)
    c = fields[:, 0]
    p = np.empty((len(fields), 8), np.float32)
    p[:, :7] = fields[:, 1:8] + np.float32(0.5) * c[:, None]
    p[:, 7] = 2 * fields[:, 8] + fields[:, 1:8].sum(axis=1) % 2 + np.float32(0.5) * c
    prod = (p.reshape(16, 256) * sig[:, None]).astype(np.float32)
    ref = torch.from_numpy(prod).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(out, ref)
    # overriding the row scales rescales the same points
    out2, _ = oracle.decode(blob, oracle.FP32, scales=np.full(16, 2.0, np.float32))
    assert np.array_equal(out2, 2.0 * p.reshape(16, 256))
