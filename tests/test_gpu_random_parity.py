"""Randomised parity: shapes, rates, tile sizes, precisions, distributions and output types drawn from a fixed
seed; every case compares the GPU decode with the oracle's decode bit for bit, and a third of them the GPU
encoder's stream with the host encoder's byte for byte."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34185_b200 as ep
from paper_2609_34185_b200 import synth

pytestmark = pytest.mark.gpu

TYPES = [(ep.BF16, oracle.BF16), (ep.FP16, oracle.FP16), (ep.FP8_E4M3, oracle.E4M3), (ep.INT8, oracle.INT8),
         (ep.FP32, oracle.FP32), (ep.FP8_E5M2, oracle.E5M2), (ep.UINT8, oracle.UINT8)]


def _draw(rng):
    R = int(rng.choice([1, 2, 3, 7, 16, 33, 64, 100, 257, 512]))
    C = 8 * int(rng.choice([1, 2, 4, 5, 16, 31, 32, 33, 64, 100, 128, 256, 511, 512]))
    bpp = float(rng.choice([2.0, 2.5, 3.0, 3.5, 4.0, 5.0, 6.0, 7.0, 8.0]))
    kind = int(rng.integers(0, 4))
    seed = int(rng.integers(1 << 30))
    if kind == 0:
        W = synth.gaussian_rows(R, C, seed)
    elif kind == 1:
        W = synth.laplace_rows(R, C, seed)
    elif kind == 2:
        W = synth.student_t_rows(R, C, seed)
    else:
        W = synth.gaussian_rows(R, C, seed, outlier_p=0.01, outlier_mag=30.0)
    if rng.random() < 0.1:
        W[rng.integers(R)] = 0
    kw = {}
    if rng.random() < 0.5:
        kw["tile_vectors"] = int(rng.choice([1, 5, 31, 32, 33, 64, 100, 455, 1000, 1792, 4000]))
    if rng.random() < 0.2:
        kw["b_start"] = int(rng.choice([9, 10, 11, 12, 13, 14]))
    if rng.random() < 0.15:
        kw["rdo_candidates"] = 5
    return W, bpp, kw


@pytest.mark.parametrize("block", range(4))
def test_random_cases_decode_and_encode_match(block):
    for it in range(25):
        rng = np.random.default_rng(7_000_003 * (block + 1) + it)
        W, bpp, kw = _draw(rng)
        blob = ep.encode(W, bpp, **kw)
        what = (W.shape, bpp, kw, blob.info.b, blob.info.V)
        if rng.random() < 0.33:
            try:
                dev = ep.encode_device(torch.from_numpy(W).cuda(), bpp, **kw)
                assert np.array_equal(dev.data, blob.data), what
            except ep.EntroPackError as e:      # coordinate range or symbol count beyond the GPU back end's limits
                assert e.status == -3, what
        d = ep.upload(blob)
        for i in rng.choice(len(TYPES), 2, replace=False):
            dt, odt = TYPES[int(i)]
            out = ep.decode(d, dt)
            torch.cuda.synchronize()
            ref, _ = oracle.decode(blob.data, odt)
            got = out.view(torch.uint8).cpu().numpy().reshape(-1)
            assert np.array_equal(got, np.ascontiguousarray(ref).view(np.uint8).reshape(-1)), (what, dt)
        assert ep.last_device_status() == 0, what
