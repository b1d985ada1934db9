"""The CUDA encoder back end against the host encoder: the same bytes for the same input, and therefore
(tests/test_library_host.py) the oracle's bytes as well."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34185_b200 as ep
from paper_2609_34185_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("maker,shape,bpp,kw", [
    (synth.gaussian_rows, (512, 512), 4.0, dict(tile_vectors=4096)),
    (synth.laplace_rows, (96, 1024), 2.0, {}),
    (synth.student_t_rows, (256, 2048), 3.0, dict(tile_vectors=455)),
    (synth.laplace_rows, (64, 4096), 6.0, {}),
    (synth.gaussian_rows, (33, 264), 5.0, dict(tile_vectors=100)),
    (synth.gaussian_rows, (8, 8), 4.0, {}),
    (synth.gaussian_rows, (128, 1024), 8.0, {}),                    # b = 12
])
def test_device_encoder_gives_the_host_encoders_bytes(maker, shape, bpp, kw):
    W = maker(shape[0], shape[1], 4242 + shape[0])
    host = ep.encode(W, bpp, **kw)
    dev = ep.encode_device(torch.from_numpy(W).cuda(), bpp, **kw)
    assert np.array_equal(dev.data, host.data)
    assert dev.report["s"] == host.report["s"] and dev.report["b"] == host.report["b"]
    assert ep.validate(dev.data) == 0


def test_device_encoder_full_size_and_round_trip():
    W = synth.config2()
    Wd = torch.from_numpy(W).cuda()
    blob = ep.encode_device(Wd, 3.0)
    ref, rep = oracle.encode(W, 3.0)
    assert np.array_equal(blob.data, ref)
    out = ep.decode(ep.upload(blob), ep.BF16)
    torch.cuda.synchronize()
    e = oracle.rel_l2(W, out.float().cpu().numpy())
    assert 0.05 < e < 0.25 and abs(blob.stored_bpp - 3.0) < 0.03


def test_device_encoder_falls_back_cleanly_on_huge_coordinates():
    # one non-zero weight per row: the normalised value is sqrt(C) = 64, and with nothing else to code the search
    # runs to the fine end of its bracket (s = 1e-3), tens of thousands of lattice steps away from zero
    W = np.zeros((16, 4096), np.float32)
    W[np.arange(16), np.arange(16) * 5] = 1.0
    with pytest.raises(ep.EntroPackError) as ei:
        ep.encode_device(torch.from_numpy(W).cuda(), 8.0)
    assert ei.value.status == -3
    assert ep.validate(ep.encode(W, 8.0).data) == 0          # the host encoder still serves it


def test_device_encoder_leaves_the_per_row_refinement_to_the_host():
    W = synth.gaussian_rows(32, 512, 11)
    with pytest.raises(ep.EntroPackError) as ei:
        ep.encode_device(torch.from_numpy(W).cuda(), 4.0, rdo_candidates=3)
    assert ei.value.status == -3
