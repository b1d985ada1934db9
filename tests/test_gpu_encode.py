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


def test_device_encoder_blobs_keep_their_bytes_while_buffers_are_reused():
    # finished blobs live in page-locked memory and a freed blob's buffer serves a later encode: a blob that is
    # still alive must never be overwritten, a reused buffer must give the same bytes as a fresh one
    import gc
    Wa, Wb = synth.gaussian_rows(256, 1024, 71), synth.laplace_rows(192, 2048, 72)
    da, db = torch.from_numpy(Wa).cuda(), torch.from_numpy(Wb).cuda()
    ref_a, ref_b = ep.encode(Wa, 4.0).data.copy(), ep.encode(Wb, 3.0).data.copy()
    a1 = ep.encode_device(da, 4.0)
    b1 = ep.encode_device(db, 3.0)                 # a1 alive: must come from another buffer
    assert np.array_equal(a1.data, ref_a) and np.array_equal(b1.data, ref_b)
    view = a1.data[100:200]
    keep = view.copy()
    del a1
    gc.collect()                                   # `view` still holds the buffer
    b2 = ep.encode_device(db, 3.0)
    assert np.array_equal(view, keep) and np.array_equal(b2.data, ref_b)
    del view, b1, b2
    gc.collect()
    for _ in range(3):                             # now buffers come back from the spare slot
        a = ep.encode_device(da, 4.0)
        assert np.array_equal(a.data, ref_a)
        del a
        gc.collect()
        b = ep.encode_device(db, 3.0)
        assert np.array_equal(b.data, ref_b)
        del b
        gc.collect()
