"""The allocation-free entry point against the regular one and against the oracle.

ep_decode_tensor_static serves callers that cannot allocate device memory at decode time (they run under a
framework that owns the allocator and hands them only input and output buffers, or in a serving loop where
an allocation would stall the device): streams that need large lookup tables get them built in a fixed
area inside the library instead of in caller scratch.  Its output must equal ep_decode_tensor's and the CPU
oracle's bit for bit, also on a second call that reuses the area with different tables, and the call must leave
the amount of free device memory as it found it.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34185_b200 as ep
from paper_2609_34185_b200 import synth


def _static(d, dt, out):
    ep.decode_tensor_static(d.info, d.d_stream, d.d_tile_index, d.d_row_scales, dt, out.data_ptr(),
                            torch.cuda.current_stream().cuda_stream)
    return out


@pytest.mark.gpu
def test_static_area_decode_equals_scratch_decode_twice_in_a_row():
    Wa = synth.laplace_rows(96, 1024, 301)
    Wb = synth.student_t_rows(64, 2048, 302)
    a = ep.encode(Wa, 4.0, b_start=12, tile_vectors=200)      # tables of 2^12 slots: need scratch
    b = ep.encode(Wb, 5.0, b_start=13)                        # the largest precision the area holds
    small = ep.encode(Wa, 4.0)                                # tables fit shared memory: no scratch at all
    assert ep.decode_scratch_bytes(a.info) > 0 and ep.decode_scratch_bytes(b.info) > 0
    assert ep.decode_scratch_bytes(small.info) == 0
    for dt, tdt, odt in ((ep.BF16, torch.bfloat16, oracle.BF16), (ep.INT8, torch.int8, oracle.INT8)):
        for blob in (a, b, a, small):                          # back to back, the area is reused and overwritten
            d = ep.upload(blob, prepare=False)
            ref = ep.decode(d, dt)                             # existing entry point, scratch from the caller
            out = torch.empty((blob.info.R, blob.info.C), dtype=tdt, device="cuda")
            _static(d, dt, out)                                # first use: looks up the area's address
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            got = _static(d, dt, out)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before  # the call took no device memory
            assert torch.equal(got.view(torch.uint8), ref.view(torch.uint8))
            want, _ = oracle.decode(blob.data, odt)             # and the independent CPU decoder agrees
            assert np.array_equal(got.view(torch.uint8).cpu().numpy().reshape(-1), want.reshape(-1).view(np.uint8))
    assert ep.last_device_status() == 0


@pytest.mark.gpu
def test_static_area_refuses_tables_it_cannot_hold():
    W = synth.gaussian_rows(32, 512, 303)
    big = ep.encode(W, 4.0, b_start=14)
    d = ep.upload(big, prepare=False)
    out = torch.empty((32, 512), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ep.EntroPackError) as ei:
        _static(d, ep.BF16, out)
    assert ei.value.status == -8 and "EP_STATIC_MAX_B" in str(ei.value)
    ref = ep.decode(d, ep.BF16)                                # the regular call with scratch still serves it
    torch.cuda.synchronize()
    assert ref.shape == (32, 512)
