"""GPU parity of the decode fused into a matrix product (ep_decode_gemm) against the oracle: the weights are the
oracle's BF16 decode of the same stream, the product is taken in float64 on the host.

Tolerance.  The kernel multiplies BF16 by BF16 (exact in fp32) and accumulates in fp32 in an order the hardware
chooses, so |y - y_ref| <= n * 2^-24 * sum_k |x_k w_k| for n additions in the worst case; with random rounding
errors it stays near sqrt(n) * 2^-24 of that sum.  The bound asserted is 2e-5 * sum_k |x_k w_k| (n <= 8192 columns
here: worst case 4.9e-4, expected 5e-6) - an operand in the wrong place of a tile changes y by the order of the sum
itself."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34185_b200 as ep
from paper_2609_34185_b200 import synth

pytestmark = pytest.mark.gpu


def _oracle_weights(blob_bytes):
    bits, _ = oracle.decode(blob_bytes, oracle.BF16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _check(blob, T, seed):
    I = blob.info
    rng = np.random.default_rng(seed)
    x = torch.from_numpy(rng.standard_normal((T, I.C)).astype(np.float32) * 0.5).to(torch.bfloat16)
    d = ep.upload(blob)
    y = ep.decode_matmul(d, x.cuda())
    torch.cuda.synchronize()
    assert ep.last_device_status() == 0
    W = _oracle_weights(blob.data)
    xd = x.double().numpy()
    ref = xd @ W.T
    bound = np.abs(xd) @ np.abs(W).T
    err = np.abs(y.double().cpu().numpy() - ref)
    assert np.all(err <= 2e-5 * bound + 1e-30), float((err / (bound + 1e-30)).max())
    return y


@pytest.mark.parametrize("R,C,T,bpp", [
    (32, 1024, 1, 5.0),       # one block of rows, one token
    (64, 2048, 16, 4.0),      # 16 staged rows of x
    (96, 2304, 17, 4.0),      # 32 staged rows, 15 of them padding
    (320, 3840, 32, 4.0),     # more blocks of rows than one round of a small grid; the layer's width
    (64, 8192, 5, 3.0),
])
def test_decode_matmul_against_the_oracle(R, C, T, bpp):
    W = synth.laplace_rows(R, C, 7000 + R + C)
    blob = ep.encode(W, bpp, tile_vectors=C // 8)
    assert blob.info.b == 11 and blob.info.V == C // 8 and blob.info.n_tiles == R
    _check(blob, T, R + T)


def test_decode_matmul_small_and_ragged_shapes():
    # hand-packed streams (b = 11, one tile per row): fewer rows than one step of a CTA, a single group per row, row
    # counts that leave the last step of a CTA ragged, more CTAs' worth of rows than SMs * 31
    rng = np.random.default_rng(74)
    for R, C, T in ((1, 256, 1), (5, 256, 32), (33, 512, 16), (157, 768, 3), (148 * 31 + 7, 256, 9)):
        n = R * C // 8
        fields = np.zeros((n, 9), np.int32)
        fields[:, 0] = rng.integers(0, 2, n)
        fields[:, 1:8] = np.rint(rng.standard_normal((n, 7)) * 6).astype(np.int32)
        fields[:, 8] = np.rint(rng.standard_normal(n) * 3).astype(np.int32)
        blob = ep.pack_fields(fields, R, C, 11, C // 8, rng.uniform(0.01, 0.05, R).astype(np.float32))
        assert blob.info.n_tiles == R
        _check(blob, T, R + C + T)


def test_decode_matmul_random_shapes():
    # 24 seeded random cases: rows 1 .. 700, 1 .. 12 groups per row, 1 .. 32 tokens, encoder-made streams (row scales,
    # tables and payload as the encoder leaves them) at 3 .. 6 bpp
    rng = np.random.default_rng(75)
    for case in range(24):
        R = int(rng.integers(1, 700))
        C = 256 * int(rng.integers(1, 13))
        T = int(rng.integers(1, 33))
        bpp = float(rng.choice([3.0, 4.0, 5.0, 6.0]))
        W = (synth.laplace_rows if case % 2 else synth.gaussian_rows)(R, C, 7600 + case)
        blob = ep.encode(W, bpp, tile_vectors=C // 8, b_start=11, b_max=11)
        assert blob.info.b == 11 and blob.info.n_tiles == R
        if ep.decode_scratch_bytes(blob.info):        # (a coordinate range beyond the shared-memory tables: not this path)
            continue
        _check(blob, T, 7700 + case)


def test_decode_matmul_more_tokens_than_one_launch_and_repeated_calls():
    W = synth.gaussian_rows(128, 1536, 71)
    blob = ep.encode(W, 4.0, tile_vectors=1536 // 8)
    y1 = _check(blob, 70, 1)              # 32 + 32 + 6 tokens
    y2 = _check(blob, 70, 1)
    assert torch.equal(y1, y2)


def test_decode_matmul_full_layer():
    # the 10240 x 3840 layer of the paper's reconstruction-cost experiment at 4 bpp, 32 tokens
    W = torch.from_numpy(synth.gaussian_rows(10240, 3840, 72)).cuda()
    blob = ep.encode_device(W, 4.0, tile_vectors=3840 // 8)
    assert blob.info.b == 11 and abs(blob.stored_bpp - 4.0) < 0.04
    _check(blob, 32, 2)


def test_decode_matmul_refuses_what_it_cannot_serve():
    W = synth.gaussian_rows(64, 2048, 73)
    d = ep.upload(ep.encode(W, 4.0, tile_vectors=100))               # not one tile per row
    x = torch.zeros((4, 2048), dtype=torch.bfloat16, device="cuda")
    y = torch.empty((4, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(ep.EntroPackError) as e:
        ep.decode_gemm(d.info, d.d_stream, d.d_tile_index, d.d_row_scales, d.tables.data_ptr(), x.data_ptr(), 4, y.data_ptr())
    assert e.value.status == -3
    d = ep.upload(ep.encode(W, 4.0, tile_vectors=256))
    x = torch.zeros((33, 2048), dtype=torch.bfloat16, device="cuda")
    y = torch.empty((33, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(ep.EntroPackError) as e:                       # more than 32 tokens in one launch
        ep.decode_gemm(d.info, d.d_stream, d.d_tile_index, d.d_row_scales, d.tables.data_ptr(), x.data_ptr(), 33, y.data_ptr())
    assert e.value.status == -3
    with pytest.raises(ep.EntroPackError):                            # misaligned x
        ep.decode_gemm(d.info, d.d_stream, d.d_tile_index, d.d_row_scales, d.tables.data_ptr(), x.data_ptr() + 2, 4, y.data_ptr())
    d8 = ep.upload(ep.encode(W, 8.0, tile_vectors=256))               # 2^12-slot stream
    with pytest.raises(ep.EntroPackError) as e:
        ep.decode_gemm(d8.info, d8.d_stream, d8.d_tile_index, d8.d_row_scales, d8.tables.data_ptr(), x.data_ptr(), 4, y.data_ptr())
    assert e.value.status == -3
    assert ep.last_device_status() == 0
