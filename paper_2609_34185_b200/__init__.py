"""B200-native EntroPack codec: host encoder + fused sm_100a rANS/E8 weight decoder.

The product is the C-ABI library declared in ``include/entropack.h``; this package is a thin
ctypes binding with the same names.  PyTorch appears only as the owner of device memory and
streams.
"""
from .binding import (  # noqa: F401
    BF16, FP16, FP8_E4M3, INT8, FP32, FP8_E5M2, UINT8, FIELDS_I32, DTYPE_BYTES, EncodeOpts, EncodeReport, Info, DecodeJob, Blob,
    EntroPackError, load, encode, encode_device, pack_fields, blob_info, validate, decode_scratch_bytes, decode_tables_bytes, prepare_tables, decode_tiles_per_sm, decode_tensor,
    decode_tiles, decode_tile_range, decode_tensor_static, decode_gemm, decode_matmul, decode_batch, last_device_status, default_tile_vectors, suggest_tile_vectors, suggest_tile_vectors_batch, strerror, DeviceBlob, upload, decode, decode_many,
)
