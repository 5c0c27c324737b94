"""B200-native boundary-tensor codec (AccEPT bit-level compression, Sec. 3.3-3.4).

The product is the C-ABI shared library declared in ``include/accept.h``; this package holds its
CUDA sources (``csrc/``), the in-tree build step and a ctypes binding with the same names.
"""
from .binding import (  # noqa: F401
    DEV_BAD_HEADER, DEV_COPY_TIMEOUT, DEV_NONFINITE, LAYOUT_BITPLANE, LAYOUT_INTERLEAVED, RANGE_ABSMAX, RANGE_MINMAX,
    ROUND_NEAREST, ROUND_STOCHASTIC, AcceptError, MbqParams, Params, accept_bitwidth_schedule, accept_check_params,
    accept_bounds_check_report, accept_compress, accept_compress_host, accept_compress_static, accept_compressed_size, accept_decompress, accept_decompress_host,
    accept_last_device_status, accept_launch_count, accept_launch_null, accept_parse_header, accept_payload_offset,
    accept_workspace_size, new_stream_buffer, new_workspace, accept_mbq_check_params, accept_mbq_compress,
    accept_mbq_compressed_size, accept_mbq_decompress, accept_mbq_payload_offset, accept_mbq_workspace_size,
)
