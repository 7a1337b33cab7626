"""CPU oracle of the session mover's data path (checksum, dirty diff, encode, decode+verify).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg
are the only callers.  It is plain C (``wm_oracle.c``) compiled with gcc and reached through
ctypes with numpy arrays; nothing here imports or links the CUDA library, and the CUDA
library never reaches this package.
"""
from .wm_oracle import (  # noqa: F401
    Result,
    build,
    checksum,
    checksum_poly,
    checksum_xxh64,
    crc32c,
    crc_bitwise,
    crc_combine,
    decode_verify,
    decode_verify_leaves,
    decode_verify_strict,
    dirty_diff,
    encode,
    encode_leaves,
    flatten_leaves,
    hw_crc_library,
    meta_end,
    num_chunks,
    num_tiles,
    wire_bound,
    xxh64,
    STATUS,
)
