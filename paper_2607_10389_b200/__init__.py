"""B200 data path of an exact-state session mover: per-chunk CRC32C, dirty-chunk diff, lossless
WM1 encode and decode+verify, as CUDA kernels behind the C ABI of ``include/wm.h``."""
