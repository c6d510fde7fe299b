"""B200-native FlashDiffusion hot path: matrix-free Gaussian-kernel block product, degree
passes, block eigensolver, bandwidth flow and out-of-sample extension behind a C ABI
(include/fd.h, built into libfd.so from csrc/), with a thin ctypes binding."""
from .binding import (  # noqa: F401
    Context, FdError, fd_workspace_bytes, fd_apply_general_static, fd_unit_peaks, FD_STATIC_MAX_N, FD_STATIC_MAX_D, FD_STATIC_MAX_B, fd_launch_count, fd_version, to_colmajor, lib, LIB_PATH, EXPORTS,
    FD_OK, FD_ERR_INVALID, FD_ERR_WORKSPACE, FD_ERR_CUDA, FD_ERR_NOT_CONVERGED, FD_ERR_PERRON_WALL,
    FD_ERR_UNSUPPORTED, FD_ERR_TIMEOUT, FD_ERR_NONFINITE, FD_ERR_COMM, FD_PREC_FP32, FD_PREC_FAST,
    FD_PATH_AUTO, FD_PATH_SIMT, FD_PATH_TC,
)
from .shard import Shard, TorchDistTransport, ThreadTransport, fd_shard_rows, fd_shard_exchange_bytes  # noqa: F401,E402
