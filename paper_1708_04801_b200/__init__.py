"""B200 (sm_100a) hot path of weighted parallel SGD (WP-SGD): thin Python binding of libwpsgd.so.

Every step of the path (sample stream, per-node SGD chains, weighted combination) runs in the
library's CUDA kernels; this package only marshals arguments. PyTorch supplies device memory
and streams. There is no CPU fallback: importing works without the built library (so that the
build step itself can import the package), but any call raises if it is missing.
"""
from .binding import (  # noqa: F401
    LOSS_HINGE, LOSS_LOGISTIC, LOSS_SQUARED, LR_CONST, LR_INV_SQRT, X_BF16, X_F32, WpsgdError, Context,
    library_path, load_library, weights, solve_static, span_valid, sample_indices_host, check_static, EXPORTED_SYMBOLS,
)
