"""B200 (sm_100a) implementation of the HIGGS quantized linear layer.

The product is the CUDA shared library built from ``csrc/`` behind the C ABI of
``include/higgs.h``; this package is its ctypes binding.  Importing it fails
loudly when the library has not been built: there is no fallback path.
"""
from .binding import (  # noqa: F401
    HIGGS_BF16, HIGGS_ERR_CUDA, HIGGS_ERR_INVALID_ARG, HIGGS_ERR_TIMEOUT, HIGGS_ERR_UNSUPPORTED, HIGGS_ERR_WORKSPACE,
    HIGGS_F16, HIGGS_F32, HIGGS_OK, HIGGS_OP_LINEAR, HIGGS_OP_MAKE_GRID, HIGGS_OP_QUANTIZE, HiggsError, LIB_PATH,
    higgs_canonical_bytes, higgs_desc, higgs_linear, higgs_make_grid, higgs_pack_codes, higgs_packed_bytes,
    higgs_quantize, higgs_rht, higgs_scales_bytes, higgs_sign, higgs_unpack_codes, higgs_workspace_bytes, make_desc,
    status_string,
)
