"""B200 (sm_100a) implementation of the ExactOBS / OBQ layer solver of "Optimal Brain Compression".

The work is done by hand-written CUDA kernels behind a C ABI (include/obc.h, built into libobc.so next to
this file by `python -m paper_2208_11580_b200.build`); this package only marshals torch tensors into that
ABI.  There is no CPU or PyTorch fallback: calling any function without the built library raises.
"""
from .binding import (  # noqa: F401
    OBCError, library_path, load_library, obc_hessian, obc_cross_gram, obc_refit, obc_hessian_inverse, obc_minmax_grid, obc_prune_apply,
    obc_prune_trace, obc_prune_nm, obc_prune_blocks, obc_quantize, obc_select_global_mask, obc_select_global_mask_static, obc_status_string, obc_workspace_bytes, obc_kernel_launches,
    obc_engine_plan, EngineOpts, engine_opts, ENGINE_AUTO, ENGINE_STREAMING, ENGINE_BLOCKED, ENGINE_WHOLE_WAVES,
    OP_HESSIAN, OP_INVERSE, OP_PRUNE_TRACE, OP_SELECT, OP_PRUNE_APPLY, OP_QUANTIZE, OP_PRUNE_BLOCKS, OP_CROSS_GRAM, OP_REFIT,
    PREC_FP32, PREC_TF32, PREC_BF16X3, FLAG_OUTLIERS, EXPORTED_SYMBOLS,
)
