"""Integer-only Q-ASR encoder inference on B200 (sm_100a): Python binding of the C-ABI library.

The arithmetic runs entirely in the CUDA library ``libqasr.so`` (built in-tree by
``python -m paper_2103_16827_b200.build``); this package only marshals arguments.
Importing it without the built library raises ImportError -- there is no CPU fallback.
"""
from .binding import (NOALLOC_SCRATCH_BYTES, tcs_block_noalloc, Context, DeviceModel, QasrError, QasrLayer, QasrRequant, lib, lib_path,
                      OPT_GRAPH, OPT_TENSOR_CORES, OPT_PROFILE, OPT_STATIC_WEIGHTS, OPT_GEMM_FRAME_TILE,
                      OPT_DW_FRAME_TILE, OPT_SIDE_BRANCH, OPT_FRAME_MAJOR_OUTPUT, MAX_TERMS)

__all__ = ["NOALLOC_SCRATCH_BYTES", "tcs_block_noalloc", "Context", "DeviceModel", "QasrError", "QasrLayer", "QasrRequant", "lib", "lib_path",
           "OPT_GRAPH", "OPT_TENSOR_CORES", "OPT_PROFILE", "OPT_STATIC_WEIGHTS", "OPT_GEMM_FRAME_TILE", "OPT_DW_FRAME_TILE", "OPT_SIDE_BRANCH", "OPT_FRAME_MAJOR_OUTPUT", "MAX_TERMS"]
