"""flexq for B200: Python binding of the C-ABI CUDA library (see include/flexq.h).

Importing the package does not load the library; the first call does, and fails loudly
if libflexq.so has not been built (there is no CPU or PyTorch fallback).
"""
from .flexq import (FQ_FMT_PACKED, FQ_FMT_PLANES, FQ_MAX_BATCH, FlexQ, FlexQError, lib, lib_path,
                    fq_store_bytes, fq_code_bytes, fq_meta_bytes, fq_quantize_layer, fq_strerror, fq_search_chain, fq_prune_chain, fq_sqdiff)

__all__ = ["FQ_FMT_PACKED", "FQ_FMT_PLANES", "FQ_MAX_BATCH", "FlexQ", "FlexQError", "lib", "lib_path",
           "fq_store_bytes", "fq_code_bytes", "fq_meta_bytes", "fq_quantize_layer", "fq_strerror", "fq_search_chain", "fq_prune_chain", "fq_sqdiff"]
