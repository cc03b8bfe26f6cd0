"""B200 (sm_100a) library for the DAB-Net inference hot path: row binarization and packed-bit contraction.

The work is done by ``libdab.so`` (CUDA, C ABI declared in ``include/dab.h``); this package is its thin
Python binding.  Build the library in-tree with ``python -m paper_1804_02941_b200.build``.
"""
from .binding import (Coded, ConvDesc, ConvDetails, DabError, DAB_MAX_N, DAB_OK, EXPORTS, LIB_PATH, ROW_DEGENERATE,
                      ROW_NONFINITE, dab_binarize, dab_binarize_into, dab_sign_binarize, dab_sign_patches, dab_binarize_patches, dab_binary_conv_contract, dab_binary_conv, dab_binary_conv_host, dab_binary_conv_host_wait, dab_binary_conv_static, dab_binary_conv_static_capacity, dab_wbin_conv, dab_wbin_conv_workspace, dab_binarize_train, dab_binarize_backward, dab_set_patch_coder, dab_get_patch_coder, PATCHES_AUTO, PATCHES_SORT, PATCHES_HIST, PATCHES_PIXEL,
                      dab_binary_conv_host_workspace, dab_binary_conv_workspace, dab_binary_gemm, dab_conv_output_size,
                      dab_default_ld, dab_pack, dab_popc_probe, dab_set_contraction, dab_get_contraction,
                      dab_contraction_wait_failures, CONTRACT_AUTO, CONTRACT_TENSOR, CONTRACT_POPC, dab_words_per_row, lib, make_desc, status_string, guards_enable, guards_check, Network, Layer, dab_network_forward, dab_network_output_shape,
                      use_library, dab_debug_bounds_enabled, dab_debug_bounds_report)

__all__ = [n for n in dir() if not n.startswith("_")]
