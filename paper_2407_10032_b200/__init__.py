"""B200 (sm_100a) implementation of the LeanQuant per-linear-layer quantisation pass.

The product is the C-ABI library ``liblq.so`` (see ``include/lq.h``); this package is its
thin ctypes binding.  PyTorch is used for device memory and streams only."""
from .binding import (LQ, LQError, Config, lq_create, lq_destroy, lq_sync_status, lq_version, lq_launch_count,
                      lq_hessian_workspace, lq_hessian_accumulate, lq_hessian_finalize,
                      lq_prepare_hinv_workspace, lq_prepare_hinv, lq_fit_grid_workspace, lq_fit_grid, lq_fit_grid_noalloc,
                      lq_quantize_layer_workspace, lq_quantize_layer, lq_pack_codes, lq_chol_diag, lq_quantize_exact_workspace, lq_quantize_exact, lq_quantize_layer_lazy_workspace, lq_quantize_layer_lazy, lq_peak_probe,
                      lq_testing_set_wait_limit_ns, lq_testing_inject_stall,
                      lq_testing_set_prepare_defer_min_blocks, lq_testing_set_prepare_slices_int8, lq_pack_layer_bytes, lq_pack_layer, lq_unpack_layer,
                      lq_zero_dead_columns, lq_act_order, lq_permute_hessian, lq_gather_columns, lq_scatter_columns,
                      StackPass, LayerPass, library_path)

__all__ = [n for n in dir() if n.startswith("lq_")] + ["LQ", "LQError", "Config", "LayerPass", "StackPass", "library_path"]
