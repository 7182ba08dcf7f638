"""B200-native best-matching-unit search for sparse binary corpora.

The product is the C-ABI CUDA library `libbmu.so` (include/bmu.h, csrc/); this
package is its thin Python binding.  Nothing here computes on the CPU.
"""
from .binding import (BmuError, Opts, bmu_codebook_norms, bmu_codebook_norms_f16,
                      bmu_search_f16_ws, bmu_release_scratch, bmu_search,
                      bmu_search_batches_host, bmu_search_host, bmu_selftest_wait_timeout, bmu_search_static, bmu_search_top2_ws,
                      bmu_search_workspace_bytes, bmu_search_ws,
                      bmu_measure_roof, bmu_validate_csr, bmu_version, load,
                      bmu_update_scatter, bmu_update_blur, bmu_update_writeback,
                      bmu_map_errors, Plan, SearchDesc, bmu_describe_search,
                      bmu_kernel_launches, bmu_last_status, bmu_score_block_argmin)

__all__ = ["BmuError", "Opts", "bmu_codebook_norms", "bmu_codebook_norms_f16",
           "bmu_search_f16_ws", "bmu_release_scratch", "bmu_search",
           "bmu_search_batches_host", "bmu_search_host", "bmu_selftest_wait_timeout", "bmu_search_static", "bmu_search_top2_ws",
           "bmu_search_workspace_bytes", "bmu_search_ws",
           "bmu_measure_roof", "bmu_validate_csr", "bmu_version", "load",
           "bmu_update_scatter", "bmu_update_blur", "bmu_update_writeback", "bmu_map_errors",
           "Plan", "SearchDesc", "bmu_describe_search", "bmu_kernel_launches", "bmu_last_status",
           "bmu_score_block_argmin"]
