"""B200-native (sm_100a) hot path of PSD, Parallel Speculative Decoding for diffusion LLMs.

A thin ctypes binding over ``libpsd_b200.so`` (C ABI in ``include/psd.h``): the fused LM-head +
confidence kernel, the unmasking policy, draft construction and hierarchical acceptance.
Importing the package loads (and, if missing, builds with nvcc) the CUDA library; there is no
other implementation behind these names.
"""
from .binding import (ACCEPT_AGREE_AND_CONF, ACCEPT_AGREE_AND_POLICY, ACCEPT_AGREE_ONLY, LIB_PATH, PSD_ERR_ALIGN,
                      PSD_ERR_CUDA, PSD_ERR_NULL, PSD_ERR_POLICY, PSD_ERR_SHAPE, PSD_ERR_TIMEOUT, PSD_ERR_INTERNAL,
                      PSD_ERR_UNSUPPORTED, PSD_ERR_WORKSPACE, PSD_MAX_DEPTH, PSD_MAX_M, PSD_OK, PsdError,
                      PsdPolicy, PsdStepIO, StepBuffers, policy, psd_build_drafts, psd_confidence, psd_confidence_static, PSD_STATIC_SCRATCH_BYTES,
                      psd_launch_count, psd_confidence_kernel_name, psd_select_unmask, psd_set_confidence_impl, psd_set_kernel_events, psd_set_tuning, PSD_TUNE_BAND_BYTES, PSD_TUNE_PDL, PSD_TUNE_TILE_ORDER, PSD_TUNE_COMPACT_ROWS, PSD_TUNE_WAIT_LIMIT, PSD_TUNE_SELFTEST_STALL, psd_compact_workspace_bytes, psd_confidence_masked, psd_confidence_partial, psd_merge_partials, psd_compact_rows_enabled, psd_step, psd_step_host,
                      psd_step_host_bytes, psd_step_host_block, host_step_buffers, psd_verify_accept, psd_workspace_bytes, status_string, psd_decode_blocks, psd_decode_scratch_bytes,
                      table_body_address, table_body_user, psd_table_body, PsdDag, psd_dag_init,
                      psd_build_drafts_dag, psd_verify_accept_dag, psd_step_dag, PsdDecodeStats, PsdTableBody, ORDER_TWO_PASSES,
                      ORDER_ONE_PASS)

__all__ = [n for n in dir() if not n.startswith("_")]
