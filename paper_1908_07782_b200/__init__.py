"""Segmented-gossip synchronization round on one B200: Python front of the
C-ABI library ``libcombo_b200.so`` (hand-written sm_100a kernels)."""
from .binding import (ComboError, combo_aggregation_divergence, combo_aggregation_divergence_noalloc,
                      combo_divergence_scratch_bytes, PATH_AUTO, PATH_DIRECT, PATH_STAGED, PATH_TILE, PATH_DIRECT_NAIVE, combo_device_status,  # noqa: F401
                      combo_last_kernel_path, combo_round_host, combo_segment_aggregate,
                      combo_segment_aggregate_bf16, combo_segment_aggregate_cols,
                      combo_segment_aggregate_members, combo_segment_aggregate_rows, combo_check_rows,
                      combo_segment_aggregate_sgd, combo_select_peers,
                      combo_select_peers_online,
                      combo_select_peers_default_stream, combo_set_kernel_path, combo_set_launch_overlap,
                      combo_set_tuning,
                      combo_validate_idx, combo_version, load, combo_max_launch_columns,
                      combo_set_launch_columns, combo_debug_dead_wait)
