"""CoSA prefill hot path (KAP + OSK) for NVIDIA B200: C-ABI CUDA library and its binding."""
from .binding import (CosaError, CosaOptions, CosaShape, cosa_budget_count, cosa_debug_set_device_status, cosa_device_status,  # noqa: F401
                      cosa_host_call_workspace_bytes, cosa_kap_select, cosa_kap_select_static,
                      cosa_kap_select_static_max_bytes, cosa_lists_to_mask, cosa_osk_attention, cosa_prefill_host, cosa_reserve_scratch,
                      cosa_reorder_lists,
                      cosa_validate_order, cosa_version, cosa_workspace_bytes, default_options, library,
                      make_shape)
