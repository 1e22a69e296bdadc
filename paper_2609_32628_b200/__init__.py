"""da2: DraftAttention2's attention hot path for NVIDIA B200, hand-written sm_100a CUDA behind a C ABI.

This package is a thin ctypes binding over ``libda2.so`` (built in-tree from ``csrc/`` by ``build.py``).
Every step of the path runs in the library's kernels; Python only marshals arguments.  There is no CPU
fallback: importing works without a GPU (so the library can be built and its symbols checked), but any
compute call requires the CUDA library and a device.
"""
from .binding import (Da2Error, Plan, PlanInfo, STATUS, load_library, da2_plan, da2_plan_info, da2_plan_slot_token, da2_prepare, da2_refresh_operands, da2_prepare_cached_scales,
                      da2_attention_fwd, da2_device_status, da2_plan_destroy, da2_status_string,
                      da2_last_launch_count, da2_probe_bounded_wait, da2_attention_host, da2_attention_host_arena_bytes, make_config, da2_tcgen05_peak, da2_selfcheck_quantiser_arithmetic, da2_draft_map_noalloc, attention, HostPipeline)

__all__ = ["Da2Error", "Plan", "PlanInfo", "STATUS", "load_library", "da2_plan", "da2_plan_info", "da2_plan_slot_token", "da2_prepare", "da2_refresh_operands", "da2_prepare_cached_scales",
           "da2_attention_fwd", "da2_device_status", "da2_plan_destroy", "da2_status_string",
           "da2_last_launch_count", "da2_probe_bounded_wait", "da2_attention_host", "da2_attention_host_arena_bytes", "make_config", "da2_tcgen05_peak", "da2_selfcheck_quantiser_arithmetic", "da2_draft_map_noalloc", "attention", "HostPipeline"]
