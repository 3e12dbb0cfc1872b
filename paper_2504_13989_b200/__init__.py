"""B200 (sm_100a) rotate-and-quantize library for arXiv 2504.13989: Python binding of the C ABI.

`binding` loads libgbs.so lazily, on first use; `synth` generates the seeded synthetic inputs.
"""
from . import binding  # noqa: F401
from .binding import (GbsError, HostPipeline, Plan, gbs_clip_error, gbs_dequantize, gbs_hadamard_m,  # noqa: F401
                      gbs_plan_create, gbs_plan_create_ex, gbs_plan_destroy, gbs_plan_device_status, gbs_plan_info,
                      gbs_rotate_quantize, gbs_rotate_quantize_static, gbs_search_clip_ratio)
