"""CPU oracle (test infrastructure only).

Plain, slow definition of what a cascade stage computes around its model: letterbox,
head decode + class-aware NMS, batch assembly and ROI crop-resize.  The arithmetic lives in
octo_oracle.c; this module only marshals numpy arrays into it.  It must not be imported by
the CUDA package, and it imports nothing from it.
"""
from .oracle import (  # noqa: F401
    DET_DTYPE, build, letterbox_geometry, resize_f64, f64_to_half, letterbox, sigmoid,
    decode, sort_candidates, iou, nms, scale_back, postprocess_image, postprocess_region, crop_rect, crop,
    assemble, StageResult, run_stage, margin_report,
)
from .queue import OracleQueue  # noqa: F401,E402
from . import coral  # noqa: F401,E402
