"""B200-native (sm_100a) tensor work of a DNN-cascade pipeline stage: batched letterbox,
detector-head decode + class-aware NMS, batch assembly and ROI crop-resize, behind a C ABI
(include/octo.h).  This package is the thin Python binding; all computation runs in the CUDA
kernels of liboctostage.so."""
from .binding import (  # noqa: F401
    DET_DTYPE, ITEM_DTYPE, EXPORTS, LIB_PATH, OctoError, Queue, QITEM_DTYPE, Stage, StageConfig, dets_to_numpy,
    load_library, make_config, octo_crop_batch, octo_postprocess_batch, octo_preprocess_batch,
    octo_stage_create, octo_stage_destroy, octo_postprocess_frame_static, octo_stage_get_stats, octo_stage_status,
    octo_coral_schedule, octo_static_status,
)
