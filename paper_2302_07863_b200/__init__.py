"""libbild: the Big Little Decoder decode loop as hand-written CUDA for sm_100a behind a
C ABI (include/bild.h), with a thin ctypes binding."""
from .binding import (  # noqa: F401
    BF16, FP32, MODE_BILD, MODE_LARGE_ONLY, MODE_SMALL_ONLY, BildError, Config, Context, lib,
    model_cfg, op_linear, op_lm_head, upload_model,
)
