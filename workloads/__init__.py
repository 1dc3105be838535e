"""Seeded synthetic inputs (model shapes, weights, token ids) shared by the CPU
oracle's tests and the CUDA library's tests.  Holds no arithmetic of the
decoding method itself: only shapes, random draws and the one-off rounding of
weights to their storage type."""
from .gen import (  # noqa: F401
    MODEL_SHAPES, WORKLOADS, ModelShape, Workload, bf16_round_bits, bf16_bits_to_f32,
    gen_model, gen_ids, gen_uniforms, tensor_names,
)
