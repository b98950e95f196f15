"""Plain CPU oracle for the NVFP4 MoE rollout forward and the trainer-side
weight fake-quant.  TEST INFRASTRUCTURE ONLY: imported by the tests, by the
smoke check and by the benchmark's CPU-baseline leg, never by the product.
It shares no code with the CUDA path."""
from . import formats, nvfp4, rac, moe  # noqa: F401
