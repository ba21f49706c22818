"""CMPQ quantization pass (arxiv 2410.13056) on one B200: CUDA library + thin Python binding.

`binding` mirrors the C ABI of include/cmpq.h one to one, `pipeline.LayerQuantizer` chains the
calls for one layer, `inputs` generates seeded synthetic layers, `build` compiles the library.
Nothing is loaded at import time; the first call into `binding` loads libcmpq.so and raises if
it has not been built.
"""
__all__ = ["binding", "pipeline", "inputs", "build"]
