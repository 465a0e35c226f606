"""Seeded synthetic inputs for the Kangaroo decode step: model shapes, weights, prompts.

This package is the one piece both the CUDA product path's tests and the CPU oracle may
use.  It holds no arithmetic of the method itself (no norms, attention, softmax, accept
rule): only a counter-based pseudo-random generator, the five workload shapes, and the
tensor naming that says which counter stream fills which tensor.

The CUDA library carries its own implementation of the same generator so that a 66 GB
model never has to cross PCIe; `tests/test_gpu_parity.py::test_device_weights_equal_host_generator`
checks the two bit for bit.
"""
from .synth import (  # noqa: F401
    splitmix64,
    stream_base,
    gauss_ints,
    gauss_f32,
    round_to_bf16_f32,
    uniform_tokens,
    fill_f32,
    TensorId,
    GAUSS_INT_STD,
)
from .configs import (KgShape, CONFIGS, get_config, make_weights, LazyWeights, make_prompt, param_counts,  # noqa: F401
                      microbench_state)
