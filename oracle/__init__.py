"""CPU oracle (test infrastructure only): fp64 definition of the attention the GPU path computes.

Only the tests, the smoke check and the benchmark's CPU-baseline / reference legs may import this
package; the product package never does.
"""
from .cpu_oracle import (  # noqa: F401
    attention,
    attention_batch,
    build,
    merge_lse,
    softmax_weights,
    xtensor_locate,
)
from .xtensor_model import PagePoolModel  # noqa: F401
