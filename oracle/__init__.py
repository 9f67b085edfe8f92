"""CPU oracle for layerwise QK-RMSNorm.  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's CPU-baseline legs may
import this package.  It imports nothing from the CUDA package and the CUDA
package imports nothing from here.
"""
from .qknorm_oracle import (  # noqa: F401
    build,
    rmsnorm,
    rmsnorm_sharded,
    bf16_to_f64,
    f64_to_bf16,
    max_threads,
    e4m3_to_f64,
    f64_to_e4m3,
    rmsnorm_e4m3,
    rmsnorm_headwise,
)
