"""CPU oracle for batch LoRA inference -- TEST INFRASTRUCTURE, not product code.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It shares nothing with the CUDA library: the arithmetic lives in
``lora_oracle.c`` (plain per-token fp64 loops, paper Section 3.4 / 4.3) and is
reached through ctypes; this file only marshals numpy arrays.

Build the shared object with ``python -m oracle.build`` (gcc, ``-O2 -fopenmp``).
"""
from .api import (  # noqa: F401
    AdapterSet,
    lora_linear,
    lora_projection,
    segments,
    groups,
    lib_path,
    num_threads,
)
