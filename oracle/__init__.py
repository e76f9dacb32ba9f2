"""CPU oracle of the MadaKV eviction pass: TEST INFRASTRUCTURE, not product code.

Only the tests, ``__graft_entry__.smoke()`` and the CPU-baseline / reference legs of ``bench.py`` may import this
package. It never imports the CUDA package and the CUDA package never imports it.
"""
from .pyoracle import (  # noqa: F401
    build,
    hardware_threads,
    score,
    allocate,
    select,
    compact,
    decode,
    topp_count_f64,
)
