"""CPU oracle for the ReST-KV eviction-scoring path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with, and never imports, the CUDA library or its binding.

`oracle.reference` wraps the plain-C fp64 implementation (`restkv_oracle.c`);
`oracle.bruteforce` holds the token-deletion definition (Eq. 6) in NumPy, used to pin it.
"""
from .reference import (  # noqa: F401
    build,
    score,
    select,
    compact,
    decode,
    num_threads,
    set_threads,
    ScoreResult,
)
