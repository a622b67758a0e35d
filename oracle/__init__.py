"""CPU oracle for the example-retrieval path.  Test infrastructure only.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library and its Python binding never do.
"""
from .ic_oracle import (  # noqa: F401
    build_oracle,
    bf16_bits_to_f32,
    f32_to_bf16_bits,
    search,
    self_similarity,
    kmeans_assign,
    kmeans_update,
    kmeans,
    search_clustered,
    utility_add,
    utility_decay,
)
from .check import accept, AcceptanceError  # noqa: F401
