"""CPU oracle of the Crystal-KV decode path: TEST INFRASTRUCTURE only.

Only tests, the smoke check and the bench's cpu-baseline leg may import this package.
The product path (the CUDA library and its binding) never does.
"""
from .oracle import Oracle, OracleConfig, attention, hit_mask, alg2  # noqa: F401
