"""TreeKV oracle: test infrastructure only.

A slow fp64 CPU statement of TreeKV (arXiv 2501.04987, Section 3.1 and
Algorithm 1) used to check the CUDA library.  Only the tests, the smoke check
and the CPU-baseline leg of the benchmark import this package; the product
never does, and this package never imports the product.
"""
from .treekv_oracle import Oracle, build_oracle, RULE_SCORES, RULE_KEEP_LEFT, RULE_EVICT_LEFT, RULE_ACCUMULATED, IDX_CYCLE, IDX_LITERAL

__all__ = ["Oracle", "build_oracle", "RULE_SCORES", "RULE_KEEP_LEFT", "RULE_EVICT_LEFT", "RULE_ACCUMULATED", "IDX_CYCLE", "IDX_LITERAL"]
