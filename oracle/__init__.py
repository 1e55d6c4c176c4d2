"""CPU oracle of the selection-resolution path — TEST INFRASTRUCTURE ONLY.

Only `tests/`, the smoke check and the benchmark's CPU-baseline / reference leg may import this
package.  It shares no code with the CUDA library and never imports it.
`oracle.attention_oracle` is the plain definition of what the sparse-attention consumer of the slot table computes.
"""
from .oracle import Oracle, build, STATUS_OUT_OF_RANGE, STATUS_DUPLICATE, FLAG_NO_BYTES, kv_footprint_bytes, POLICY_LRU, POLICY_FIFO, POLICY_RANDOM  # noqa: F401
