"""CPU oracle of the R-KV compression step.  Test infrastructure only: nothing in
the product package imports it, and it imports nothing from the product."""
from .rkv_oracle import (build, oracle_head, oracle_batch, oracle_gather, oracle_append, oracle_push_query,  # noqa: F401
                         oracle_decode_attention, e4m3_to_f32,
                         HeadResult, BatchResult)
