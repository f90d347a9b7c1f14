"""fp64 CPU oracle for the gated delta-rule prefill — test infrastructure only.

Nothing in the product package may import this; only the tests, the smoke check
and the CPU-baseline leg of the benchmark do.
"""
from .gdn_oracle import (chunked, chunked_stages, dense, epilogue, num_threads, prologue, sequential)  # noqa: F401
from .attn_oracle import attention_causal, attention_causal_rows, attention_gemm_form  # noqa: F401
