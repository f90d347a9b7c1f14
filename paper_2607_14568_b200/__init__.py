"""B200-native chunked gated delta-rule prefill: Python binding of the C-ABI library.

The functions here only marshal arguments (pointers, sizes, the stream) into
``libgdn.so``; every step of the computation runs in the library's CUDA kernels.
There is no CPU fallback: importing works without the shared object (so that the
build step can run), but any call raises if it is missing.
"""
from .binding import (GdnError, gdn_chunk_prefill, gdn_chunk_prefill_bf16_simt,  # noqa: F401
                      gdn_chunk_prefill_f32, gdn_chunk_prefill_host, gdn_chunk_prefill_noalloc, gdn_attn_causal_prefill, gdn_chunk_prefill_raw, gdn_chunk_prefill_gated, gdn_chunk_prefill_snapshots, gdn_decode_step, gdn_host_staging_bytes,
                      gdn_launch_count, gdn_query_status, gdn_query_status_stream, gdn_set_workspace, gdn_status_string,
                      gdn_workspace_bytes, lib, lib_path)
