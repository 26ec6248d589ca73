"""KV-cache compression event of the alpha retainer (score -> greedy set-conditioned
selection -> in-place compaction) as hand-written CUDA for sm_100a behind a C ABI.

``api`` holds the Python binding (same names as the C entry points); ``synth`` the
seeded input generators; ``build`` compiles the library in-tree. The binding needs the
compiled library and a CUDA device; nothing here falls back to the CPU.
"""
from .api import (AkvError, Layout, Options, Selection, alpha_compress_event, alpha_compress_event_static, alpha_score, alpha_select,  # noqa: F401
                  alpha_gram_shared, alpha_signature_flat, alpha_signature_layer, kv_compact, launch_count, load_library, to_device,
                  to_host_bits, workspace_bytes, FLAG_FORCE_GREEDY, GQA_MAX, GQA_MEAN, FLAG_NO_CHAIN, FLAG_NO_PRUNE, FLAG_TEST_STARVE_WAIT, SIG_FLAT,
                  SIG_PER_HEAD, SIG_PER_LAYER)
