"""CPU oracle of the MAGE per-block attention path.  TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / reference
legs of ``bench.py`` may import this package.  It shares no code with the CUDA
library and never imports it.
"""
from .oracle import (build, exact_block_attn, block_score, topk, sparse_block_attn, recall,  # noqa: F401
                     num_threads, run_block, quest_page_summaries, quest_page_scores, quest_select,
                     e4m3_round, k8_scale, k8_codes, k8_quantize_block, k8_exact_block_attn, k8_block_score,
                     k8_sparse_block_attn, E4M3_MAX)
