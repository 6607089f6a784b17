"""CPU oracle of the LVSpec verify step (test infrastructure, fp64, plain C)."""
from .oracle import (build, verify_attention, loose_accept, n_loose, set_threads,
                     max_threads, visual_relevance, emit, select_branch,
                     verify_attention_fp8, e4m3_decode)

__all__ = ["build", "verify_attention", "loose_accept", "n_loose", "set_threads",
           "max_threads", "visual_relevance", "emit", "select_branch",
           "verify_attention_fp8", "e4m3_decode"]
