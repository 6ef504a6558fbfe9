"""Seeded synthetic inputs for the DISC + PPV hot path.

This package only PRODUCES inputs (constraint sets, query contexts, prefixes,
stand-in language-model weights and logits).  It contains none of the method's
arithmetic: no masks, no log-softmax, no sampling, no resampling.  Both the CPU
oracle's tests and the CUDA path's tests/bench draw their inputs from here.
"""
from .gen import (CONFIGS, Workload, scaled, make_set, make_contexts,
                  make_prefixes, make_lm_weights, BASE_SEED)

__all__ = ["CONFIGS", "Workload", "scaled", "make_set", "make_contexts",
           "make_prefixes", "make_lm_weights", "BASE_SEED"]
