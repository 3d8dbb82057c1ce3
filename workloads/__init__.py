"""Seeded synthetic inputs shaped like the retrieval workloads of RaLMSpec's evaluation.

This module only draws random inputs (corpora, queries, cache contents, speculated id
streams). It holds none of the retrieval arithmetic: no scoring, no top-k, no
verification. Both the CUDA library and the CPU oracle are fed the bytes produced here.

Everything is generated in chunks of at most `CHUNK_ROWS` rows; chunk b of a tensor with
seed S is drawn from a generator seeded with S * 1000003 + b, so any chunk can be
regenerated on its own. The same seed gives the same bytes on one device type; CPU and
CUDA generators are different streams (the recipe is the same).
"""
from .synth import (CHUNK_ROWS, CONFIGS, WorkloadConfig, unit_gaussian_corpus, mixture_corpus,
                    noisy_copy_queries, speculation_cache_ids, bernoulli_speculation,
                    integer_valued, seed_for)

__all__ = ["CHUNK_ROWS", "CONFIGS", "WorkloadConfig", "unit_gaussian_corpus", "mixture_corpus",
           "noisy_copy_queries", "speculation_cache_ids", "bernoulli_speculation",
           "integer_valued", "seed_for"]
