"""Seeded synthetic inputs for Superposed Decoding experiments.

This package only *generates data*: model weights, token streams, prefixes and
n-gram frequency tables (unique n-gram -> count, the store of Section 4 of the
paper).  It contains none of the decoding method's arithmetic, so that the CPU
oracle and the CUDA path can both consume what it emits without sharing code.
"""
from .rng import splitmix64_scalar, hash_u64, uniform01
from .model import ModelShape, SHAPES, make_weights
from .text import zipf_cdf, zipf_tokens, make_prefix, count_ngrams, make_ngram_tables
from .workloads import Workload, WORKLOADS, get_workload

__all__ = [
    "splitmix64_scalar", "hash_u64", "uniform01",
    "ModelShape", "SHAPES", "make_weights",
    "zipf_cdf", "zipf_tokens", "make_prefix", "count_ngrams", "make_ngram_tables",
    "Workload", "WORKLOADS", "get_workload",
]
