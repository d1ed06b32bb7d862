"""Seeded synthetic corpora and queries (inputs only).

This package produces the arrays that both the CPU oracle and the CUDA
library consume.  It holds none of the retrieval method's arithmetic: no
scoring, no selection, no decoding.  It imports neither `oracle` nor the
CUDA package.
"""
from .corpus import (CONFIGS, CorpusConfig, Corpus, make_corpus, make_queries, doc_lengths,  # noqa: F401
                     random_rotation, encode_rabitq_1bit)
