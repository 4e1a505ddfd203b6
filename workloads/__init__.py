"""Seeded synthetic inputs: graphs, feature matrices and seed batches.

This package only *produces inputs* (CSR graphs, feature bits, seed lists).  It
contains none of the sampler's arithmetic (no Philox keys, no selection, no
relabelling) and is the one module that both the CPU oracle's tests and the
CUDA path's tests/benchmark are allowed to share.
"""
from .configs import CONFIGS, config_names, get_config  # noqa: F401
from .graphs import build_graph, Graph  # noqa: F401
from .features import build_features, feature_rows  # noqa: F401
from .seeds import seed_permutation, batch_seeds  # noqa: F401
