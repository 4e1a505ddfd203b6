"""Small helpers shared by the tests (no sampler arithmetic)."""
import json
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def golden_json(name):
    with open(os.path.join(GOLDEN, name)) as fh:
        return json.load(fh)


def csr_from_rows(rows):
    indptr = np.zeros(len(rows) + 1, dtype=np.int64)
    for v, r in enumerate(rows):
        indptr[v + 1] = indptr[v] + len(r)
    indices = np.array([u for r in rows for u in r], dtype=np.int32)
    return indptr, indices


def star_graph(d, extra=0):
    """Node 0 has in-neighbours 1..d; all other rows are empty."""
    rows = [list(range(1, d + 1))] + [[] for _ in range(d + extra)]
    return csr_from_rows(rows)
