"""Plain statement of the paged KV swap: moving one request's pages between the pool and a
contiguous host image (paper Section 3, "Request Multiplexing with Mixed Instances": an evicted
batch request's KV cache is saved by migrating it to CPU memory for a fast restart).

TEST INFRASTRUCTURE ONLY.  numpy fancy indexing, nothing else; shares no code with the library.

Host image layout: bf16 [num_layers][n_pages][num_kv_heads][2][page_size][head_dim] -- for every
layer, the request's pages in block-table order.
"""
from __future__ import annotations

import numpy as np


def swap_out(pool6: np.ndarray, page_ids: np.ndarray) -> np.ndarray:
    """pool6: uint16 [layers][pages][Hkv][2][P][d]; returns the image [layers][n][Hkv][2][P][d]."""
    return np.ascontiguousarray(pool6[:, np.asarray(page_ids, dtype=np.int64)])


def swap_in(pool6: np.ndarray, page_ids: np.ndarray, image: np.ndarray) -> None:
    """Scatter the image back into (possibly different) physical pages, in place."""
    pool6[:, np.asarray(page_ids, dtype=np.int64)] = image
