"""Access contiguity of a decode step's gather list (the quantity behind the paper's comparison of placements,
arXiv 2511.07427 Section 5.1 and its evaluation of continuous access lengths): how many rows the attention kernel reads
per contiguous stretch of the page pool."""
from __future__ import annotations

import numpy as np


def mean_contiguous_rows(n_entries: np.ndarray, entries: np.ndarray) -> float:
    """n_entries [U], entries [U, W, 2] as returned by DynaKV.get_work_list().  The store is made of 32-row pages and a
    cluster's last page is usually part-filled, so a stretch is a run of CONSECUTIVE PAGES of the pool: per unit the
    runs are sorted by their first row, and a run on the page right after the previous run's page continues the
    stretch.  Returns rows read / number of stretches, over all units."""
    rows_total, stretches = 0, 0
    for u in range(len(n_entries)):
        e = entries[u, : n_entries[u]]
        if len(e) == 0:
            continue
        e = e[np.argsort(e[:, 0], kind="stable")]
        first, rows = e[:, 0].astype(np.int64), e[:, 1].astype(np.int64)
        page = first // 32
        joined = page[1:] <= page[:-1] + 1
        rows_total += int(rows.sum())
        stretches += 1 + int((~joined).sum())
    return rows_total / max(stretches, 1)
