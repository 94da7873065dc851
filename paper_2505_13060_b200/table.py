"""Saving and loading the per-layer table of a calibration.

The sensitivities are computed once and reused for any threshold, performance
metric or grouping (Algorithm 1: step 2 does not depend on steps 3 and 4), so a
calibration is worth keeping.  The table is the one ``shard.layer_row`` builds:
per layer ``[s_mean, d_model[0..F-1], d_meas[0..F-1]]``.  Numbers are stored as
hexadecimal floating-point strings, so a table read back is bit-identical and
selections made from it (``shard.select_from_table``) do not change.
"""
from __future__ import annotations

import json

import numpy as np

FORMAT = "ampq-layer-table-1"


def save_table(path: str, names, formats, table, meta: dict | None = None) -> None:
    """``names[L]`` layer names, ``formats[F]`` the context's format list,
    ``table[L, 1 + 2F]``."""
    tab = np.asarray(table, dtype=np.float64)
    F = len(formats)
    if tab.ndim != 2 or tab.shape != (len(names), 1 + 2 * F):
        raise ValueError("table must be [len(names), 1 + 2 * len(formats)]")
    doc = {"format": FORMAT, "formats": [int(f) for f in formats], "meta": meta or {},
           "layers": [{"name": str(n), "row": [float(x).hex() for x in row]} for n, row in zip(names, tab)]}
    with open(path, "w") as f:
        json.dump(doc, f, indent=1)


def load_table(path: str):
    """Returns (names, formats, table, meta)."""
    with open(path) as f:
        doc = json.load(f)
    if doc.get("format") != FORMAT:
        raise ValueError("%s is not a saved layer table" % path)
    formats = [int(x) for x in doc["formats"]]
    names = [l["name"] for l in doc["layers"]]
    table = np.array([[float.fromhex(x) for x in l["row"]] for l in doc["layers"]], dtype=np.float64)
    table = table.reshape(len(names), 1 + 2 * len(formats))
    return names, formats, table, doc.get("meta", {})
