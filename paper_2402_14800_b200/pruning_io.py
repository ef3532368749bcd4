"""Saving and reloading the result of the layer-wise pruning search.

The search is run once per model on a calibration set; afterwards the pruned layers are built
straight from the kept-expert masks (Sec. 3.2, last paragraph: the pruned model is saved and
loaded as a smaller model).  The file is JSON: a ``meta`` object that names what was searched
(shape, number of layers, subset size, calibration recipe) and one record per layer with the
kept-expert bitmask, the loss of every subset in enumeration order, and the layer's calibrated
skipping threshold beta (Sec. 3.3)."""
from __future__ import annotations

import json
import os
from math import comb

FORMAT = "moe-pruning-v1"


def save_pruning(path: str, meta: dict, layers: list) -> None:
    """``layers``: dicts with ``kept_mask`` (int), ``losses`` (list of floats, may be empty when
    nothing was searched), ``beta`` (float)."""
    E, r = int(meta["E"]), int(meta["r"])
    recs = []
    for i, rec in enumerate(layers):
        mask, losses = int(rec["kept_mask"]), [float(v) for v in rec.get("losses", [])]
        if bin(mask).count("1") != r or mask >> E:
            raise ValueError("layer %d: mask %#x does not keep %d of %d experts" % (i, mask, r, E))
        if losses and len(losses) != comb(E, r):
            raise ValueError("layer %d: %d losses for C(%d, %d) subsets" % (i, len(losses), E, r))
        recs.append({"layer": i, "kept_mask": mask, "losses": losses, "beta": float(rec.get("beta", 0.0))})
    tmp = path + ".tmp"
    with open(tmp, "w") as fh:
        json.dump({"format": FORMAT, "meta": dict(meta), "layers": recs}, fh)
    os.replace(tmp, path)


def load_pruning(path: str, expect_meta: dict | None = None) -> list:
    """The per-layer records of ``path``.  Raises ValueError when the file is not of this format,
    is inconsistent, or (with ``expect_meta``) describes another search: every key of
    ``expect_meta`` must be present in the file's meta with the same value."""
    with open(path) as fh:
        doc = json.load(fh)
    if doc.get("format") != FORMAT:
        raise ValueError("%s is not a %s file" % (path, FORMAT))
    meta, recs = doc["meta"], doc["layers"]
    if expect_meta is not None:
        for k, v in expect_meta.items():
            if meta.get(k) != v:
                raise ValueError("%s was written for %s = %r, not %r" % (path, k, meta.get(k), v))
    E, r = int(meta["E"]), int(meta["r"])
    if "n_layers" in meta and len(recs) != int(meta["n_layers"]):
        raise ValueError("%s holds %d layers, its meta says %s" % (path, len(recs), meta["n_layers"]))
    for i, rec in enumerate(recs):
        mask = int(rec["kept_mask"])
        if rec.get("layer") != i or bin(mask).count("1") != r or mask >> E:
            raise ValueError("%s: bad record for layer %d" % (path, i))
        if rec["losses"] and len(rec["losses"]) != comb(E, r):
            raise ValueError("%s: layer %d has %d losses" % (path, i, len(rec["losses"])))
    return recs
