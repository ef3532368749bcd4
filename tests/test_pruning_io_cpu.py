"""The saved result of the layer-wise search round-trips through its file and is refused when it
describes another search or is damaged (no GPU needed)."""
import json
from math import comb

import pytest

from paper_2402_14800_b200 import pruning_io as io


def records(E, r, n):
    subsets = comb(E, r)
    out = []
    for l in range(n):
        mask = ((1 << r) - 1) << (l % (E - r + 1))
        out.append({"kept_mask": mask, "losses": [0.5 + 0.01 * ((7 * l + s) % subsets) for s in range(subsets)],
                    "beta": 0.2 + 0.01 * l})
    return out


def test_round_trip(tmp_path):
    meta = {"E": 8, "r": 6, "n_layers": 5, "h": 4096, "f": 14336, "calibration_tokens": 4096,
            "search_mode": "layerwise", "weight_seed0": 100}
    recs = records(8, 6, 5)
    p = str(tmp_path / "pruning.json")
    io.save_pruning(p, meta, recs)
    got = io.load_pruning(p, expect_meta=meta)
    assert [g["kept_mask"] for g in got] == [r["kept_mask"] for r in recs]
    assert [g["losses"] for g in got] == [r["losses"] for r in recs]
    assert [g["beta"] for g in got] == [r["beta"] for r in recs]
    assert [g["layer"] for g in got] == list(range(5))
    # written atomically: no temporary file is left behind
    assert [f.name for f in tmp_path.iterdir()] == ["pruning.json"]


def test_a_file_of_another_search_is_refused(tmp_path):
    meta = {"E": 8, "r": 4, "n_layers": 2, "calibration_tokens": 4096, "search_mode": "layerwise"}
    p = str(tmp_path / "p.json")
    io.save_pruning(p, meta, records(8, 4, 2))
    for key, other in (("r", 6), ("calibration_tokens", 1024), ("search_mode", "progressive"), ("n_layers", 3)):
        with pytest.raises(ValueError):
            io.load_pruning(p, expect_meta=dict(meta, **{key: other}))
    assert len(io.load_pruning(p)) == 2


def test_inconsistent_records_are_refused(tmp_path):
    meta = {"E": 8, "r": 6, "n_layers": 2}
    with pytest.raises(ValueError):
        io.save_pruning(str(tmp_path / "a.json"), meta, [{"kept_mask": 0x0F, "losses": [], "beta": 0.0}] * 2)
    with pytest.raises(ValueError):
        io.save_pruning(str(tmp_path / "b.json"), meta, [{"kept_mask": 0x3F, "losses": [1.0, 2.0], "beta": 0.0}] * 2)
    p = str(tmp_path / "c.json")
    io.save_pruning(p, meta, records(8, 6, 2))
    doc = json.load(open(p))
    doc["layers"][1]["kept_mask"] = 0x1FF
    json.dump(doc, open(p, "w"))
    with pytest.raises(ValueError):
        io.load_pruning(p)
    doc["format"] = "something else"
    json.dump(doc, open(p, "w"))
    with pytest.raises(ValueError):
        io.load_pruning(p)
