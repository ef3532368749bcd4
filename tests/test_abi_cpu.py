"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2402_14800_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_symbols():
    import glob
    names = set()
    for path in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):
        src = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names |= set(re.findall(r"\b(moe_[a-z_0-9]+)\s*\(", src))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"moe_layer_create", "moe_forward", "moe_prune_search", "moe_reserve",
            "moe_test_wait_expiry", "moe_test_set_free_bytes_limit"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_routing_stats_layout():
    total, off = binding.routing_stats_layout(256, 8)
    assert off[0] == 0 and all(o % 16 == 0 for o in off)
    assert off[1] >= 256 * 8 and off[2] >= off[1] + 256 * 8 and off[3] >= off[2] + 256 * 4
    assert off[4] >= off[3] + 256 and off[5] >= off[4] + 64 and off[6] >= off[5] + 4
    assert total >= off[6] + 4
    assert binding.load_library().moe_routing_stats_bytes(256, 8) == total
    t1, o1 = binding.routing_stats_layout(1, 8)
    assert t1 > 0 and sorted(o1) == o1


def test_num_subsets():
    assert binding.num_subsets(8, 6) == 28 and binding.num_subsets(8, 4) == 70
    assert binding.num_subsets(8, 8) == 1 and binding.num_subsets(16, 8) == 12870
    assert binding.num_subsets(8, 1) == 0 and binding.num_subsets(8, 9) == 0 and binding.num_subsets(17, 4) == 0


def test_create_rejects_bad_arguments_without_a_device(lib):
    p = ctypes.c_void_p(0x1000)
    assert not lib.moe_layer_create(None, p, p, p, 128, 448, 8, 0xFF)
    assert "NULL" in binding.last_error()
    assert not lib.moe_layer_create(ctypes.c_void_p(0x1001), p, p, p, 128, 448, 8, 0xFF)
    assert "aligned" in binding.last_error()
    assert not lib.moe_layer_create(p, p, p, p, 128, 448, 17, 0xFF)
    assert not lib.moe_layer_create(p, p, p, p, 100, 448, 8, 0xFF)
    assert "multiples of 64" in binding.last_error()
    assert not lib.moe_layer_create(p, p, p, p, 128, 448, 8, 0x1)
    assert "fewer than 2" in binding.last_error()
    assert not lib.moe_layer_create(p, p, p, p, 128, 448, 8, 0x1FF)


def test_null_handle_is_an_error(lib):
    assert lib.moe_forward(None, None, 4, 0.0, None, None) == -1
    assert lib.moe_prune_search(None, None, 4, 6, None, None) == -1
    assert lib.moe_prune_search_multi(None, None, 4, None, 2, None, None) == -1
    assert lib.moe_calibrate_beta(None, None, 4, None) == -1
    assert lib.moe_device_status(None) == -1
    assert lib.moe_reserve(None, 16) == -1
    assert lib.moe_test_wait_expiry(None, 1000, 0) == -1
    assert lib.moe_layer_weight_bytes(None) == 0
    lib.moe_layer_destroy(None)


def test_binding_fails_loudly_without_the_library(tmp_path):
    with pytest.raises(binding.MoeError):
        binding.load_library(str(tmp_path / "libmoe.so"))


def test_frequency_subset_on_the_host(lib):
    # the activation-frequency baseline: the r most used experts (row + column sums of the
    # co-selection map), equal use resolved towards the lower index; host code, no device
    import numpy as np
    rng = np.random.default_rng(5)
    for E, r in ((8, 6), (8, 4), (16, 9), (4, 2), (5, 5)):
        counts = rng.integers(0, 50, size=(E, E)).astype(np.int32)
        np.fill_diagonal(counts, 0)
        if E == 8:
            counts[3, :] = counts[5, :]      # make two experts tie
            counts[:, 3] = counts[:, 5]
            counts[3, 5] = counts[5, 3] = 7
        freq = counts.sum(0).astype(np.int64) + counts.sum(1)
        order = sorted(range(E), key=lambda e: (-int(freq[e]), e))
        want = sum(1 << e for e in order[:r])
        buf = (ctypes.c_int32 * (E * E))(*[int(v) for v in counts.ravel()])
        assert lib.moe_frequency_subset(buf, E, r) == want
    assert lib.moe_frequency_subset(None, 8, 4) == 0
