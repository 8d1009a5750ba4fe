"""CPU-side checks of the boundary: the library builds for sm_100a, loads without a GPU and
exports every function include/atomo.h declares; size queries (host-only) behave."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1806_04090_b200 import api, build
    build.build()
    return api.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "atomo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(atomo_[a-z_0-9]+)\s*\(", text)))


def test_header_functions_are_exported(lib):
    from paper_1806_04090_b200 import api
    names = _declared_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/atomo.h but not exported"
    assert sorted(api.EXPORTS) == names


def test_header_struct_sizes_match_binding():
    from paper_1806_04090_b200 import api
    assert ctypes.sizeof(api.PayloadHeader) == 64
    assert ctypes.sizeof(api.LayerHeader) == 80


def test_payload_size_queries(lib):
    from paper_1806_04090_b200 import api
    # header 64 + 80 per layer, then idx, coef, short, long per layer, 16-byte aligned
    b = api.payload_bytes_spectral([(64, 64)], 4)
    assert b == 64 + 80 + 16 + 16 + 4 * 64 * 4 + 4 * 64 * 4
    # k_cap is clamped to the number of atoms
    assert api.payload_bytes_spectral([(3, 500)], 100) == api.payload_bytes_spectral([(3, 500)], 3)
    b2 = api.payload_bytes_spectral([(64, 64), (10, 512)], 4)
    assert b2 > b and b2 % 16 == 0
    e = api.payload_bytes_entrywise([4096], 100)
    assert e == 64 + 80 + 400 + 400 + 16       # + per-tile offset table (2 entries, 16-byte aligned)
    # compact format: 2 bytes per entry, then values and indices of the saturated list (here 8 of them)
    assert api.payload_bytes_entrywise_compact([4096], 100, 8) == 64 + 80 + 208 + 32 + 16 + 32
    assert api.payload_bytes_entrywise_compact([4096], 100, 0) == 64 + 80 + 208 + 16
    assert api.payload_bytes_entrywise_compact([4096], 100, 10 ** 9) == api.payload_bytes_entrywise_compact([4096], 100, 4096)
    assert api.payload_bytes_entrywise_compact([100], 10, -1) == -1
    n, k_cap = 25_600_000, 300_000                       # a quarter of the explicit format's bytes per kept atom
    assert api.payload_bytes_entrywise_compact([n], k_cap, 0) < 0.3 * api.payload_bytes_entrywise([n], k_cap)
    assert api.payload_bytes_entrywise([0], 10) == -1
    assert api.payload_bytes_entrywise([2 ** 32], 10) == -1
    assert api.payload_bytes_spectral([(0, 5)], 10) == -1
    assert api.default_k_cap(2.0, 512) == 22 and api.default_k_cap(2.0, 10) == 10


def test_no_cpu_fallback():
    import torch
    from paper_1806_04090_b200 import api
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        api.Atomo(0)


def test_product_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_1806_04090_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|#include.*oracle|oracle/", text, flags=re.M), \
                    f"{f} reaches into the oracle"
