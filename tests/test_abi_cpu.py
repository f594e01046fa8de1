"""Host-only checks of the C-ABI library: it builds, loads, exports every
declared symbol, and rejects bad arguments before touching a device."""
import os
import re

import pytest

from paper_2502_15572_b200 import binding, build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return binding.load()


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names.update(re.findall(r"\b(dresd_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"
    assert set(binding.EXPORTS) <= set(names)


def test_validation_needs_no_device(lib):
    with pytest.raises(binding.DresdError) as e:
        binding.dresd_store_create(0, 0, 10, 64, binding.DRESD_F16, 4)
    assert e.value.status == -1 and "NULL" in e.value.message
    for kwargs, status in [
        (dict(N=2 ** 31 - 1023, d=64, dtype=1, stored_len=4), -1),   # last tile's row coordinate would pass 2^31
        (dict(N=0, d=64, dtype=1, stored_len=4), -1),
        (dict(N=2 ** 31, d=64, dtype=1, stored_len=4), -1),
        (dict(N=10, d=12, dtype=1, stored_len=4), -1),        # 24-byte rows
        (dict(N=10, d=64, dtype=7, stored_len=4), -1),
        (dict(N=10, d=64, dtype=1, stored_len=0), -1),
        (dict(N=10, d=8192, dtype=1, stored_len=4), -2),
        (dict(N=10, d=64, dtype=1, stored_len=4, keys_ptr=0x1008), -1),   # misaligned base
    ]:
        with pytest.raises(binding.DresdError) as e:
            binding.dresd_store_create(kwargs.pop("keys_ptr", 0x1000), 0x2000, kwargs["N"], kwargs["d"],
                                       kwargs["dtype"], kwargs["stored_len"])
        assert e.value.status == status, (kwargs, e.value)
    with pytest.raises(binding.DresdError) as e:
        binding.dresd_retrieve(0, 0, 1, 1, 1, 0, 0, 0, 0)
    assert e.value.status == -1
    with pytest.raises(binding.DresdError):
        binding.dresd_store_status(0)
    with pytest.raises(binding.DresdError):
        binding.dresd_store_set_option(0, "grid", 1)
    binding.dresd_store_destroy(0)                      # NULL is allowed
    assert binding.dresd_store_last_launches(0) == 0


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(binding.DresdError) as e:
        binding.load(str(tmp_path / "nope.so"))
    assert "no CPU fallback" in str(e.value)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2502_15572_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "import oracle" not in text and "from oracle" not in text, fn
                assert "dresd_oracle" not in text, fn
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", fn)).read()
            assert "paper_2502_15572_b200" not in text, fn
