"""The C-ABI library loads without a GPU and exports every function include/onela.h declares."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import binding, build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    build.build()
    return P.load_library()


def _declared():
    text = (ROOT / "include" / "onela.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(onela_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "onela_init_shared_state" in names and "onela_append_records" in names
    assert "onela_reorder_beams" in names and "onela_decode_step" in names
    for n in names:
        assert isinstance(getattr(lib, n), ctypes._CFuncPtr), n


def test_binding_covers_the_header(lib):
    assert sorted(binding.PROTOTYPES) == _declared()


def test_status_strings(lib):
    seen = {P.status_string(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert P.status_string(-99) == "unknown status"


def test_header_constants_match_binding():
    text = (ROOT / "include" / "onela.h").read_text()
    defs = dict(re.findall(r"#define\s+(ONELA_[A-Z_0-9]+)\s+\(?(-?\d+)u?\)?", text))
    assert int(defs["ONELA_E_ORDER"]) == binding.E_ORDER and int(defs["ONELA_E_TIMEOUT"]) == binding.E_TIMEOUT
    assert int(defs["ONELA_DTYPE_BF16"]) == binding.DTYPE_BF16 and int(defs["ONELA_MAX_BATCH"]) == binding.MAX_BATCH
    assert int(defs["ONELA_FLAG_DRY_RUN"]) == binding.FLAG_DRY_RUN
    assert int(defs["ONELA_FLAG_FORCE_GENERIC"]) == binding.FLAG_FORCE_GENERIC
