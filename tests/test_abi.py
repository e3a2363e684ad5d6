"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import re
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def _declared():
    names = set()
    for h in (ROOT / "include").glob("*.h"):
        text = re.sub(r"/\*.*?\*/", "", h.read_text(), flags=re.S)
        names |= set(re.findall(r"\b(first_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2410_12513_b200 import build
    lib = ctypes.CDLL(str(build.build()))
    names = _declared()
    assert {"first_create", "first_destroy", "first_prefill_route", "first_set_mask", "first_decode_step",
            "first_last_device_flags"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings_and_null_argument_errors_need_no_gpu():
    from paper_2410_12513_b200 import lib
    L = lib()
    assert L.first_status_string(0) == b"ok"
    assert L.first_status_string(-4) == b"capacity exceeded"
    assert L.first_create(None, None, None) == -1
    assert L.first_decode_step(None, None, None, None, None, None, None) == -1
    assert L.first_set_mask(None, None, 1, None) == -1
    assert L.first_prefill_route(None, 0, None, 0, None, 1, 1, None, None, 0.5, 0, None, None, None) == -1
    assert L.first_prefill(None, None, None, 1, None, None, None, 0.5, 0, None, None, None, None, None) == -1
    assert L.first_destroy(None) == 0
    # the entry points for changing batches and the measurement aids reject missing arguments the same way
    assert L.first_set_mask_host(None, None, 1, None) == -1
    assert L.first_pool_create(None, 4, None, None, None, None) == -1
    assert L.first_seq_join(None, None, 8, None, 0, 0, None, None) == -1
    assert L.first_seq_leave(None, 0, None) == -1
    assert L.first_pool_commit(None, None) == -1
    assert L.first_pool_kv(None, None) == -1
    assert L.first_pool_stats(None, None, None, None) == -1
    assert L.first_pool_destroy(None) == 0
    assert L.first_step_trace(None, 0, None, None, None, None, None) == -1
    assert L.first_selftest_wait_expiry(None, 10, None, None, None) == -1
    assert L.first_graph_count(None) == 0
    assert {"first_pool_create", "first_seq_join", "first_seq_leave", "first_pool_commit", "first_set_mask_host",
            "first_step_trace", "first_prefill_route_static"} <= set(_declared())


def test_product_package_does_not_import_the_oracle():
    for p in (ROOT / "paper_2410_12513_b200").rglob("*"):
        if p.suffix in (".py", ".cu", ".cuh", ".h"):
            assert "oracle" not in p.read_text(), p
