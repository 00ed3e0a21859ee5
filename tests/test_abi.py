"""The C-ABI library builds, loads, and exports every entry point that include/flashmesh.h declares.
No compute call is made (this file runs without a GPU)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "flashmesh.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fm_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_six_calls_of_the_path():
    names = _declared_symbols()
    for want in ("fm_create", "fm_prefill", "fm_draft", "fm_verify", "fm_accept", "fm_generate"):
        assert want in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2511_15618_b200.build import build
    lib = ctypes.CDLL(build())
    for name in _declared_symbols():
        assert hasattr(lib, name), f"{name} is declared in flashmesh.h but not exported"


def test_host_side_argument_checks_need_no_device():
    from paper_2511_15618_b200 import binding as B
    import fm_synth as S
    cfg = B.make_config(S.get_config("tiny"))
    assert B.fm_workspace_bytes(cfg) > 0
    bad = B.make_config(S.get_config("tiny"))
    bad.head_dim = 48
    assert B.fm_workspace_bytes(bad) == 0
    assert B.fm_strerror(-3) == "capacity exceeded"
    assert B.fm_verify_bytes(None, 1, [[1, 1, 1]]) == 0.0
