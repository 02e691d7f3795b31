"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares;
host-only validation works without any CUDA call."""
import ctypes
import os
import re

import pytest

from paper_2511_05534_b200 import binding as F
from paper_2511_05534_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return F.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "flowmm.h")).read()
    declared = set(re.findall(r"\b(flowmm_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(F.EXPORTS)


def test_params_struct_matches_header():
    header = open(os.path.join(ROOT, "include", "flowmm.h")).read()
    body = header[header.index("typedef struct {"):header.index("} flowmm_params;")]
    fields = re.findall(r"(?:int32_t|float|int64_t)\s+([^;]+);", body)
    names = [n.strip().split("[")[0] for group in fields for n in group.split(",")]
    assert names == [f[0] for f in F._CParams._fields_]


def test_workspace_bytes_and_validation_need_no_gpu(lib):
    p = F.Params(4, 8, 2, 128, 1000, 16, 100)
    n = F.flowmm_workspace_bytes(p)
    assert n > 0 and n % 256 == 0
    bigger = F.flowmm_workspace_bytes(F.Params(8, 8, 2, 128, 1000, 16, 100))
    assert bigger > n
    cases = [
        (dict(n_q_heads=7), 2), (dict(head_dim=96), 2), (dict(window=2000), 2), (dict(n_keep=0), 3),
        (dict(n_keep=1001), 3), (dict(keep_window=1, n_keep=8), 3), (dict(dtype=5), 4), (dict(n_units=0), 2),
    ]
    for change, code in cases:
        kw = dict(n_units=4, n_q_heads=8, n_kv_heads=2, head_dim=128, seq_len=1000, window=16, n_keep=100)
        kw.update(change)
        with pytest.raises(F.FlowmmError) as e:
            F.flowmm_workspace_bytes(F.Params(**kw))
        assert e.value.code == code, change
    assert F.status_string(0) == "ok" and "workspace" in F.status_string(5)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(F, "_lib", None)
    monkeypatch.setattr(F, "LIB_PATH", str(tmp_path / "libflowmm.so"))
    with pytest.raises(FileNotFoundError):
        F.load()
