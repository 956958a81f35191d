"""CPU tests: the library loads, exports what the header declares, and its host policy
(admission, Eq. 4, Eq. 5) agrees with the oracle.  No GPU compute is called."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def E():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara
    return epara


def test_library_exports_every_declared_symbol(E):
    hdr = open(os.path.join(ROOT, "include", "epara.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(epara_[a-z_0-9]+)\s*\(", hdr))
    assert {"epara_register_model", "epara_submit", "epara_step", "epara_collect"} <= declared
    for name in declared:
        assert hasattr(E.lib, name), name
    assert declared == set(E.EXPORTS)


def test_strerror_and_null_arguments(E):
    assert E.lib.epara_strerror(E.E_TIMEOUT) == b"timeout"
    assert E.lib.epara_strerror(E.E_RESOURCE) == b"resource insufficiency"
    assert E.lib.epara_init(None, None) == E.E_INVALID
    assert E.lib.epara_submit(None, 0, 0, None, None) == E.E_INVALID
    assert E.lib.epara_step(None, None, 0, None) == E.E_INVALID
    assert E.lib.epara_collect(None, 1, None) == E.E_INVALID
    assert E.lib.epara_destroy(None) == E.E_INVALID


def test_eq4_eq5_match_oracle(E):
    from oracle import epara_oracle as O
    for req, grp in [(97, 49), (98, 49), (99, 49), (60, 60), (1, 100), (120.5, 30)]:
        assert E.epara_dp_group_count(req, grp) == O.dp_group_count(req, grp)
    for bs in [0, 1, 4, 7, 256, 512]:
        for mf in [1, 2, 3, 8, 300]:
            assert E.epara_inter_request_count(bs, mf) == O.inter_request_count(bs, mf)
    assert E.epara_inter_request_count(4, 0) == E.E_INVALID
    assert E.epara_dp_group_count(10, 0) == E.E_INVALID


def test_admission_matches_oracle_on_random_queues(E):
    from oracle import epara_oracle as O
    rng = np.random.default_rng(0)
    for trial in range(300):
        n = int(rng.integers(0, 40))
        now = int(rng.integers(0, 1000))
        q = [{"ticket": 100 + i, "deadline_ns": int(rng.choice([0, 0, rng.integers(1, 1000)])),
              "stream": int(rng.integers(0, 6))} for i in range(n)]
        cap = int(rng.integers(0, 20))
        mf = int(rng.choice([0, 0, 1, 2, 3, 5, 30]))
        exp = O.admit(q, now, cap, mf)
        got = E.epara_admit_queue([r["ticket"] for r in q], [r["deadline_ns"] for r in q],
                                  [r["stream"] for r in q], now, cap, mf)
        assert (list(exp[0]), list(exp[1])) == got, (trial, q, now, cap, mf)


def test_binding_refuses_to_import_without_the_library(E, tmp_path):
    """The product path has no fallback: a missing libepara.so is an ImportError."""
    code = ("import importlib.util, sys, os\n"
            "spec = importlib.util.spec_from_file_location('epara_copy', sys.argv[1])\n"
            "m = importlib.util.module_from_spec(spec)\n"
            "try:\n    spec.loader.exec_module(m)\nexcept ImportError as e:\n    print('IMPORTERROR'); sys.exit(0)\n"
            "sys.exit(1)\n")
    src = open(os.path.join(ROOT, "paper_2511_00603_b200", "epara.py")).read()
    p = tmp_path / "epara_copy.py"
    p.write_text(src)
    r = subprocess.run([sys.executable, "-c", code, str(p)], capture_output=True, text=True)
    assert r.returncode == 0 and "IMPORTERROR" in r.stdout


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2511_00603_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|epara_oracle|oracle[/.]", txt, flags=re.M), f
    otxt = open(os.path.join(ROOT, "oracle", "epara_oracle.py")).read()
    assert "paper_2511_00603_b200" not in otxt and "ctypes" not in otxt
