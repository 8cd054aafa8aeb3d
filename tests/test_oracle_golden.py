"""The oracle against its own stored digest (tests/golden/oracle_tiny.json, written by tests/golden/make_golden.py,
which calls the oracle and the seeded generator only).  Not a pin against the paper -- the paper prints no worked
example -- but a guard: any change to the oracle's arithmetic shows up here and has to be justified."""
import importlib.util
import json
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def _close(a, b, path):
    if isinstance(a, dict):
        assert set(a) == set(b), path
        for k in a:
            _close(a[k], b[k], f"{path}.{k}")
    elif isinstance(a, list):
        assert len(a) == len(b), path
        for i, (x, y) in enumerate(zip(a, b)):
            _close(x, y, f"{path}[{i}]")
    elif isinstance(a, float):
        assert abs(a - b) <= 1e-9 * max(1.0, abs(a)), f"{path}: {a} != {b}"
    else:
        assert a == b, f"{path}: {a} != {b}"


def test_oracle_reproduces_its_stored_digest():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    want = json.load(open(os.path.join(HERE, "golden", "oracle_tiny.json")))
    got = json.loads(json.dumps(mod.compute()))
    _close(want, got, "golden")
    # the stream's structure on the tiny workload, stated in words as well: capacity 4, 8 frames -> 4 evictions
    assert len(want["evict_log"]) == 4 and len(want["bank_frame_ids"]) == 4
