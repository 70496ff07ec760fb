"""The oracle still produces the arrays whose digests were frozen by tests/golden/make_digests.py."""
import importlib.util
import json
import os

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
spec = importlib.util.spec_from_file_location("make_digests", os.path.join(HERE, "golden", "make_digests.py"))
md = importlib.util.module_from_spec(spec)
spec.loader.exec_module(md)


@pytest.mark.parametrize("name", md.DIGEST_CASES)
def test_oracle_digest(name):
    with open(os.path.join(HERE, "golden", "digests.json")) as f:
        golden = json.load(f)[name]
    got = {k: md.fnv1a64(v) for k, v in md.run_case(md.PARITY_CASES[name]).items()}
    assert got == golden
