"""The oracle still produces the stored small case (tests/golden/, written by a script that calls only the
oracle).  A guard against unintended change, not a pin to the paper."""
import importlib.util
import json
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_reproduces_the_stored_small_case():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with open(os.path.join(HERE, "golden", "oracle_small_case.json")) as f:
        want = json.load(f)
    got = json.loads(json.dumps(mod.compute()))
    assert got == want
    # sanity of the stored case itself: the dominant coordinate of every step was selected
    for t, step in enumerate(want["steps"]):
        assert (t * 7 + 3) % want["shape"]["d"] in step["out_idx"]
