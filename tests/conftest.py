import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def load_accept_cases():
    import json
    import numpy as np

    path = os.path.join(ROOT, "tests", "golden", "accept_cases.json")
    with open(path) as f:
        doc = json.load(f)
    out = []
    for c in doc["cases"]:
        state = np.array([[99 if v == "M" else v for v in row] for row in c["state"]], dtype=np.int32)
        base = dict(
            name=c["name"],
            parent=np.array(c["parent"], dtype=np.int32)[None],
            state=state[None],
            conf=np.array(c["conf"], dtype=np.float32)[None],
            top1=np.array(c["top1"], dtype=np.int32)[None],
            tau=float(c["tau"]),
            mask_id=99,
            topk=None if "topk" not in c else np.array(c["topk"], dtype=np.int32)[None],
            topk_m=int(c.get("topk_m", 1)),
            draft_prob=None if "draft_prob" not in c else np.array(c["draft_prob"], dtype=np.float32)[None],
        )
        for run in c["runs"]:
            out.append(dict(base, rule={"EXACT": 0, "TOP1": 1, "TOPK": 2, "PROB": 3}[run["rule"]],
                            search={"GREEDY": 0, "LONGEST": 1}[run["search"]],
                            expect=run, id="%s-%s-%s" % (c["name"], run["rule"], run["search"])))
    return out


@pytest.fixture(scope="session")
def accept_cases():
    return load_accept_cases()
