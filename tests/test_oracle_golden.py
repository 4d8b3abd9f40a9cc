"""The oracle against its own stored outputs on tiny seeded cases (tests/golden/oracle_small_cases.json,
written by tests/golden/make_golden.py, which calls only the oracle): a regression anchor for the oracle's
arithmetic, next to the pins that tie it to library routines and closed forms."""
import json
import os

import numpy as np

import oracle

PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "oracle_small_cases.json")


def close(a, b):
    return np.max(np.abs(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64))) < 1e-12


def test_oracle_reproduces_its_stored_outputs():
    cases = json.load(open(PATH))["cases"]
    kinds = set()
    for c in cases:
        i, e = c["inputs"], c["expected"]
        kinds.add(c["kind"])
        if c["kind"] == "attn":
            out, lse = oracle.attn_fwd(i["q"], i["pk"], i["pv"], i["sk"], i["sv"], c["scale"])
            dq, dk, dv = oracle.attn_bwd(i["dout"], i["q"], i["pk"], i["pv"], i["sk"], i["sv"], c["scale"])
            assert close(out, e["out"]) and close(lse, e["lse"])
            assert close(dq, e["dq"]) and close(dk, e["dk"]) and close(dv, e["dv"])
        elif c["kind"] == "decode":
            out, lse = oracle.attn_fwd_decode(i["q"], i["pk"], i["pv"], i["sk"], i["sv"], c["scale"], c["suffix_len"])
            assert close(out, e["out"]) and close(lse, e["lse"])
        elif c["kind"] == "target_ce":
            nll, lse, loss = oracle.target_ce_fwd(i["hidden"], i["weight"], np.asarray(i["target"], dtype=np.int32), i["mask"])
            assert close(nll, e["nll"]) and close(lse, e["lse"]) and close(loss, e["loss"])
    assert kinds == {"attn", "decode", "target_ce"}
