"""Writes tests/golden/oracle_small_cases.json: outputs of the fp64 oracle on a few tiny seeded cases.

The file is a regression anchor for the ORACLE itself (so that an accidental change to its arithmetic shows
up as a diff against stored numbers, not only against the pins); it is produced by this script, which
calls nothing but `oracle/` and numpy.  The paper prints no worked numeric example of Eq. 2 on the shared
prefix cache, so there are no paper-printed values to store here; the hand-computable cases live in
tests/test_oracle_pins.py.  Run from the repository root:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", ".."))
import oracle  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def small(rng, *shape):
    # multiples of 1/8 in [-2, 2]: exactly representable in bf16 / fp32 / fp64 and in JSON
    return rng.integers(-16, 17, size=shape).astype(np.float64) / 8.0


def main():
    rng = np.random.default_rng(260313420)
    cases = []
    # full-suffix operator (Eq. 2 over prefix (+) suffix, GQA): forward and backward
    B, Hq, Hkv, S, P, d = 2, 4, 2, 3, 4, 4
    t = dict(q=small(rng, B, Hq, S, d), pk=small(rng, Hkv, P, d), pv=small(rng, Hkv, P, d),
             sk=small(rng, B, Hkv, S, d), sv=small(rng, B, Hkv, S, d), dout=small(rng, B, Hq, S, d))
    out, lse = oracle.attn_fwd(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.5)
    dq, dk, dv = oracle.attn_bwd(t["dout"], t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.5)
    cases.append(dict(kind="attn", scale=0.5, inputs={k: v.tolist() for k, v in t.items()},
                      expected=dict(out=out.tolist(), lse=lse.tolist(), dq=dq.tolist(), dk=dk.tolist(), dv=dv.tolist())))
    # decode-shaped operator with ragged cache lengths
    B, Hq, Hkv, Sq, Skv, P, d = 3, 2, 1, 2, 5, 3, 4
    t = dict(q=small(rng, B, Hq, Sq, d), pk=small(rng, Hkv, P, d), pv=small(rng, Hkv, P, d),
             sk=small(rng, B, Hkv, Skv, d), sv=small(rng, B, Hkv, Skv, d))
    lens = [2, 5, 3]
    out, lse = oracle.attn_fwd_decode(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.75, lens)
    cases.append(dict(kind="decode", scale=0.75, suffix_len=lens, inputs={k: v.tolist() for k, v in t.items()},
                      expected=dict(out=out.tolist(), lse=lse.tolist())))
    # masked target cross-entropy on top of the output head
    N, Lr, Dm, V = 2, 3, 4, 6
    h, w = small(rng, N, Lr, Dm), small(rng, V, Dm)
    tg = rng.integers(0, V, size=(N, Lr)).astype(np.int32)
    mk = np.array([[1.0, 0.0, 1.0], [1.0, 1.0, 1.0]])
    nll, lse, loss = oracle.target_ce_fwd(h, w, tg, mk)
    cases.append(dict(kind="target_ce", inputs=dict(hidden=h.tolist(), weight=w.tolist(), target=tg.tolist(), mask=mk.tolist()),
                      expected=dict(nll=nll.tolist(), lse=lse.tolist(), loss=loss.tolist())))
    with open(os.path.join(HERE, "oracle_small_cases.json"), "w") as f:
        json.dump(dict(written_by="tests/golden/make_golden.py (oracle only)", cases=cases), f, indent=1)


if __name__ == "__main__":
    main()
