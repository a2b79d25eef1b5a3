"""Writes tests/golden/comm_words.json from the oracle's statement of Eq. 8 /
Eq. 9 (calls nothing but `oracle/`).  Run from the repository root:

    python tests/golden/make_comm_words_golden.py
"""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import comm_words as CW  # noqa: E402


def fc(dims):
    return [dict(kind="fc", split="model", d_in=dims[i - 1], d_out=dims[i]) for i in range(1, len(dims))]


def conv2():
    return [dict(kind="conv", split="domain", C_in=64, C_out=64, H=224, W=224, kh=3, kw=3)] * 2


CASES = {
    "cfg1": (fc((784, 512, 512, 10)), 64, [(1, 1), (2, 2), (4, 1), (1, 4)]),
    "cfg2": (fc((9216, 4096, 4096, 1000)), 256, [(1, 1), (8, 1), (1, 8), (2, 4), (4, 2)]),
    "cfg3": (fc((25088, 4096, 4096, 1000)), 512, [(1, 1), (4, 4), (16, 1), (1, 16)]),
    "cfg4": (conv2(), 32, [(1, 1), (2, 1), (4, 1), (8, 1)]),
    "cfg5": (fc((8192,) * 9), 8192, [(1, 1), (16, 16), (64, 4), (4, 64)]),
}

out = {"_source": "Eq. 8 and Eq. 9 bandwidth terms, evaluated by oracle/comm_words.py", "cases": []}
for name, (layers, B, grids) in CASES.items():
    for (P_r, P_c) in grids:
        rows = CW.layer_words(layers, B, P_r, P_c)
        out["cases"].append(dict(workload=name, layers=layers, B=B, P_r=P_r, P_c=P_c, rows=rows,
                                 total=CW.total_words(layers, B, P_r, P_c)))

with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "comm_words.json"), "w") as f:
    json.dump(out, f, indent=1)
print("wrote", len(out["cases"]), "cases")
