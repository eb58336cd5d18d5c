"""Writes tests/golden/toy_decode.json from the CPU oracle alone (float64).

The paper prints no worked numerical example, so this fixture is not a value of the
paper: it is the oracle's own greedy decode of the toy workload, stored so that a change
in the oracle's arithmetic shows up as a diff.  It calls nothing but `oracle/` and the
seeded input generators.   Run:  python tests/golden/make_toy_golden.py
"""
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from tests.util_oracle import make_oracle  # noqa: E402
from paper_2505_19201_b200 import synth    # noqa: E402


def main():
    p, orc = make_oracle("toy", torch.float64)
    vis, ids = synth.request_inputs(p, 0)
    st, tok, margin = orc.prefill(vis.to(torch.float64), 0, ids.tolist())
    kept, scores, _ = orc.compress_visual(st, p["k_visual"])
    ar, margins = orc.ar_decode(vis.to(torch.float64), 0, ids.tolist(), 24)
    out = dict(first_token=tok, first_margin=margin, entropy=[float(e) for e in st.entropy],
               kept=kept.tolist(), ar_tokens=ar, min_ar_margin=min(margins))
    with open(os.path.join(os.path.dirname(__file__), "toy_decode.json"), "w") as f:
        json.dump(out, f, indent=1)
    print(out)


if __name__ == "__main__":
    main()
