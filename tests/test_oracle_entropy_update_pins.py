"""Pins of the oracle's running form of Eq. 2 (Section 3.2 selects the layer "during each decoding
step"): the per-layer entropy sums are extended by the rows each acceptance commits, nothing is
recomputed.  Held against the full recomputation (a fresh prefill of prompt + emitted tokens), against
the closed form for uniform attention, and against the tree's shape (only the accepted path counts).
None needs a GPU."""
import math

import pytest
import torch

from oracle import dream_oracle as O
from paper_2505_19201_b200 import synth
from tests.util_oracle import make_oracle, tiny_preset

D64, BF = torch.float64, torch.bfloat16


def _setup(kv_dtype=None, scale=30.0, **over):
    p, orc = make_oracle(tiny_preset(**over), D64, kv_dtype=kv_dtype)
    orc.tw["lm_head"] = orc.tw["lm_head"] * scale
    vis, ids = synth.request_inputs(p, 0)
    vis, ids = vis.to(D64), ids.tolist()
    st, _, _ = orc.prefill(vis, 0, ids)
    orc.compress_visual(st, p["k_visual"])
    return p, orc, st, vis, ids


def _rounds(p, orc, st, vis, ids, lengths, distractors=True):
    """Rounds whose trees hold the target's own continuation as a chain of the given lengths, each
    chain node with a sibling that is refused."""
    ref, _ = orc.ar_decode(vis, 0, ids, sum(lengths) + len(lengths) + 2)
    emitted = [st.pending]
    for a in lengths:
        toks, par, last = [st.pending], [-1], 0
        for j in range(a):
            toks.append(ref[len(emitted) + j]); par.append(last)
            if distractors:
                toks.append((ref[len(emitted) + j] + 3) % p["vocab"]); par.append(last)
                last = len(toks) - 2
            else:
                last = len(toks) - 1
        r = orc.step(st, O.make_tree(toks, par))
        assert r["A"] == a
        emitted += r["out"]
    return emitted


@pytest.mark.parametrize("kv_dtype", [None, BF])
def test_running_sums_equal_the_full_recomputation(kv_dtype):
    p, orc, st, vis, ids = _setup(kv_dtype)
    before, _, _ = orc.layer_entropy(st)
    assert torch.allclose(before, st.entropy, atol=1e-14)              # nothing committed yet: the prefill's AE
    emitted = _rounds(p, orc, st, vis, ids, (2, 0, 3))
    st2, tok2, _ = orc.prefill(vis, 0, ids, extra_ids=emitted[:-1])
    assert st2.P == st.P and tok2 == st.pending
    ae, layer, _ = orc.layer_entropy(st)
    assert torch.allclose(ae, st2.entropy, atol=1e-12)
    assert layer == orc.select_tap(st2.entropy)[0]
    assert float((ae - before).abs().max()) > 1e-6                    # the new rows moved it


def test_only_the_accepted_path_counts():
    """The same continuation verified as a bare chain and inside a tree with refused siblings gives
    the same sums: a refused node's row adds nothing, and an accepted row does not see it."""
    p, orc, st, vis, ids = _setup()
    _rounds(p, orc, st, vis, ids, (3, 1), distractors=True)
    p2, orc2, st2, vis2, ids2 = _setup()
    _rounds(p2, orc2, st2, vis2, ids2, (3, 1), distractors=False)
    assert torch.allclose(orc.layer_entropy(st)[0], orc2.layer_entropy(st2)[0], atol=1e-12)


def test_uniform_attention_has_the_closed_form():
    """With the query projection zeroed every score is 0, row i attends uniformly to its i + 1 keys and
    its entropy is ln(i + 1) in every head and layer: AE over P rows = (1/P) sum_i ln(i + 1), before
    and after rows are committed."""
    p, orc = make_oracle(tiny_preset(), D64)
    c = orc.cfg
    for l in range(c.n_layers):
        orc.tw["wqkv"][l][:c.n_heads * c.head_dim] = 0
    orc.tw["lm_head"] = orc.tw["lm_head"] * 30
    vis, ids = synth.request_inputs(p, 0)
    vis, ids = vis.to(D64), ids.tolist()
    st, _, _ = orc.prefill(vis, 0, ids)
    orc.compress_visual(st, p["k_visual"])
    want = lambda P: sum(math.log(i + 1) for i in range(P)) / P
    assert torch.allclose(orc.layer_entropy(st)[0], torch.full((c.n_layers,), want(st.P), dtype=D64), atol=1e-12)
    _rounds(p, orc, st, vis, ids, (2, 1))
    assert st.P == p["n_visual"] + p["n_prompt"] + 5
    assert torch.allclose(orc.layer_entropy(st)[0], torch.full((c.n_layers,), want(st.P), dtype=D64), atol=1e-12)
