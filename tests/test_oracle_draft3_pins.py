"""Pins of the oracle's three-block draft (Section 4: an initial decoder block, an intermediate
cross-attention block and a final decoder block; Eq. 1 in the middle one).

Nothing here re-types the blocks.  The draft is held against things fixed elsewhere:
  * the target path of the same oracle (itself pinned against goldens, chain = causal decoding and
    brute force): with the middle block switched off the draft is a two-layer causal decoder, and a
    two-layer target built from the draft's own tensors must give the same logits;
  * the single-block draft (pinned on its own): with both decoder blocks switched off only Eq. 1 and
    its MLP remain, and the two drafts must agree;
  * invariants: a tree node's feature depends on its own root path only (every path re-drafted as a
    chain), the rows appended round by round equal the rows of a fresh draft prefill over the longer
    context, a memory row is seen by strictly later positions only, greedy speculative output equals
    autoregressive decoding, and the parameter counts the paper prints for its draft models.
None needs a GPU.
"""
import pytest
import torch

from oracle import dream_oracle as O
from paper_2505_19201_b200 import configs, synth
from tests.util_oracle import make_oracle, tiny_preset

D64 = torch.float64


def _inputs(p, seed=0):
    vis, ids = synth.request_inputs(p, seed)
    return vis.to(D64), ids.tolist()


def _ready(p, orc, scale=30.0, k=None):
    orc.tw["lm_head"] = orc.tw["lm_head"] * scale
    vis, ids = _inputs(p)
    st, _, _ = orc.prefill(vis, 0, ids)
    orc.compress_visual(st, p["k_visual"] if k is None else k)
    return st, vis, ids


def _zero(orc, *names):
    for n in names:
        orc.dw[n] = torch.zeros_like(orc.dw[n])


def test_parameter_counts_match_the_sizes_the_paper_prints():
    """Section 4 gives 0.65B for the 7B target's draft and 0.98B for the 13B one.  Three blocks of
    the target's widths, each with an MLP, give 0.61B and 0.95B; with one block it would be a third,
    and with MLP-less attention blocks less than half."""
    for preset, printed in (("llava7b", 0.65e9), ("llava13b", 0.98e9)):
        p = configs.scaled(preset, draft_blocks=3)
        d, H, Hkv, hd, ff = (p[k] for k in ("d_model", "n_heads", "n_kv_heads", "head_dim", "d_ff"))
        shapes = {"ln1": d, "wqkv": (H + 2 * Hkv) * hd * d, "wo": d * H * hd, "i_ln2": d, "i_wgu": 2 * ff * d,
                  "i_wd": d * ff, "lnx": d, "xq": H * hd * d, "xkv": 2 * Hkv * hd * d, "xo": d * H * hd, "ln2": d,
                  "wgu": 2 * ff * d, "wd": d * ff, "f_ln1": d, "f_wqkv": (H + 2 * Hkv) * hd * d, "f_wo": d * H * hd,
                  "f_ln2": d, "f_wgu": 2 * ff * d, "f_wd": d * ff}
        # the generator makes exactly these tensors (checked on a narrow model, same key set)
        small = synth.draft_weights(tiny_preset(draft_blocks=3))
        assert set(small) == set(shapes)
        total = sum(shapes.values())
        assert 0.9 * printed < total < 1.0 * printed, (preset, total)


def test_one_block_draft_is_untouched_by_the_extra_tensors():
    p1, a = make_oracle(tiny_preset(), D64)
    p3, b = make_oracle(tiny_preset(draft_blocks=3), D64)
    for k in a.dw:
        assert torch.equal(a.dw[k], b.dw[k])            # the shared tensors are the same numbers
    b.cfg.draft_blocks = 1                               # extra tensors present, single-block path taken
    sa, _, _ = _ready(p1, a)
    sb, _, _ = _ready(p3, b)
    ta, tb = a.draft_tree(sa), b.draft_tree(sb)
    assert ta["tokens"] == tb["tokens"] and ta["parent"] == tb["parent"]
    assert all(torch.equal(x, y) for x, y in zip(ta["feats"], tb["feats"]))


def test_without_the_middle_block_the_draft_is_a_two_layer_causal_decoder():
    """xo = 0 and the middle MLP's down projection = 0 make the cross-attention block the identity.
    What is left must equal the oracle's target path run with two layers made of the draft's initial
    and final tensors: same logits for the root and along a chain, keep-all context so that the
    draft's positions are 0..n-1 as in the target."""
    p, orc = make_oracle(tiny_preset(draft_blocks=3, tree_topk=1, tree_beam=1, tree_max_nodes=3), D64)
    _zero(orc, "xo", "wd")
    st, vis, ids = _ready(p, orc, k=p["n_visual"])
    dw, tw = orc.dw, orc.tw
    tw2 = {"embed": tw["embed"], "ln_f": tw["ln_f"], "lm_head": tw["lm_head"],
           "ln1": [dw["ln1"], dw["f_ln1"]], "wqkv": [dw["wqkv"], dw["f_wqkv"]], "wo": [dw["wo"], dw["f_wo"]],
           "ln2": [dw["i_ln2"], dw["f_ln2"]], "wgu": [dw["i_wgu"], dw["f_wgu"]], "wd": [dw["i_wd"], dw["f_wd"]]}
    p2 = dict(p, n_layers=2, tap_lo=1, tap_hi=2)
    two = O.DreamOracle(O.OracleConfig.from_preset(p2), tw2, dw, D64)
    tree = orc.draft_tree(st)
    chain = tree["in_tok"]                                # pending token, then the draft's own chain
    assert len(chain) == p["tree_depth"]
    st2, _, _ = two.prefill(vis, 0, ids, extra_ids=chain)
    n = st.P
    want = torch.log_softmax(two._logits(two._last_hidden[n:]), dim=-1)
    got = torch.stack(tree["logp_rows"])
    assert torch.allclose(got, want, atol=1e-10)
    # and the cached rows of both self-attention blocks are the two layers' K/V rows of the prompt
    assert torch.allclose(st.dK, st2.K[0][:n], atol=1e-12) and torch.allclose(st.fK, st2.K[1][:n], atol=1e-10)
    assert torch.allclose(st.dV, st2.V[0][:n], atol=1e-12) and torch.allclose(st.fV, st2.V[1][:n], atol=1e-10)


def test_without_the_decoder_blocks_the_draft_is_the_single_block_one():
    """wo = 0 and a zero down projection make a decoder block the identity; with both switched off
    the three-block draft keeps Eq. 1 and its MLP, which is the single-block draft with wo = 0."""
    p3, b = make_oracle(tiny_preset(draft_blocks=3), D64)
    p1, a = make_oracle(tiny_preset(), D64)
    _zero(b, "wo", "i_wd", "f_wo", "f_wd")
    _zero(a, "wo")
    sa, _, _ = _ready(p1, a)
    sb, _, _ = _ready(p3, b)
    for _ in range(3):
        ta, tb = a.draft_tree(sa), b.draft_tree(sb)
        assert ta["tokens"] == tb["tokens"] and ta["parent"] == tb["parent"]
        assert max(float((x - y).abs().max()) for x, y in zip(ta["feats"], tb["feats"])) < 1e-12
        a.step(sa, ta)
        b.step(sb, tb)


def test_every_tree_node_equals_its_own_path_drafted_as_a_chain():
    """Brute force over paths: for each input node of the tree pass, a chain draft forced along its
    root path gives the same feature, so nothing off the path leaks into a row."""
    p, orc = make_oracle(tiny_preset(draft_blocks=3), D64)
    st, _, _ = _ready(p, orc)
    tree = orc.draft_tree(st)
    in_tok, in_anc = tree["in_tok"], tree["in_anc"]
    assert len(tree["feats"]) == len(in_tok) > p["tree_depth"]          # some pass expanded several nodes
    for r in range(len(in_tok)):
        assert in_anc[r][0] == 0 and in_anc[r][-1] == r
        feat = chain_feature(orc, st, [in_tok[a] for a in in_anc[r]])
        assert torch.allclose(feat, tree["feats"][r], atol=1e-11), r
    # the rows of two siblings differ (the check above is not vacuous)
    assert not torch.allclose(tree["feats"][1], tree["feats"][2], atol=1e-6)


def chain_feature(orc, st, path):
    """e^M of the last token of `path` when the draft runs it as a chain from the same state."""
    import copy
    s2 = copy.deepcopy(st)
    c = orc.cfg
    empty = torch.empty(0, c.n_kv_heads, c.head_dim, dtype=D64)
    tr = {n: empty.clone() for n in ("K", "V", "mK", "mV", "fK", "fV")}
    h = None
    for j, tok in enumerate(path):
        h = orc._draft_pass3(s2, tr, [j], [tok], [s2.P + j], [list(range(j + 1))])
    return h[0]


def test_rows_appended_round_by_round_equal_a_fresh_draft_prefill():
    """After some rounds the two self-attention caches and the memory hold what compressing a fresh
    prefill of prompt + emitted tokens (same kept visual tokens) builds in one go."""
    p, orc = make_oracle(tiny_preset(draft_blocks=3), D64)
    st, vis, ids = _ready(p, orc)
    emitted = [st.pending]
    for _ in range(4):
        emitted += orc.step(st)["out"]
    orc.draft_tree(st)                                    # catches up with the last acceptance
    assert len(emitted) > 5                               # some round accepted more than the bonus token
    _, fresh = make_oracle(tiny_preset(draft_blocks=3), D64)
    fresh.tw["lm_head"] = orc.tw["lm_head"]
    st2, tok2, _ = fresh.prefill(vis, 0, ids, extra_ids=emitted[:-1])
    st2.tap = st.tap
    fresh.compress_visual(st2, p["k_visual"], forced_idx=st.kept)
    assert tok2 == st.pending and torch.equal(st2.dpos, st.dpos) and torch.equal(st2.mpos, st.mpos)
    for a, b in ((st.dK, st2.dK), (st.dV, st2.dV), (st.fK, st2.fK), (st.fV, st2.fV), (st.mK, st2.mK)):
        assert a.shape == b.shape and torch.allclose(a, b, atol=1e-10)


def test_a_memory_row_is_seen_by_strictly_later_positions_only():
    """Perturb the tapped feature of one context position j: the final block's rows at positions
    <= j stay bit-identical, the row at the next context position moves."""
    p, orc = make_oracle(tiny_preset(draft_blocks=3), D64)
    st, vis, ids = _ready(p, orc)
    base = st.fK.clone()
    C = st.ctx_pos.tolist()
    i = len(C) // 2
    j = C[i]
    st.taps[st.tap][j] += 0.5
    orc.compress_visual(st, p["k_visual"], forced_idx=st.kept)
    assert torch.equal(st.fK[:i + 1], base[:i + 1])
    assert float((st.fK[i + 1] - base[i + 1]).abs().max()) > 1e-9
    # position 0 sees no memory at all: its middle block adds only the MLP term
    assert int((st.mpos < st.dpos[0]).sum()) == 0


def test_speculative_output_equals_greedy_autoregressive():
    p, orc = make_oracle(tiny_preset(draft_blocks=3), D64)
    st, vis, ids = _ready(p, orc)
    ref, margins = orc.ar_decode(vis, 0, ids, 24)
    assert min(margins) > 1e-9
    out, acc = [st.pending], []
    while len(out) < 20:
        r = orc.step(st)
        out += r["out"]
        acc.append(r["A"])
    assert out[:20] == ref[:20]
