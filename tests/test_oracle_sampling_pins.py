"""Pins of the oracle's sampling form of the acceptance (Section 2.1 acceptance rule at a
temperature above zero) against hand-computed cases and against the fact that fixes it: the
emitted tokens follow the target's own sampling distribution, whatever tree was proposed."""
import math

import torch

from oracle import dream_oracle as O

LOG = lambda ps: [math.log(p) for p in ps]


def _accept(tree, rows, temp, u):
    return O.DreamOracle.accept_sample(tree, torch.tensor(rows, dtype=torch.float64), temp, u)


def test_hand_example_refusal_renormalises():
    # root distribution (0.5, 0.3, 0.2); children propose token 0 then token 1
    tree = O.make_tree([7, 0, 1], [-1, 0, 0])
    rows = [LOG([0.5, 0.3, 0.2])] * 3
    # 0.6 >= 0.5 refuses token 0; token 1 then has 0.3 / 0.5 = 0.6 > 0.59: kept
    A, out, path, _ = _accept(tree, rows, 1.0, [[0.6, 0.59, 0.0], [0.0, 0.0, 0.0]])
    assert (A, path, out[0]) == (1, [0, 2], 1)
    # 0.61 refuses it too; what is left is token 2 alone
    A, out, path, _ = _accept(tree, rows, 1.0, [[0.6, 0.61, 0.3], [0.0, 0.0, 0.0]])
    assert (A, out, path) == (0, [2], [0])
    # below 0.5 the first child is kept and the walk goes on from its row
    A, out, path, _ = _accept(tree, rows, 1.0, [[0.49, 0.0, 0.0], [0.0, 0.0, 0.55]])
    assert (A, path, out) == (1, [0, 1], [0, 1])        # 0.55 falls in [0.5, 0.8): token 1


def test_final_draw_inverts_the_cumulative_sum_in_token_order():
    tree = O.make_tree([3], [-1])
    rows = [LOG([0.1, 0.2, 0.3, 0.4])]
    for u, want in ((0.0, 0), (0.0999, 0), (0.1001, 1), (0.2999, 1), (0.3001, 2), (0.5999, 2), (0.6001, 3), (0.9999, 3)):
        A, out, path, _ = _accept(tree, rows, 1.0, [[u]])
        assert (A, out, path) == (0, [want], [0])


def test_temperature_scales_the_logits():
    tree = O.make_tree([3], [-1])
    # at temp 2 the distribution is proportional to sqrt of (1/9, 4/9, 4/9)... = (1, 2, 2) / 5
    rows = [LOG([1 / 9, 4 / 9, 4 / 9])]
    for u, want in ((0.19, 0), (0.21, 1), (0.59, 1), (0.61, 2)):
        assert _accept(tree, rows, 2.0, [[u]])[1] == [want]


def test_refused_tokens_are_never_emitted_at_that_node():
    tree = O.make_tree([9, 2, 0, 3], [-1, 0, 0, 0])
    g = torch.Generator().manual_seed(5)
    for _ in range(200):
        rows = torch.randn(4, 6, dtype=torch.float64, generator=g)
        u = torch.rand(2, 4, dtype=torch.float64, generator=g)
        u[0, :3] = 1.0 - 1e-12                                  # every child refused
        A, out, path, _ = _accept(tree, rows.tolist(), 1.0, u.tolist())
        assert A == 0 and out[0] in (1, 4, 5)


def test_low_temperature_is_greedy_acceptance():
    g = torch.Generator().manual_seed(6)
    tokens, parent = [5, 0, 1, 2, 0, 1, 2, 3], [-1, 0, 0, 0, 1, 1, 2, 3]
    tree = O.make_tree(tokens, parent)
    for _ in range(100):
        rows = torch.randn(8, 4, dtype=torch.float64, generator=g)
        am = [int(torch.argmax(r)) for r in rows]
        want = O.DreamOracle.accept(tree, am)
        u = (torch.rand(4, 4, dtype=torch.float64, generator=g) * 0.98 + 0.01).tolist()
        A, out, path, _ = _accept(tree, rows.tolist(), 1e-3, u)
        assert (A, out, path) == want


def test_emitted_tokens_follow_the_target_distribution():
    """The first emitted token is distributed as softmax(root row / temp) and, given that it
    was child c's token, the second as softmax(row of c / temp): the acceptance rule samples
    from the target.  20000 draws; bound = 4.5 standard deviations of a frequency."""
    g = torch.Generator().manual_seed(7)
    V, temp, n = 5, 1.3, 20000
    tokens, parent = [0, 3, 1, 4, 2, 0], [-1, 0, 0, 0, 1, 1]       # three proposals under the root, two under node 1
    tree = O.make_tree(tokens, parent)
    rows = torch.randn(6, V, dtype=torch.float64, generator=g) * 1.5
    p0 = torch.softmax(rows[0] / temp, 0)
    p1 = torch.softmax(rows[1] / temp, 0)
    first, second, n1 = torch.zeros(V), torch.zeros(V), 0
    us = torch.rand(n, 3, 4, dtype=torch.float64, generator=g)
    for i in range(n):
        A, out, path, _ = O.DreamOracle.accept_sample(tree, rows, temp, us[i].tolist())
        first[out[0]] += 1
        if len(path) > 1 and path[1] == 1:
            second[out[1]] += 1
            n1 += 1
    for v in range(V):
        sd = math.sqrt(float(p0[v]) * (1 - float(p0[v])) / n)
        assert abs(float(first[v]) / n - float(p0[v])) < 4.5 * sd
        sd = math.sqrt(float(p1[v]) * (1 - float(p1[v])) / n1)
        assert abs(float(second[v]) / n1 - float(p1[v])) < 4.5 * sd
    # node 1 proposes token 3: it is walked into exactly when token 3 is emitted first
    assert n1 == int(first[3])


def test_sampled_rounds_leave_the_state_of_a_fresh_prefill():
    """Whole loop with the sampling rule: after several rounds whose trees hold plausible
    proposals, the target KV cache equals that of a fresh prefill of prompt + emitted tokens, and
    every emitted token was drawn from the target's row at its position (it has non-zero
    probability there and the pending token is the last one emitted)."""
    from tests.test_oracle_pins import _setup
    p, orc, st, vis, ids = _setup(scale=30.0)
    g = torch.Generator().manual_seed(21)
    D, V = p["tree_depth"], p["vocab"]
    emitted, lens = [st.pending], []
    for _ in range(5):
        # proposals: the two most likely tokens under the target at each level of a depth-D chain
        toks, par, last = [st.pending], [-1], 0
        for _lvl in range(D):
            ver = orc.verify_tree(st, O.make_tree(toks, par))
            top = torch.topk(ver["logits"][last], 2).indices.tolist()
            toks += top
            par += [last, last]
            last = len(toks) - 2
        T = len(toks)
        u = torch.rand(D + 1, T, dtype=torch.float64, generator=g)
        r = orc.step(st, O.make_tree(toks, par), temp=0.7, uniforms=u.tolist())
        assert len(r["out"]) == r["A"] + 1 and r["out"][-1] == st.pending
        emitted += r["out"]
        lens.append(r["A"])
    assert max(lens) >= 1
    st2, tok2, _ = orc.prefill(vis, 0, ids, extra_ids=emitted[:-1])
    assert st2.P == st.P
    for l in range(p["n_layers"]):
        assert torch.allclose(st.K[l], st2.K[l], atol=1e-10)
        assert torch.allclose(st.V[l], st2.V[l], atol=1e-10)
