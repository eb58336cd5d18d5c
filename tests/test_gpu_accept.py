"""Acceptance on the GPU with accept lengths above zero: trees that contain the target's own greedy
continuation are injected into both sides (a randomly initialised draft is almost never right),
for the greedy rule and for the sampling rule at several temperatures."""
import json

import pytest
import torch

pytestmark = pytest.mark.gpu


def continuation_tree(pr, seq, depth):
    """Tokens and parents of a T-node tree whose nodes 1..depth are the oracle's greedy
    continuation of the pending token (a chain); the remaining nodes are further children of the
    root with other tokens."""
    from oracle.dream_oracle import make_tree
    st, T, V = pr.st[seq], pr.T, pr.p["vocab"]

    def padded(chain):
        tokens, parent = [st.pending] + chain, [-1] + list(range(len(chain)))
        first = chain[0] if chain else -1
        t = 0
        while len(tokens) < T:
            if t != first:
                tokens.append(t)
                parent.append(0)
            t += 1
        return tokens, parent

    chain = []
    for _ in range(depth):
        tokens, parent = padded(chain)
        ver = pr.orc.verify_tree(st, make_tree(tokens, parent))
        chain.append(ver["argmax"][len(chain)])
    tokens, parent = padded(chain)
    return dict(tokens=tokens, parent=parent)


def test_toy_greedy_accepts_injected_continuation():
    from tests.parity import Pair
    pr = Pair("toy")
    try:
        pr.prefill()
        got = []
        for depth in (1, 2, 3, 0, 3):
            got.append(pr.step(inject={0: continuation_tree(pr, 0, depth)})[0]["A"])
        print(json.dumps(dict(pr.summary(), accepted=got), default=float))
        if pr.summary()["exempt"] == 0:
            assert got == [1, 2, 3, 0, 3]
        assert max(got) == 3
    finally:
        pr.close()


def test_toy_sampled_acceptance():
    """Sampling rule at temperatures from near-greedy to 1: kept children, refusals with the
    renormalised rest, and final draws all occur; state and caches stay equal to the oracle's."""
    from tests.parity import Pair
    pr = Pair("toy")
    try:
        pr.prefill()
        gen = torch.Generator().manual_seed(11)
        got = []
        for i in range(12):
            temp = (0.01, 0.05, 0.2, 1.0)[i % 4]
            got.append(pr.step(inject={0: continuation_tree(pr, 0, 3)}, temp=temp, gen=gen)[0]["A"])
        print(json.dumps(dict(pr.summary(), accepted=got), default=float))
        assert max(got) >= 1 and min(got) == 0
        assert pr.summary()["exempt"] <= 2
    finally:
        pr.close()


@pytest.mark.parametrize("preset", ["llava7b", "smolvlm2b"])
def test_bf16_shapes_sampled_and_greedy_acceptance(preset):
    """LLaVA-7B-shaped (vocab 32000: the sampling kernel keeps a row's exponentials in registers) and
    SmolVLM-2B-shaped widths (vocab 49152: it re-reads the row per trial), 61 tree rows, 2 layers:
    injected continuation of depth 2, greedy rule, then the sampling rule near greedy and at
    temperature 1."""
    from tests.parity import Pair
    pr = Pair(preset, n_layers=2, n_visual=96, k_visual=24, n_prompt=32, decode_steps=8)
    try:
        pr.prefill()
        gen = torch.Generator().manual_seed(12)
        got = [pr.step(inject={0: continuation_tree(pr, 0, 2)})[0]["A"]]
        for temp in (0.002, 0.05, 1.0):
            got.append(pr.step(inject={0: continuation_tree(pr, 0, 2)}, temp=temp, gen=gen)[0]["A"])
        print(json.dumps(dict(pr.summary(), accepted=got), default=float))
        assert got[0] >= 1
    finally:
        pr.close()
