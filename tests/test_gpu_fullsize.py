"""The LLaVA-7B-shaped workload at its full size (32 layers, 576 visual + 256 text tokens, 61 tree
rows, batch 1), the configuration the benchmark times."""
import json

import pytest
import torch

pytestmark = pytest.mark.gpu


def test_llava_full_size_against_the_oracle():
    """Prefill, compression and one whole round at full size against the oracle, element by element
    (about two minutes of CPU time for the oracle's prefill and round)."""
    from tests.test_gpu_parity import _run
    _run("llava7b", 1, decode_steps=4, stated_miss=FULL_SIZE_MISS)


def test_llava_full_size_three_block_draft_against_the_oracle():
    """The same workload with the draft of Section 4 (initial decoder block, cross-attention block,
    final decoder block): the draft's run over the 400-row compressed context, one round, and the
    draft call after it (catch-up row), element by element."""
    from tests.test_gpu_parity import _run
    # Stated misses of the flat 3e-2 (all with relative L2 below 1e-2): the tree this draft proposes holds a
    # node whose verify logits are off by 3.4e-2 (one of 61 x 32000 values; relative L2 2.1e-3; target path);
    # the final decoder block's cache rows inherit the memory rows' relative difference (2e-3 at the
    # tapped layer 20, rms 12.6) through the peaked softmax of Eq. 1: 3.9e-2 / 4.9e-2 on K / V rows
    # (a row that sees a single memory row differs by exactly that 2e-3; the row that sees none by 8e-6)
    miss = dict(FULL_SIZE_MISS, **{"verify logits": 5e-2, "draft final-block K row": 8e-2, "draft final-block V row": 8e-2})
    pr, s = _run("llava7b", 1, decode_steps=4, stated_miss=miss, draft_blocks=3)
    assert any("final-block" in what for what in s["worst"])


def test_llava_full_size_output_does_not_depend_on_the_tree():
    """Section 2.1: whatever the draft proposes, the emitted tokens are the target's own greedy
    continuation.  At full size three decodes of the same request must therefore emit the same
    token sequence, position by position, up to the first decision whose top-1/top-2 margin is
    below the decision tolerance: (a) rounds that verify a tree with nothing to accept (every node
    a child of the root carrying a token the target does not choose: one token per round), (b)
    rounds with the library's own draft trees, (c) rounds whose tree holds the continuation found
    in (a) as a chain of depth D, which must be accepted in full and compacted."""
    from paper_2505_19201_b200 import api, configs, synth
    dev = "cuda:0"
    p = configs.scaled("llava7b", decode_steps=40)
    tw, dw = synth.target_weights(p, 0, dev), synth.draft_weights(p, 0, dev)
    ctx = api.Context(api.make_config(p), tw, dw, dev)
    try:
        T, D = ctx.T, p["tree_depth"]
        vis, ids = synth.request_inputs(p, 0, dev)
        am = torch.zeros(T, dtype=torch.int32, device=dev)
        mg = torch.zeros(T, dtype=torch.float32, device=dev)
        alen = torch.zeros(1, dtype=torch.int32, device=dev)
        outt = torch.zeros(D + 1, dtype=torch.int32, device=dev)
        csrc = torch.zeros(D + 1, dtype=torch.int32, device=dev)

        def star(pending, avoid):
            toks = [pending] + [t if t != avoid else T + 1 for t in range(1, T)]
            return toks, [-1] + [0] * (T - 1)

        def decode(rounds, mode, known=None):
            first = torch.zeros(1, dtype=torch.int32, device=dev)
            ctx.dream_seq_reset(0)
            ctx.dream_prefill(0, vis, 0, ids, first)
            ctx.dream_compress_visual(0, p["k_visual"])
            toks, margins, lens = [int(first)], [], []
            tree = ctx.new_tree()
            for _ in range(rounds):
                P0, pending, _ = ctx.dream_seq_state(0)
                assert pending == toks[-1]
                if mode == "own":
                    ctx.dream_draft_tree([0], [tree])
                    ctx.dream_verify_tree([0], [tree], am, mg)
                else:
                    ctx.dream_draft_tree([0], None)             # keeps the draft's caches in step
                    if mode == "chain":
                        nxt = known[len(toks):len(toks) + D]
                        tk, par = star(pending, nxt[0])
                        tk[1:1 + D], par[1:1 + D] = nxt, list(range(D))
                        tree.load(tk, par)
                        ctx.dream_verify_tree([0], [tree], am, mg)
                    else:
                        tree.load(*star(pending, -1))
                        ctx.dream_verify_tree([0], [tree], am, mg)
                        # the root's row does not depend on its children: take the target's choice
                        # out of the proposals before the acceptance reads them
                        tree.load(*star(pending, int(am[0])))
                ctx.dream_accept([0], [tree], am, alen, outt, csrc)
                ctx.dream_poll()
                A = int(alen[0])
                path = csrc.cpu().tolist()[:A + 1]
                host = tree.to_host()
                assert path[0] == 0 and all(host["parent"][c] == q for q, c in zip(path, path[1:]))
                out = outt.cpu().tolist()[:A + 1]
                assert out[:-1] == [host["tokens"][c] for c in path[1:]]
                assert out == [int(am[c]) for c in path]        # every emitted token is a target argmax
                P1, _, _ = ctx.dream_seq_state(0)
                assert P1 == P0 + A + 1
                toks += out
                margins += [float(mg[c]) for c in path]
                lens.append(A)
            return toks, margins, lens

        def same_until_near_tie(a, ma, b, mb, what):
            for i in range(1, min(len(a), len(b))):
                if a[i] != b[i]:
                    assert min(ma[i - 1], mb[i - 1]) < 1e-2, f"{what}: token {i}: {a[i]} vs {b[i]}, margins {ma[i - 1]}, {mb[i - 1]}"
                    return i
            return min(len(a), len(b))

        n_tok = 3 * (D + 1) + D
        sa, ma, la = decode(n_tok, "star")
        assert la == [0] * n_tok and len(sa) == n_tok + 1
        sb, mb, lb = decode(6, "own")
        sc, mc, lc = decode(3, "chain", known=sa)
        nb = same_until_near_tie(sa, ma, sb, mb, "own trees")
        nc = same_until_near_tie(sa, ma, sc, mc, "continuation chains")
        if nc == len(sc):
            assert lc == [D] * 3, f"accept lengths {lc}"
        print(json.dumps(dict(tokens=len(sa), own_accept_lengths=lb, chain_accept_lengths=lc, compared=[nb, nc],
                              min_margin=min(ma))))
    finally:
        ctx.close()


# The draft's per-level log-probabilities are the one quantity that misses the flat max-abs 3e-2 at
# full size: the cross-attention memory of Eq. 1 holds unnormalised rows of a deep layer (rms about 13
# at layer 20 of 32), the softmax over it is sharply peaked, and the 2e-3 relative difference of the
# tapped features (within the rel-L2 bound) moves the draft's output by up to this much.  Measured:
# 1.7e-2 .. 4.9e-2 on the LLaVA-7B shape (memory rms 12.6), 1.2e-1 on the Pixtral shape (rms 23).
FULL_SIZE_MISS = {"draft logp (per level)": 8e-2}
FULL_SIZE_MISS_BY_PRESET = {"pixtral12b": {"draft logp (per level)": 2e-1}, "gemma3_12b": FULL_SIZE_MISS}


def test_llava_full_size_batch_4_against_the_oracle():
    """Config 3 with batch 4 at its full depth: four requests (input seeds 0..3) prefilled one by one,
    then one round of all four in one call (244 rows: two token tiles per weight panel), every
    sequence against its own oracle run."""
    from tests.parity import Pair
    pr = Pair("llava7b_b4", decode_steps=4, stated_miss=FULL_SIZE_MISS)
    try:
        seqs = (0, 1, 2, 3)
        for s in seqs:
            pr.prefill(seq=s, seq_seed=s)
        pr.step(seqs=seqs)
        print(json.dumps(pr.summary(), default=float))
    finally:
        pr.close()


@pytest.mark.parametrize("preset", ["pixtral12b", "gemma3_12b"])
def test_large_presets_full_size_against_the_oracle(preset):
    """The Pixtral-12B-shaped and Gemma3-12B-shaped workloads at full size (40 / 48 layers, prefixes
    of 1536 / 4352 tokens) against the oracle: prefill, compression and one round, element by
    element (about one and two minutes of oracle time on 16 cores)."""
    from tests.test_gpu_parity import _run
    _run(preset, 1, decode_steps=4, stated_miss=FULL_SIZE_MISS_BY_PRESET[preset])
