"""The three-block draft (Section 4: an initial decoder block, an intermediate cross-attention block,
a final decoder block) through the C ABI against the oracle: the draft's run over the compressed
context at set-up, the catch-up rows of accepted tokens, and the tree passes, at the toy widths in
fp32 and at LLaVA-7B- and SmolVLM-shaped widths in bf16."""
import json

import pytest

pytestmark = pytest.mark.gpu


def _run(preset, steps, prefill=None, **over):
    from tests.parity import Pair
    pr = Pair(preset, draft_blocks=3, **over)
    try:
        pr.prefill(**(prefill or {}))
        accepted = []
        for _ in range(steps):
            accepted.append(pr.step()[0]["A"])
        pr.orc.draft_tree(pr.st[0])
        pr.ctx.dream_draft_tree([0])
        pr.ctx.dream_poll()
        pr.check_draft_cache()
        s = pr.summary()
        s["accepted"] = accepted
        print(json.dumps(s, default=float))
        assert any("final-block" in what for what in s["worst"]), "the final block's rows were not compared"
        return s
    finally:
        pr.close()


def test_toy_fp32_full_decode():
    """Config 1 widths in fp32, 16 rounds: every catch-up length the acceptances produce."""
    _run("toy", 16)


def test_llava_shape_4_layers_bf16():
    """d 4096, 32 heads of 128, MLP 11008, vocab 32000; four target layers under the draft; the
    context (35 text + 432 kept visual tokens) spans several row chunks of the draft's set-up run."""
    _run("llava7b", 3, n_layers=4, decode_steps=8)


def test_smolvlm_shape_bf16():
    """Heads of 64 (d 2048), 4 target layers."""
    _run("smolvlm2b", 2, n_layers=4, decode_steps=6)


def test_memory_keeps_every_prompt_position():
    """xattn_full_memory = 1: a context row at position p sees p memory rows, not its own index."""
    _run("llava7b", 2, n_layers=2, n_visual=96, k_visual=24, n_prompt=40, decode_steps=6, xattn_full_memory=1)


def test_visual_span_after_the_text_and_no_kept_visual_token():
    _run("llava7b", 1, prefill=dict(vis_start=40), n_layers=2, n_visual=96, k_visual=0, n_prompt=40, decode_steps=6)


@pytest.mark.parametrize("preset,over", [("toy", {}), ("llava7b", dict(n_layers=2, n_visual=96, k_visual=24, n_prompt=32, decode_steps=8))])
def test_catch_up_rows_after_accepted_tokens(preset, over):
    """A randomly initialised draft is almost never right, so trees holding the target's own greedy
    continuation are injected: accept lengths 1, 3, 0, 2 leave 2, 4, 1, 3 tokens for the next draft call
    to run through the three blocks before its tree passes, each seeing the rows and the memory of
    earlier positions only.  The rows they leave in both decoder blocks' caches are compared."""
    from tests.parity import Pair
    from tests.test_gpu_accept import continuation_tree
    pr = Pair(preset, draft_blocks=3, **over)
    try:
        pr.prefill()
        got = []
        for depth in (1, 3, 0, 2):
            got.append(pr.step(inject={0: continuation_tree(pr, 0, min(depth, pr.p["tree_depth"]))})[0]["A"])
        pr.step()                                       # the draft after the last acceptance
        pr.check_draft_cache()
        n = pr.st[0].fK.shape[0]
        for row in range(n - 6, n):                     # the rows the catch-up passes appended
            from tests.parity import close
            close(pr.ctx.dream_debug_read(0, 8, 0, row), pr.st[0].fK[row].flatten(), pr.tol, "draft final-block K row", pr.report)
            close(pr.ctx.dream_debug_read(0, 4, 0, row), pr.st[0].dK[row].flatten(), pr.tol, "draft K row", pr.report)
        s = dict(pr.summary(), accepted=got)
        print(json.dumps(s, default=float))
        assert max(got) >= 2, got
    finally:
        pr.close()


def test_two_sequences():
    from tests.parity import Pair
    pr = Pair("llava7b", draft_blocks=3, max_batch=2, n_layers=2, n_visual=96, k_visual=24, n_prompt=40, decode_steps=6)
    try:
        pr.prefill(seq=0, seq_seed=0)
        pr.prefill(seq=1, seq_seed=1, n_visual=48, n_prompt=21, k=12)
        for _ in range(2):
            pr.step(seqs=(0, 1))
        pr.step(seqs=(1, 0))
        print(json.dumps(pr.summary(), default=float))
    finally:
        pr.close()


def test_chain_shaped_three_block_draft_with_running_entropy_and_sampling():
    """The options together: one child per node (a chain of depth D), Eq. 2 kept up to date, and an
    acceptance by the sampling rule at temperature 1 after a greedy one."""
    import torch
    from tests.parity import Pair
    from tests.test_gpu_accept import continuation_tree
    pr = Pair("llava7b", draft_blocks=3, track_entropy=1, tree_topk=1, tree_beam=1, tree_max_nodes=6,
              n_layers=2, n_visual=96, k_visual=24, n_prompt=40, decode_steps=8)
    try:
        pr.prefill()
        gen = torch.Generator().manual_seed(5)
        got = [pr.step(inject={0: continuation_tree(pr, 0, 2)})[0]["A"]]
        got.append(pr.step(inject={0: continuation_tree(pr, 0, 3)}, temp=1.0, gen=gen)[0]["A"])
        pr.step()
        pr.check_draft_cache()
        ae_g, _ = pr.ctx.dream_layer_entropy(0)
        ae_o, _, _ = pr.orc.layer_entropy(pr.st[0])
        assert float((ae_g.double() - ae_o.double()).abs().max()) <= 1e-3
        print(json.dumps(dict(pr.summary(), accepted=got), default=float))
    finally:
        pr.close()
