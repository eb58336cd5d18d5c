"""Eq. 2 kept up to date while decoding (Section 3.2: the layer is selected "during each decoding
step"): with track_entropy = 1 the verification leaves every tree row's attention entropy and the
acceptance adds those of the committed rows to the prefill's per-layer sums.  Compared with the
oracle's running sums (which are pinned on the CPU against a full recomputation) after rounds with
accept lengths above zero, on the fp32 toy and at bf16 widths with one and with several key chunks."""
import json

import pytest
import torch

pytestmark = pytest.mark.gpu

AE_TOL = 1e-3          # absolute, as for the prefill's AE


def _check(pr, seq=0):
    ae_g, layer_g = pr.ctx.dream_layer_entropy(seq)
    ae_o, layer_o, margin = pr.orc.layer_entropy(pr.st[seq])
    gap = float((ae_g.double() - ae_o.double()).abs().max())
    assert gap <= AE_TOL, f"AE gap {gap:.3e}"
    if margin > 2 * AE_TOL:
        assert layer_g == layer_o
    return gap


@pytest.mark.parametrize("preset,over", [
    ("toy", {}),
    ("llava7b", dict(n_layers=4, n_visual=96, k_visual=24, n_prompt=32, decode_steps=10)),       # 3 key blocks
    ("llava7b", dict(n_layers=2, decode_steps=10)),                                            # 832-row prefix: several chunks
    ("smolvlm2b", dict(n_layers=3, n_visual=192, k_visual=48, n_prompt=64, decode_steps=10)),   # heads of 64
])
def test_running_entropy_follows_the_oracle(preset, over):
    from tests.parity import Pair
    from tests.test_gpu_accept import continuation_tree
    pr = Pair(preset, track_entropy=1, **over)
    try:
        pr.prefill()
        gaps = [_check(pr)]                                     # nothing committed yet: the prefill's AE
        got = []
        for depth in (2, 0, 3, 1):
            got.append(pr.step(inject={0: continuation_tree(pr, 0, min(depth, pr.p["tree_depth"]))})[0]["A"])
            gaps.append(_check(pr))
        pr.step()
        gaps.append(_check(pr))
        P, _, _ = pr.ctx.dream_seq_state(0)
        assert P == pr.st[0].P
        print(json.dumps(dict(accepted=got, ae_gaps=gaps, exempt=pr.report["exempt"]), default=float))
        assert max(got) >= 2
    finally:
        pr.close()


def test_two_sequences_keep_their_own_sums():
    from tests.parity import Pair
    pr = Pair("llava7b", track_entropy=1, max_batch=2, n_layers=2, n_visual=96, k_visual=24, n_prompt=40, decode_steps=6)
    try:
        pr.prefill(seq=0, seq_seed=0)
        pr.prefill(seq=1, seq_seed=1, n_visual=48, n_prompt=21, k=12)
        for _ in range(2):
            pr.step(seqs=(0, 1))
        pr.step(seqs=(1, 0))
        _check(pr, 0)
        _check(pr, 1)
    finally:
        pr.close()


def test_the_call_needs_the_flag():
    from paper_2505_19201_b200 import api
    from tests.parity import Pair
    pr = Pair("toy")
    try:
        pr.prefill()
        with pytest.raises(api.DreamError) as e:
            pr.ctx.dream_layer_entropy(0)
        assert e.value.code == -2
    finally:
        pr.close()
