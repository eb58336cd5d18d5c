"""CUDA path vs CPU oracle through the C ABI, element by element, on seeded inputs."""
import json
import os

import pytest
import torch

pytestmark = pytest.mark.gpu


def _run(preset, steps, **over):
    from tests.parity import Pair
    pr = Pair(preset, **over)
    try:
        pr.prefill()
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
        return pr, s
    finally:
        pr.close()


def test_toy_fp32_full_decode():
    """Config 1: toy VLM in fp32, complete binary tree of depth 3, 16 decode steps."""
    pr, s = _run("toy", 16)
    assert s["exempt"] <= 2
