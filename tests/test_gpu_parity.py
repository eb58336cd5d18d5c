"""CUDA path vs CPU oracle through the C ABI, element by element, on seeded inputs."""
import json
import os

import pytest
import torch

pytestmark = pytest.mark.gpu


def _run(preset, steps, stated_miss=None, **over):
    from tests.parity import Pair
    pr = Pair(preset, stated_miss=stated_miss, **over)
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


def test_llava_shape_4_layers_bf16():
    """LLaVA-7B-shaped widths (d 4096, 32 heads of 128, MLP 11008, vocab 32000), 4 layers."""
    pr, s = _run("llava7b", 3, n_layers=4, decode_steps=8)


def test_smolvlm_shape_full_bf16():
    """Config 2: SmolVLM-2B-shaped target, all 24 layers, 4 decode steps."""
    pr, s = _run("smolvlm2b", 4)


def test_llava_shape_full_depth_bf16():
    """Config 3 at its full depth (32 layers, 61 tree nodes) with a shortened prompt so that the
    oracle's prefill stays cheap; two rounds."""
    pr, s = _run("llava7b", 2, n_visual=192, k_visual=48, n_prompt=64, decode_steps=4)


def test_pixtral_shape_gqa_bf16():
    """Config 4 widths (d 5120, 32 query / 8 KV heads of 128, MLP 14336, vocab 131072), 2 layers,
    shortened prompt."""
    pr, s = _run("pixtral12b", 2, n_layers=2, n_visual=256, k_visual=64, n_prompt=96, decode_steps=4)


def test_gemma_shape_hd256_bf16():
    """Config 5 widths (d 3840, 16 query / 8 KV heads of 256, MLP 15360, vocab 262144, 81 tree rows:
    the two-plane GEMM input layout), 2 layers, shortened prompt."""
    pr, s = _run("gemma3_12b", 2, n_layers=2, n_visual=128, k_visual=32, n_prompt=192, decode_steps=4)


@pytest.mark.parametrize("batch", [2, 4])
def test_llava_shape_batched(batch):
    """Several sequences per call: 2 x 61 tree rows take the two-plane GEMM input layout, 4 x 61 rows
    are cut into 64-row launches; every sequence is checked against its own oracle run."""
    from tests.parity import Pair
    pr = Pair("llava7b", max_batch=batch, n_layers=2, n_visual=192, k_visual=48, n_prompt=64, decode_steps=4)
    try:
        seqs = tuple(range(batch))
        for s in seqs:
            pr.prefill(seq=s, seq_seed=s)
        for _ in range(2):
            pr.step(seqs=seqs)
        print(json.dumps(pr.summary(), default=float))
    finally:
        pr.close()
