"""Helpers shared by the oracle tests: build an oracle for a preset on the CPU."""
import torch

from oracle.dream_oracle import DreamOracle, OracleConfig
from paper_2505_19201_b200 import configs, synth


def make_oracle(preset, dtype=torch.float64, seed=0, kv_dtype=None, **over):
    p = configs.scaled(preset, **over) if isinstance(preset, str) else dict(preset, **over)
    tw = synth.target_weights(p, seed)
    dw = synth.draft_weights(p, seed)
    return p, DreamOracle(OracleConfig.from_preset(p), tw, dw, dtype, kv_dtype=kv_dtype)


def tiny_preset(**over):
    """A model small enough for pure-Python brute force."""
    p = configs.scaled("toy", n_layers=2, d_model=32, n_heads=4, n_kv_heads=2, head_dim=8,
                       d_ff=48, vocab=50, n_visual=6, k_visual=3, n_prompt=5,
                       tree_depth=3, tree_topk=2, tree_beam=4, tree_max_nodes=14)
    p.update(over)
    return p
