"""Named model/tree shapes of the five benchmark workloads.

Shapes only: this module holds no arithmetic of the method.  Each preset is a
plain dict so that both the CPU oracle's tests and the CUDA binding can build
their own configuration objects from it.

Notation follows the paper (Section 3): the target has L blocks, the prompt has
q text tokens and v visual tokens, k visual tokens are kept by the compression
step, the draft tree has depth D, K children per expanded node and at most N
draft nodes.
"""

TAP_FIXED, TAP_ENTROPY_MIN, TAP_ENTROPY_MAX = 0, 1, 2


def _mid(L):
    """Middle-layer range used by the entropy tap modes: [ceil(L/4), floor(3L/4)], 1-based."""
    lo = (L + 3) // 4
    return lo, max(lo, (3 * L) // 4)


def _preset(name, dtype, L, d, H, Hkv, hd, ff, V, v, k, q, D, K, N, steps, batch,
            tap_mode, tap_layer=0):
    lo, hi = _mid(L)
    return dict(name=name, dtype=dtype, n_layers=L, d_model=d, n_heads=H, n_kv_heads=Hkv,
                head_dim=hd, d_ff=ff, vocab=V, n_visual=v, k_visual=k, n_prompt=q,
                tree_depth=D, tree_topk=K, tree_beam=K, tree_max_nodes=N,
                decode_steps=steps, batch=batch, tap_mode=tap_mode, tap_layer=tap_layer,
                tap_lo=lo, tap_hi=hi, rms_eps=1e-5, rope_theta=10000.0,
                score_include_self=0, xattn_full_memory=0, vis_start=0)


PRESETS = {
    # Toy VLM, fp32.  The tree is the complete K-ary tree of depth D (beam unbounded).
    "toy": dict(_preset("toy", "f32", 2, 256, 4, 4, 64, 1024, 1024, 64, 16, 32,
                        3, 2, 14, 16, 1, TAP_FIXED, 1), tree_beam=4),
    "smolvlm2b": _preset("smolvlm2b", "bf16", 24, 2048, 32, 32, 64, 8192, 49152,
                         1024, 256, 128, 5, 4, 60, 128, 1, TAP_ENTROPY_MIN),
    "llava7b": _preset("llava7b", "bf16", 32, 4096, 32, 32, 128, 11008, 32000,
                       576, 144, 256, 6, 8, 60, 256, 1, TAP_ENTROPY_MAX),
    "llava7b_b4": _preset("llava7b_b4", "bf16", 32, 4096, 32, 32, 128, 11008, 32000,
                          576, 144, 256, 6, 8, 60, 256, 4, TAP_ENTROPY_MAX),
    "pixtral12b": _preset("pixtral12b", "bf16", 40, 5120, 32, 8, 128, 14336, 131072,
                          1024, 256, 512, 6, 8, 60, 64, 1, TAP_ENTROPY_MIN),
    # LLaVA-1.5-13B-shaped target (Section 4 lists the 13B model among the targets): same prompt and
    # tree as the 7B-shaped workload.
    "llava13b": _preset("llava13b", "bf16", 40, 5120, 40, 40, 128, 13824, 32000,
                        576, 144, 256, 6, 8, 60, 256, 1, TAP_ENTROPY_MAX),
    "gemma3_12b": _preset("gemma3_12b", "bf16", 48, 3840, 16, 8, 256, 15360, 262144,
                          256, 64, 4096, 7, 10, 80, 64, 1, TAP_ENTROPY_MIN),
}


def scaled(name, **over):
    """A preset with some fields replaced (used for reduced-size parity cases)."""
    p = dict(PRESETS[name])
    p.update(over)
    if "n_layers" in over and "tap_lo" not in over:
        p["tap_lo"], p["tap_hi"] = _mid(p["n_layers"])
    return p
