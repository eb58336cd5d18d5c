"""Pins of the oracle's bf16 key/value store (`kv_dtype=torch.bfloat16`).

Section 4 runs every model with KV caching enabled; for the bf16 model shapes the cache is a
bf16 store.  The reading pinned here: a K/V row is rounded to bf16 exactly once, after the
rotary embedding, when it enters the cache, and before any query attends to it (its own row's
query included); queries are never rounded; everything computed from the cache stays in the
arithmetic type.  Each test below fails for one of the plausible mistakes: rounding before the
rotary embedding, rounding the queries too, or attending to the new rows before they are rounded.
None needs a GPU.
"""
import pytest
import torch

from oracle import dream_oracle as O
from tests.util_oracle import make_oracle, tiny_preset

D64, BF = torch.float64, torch.bfloat16


def _inputs(p, dtype, seed=0):
    from paper_2505_19201_b200 import synth
    vis, ids = synth.request_inputs(p, seed)
    return vis.to(dtype), ids.tolist()


def _round(t):
    return t.to(BF).to(t.dtype)


@pytest.mark.parametrize("dtype", [torch.float32, D64])
def test_first_layer_rows_are_the_unrounded_rows_rounded_once(dtype):
    """Layer 1's K/V rows depend on the inputs only, so the bf16 store must hold exactly the
    rounded rows of the plain oracle; deeper layers see the rounded rows and drift apart."""
    p, plain = make_oracle(tiny_preset(n_visual=8, n_prompt=6), dtype)
    _, store = make_oracle(tiny_preset(n_visual=8, n_prompt=6), dtype, kv_dtype=BF)
    vis, ids = _inputs(p, dtype)
    a, tok_a, _ = plain.prefill(vis, 0, ids)
    b, tok_b, _ = store.prefill(vis, 0, ids)
    assert torch.equal(b.K[0], _round(a.K[0])) and torch.equal(b.V[0], _round(a.V[0]))
    assert not torch.equal(a.K[0], _round(a.K[0]))                      # the rounding does something
    for l in range(p["n_layers"]):                                       # every stored row is a bf16 value
        assert torch.equal(b.K[l], _round(b.K[l])) and torch.equal(b.V[l], _round(b.V[l]))
    assert not torch.equal(b.K[1], _round(a.K[1]))                      # layer 2 has seen rounded rows


def test_rounding_follows_the_rotary_embedding():
    """round(rope(k)) is what is stored; rope(round(k)) is in general not a bf16 value."""
    p, store = make_oracle(tiny_preset(n_visual=8, n_prompt=6), D64, kv_dtype=BF)
    vis, ids = _inputs(p, D64)
    st, _, _ = store.prefill(vis, 0, ids)
    c, w = store.cfg, store.tw
    H, Hkv, hd = c.n_heads, c.n_kv_heads, c.head_dim
    qkv = O.linear(O.rmsnorm(st.x0, w["ln1"][0], c.rms_eps), w["wqkv"][0])
    k = qkv[:, H * hd:(H + Hkv) * hd].reshape(-1, Hkv, hd)
    pos = torch.arange(st.P)
    assert torch.equal(st.K[0], _round(O.rope(k, pos, c.rope_theta)))
    wrong = O.rope(_round(k), pos, c.rope_theta)
    assert not torch.equal(st.K[0][1:], wrong[1:])                      # position 0 is the identity rotation


def test_queries_stay_unrounded_and_rows_are_rounded_before_they_are_attended():
    """The first block's output, recomputed step by step: exact queries against the rounded K/V
    rows of every position up to and including the query's own."""
    p, store = make_oracle(tiny_preset(n_visual=8, n_prompt=6), D64, kv_dtype=BF)
    for l in range(p["n_layers"]):          # larger weights: peaked attention, so a rounded operand shows
        store.tw["wqkv"][l] = store.tw["wqkv"][l] * 20
    vis, ids = _inputs(p, D64)
    st, _, _ = store.prefill(vis, 0, ids, keep_all_taps=True)
    c, w = store.cfg, store.tw
    H, Hkv, hd, n = c.n_heads, c.n_kv_heads, c.head_dim, st.P
    pos = torch.arange(n)
    qkv = O.linear(O.rmsnorm(st.x0, w["ln1"][0], c.rms_eps), w["wqkv"][0])
    q = O.rope(qkv[:, :H * hd].reshape(-1, H, hd), pos, c.rope_theta)

    def block_out(q_used, K_used, V_used):
        o, _ = O.attention(q_used, K_used, V_used, torch.ones(n, n, dtype=torch.bool).tril())
        x = st.x0 + O.linear(o, w["wo"][0])
        return x + O.mlp(O.rmsnorm(x, w["ln2"][0], c.rms_eps), w["wgu"][0], w["wd"][0], c.d_ff)

    want = block_out(q, st.K[0], st.V[0])
    assert torch.allclose(st.taps[1], want, atol=1e-12)
    # the two mistakes this guards against give visibly different outputs
    k_raw = O.rope(qkv[:, H * hd:(H + Hkv) * hd].reshape(-1, Hkv, hd), pos, c.rope_theta)
    v_raw = qkv[:, (H + Hkv) * hd:].reshape(-1, Hkv, hd)
    assert float((block_out(_round(q), st.K[0], st.V[0]) - want).abs().max()) > 1e-6
    assert float((block_out(q, k_raw, v_raw) - want).abs().max()) > 1e-6


def _setup(scale=30.0, **over):
    p, orc = make_oracle(tiny_preset(**over), D64, kv_dtype=BF)
    orc.tw["lm_head"] = orc.tw["lm_head"] * scale
    vis, ids = _inputs(p, D64)
    st, _, _ = orc.prefill(vis, 0, ids)
    orc.compress_visual(st, p["k_visual"])
    return p, orc, st, vis, ids


def test_chain_tree_equals_causal_decoding_under_the_bf16_store():
    """Verifying a chain on top of the cached (rounded) prefix gives the logits and the stored
    rows of a fresh causal pass over prompt + chain: every row was rounded before anything saw it."""
    p, orc, st, vis, ids = _setup()
    toks = [st.pending, 7, 3, 11, 5]
    ver = orc.verify_tree(st, O.make_tree(toks, [-1, 0, 1, 2, 3]))
    st2, _, _ = orc.prefill(vis, 0, ids, extra_ids=toks)
    n = st.P
    assert torch.allclose(ver["logits"], orc._logits(orc._last_hidden[n:]), atol=1e-10)
    for l in range(p["n_layers"]):
        assert torch.equal(ver["tailK"][l], st2.K[l][n:]) and torch.equal(ver["tailV"][l], st2.V[l][n:])


def test_speculative_output_equals_greedy_autoregressive_under_the_bf16_store():
    p, orc, st, vis, ids = _setup()
    ref, margins = orc.ar_decode(vis, 0, ids, 24)
    assert min(margins) > 1e-9
    out = [st.pending]
    while len(out) < 16:
        out += orc.step(st)["out"]
    assert out[:16] == ref[:16]


def test_commit_equals_fresh_prefill_under_the_bf16_store():
    """After rounds with accept lengths 2, 0, 3 the compacted cache holds, bit for bit, the rows
    a fresh prefill of the emitted sequence stores."""
    p, orc, st, vis, ids = _setup()
    ref, _ = orc.ar_decode(vis, 0, ids, 12)
    emitted = [st.pending]
    for a in (2, 0, 3):
        toks, par, last = [st.pending], [-1], 0
        for j in range(a):
            toks += [ref[len(emitted) + j], (ref[len(emitted) + j] + 3) % p["vocab"]]
            par += [last, last]
            last = len(toks) - 2
        r = orc.step(st, O.make_tree(toks, par))
        assert r["A"] == a
        emitted += r["out"]
    assert emitted == ref[:len(emitted)]
    st2, tok2, _ = orc.prefill(vis, 0, ids, extra_ids=emitted[:-1])
    assert tok2 == st.pending and st2.P == st.P
    for l in range(p["n_layers"]):
        assert torch.allclose(st.K[l], st2.K[l], atol=1e-10) and torch.allclose(st.V[l], st2.V[l], atol=1e-10)
        assert torch.equal(st.K[l], _round(st.K[l]))
