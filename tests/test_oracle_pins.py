"""Pins of the CPU oracle against what the paper and the mathematics fix.

The paper prints no intermediate numerical value (no example entropy, score, tree or
logit), so every pin here is a closed form, an invariant of the method, a reduction to a
library routine, or brute force on tiny inputs.  None needs a GPU.
"""
import itertools
import math

import pytest
import torch
import torch.nn.functional as F

from oracle import dream_oracle as O
from tests.util_oracle import make_oracle, tiny_preset

D64 = torch.float64


# ------------------------------------------------------------------ primitives vs library routines

def test_rmsnorm_matches_library():
    g = torch.Generator().manual_seed(1)
    x = torch.randn(5, 24, dtype=D64, generator=g)
    w = torch.rand(24, dtype=D64, generator=g) + 0.5
    assert torch.allclose(O.rmsnorm(x, w, 1e-5), F.rms_norm(x, (24,), w, 1e-5), atol=1e-13)


def test_linear_is_x_times_w_transposed():
    g = torch.Generator().manual_seed(2)
    x, w = torch.randn(3, 7, dtype=D64, generator=g), torch.randn(4, 7, dtype=D64, generator=g)
    ref = [[sum(float(x[i, k]) * float(w[j, k]) for k in range(7)) for j in range(4)] for i in range(3)]
    assert torch.allclose(O.linear(x, w), torch.tensor(ref, dtype=D64), atol=1e-13)


def test_attention_matches_library_with_grouped_heads_and_mask():
    g = torch.Generator().manual_seed(3)
    m, r, H, Hkv, hd = 5, 9, 4, 2, 8
    q = torch.randn(m, H, hd, dtype=D64, generator=g)
    K = torch.randn(r, Hkv, hd, dtype=D64, generator=g)
    V = torch.randn(r, Hkv, hd, dtype=D64, generator=g)
    mask = torch.rand(m, r, generator=g) > 0.4
    mask[:, 0] = True
    out, probs = O.attention(q, K, V, mask)
    Kr = K.repeat_interleave(H // Hkv, dim=1).permute(1, 0, 2)
    Vr = V.repeat_interleave(H // Hkv, dim=1).permute(1, 0, 2)
    ref = F.scaled_dot_product_attention(q.permute(1, 0, 2), Kr, Vr, attn_mask=mask[None])
    assert torch.allclose(out, ref.permute(1, 0, 2).reshape(m, H * hd), atol=1e-12)
    assert torch.allclose(probs.sum(-1), torch.ones(H, m, dtype=D64), atol=1e-12)
    assert float(probs[:, ~mask].abs().max()) == 0.0


def test_cross_attention_with_one_memory_row_returns_its_value():
    g = torch.Generator().manual_seed(4)
    q = torch.randn(3, 4, 8, dtype=D64, generator=g)
    K, V = torch.randn(1, 2, 8, dtype=D64, generator=g), torch.randn(1, 2, 8, dtype=D64, generator=g)
    out, _ = O.attention(q, K, V, torch.ones(3, 1, dtype=torch.bool))
    want = V[0].repeat_interleave(2, dim=0).reshape(-1)
    assert torch.allclose(out, want.expand(3, -1), atol=1e-14)


def test_mlp_is_gated_silu():
    g = torch.Generator().manual_seed(5)
    b = torch.randn(2, 6, dtype=D64, generator=g)
    wgu, wd = torch.randn(10, 6, dtype=D64, generator=g), torch.randn(6, 5, dtype=D64, generator=g)
    gate, up = F.linear(b, wgu[:5]), F.linear(b, wgu[5:])
    ref = F.linear(gate * torch.sigmoid(gate) * up, wd)
    assert torch.allclose(O.mlp(b, wgu, wd, 5), ref, atol=1e-13)


def test_rope_identity_norm_and_relative_phase():
    g = torch.Generator().manual_seed(6)
    x = torch.randn(4, 2, 8, dtype=D64, generator=g)
    y = torch.randn(4, 2, 8, dtype=D64, generator=g)
    assert torch.equal(O.rope(x, torch.zeros(4, dtype=torch.long), 10000.0), x)
    pos = torch.tensor([3, 17, 0, 250])
    rx = O.rope(x, pos, 10000.0)
    assert torch.allclose(rx.norm(dim=-1), x.norm(dim=-1), atol=1e-12)
    # <R_m x, R_n y> depends on m - n only
    a = (O.rope(x, pos, 1e4) * O.rope(y, pos + 5, 1e4)).sum(-1)
    b = (O.rope(x, pos + 40, 1e4) * O.rope(y, pos + 45, 1e4)).sum(-1)
    assert torch.allclose(a, b, atol=1e-11)
    # complex-number form on one vector: (x_i + i x_{i+hd/2}) * exp(i pos theta^(-2i/hd))
    hd, p = 8, 17
    v = [float(t) for t in x[1, 0]]
    for i in range(hd // 2):
        z = complex(v[i], v[i + hd // 2]) * complex(math.cos(p * 10000.0 ** (-2 * i / hd)),
                                                    math.sin(p * 10000.0 ** (-2 * i / hd)))
        assert abs(z.real - float(rx[1, 0, i])) < 1e-12
        assert abs(z.imag - float(rx[1, 0, i + hd // 2])) < 1e-12


def test_row_entropy_closed_forms():
    for n in (1, 2, 7, 100):
        assert abs(float(O.row_entropy(torch.full((n,), 1.0 / n, dtype=D64))) - math.log(n)) < 1e-12
    onehot = torch.zeros(5, dtype=D64)
    onehot[3] = 1.0
    assert float(O.row_entropy(onehot)) == 0.0
    p = torch.tensor([0.5, 0.25, 0.25, 0.0], dtype=D64)
    assert abs(float(O.row_entropy(p)) - 1.5 * math.log(2)) < 1e-12


def test_argmax_and_topk_tie_to_lower_index():
    x = torch.tensor([1.0, 3.0, 3.0, 2.0, 3.0])
    assert O.argmax_low(x) == (1, 0.0)
    v, i = O.topk_low(x, 3)
    assert i.tolist() == [1, 2, 4]


# ------------------------------------------------------------------ Eq. 2 and Section 3.3 closed forms

def _zero_queries(orc):
    c = orc.cfg
    for l in range(c.n_layers):
        orc.tw["wqkv"][l] = orc.tw["wqkv"][l].clone()
        orc.tw["wqkv"][l][:c.n_heads * c.head_dim] = 0


def test_uniform_attention_entropy_and_importance_closed_forms():
    """W_Q = 0 makes every causal row uniform: row i has entropy ln(i+1), so
    AE = ln(n!)/n; visual token j then receives sum_{i>j} 1/(i+1) per head."""
    p, orc = make_oracle(tiny_preset())
    _zero_queries(orc)
    vis, ids = _inputs(p)
    st, _, _ = orc.prefill(vis, 0, ids, keep_all_taps=True)
    n, H = p["n_visual"] + p["n_prompt"], p["n_heads"]
    want = math.lgamma(n + 1) / n
    assert torch.allclose(st.entropy, torch.full((p["n_layers"],), want, dtype=D64), atol=1e-12)
    harm = lambda m: sum(1.0 / t for t in range(1, m + 1))
    for l in (1, 2):
        for j in range(p["n_visual"]):
            assert abs(float(st.scores[l][j]) - H * (harm(n) - harm(j + 1))) < 1e-11
    # the last causal row sees all n keys: its entropy is ln n
    assert abs(math.log(n) - (math.lgamma(n + 1) - math.lgamma(n))) < 1e-12


def test_importance_with_self_sums_to_rows_times_heads():
    """Every attention row sums to 1, so the column sums over all n columns total n*H."""
    p, orc = make_oracle(tiny_preset(n_prompt=0, n_visual=11, score_include_self=1))
    vis, ids = _inputs(p)
    st, _, _ = orc.prefill(vis, 0, ids, keep_all_taps=True)
    for l in (1, 2):
        assert abs(float(st.scores[l].sum()) - 11 * p["n_heads"]) < 1e-10


def test_visual_span_may_follow_the_text():
    """Importance scores are taken on the visual span wherever it sits in the sequence."""
    p, orc = make_oracle(tiny_preset())
    _zero_queries(orc)
    vis, ids = _inputs(p)
    q, v = p["n_prompt"], p["n_visual"]
    st, _, _ = orc.prefill(vis, q, ids)
    n = q + v
    harm = lambda m: sum(1.0 / t for t in range(1, m + 1))
    for j in range(v):
        assert abs(float(st.scores[1][j]) - p["n_heads"] * (harm(n) - harm(q + j + 1))) < 1e-11


def test_tap_selection_modes():
    p, orc = make_oracle(tiny_preset(n_layers=2))
    ent = torch.tensor([0.9, 0.3, 0.3, 0.7, 1.2], dtype=D64)
    orc.cfg.tap_lo, orc.cfg.tap_hi = 1, 5
    orc.cfg.tap_mode = O.TAP_ENTROPY_MIN
    assert orc.select_tap(ent)[0] == 2          # tie -> lower layer
    orc.cfg.tap_mode = O.TAP_ENTROPY_MAX
    assert orc.select_tap(ent)[0] == 5
    orc.cfg.tap_lo, orc.cfg.tap_hi = 2, 4
    assert orc.select_tap(ent)[0] == 4
    orc.cfg.tap_mode, orc.cfg.tap_layer = O.TAP_FIXED, 3
    assert orc.select_tap(ent)[0] == 3


# ------------------------------------------------------------------ a block, by brute force

def _inputs(p, seed=0):
    from paper_2505_19201_b200 import synth
    vis, ids = synth.request_inputs(p, seed)
    return vis.to(D64), ids.tolist()


def _py_block(orc, l, xs, positions):
    """One causal decoder block in pure Python lists (no tensor ops)."""
    c = orc.cfg
    H, Hkv, hd, d, ff = c.n_heads, c.n_kv_heads, c.head_dim, c.d_model, c.d_ff
    W = lambda t: [[float(a) for a in row] for row in t.to(D64)]
    wqkv, wo, wgu, wd = W(orc.tw["wqkv"][l]), W(orc.tw["wo"][l]), W(orc.tw["wgu"][l]), W(orc.tw["wd"][l])
    g1 = [float(a) for a in orc.tw["ln1"][l].to(D64)]
    g2 = [float(a) for a in orc.tw["ln2"][l].to(D64)]
    mv = lambda M, x: [sum(M[o][i] * x[i] for i in range(len(x))) for o in range(len(M))]

    def norm(x, g):
        r = math.sqrt(sum(t * t for t in x) / len(x) + c.rms_eps)
        return [t / r * gg for t, gg in zip(x, g)]

    def rot(vec, pos):
        out = list(vec)
        for i in range(hd // 2):
            a = pos * c.rope_theta ** (-2.0 * i / hd)
            out[i] = vec[i] * math.cos(a) - vec[i + hd // 2] * math.sin(a)
            out[i + hd // 2] = vec[i + hd // 2] * math.cos(a) + vec[i] * math.sin(a)
        return out

    qs, ks, vs = [], [], []
    for x, pos in zip(xs, positions):
        qkv = mv(wqkv, norm(x, g1))
        qs.append([rot(qkv[h * hd:(h + 1) * hd], pos) for h in range(H)])
        ks.append([rot(qkv[(H + h) * hd:(H + h + 1) * hd], pos) for h in range(Hkv)])
        vs.append([qkv[(H + Hkv + h) * hd:(H + Hkv + h + 1) * hd] for h in range(Hkv)])
    out, ent_sum = [], 0.0
    for i, x in enumerate(xs):
        o = []
        for h in range(H):
            kvh = h // (H // Hkv)
            s = [sum(qs[i][h][t] * ks[j][kvh][t] for t in range(hd)) / math.sqrt(hd) for j in range(i + 1)]
            mx = max(s)
            e = [math.exp(t - mx) for t in s]
            z = sum(e)
            pr = [t / z for t in e]
            ent_sum -= sum(t * math.log(t) for t in pr if t > 0)
            o += [sum(pr[j] * vs[j][kvh][t] for j in range(i + 1)) for t in range(hd)]
        y = [a + b for a, b in zip(x, mv(wo, o))]
        gu = mv(wgu, norm(y, g2))
        act = [gu[t] / (1 + math.exp(-gu[t])) * gu[ff + t] for t in range(ff)]
        out.append([a + b for a, b in zip(y, mv(wd, act))])
    return out, ent_sum / (len(xs) * H)


def test_prefill_block_and_entropy_by_brute_force():
    p, orc = make_oracle(tiny_preset(n_visual=4, n_prompt=3))
    for l in range(2):   # larger weights -> peaked, non-uniform attention
        orc.tw["wqkv"][l] = orc.tw["wqkv"][l] * 20
    vis, ids = _inputs(p)
    st, tok, _ = orc.prefill(vis, 0, ids, keep_all_taps=True)
    xs = [[float(a) for a in row] for row in st.x0]
    pos = list(range(len(xs)))
    y1, e1 = _py_block(orc, 0, xs, pos)
    y2, e2 = _py_block(orc, 1, y1, pos)
    assert torch.allclose(st.taps[1], torch.tensor(y1, dtype=D64), atol=1e-11)
    assert torch.allclose(st.taps[2], torch.tensor(y2, dtype=D64), atol=1e-11)
    assert abs(float(st.entropy[0]) - e1) < 1e-12 and abs(float(st.entropy[1]) - e2) < 1e-12
    # first token = argmax of the LM head on the last row
    h = O.rmsnorm(torch.tensor(y2[-1], dtype=D64), orc.tw["ln_f"], p["rms_eps"])
    assert tok == int(torch.argmax(orc.tw["lm_head"].to(D64) @ h))


# ------------------------------------------------------------------ compression (Section 3.3)

def test_keep_all_visual_tokens_is_identity():
    p, orc = make_oracle(tiny_preset())
    vis, ids = _inputs(p)
    st, _, _ = orc.prefill(vis, 0, ids)
    kept, sc, _ = orc.compress_visual(st, p["n_visual"])
    assert kept.tolist() == list(range(p["n_visual"]))
    assert st.ctx_pos.tolist() == list(range(p["n_visual"] + p["n_prompt"]))
    full_K, full_m = st.dK.clone(), st.mK.clone()
    # with xattn_full_memory the memory is over all n positions regardless of k
    orc.cfg.xattn_full_memory = 1
    orc.compress_visual(st, 2)
    assert torch.equal(st.mK, full_m) and st.dK.shape[0] == 2 + p["n_prompt"]
    assert torch.equal(st.dK, full_K[st.ctx_pos])


def test_topk_agrees_with_full_sort_and_context_is_sorted_union():
    p, orc = make_oracle(tiny_preset(n_visual=9, n_prompt=4))
    vis, ids = _inputs(p)
    st, _, _ = orc.prefill(vis, 2, ids)           # visual span in the middle of the text
    for k in (1, 4, 8):
        kept, sc, margin = orc.compress_visual(st, k)
        order = sorted(range(9), key=lambda j: (-float(sc[j]), j))
        assert kept.tolist() == sorted(order[:k])
        assert margin >= 0
        text = [0, 1] + list(range(11, 13))
        assert st.ctx_pos.tolist() == sorted(text + [2 + j for j in kept.tolist()])
        # memory rows are the tapped features at C, projected with no norm (Eq. 1)
        kv = st.taps[st.tap][st.ctx_pos] @ orc.dw["xkv"].to(D64).t()
        assert torch.allclose(st.mK.reshape(len(st.ctx_pos), -1), kv[:, :kv.shape[1] // 2], atol=1e-13)


# ------------------------------------------------------------------ verification (tree mask)

def _setup(p=None, scale=1.0, **over):
    p, orc = make_oracle(p or tiny_preset(**over))
    if scale != 1.0:
        orc.tw["lm_head"] = orc.tw["lm_head"] * scale
    vis, ids = _inputs(p)
    st, tok, _ = orc.prefill(vis, 0, ids)
    orc.compress_visual(st, p["k_visual"])
    return p, orc, st, vis, ids


def test_chain_tree_equals_causal_decoding():
    p, orc, st, vis, ids = _setup()
    toks = [st.pending, 7, 3, 11, 5]
    tree = O.make_tree(toks, [-1, 0, 1, 2, 3])
    ver = orc.verify_tree(st, tree)
    # reference: a fresh causal prefill over prompt + those tokens
    st2, _, _ = orc.prefill(vis, 0, ids, extra_ids=toks)
    n = st.P
    ref = orc._logits(orc._last_hidden[n:])
    assert torch.allclose(ver["logits"], ref, atol=1e-10)
    for l in range(p["n_layers"]):
        assert torch.allclose(ver["tailK"][l], st2.K[l][n:], atol=1e-11)


def test_star_tree_gives_one_token_continuations():
    p, orc, st, vis, ids = _setup()
    kids = [4, 9, 21]
    tree = O.make_tree([st.pending] + kids, [-1, 0, 0, 0])
    ver = orc.verify_tree(st, tree)
    for i, t in enumerate(kids):
        orc.prefill(vis, 0, ids, extra_ids=[st.pending, t])
        ref = orc._logits(orc._last_hidden[-1:])[0]
        assert torch.allclose(ver["logits"][1 + i], ref, atol=1e-10)


# ------------------------------------------------------------------ acceptance

def test_accept_is_the_longest_matching_root_path_brute_force():
    g = torch.Generator().manual_seed(11)
    for trial in range(200):
        T = int(torch.randint(2, 12, (1,), generator=g))
        parent = [-1] + [int(torch.randint(0, i, (1,), generator=g)) for i in range(1, T)]
        tokens = [0] * T
        for i in range(T):          # children of one node get distinct tokens from a small alphabet
            kids = [j for j in range(T) if parent[j] == i]
            perm = torch.randperm(6, generator=g).tolist()
            for j, kk in enumerate(kids):
                tokens[kk] = perm[j % 6] if j < 6 else 6 + j
        argmax = torch.randint(0, 4, (T,), generator=g).tolist()
        tree = O.make_tree(tokens, parent)
        A, out, path = O.DreamOracle.accept(tree, argmax)
        best = [0]
        for i in range(T):          # every root path
            chain = [i]
            while parent[chain[-1]] >= 0:
                chain.append(parent[chain[-1]])
            chain.reverse()
            if all(tokens[c] == argmax[pp] for pp, c in zip(chain, chain[1:])) and len(chain) > len(best):
                best = chain
        assert path == best and A == len(best) - 1
        assert out == [tokens[c] for c in best[1:]] + [argmax[best[-1]]]


# ------------------------------------------------------------------ the whole loop

def _decode(orc, st, n_new, tree_fn=None):
    out = [st.pending]
    stats = []
    while len(out) < n_new:
        r = orc.step(st, tree_fn(st) if tree_fn else None)
        out += r["out"]
        stats.append(r["A"])
    return out[:n_new], stats


@pytest.mark.parametrize("mode", ["draft", "adversarial", "oracle_path"])
def test_speculative_output_equals_greedy_autoregressive(mode):
    """Greedy speculative decoding emits exactly the target's greedy sequence, for any tree."""
    p, orc, st, vis, ids = _setup(scale=30.0)
    n_new = 20
    ref, margins = orc.ar_decode(vis, 0, ids, n_new + 8)
    assert min(margins) > 1e-9
    g = torch.Generator().manual_seed(5)
    D, V = p["tree_depth"], p["vocab"]

    def adversarial(st_):
        T = 1 + int(torch.randint(1, 12, (1,), generator=g))
        par = [-1] + [int(torch.randint(0, i, (1,), generator=g)) for i in range(1, T)]
        toks = [st_.pending] + [(7 * i + int(torch.randint(0, V, (1,), generator=g))) % V for i in range(1, T)]
        return O.make_tree(toks, par)

    produced = [1]      # tokens emitted so far, the first one by the prefill
    stats = []

    def with_truth(st_):
        # a tree that contains the true continuation for `a` levels plus distractor siblings
        a = 1 + (len(stats) % D)
        cur, toks, par = produced[0], [st_.pending], [-1]
        last = 0
        for j in range(a):
            toks += [ref[cur + j], (ref[cur + j] + 1) % V]
            par += [last, last]
            last = len(toks) - 2
        return O.make_tree(toks, par)

    fn = {"draft": None, "adversarial": adversarial, "oracle_path": with_truth}[mode]
    out = [st.pending]
    while len(out) < n_new:
        r = orc.step(st, fn(st) if fn else None)
        out += r["out"]
        produced[0] = len(out)
        stats.append(r["A"])
    assert out[:n_new] == ref[:n_new]
    if mode == "oracle_path":
        assert set(stats) >= set(range(1, D + 1))      # every accept length 1..D is exercised


def test_commit_equals_fresh_prefill_of_emitted_sequence():
    p, orc, st, vis, ids = _setup(scale=30.0)
    ref, _ = orc.ar_decode(vis, 0, ids, 12)
    kept = st.kept.clone()
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
    # tokens in the KV cache are all emitted tokens except the pending one
    st2, tok2, _ = orc.prefill(vis, 0, ids, extra_ids=emitted[:-1])
    assert tok2 == st.pending and st2.P == st.P
    for l in range(p["n_layers"]):
        assert torch.allclose(st.K[l], st2.K[l], atol=1e-10)
        assert torch.allclose(st.V[l], st2.V[l], atol=1e-10)
    st2.tap = st.tap
    orc.compress_visual(st2, p["k_visual"], forced_idx=kept)
    # the appended text positions count as context in the fresh prefill, so its memory and
    # draft self-attention rows must equal the incrementally grown ones, row for row
    assert torch.allclose(st.mK, st2.mK, atol=1e-10) and torch.allclose(st.mV, st2.mV, atol=1e-10)
    orc.draft_tree(st)                      # catch-up rows of the draft's self-attention cache
    assert torch.allclose(st.dK, st2.dK, atol=1e-10) and torch.allclose(st.dV, st2.dV, atol=1e-10)


# ------------------------------------------------------------------ tree drafting by brute force

def _draft_chain_logp(orc, st, toks):
    """log-probabilities after each token of a single root path, evaluated on its own."""
    c, dw = orc.cfg, orc.dw
    H, Hkv, hd = c.n_heads, c.n_kv_heads, c.head_dim
    P = st.P
    dK, dV, mK, mV = st.dK, st.dV, st.mK, st.mV
    rows = []
    for j, t in enumerate(toks):
        x = orc.tw["embed"][t].to(D64)[None]
        qkv = O.linear(O.rmsnorm(x, dw["ln1"], c.rms_eps), dw["wqkv"])
        pos = torch.tensor([P + j])
        q = O.rope(qkv[:, :H * hd].reshape(1, H, hd), pos, c.rope_theta)
        k = O.rope(qkv[:, H * hd:(H + Hkv) * hd].reshape(1, Hkv, hd), pos, c.rope_theta)
        v = qkv[:, (H + Hkv) * hd:].reshape(1, Hkv, hd)
        dK, dV = torch.cat([dK, k]), torch.cat([dV, v])
        o, _ = O.attention(q, dK, dV, torch.ones(1, dK.shape[0], dtype=torch.bool))
        h = x + O.linear(o, dw["wo"])
        qx = O.linear(O.rmsnorm(h, dw["lnx"], c.rms_eps), dw["xq"]).reshape(1, H, hd)
        o, _ = O.attention(qx, mK, mV, torch.ones(1, mK.shape[0], dtype=torch.bool))
        h = h + O.linear(o, dw["xo"])
        h = h + O.mlp(O.rmsnorm(h, dw["ln2"], c.rms_eps), dw["wgu"], dw["wd"], c.d_ff)
        kv = O.linear(h, dw["xkv"])
        mK = torch.cat([mK, kv[:, :Hkv * hd].reshape(1, Hkv, hd)])
        mV = torch.cat([mV, kv[:, Hkv * hd:].reshape(1, Hkv, hd)])
        rows.append(torch.log_softmax(orc._logits(h)[0], -1))
    return rows


def test_complete_tree_agrees_with_brute_force_path_enumeration():
    p, orc, st, vis, ids = _setup(scale=30.0)          # beam 4 >= K^(D-1): complete binary tree
    K, D = p["tree_topk"], p["tree_depth"]
    tree = orc.draft_tree(st)
    assert len(tree["tokens"]) == 1 + sum(K ** j for j in range(1, D + 1))
    # brute force: expand every root path on its own
    want = {}
    frontier = [((st.pending,), 0.0)]
    for depth in range(1, D + 1):
        nxt = []
        for path, cum in frontier:
            lp = _draft_chain_logp(orc, st, list(path))[-1]
            assert abs(float(torch.exp(lp).sum()) - 1.0) < 1e-12
            v, i = torch.sort(lp, descending=True, stable=True)
            for j in range(K):
                want[path + (int(i[j]),)] = cum + float(v[j])
                nxt.append((path + (int(i[j]),), cum + float(v[j])))
        frontier = nxt
    got = {}
    for i in range(1, len(tree["tokens"])):
        chain = [i]
        while tree["parent"][chain[-1]] > 0:
            chain.append(tree["parent"][chain[-1]])
        got[(st.pending,) + tuple(tree["tokens"][c] for c in reversed(chain))] = tree["cum"][i]
    assert set(got) == set(want)
    for k in want:
        assert abs(got[k] - want[k]) < 1e-9


@pytest.mark.parametrize("beam,N,K,Dp", [(2, 7, 2, 4), (3, 9, 3, 3), (1, 3, 1, 3), (2, 100, 2, 3)])
def test_tree_structure_invariants(beam, N, K, Dp):
    p, orc, st, vis, ids = _setup(scale=30.0, tree_beam=beam, tree_max_nodes=N, tree_topk=K, tree_depth=Dp)
    tree = orc.draft_tree(st)
    T = len(tree["tokens"])
    ncand = K + (Dp - 1) * min(beam, K) * K if beam <= K else None
    if ncand is not None:
        assert len(tree["cands"]) == ncand and T == 1 + min(N, ncand)
    assert tree["parent"][0] == -1 and tree["depth"][0] == 0
    for i in range(1, T):
        pa = tree["parent"][i]
        assert 0 <= pa < i                                      # parents precede children
        assert tree["depth"][i] == tree["depth"][pa] + 1
        assert tree["cum"][i] <= tree["cum"][pa] + 1e-12         # log-probabilities are <= 0
        anc, a = {i}, i
        while a > 0:
            a = tree["parent"][a]
            anc.add(a)
        assert tree["mask"][i] == anc                            # mask = transitive closure
        sib = [tree["tokens"][j] for j in range(1, T) if tree["parent"][j] == pa]
        assert len(sib) == len(set(sib))                         # siblings carry distinct tokens
    # the selected set is the N best candidates by cumulative score
    cums = sorted((cd[3] for cd in tree["cands"]), reverse=True)
    assert sorted(tree["cum"][1:], reverse=True) == pytest.approx(cums[:T - 1])
    # each node's cum equals the single-path evaluation of its root path
    for i in range(1, T):
        chain = [i]
        while tree["parent"][chain[-1]] > 0:
            chain.append(tree["parent"][chain[-1]])
        toks = [st.pending] + [tree["tokens"][c] for c in reversed(chain)]
        rows = _draft_chain_logp(orc, st, toks[:-1])
        want = sum(float(rows[j][toks[j + 1]]) for j in range(len(toks) - 1))
        assert abs(tree["cum"][i] - want) < 1e-9


def test_chain_draft_is_greedy_draft_decoding():
    """K = 1 reduces the tree to a chain whose tokens are the draft's own greedy tokens."""
    p, orc, st, vis, ids = _setup(scale=30.0, tree_beam=1, tree_max_nodes=3, tree_topk=1, tree_depth=3)
    tree = orc.draft_tree(st)
    assert tree["parent"] == [-1, 0, 1, 2]
    toks = [st.pending]
    for _ in range(3):
        toks.append(int(torch.argmax(_draft_chain_logp(orc, st, toks)[-1])))
    assert tree["tokens"] == toks


def test_draft_uses_catch_up_rows_after_accept():
    """After an accept the draft's self-attention rows cover every verified token."""
    p, orc, st, vis, ids = _setup(scale=30.0)
    n0 = st.dK.shape[0]
    r = orc.step(st)
    orc.draft_tree(st)
    assert st.dK.shape[0] == n0 + r["A"] + 1 and st.mK.shape[0] == n0 + r["A"] + 1


def test_toy_decode_matches_stored_oracle_run():
    """The stored toy decode (written by tests/golden/make_toy_golden.py from the oracle
    alone) still comes out of the oracle, and speculative decoding reproduces it."""
    import json, os
    from paper_2505_19201_b200 import synth
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "toy_decode.json")))
    p, orc = make_oracle("toy", D64)
    vis, ids = synth.request_inputs(p, 0)
    st, tok, _ = orc.prefill(vis.to(D64), 0, ids.tolist())
    assert tok == gold["first_token"]
    assert torch.allclose(st.entropy, torch.tensor(gold["entropy"], dtype=D64), atol=1e-12)
    kept, _, _ = orc.compress_visual(st, p["k_visual"])
    assert kept.tolist() == gold["kept"]
    out = [tok]
    while len(out) < 24:
        out += orc.step(st)["out"]
    assert out[:24] == gold["ar_tokens"]
