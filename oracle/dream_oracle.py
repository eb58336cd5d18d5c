"""CPU oracle for the DREAM draft-and-verify loop.  TEST INFRASTRUCTURE ONLY.

A plain, slow, step-by-step implementation of what the hot path computes,
written from the paper's method section with plain PyTorch CPU tensor ops
(matmul, softmax, sort are used as library steps; no blocking, no fusion).
It shares no code with the CUDA path and imports nothing from it.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may call it.

Precision: `dtype` is the arithmetic and activation storage type.  float64 is
used for the pins and the toy model; float32 is used for the bf16 model shapes
(weights are taken as given, i.e. bf16-rounded values, and up-converted).  For
those shapes the target KV cache is a bf16 store: `kv_dtype=torch.bfloat16` rounds
each K/V row once on entry to the cache; everything computed from it stays fp32.

Readings taken where the paper is silent (each is listed in the design notes):
pre-norm decoder blocks with RMSNorm, rotary positions (half-split pairing) on
self-attention only, gated SiLU MLP, no biases, softmax scale 1/sqrt(head_dim),
grouped KV heads, causal mask in the entropy and importance sums, natural log,
ties broken toward the lower index everywhere.

Paper anchors: Section 2.1 (draft-then-verify, acceptance), Section 3.1 and
Eq. 1 (cross-attention fusion, growing key/value memory, tree drafting),
Section 3.2 and Eq. 2 (average attention entropy, layer selection),
Section 3.3 (visual-token importance and top-k subsampling), Section 4 setup
(tree depth/width, bonus token, KV caching).

Parity unpinned: acceptance length tau and speedup S (need trained weights).

Weight layout: every matrix is [out_features, in_features]; wqkv stacks the
query/key/value projections by rows, wgu stacks gate then up, xkv stacks the
cross-attention key then value projections.
"""
from dataclasses import dataclass, field
import math
import torch

TAP_FIXED, TAP_ENTROPY_MIN, TAP_ENTROPY_MAX = 0, 1, 2


@dataclass
class OracleConfig:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    tree_depth: int = 3
    tree_topk: int = 2
    tree_beam: int = 2
    tree_max_nodes: int = 14
    tap_mode: int = TAP_FIXED
    tap_layer: int = 1          # 1-based: S^l is the residual stream after block l
    tap_lo: int = 1
    tap_hi: int = 1
    score_include_self: int = 0
    xattn_full_memory: int = 0
    draft_blocks: int = 1       # 1: one layer (self-attention, cross-attention, MLP); 3: the paper's three blocks

    @staticmethod
    def from_preset(p):
        names = ("n_layers d_model n_heads n_kv_heads head_dim d_ff vocab rms_eps rope_theta "
                 "tree_depth tree_topk tree_beam tree_max_nodes tap_mode tap_layer tap_lo tap_hi "
                 "score_include_self xattn_full_memory").split()
        return OracleConfig(draft_blocks=int(p.get("draft_blocks", 1)), **{k: p[k] for k in names})


# --------------------------------------------------------------------------- primitives

def rmsnorm(x, g, eps):
    """x * g / sqrt(mean(x^2) + eps) over the last axis."""
    ms = (x * x).mean(dim=-1, keepdim=True)
    return x / torch.sqrt(ms + eps) * g.to(x.dtype)


def rope(x, pos, theta):
    """Rotary position embedding on x [rows, heads, hd] at integer positions pos [rows].

    Pair (i, i + hd/2) is rotated by the angle pos * theta^(-2i/hd).
    """
    hd = x.shape[-1]
    half = hd // 2
    i = torch.arange(half, dtype=torch.float64)
    inv = theta ** (-2.0 * i / hd)
    ang = pos.to(torch.float64)[:, None] * inv[None, :]
    c = torch.cos(ang).to(x.dtype)[:, None, :]
    s = torch.sin(ang).to(x.dtype)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return torch.cat([a * c - b * s, b * c + a * s], dim=-1)


def linear(x, w):
    """x [rows, in] times W^T for W [out, in]."""
    return x @ w.to(x.dtype).t()


def attention(q, K, V, mask):
    """softmax(q K^T / sqrt(hd)) V with a boolean mask (Eq. 1 with several heads).

    q [m, H, hd]; K, V [r, Hkv, hd]; mask [m, r] True = visible.  Query head h reads
    KV head h // (H / Hkv).  Returns (out [m, H*hd], probs [H, m, r]).
    """
    m, H, hd = q.shape
    Hkv = K.shape[1]
    g = H // Hkv
    outs, probs = [], []
    for h in range(H):
        kh, vh = K[:, h // g, :], V[:, h // g, :]
        s = (q[:, h, :] @ kh.t()) / math.sqrt(hd)
        s = s.masked_fill(~mask, float("-inf"))
        p = torch.softmax(s, dim=-1)
        outs.append(p @ vh)
        probs.append(p)
    return torch.cat(outs, dim=-1), torch.stack(probs, 0)


def mlp(b, wgu, wd, ff):
    gu = linear(b, wgu)
    gate, up = gu[:, :ff], gu[:, ff:]
    return linear(torch.nn.functional.silu(gate) * up, wd)


def row_entropy(p):
    """-sum_j p_j ln p_j per row with 0 ln 0 = 0 (inner sum of Eq. 2)."""
    t = torch.where(p > 0, p * torch.log(torch.where(p > 0, p, torch.ones_like(p))),
                    torch.zeros_like(p))
    return -t.sum(dim=-1)


def argmax_low(x):
    """Index of the maximum, ties to the lower index; also the top-1 minus top-2 margin."""
    v, i = torch.sort(x, descending=True, stable=True)
    return int(i[0]), float(v[0] - v[1]) if x.numel() > 1 else float("inf")


def topk_low(x, k):
    """The k largest entries, ties to the lower index, in descending order."""
    v, i = torch.sort(x, descending=True, stable=True)
    return v[:k], i[:k]


# --------------------------------------------------------------------------- state

@dataclass
class SeqState:
    """Everything the loop keeps for one sequence."""
    K: list = field(default_factory=list)       # per target layer [rows, Hkv, hd]
    V: list = field(default_factory=list)
    P: int = 0                                  # verified length: positions 0..P-1 are in K/V
    pending: int = -1                           # token at position P, not yet run through the target
    n_prompt_total: int = 0                     # n = q + v
    taps: dict = field(default_factory=dict)    # layer -> S^layer over the prompt [n, d]
    x0: torch.Tensor = None                     # input embeddings of the prompt [n, d]
    entropy: torch.Tensor = None                # AE per layer [L]
    scores: dict = field(default_factory=dict)  # layer -> importance of visual tokens [v]
    vis_start: int = 0
    n_visual: int = 0
    tap: int = 0                                # selected layer l*
    kept: torch.Tensor = None                   # kept visual indices, ascending, relative to vis_start
    ctx_pos: torch.Tensor = None                # positions of the compressed context C
    dK: torch.Tensor = None                     # draft self-attention K rows [rows, Hkv, hd]
    dV: torch.Tensor = None
    mK: torch.Tensor = None                     # cross-attention memory K rows
    mV: torch.Tensor = None
    new_tokens: list = field(default_factory=list)   # tokens verified since the last draft call
    new_pos: list = field(default_factory=list)
    # three-block draft only: the final block's self-attention rows, and the position of every
    # permanent row of the draft's caches and of the memory
    fK: torch.Tensor = None
    fV: torch.Tensor = None
    dpos: torch.Tensor = None
    mpos: torch.Tensor = None
    # Eq. 2 kept up to date over the verified sequence: per layer the sum over rows and heads of the
    # row entropies (fp64), over the P rows verified so far
    ent_sum: torch.Tensor = None


class DreamOracle:
    def __init__(self, cfg, tw, dw, dtype=torch.float64, kv_dtype=None):
        """kv_dtype: storage type of the target KV cache (None = same as dtype).  With
        torch.bfloat16 every K/V row is rounded once, when it enters the cache, and read
        back from there by all later arithmetic (which stays in `dtype`)."""
        self.cfg, self.tw, self.dw, self.dtype, self.kv_dtype = cfg, tw, dw, dtype, kv_dtype

    # ------------------------------------------------------------------ target block
    def _block(self, x, l, pos, Kc, Vc, mask, want_probs=False):
        """One pre-norm decoder block of the target on rows x at positions pos.

        Kc/Vc are the cached rows visible to these queries (may be empty); the new
        rows' K/V are appended after them and mask [m, cached + m] covers both.
        """
        c, w = self.cfg, self.tw
        H, Hkv, hd = c.n_heads, c.n_kv_heads, c.head_dim
        a = rmsnorm(x, w["ln1"][l], c.rms_eps)
        qkv = linear(a, w["wqkv"][l])
        q = qkv[:, :H * hd].reshape(-1, H, hd)
        k = qkv[:, H * hd:(H + Hkv) * hd].reshape(-1, Hkv, hd)
        v = qkv[:, (H + Hkv) * hd:].reshape(-1, Hkv, hd)
        q, k = rope(q, pos, c.rope_theta), rope(k, pos, c.rope_theta)
        if self.kv_dtype is not None:           # the cache's storage format
            k, v = k.to(self.kv_dtype).to(self.dtype), v.to(self.kv_dtype).to(self.dtype)
        Kall = torch.cat([Kc, k], 0) if Kc is not None and Kc.shape[0] else k
        Vall = torch.cat([Vc, v], 0) if Vc is not None and Vc.shape[0] else v
        o, probs = attention(q, Kall, Vall, mask)
        x = x + linear(o, w["wo"][l])
        b = rmsnorm(x, w["ln2"][l], c.rms_eps)
        x = x + mlp(b, w["wgu"][l], w["wd"][l], c.d_ff)
        return x, k, v, (probs if want_probs else None)

    def _logits(self, x):
        return linear(rmsnorm(x, self.tw["ln_f"], self.cfg.rms_eps), self.tw["lm_head"])

    def embed_rows(self, ids):
        return self.tw["embed"][torch.as_tensor(ids, dtype=torch.long)].to(self.dtype)

    # ------------------------------------------------------------------ O1 + O2 + scores
    def prefill(self, visual, vis_start, ids, extra_ids=(), keep_all_taps=False):
        """Causal forward of the n = q + v prompt tokens (Section 3, inference).

        The sequence holds the visual embeddings at [vis_start, vis_start+v) and
        embed[id] elsewhere; `extra_ids` are further text tokens appended at the end.
        Keeps per-layer K/V, S^l for every layer, the per-layer average attention
        entropy (Eq. 2) and, per layer, the importance of each visual token
        (Section 3.3).  Returns the state and (first token, margin).
        """
        c = self.cfg
        ids = [int(t) for t in ids] + [int(t) for t in extra_ids]
        v = visual.shape[0]
        n = v + len(ids)
        x = torch.empty(n, c.d_model, dtype=self.dtype)
        emb = self.embed_rows(ids) if ids else torch.empty(0, c.d_model, dtype=self.dtype)
        x[:vis_start] = emb[:vis_start]
        x[vis_start:vis_start + v] = visual.to(self.dtype)
        x[vis_start + v:] = emb[vis_start:]
        st = SeqState(P=n, n_prompt_total=n, vis_start=vis_start, n_visual=v, x0=x.clone())
        pos = torch.arange(n)
        causal = torch.ones(n, n, dtype=torch.bool).tril()
        ent = torch.zeros(c.n_layers, dtype=torch.float64)
        ent_sum = torch.zeros(c.n_layers, dtype=torch.float64)
        for l in range(c.n_layers):
            x, k, vv, probs = self._block(x, l, pos, None, None, causal, want_probs=True)
            st.K.append(k)
            st.V.append(vv)
            if keep_all_taps or c.tap_mode != TAP_FIXED and c.tap_lo <= l + 1 <= c.tap_hi \
                    or c.tap_mode == TAP_FIXED and l + 1 == c.tap_layer:
                st.taps[l + 1] = x.clone()
            ent[l] = row_entropy(probs).to(torch.float64).mean()       # mean over rows and heads
            ent_sum[l] = row_entropy(probs).to(torch.float64).sum()
            col = probs.sum(dim=0)                                      # sum over heads [n, n]
            if not c.score_include_self:
                col = col - torch.diag(torch.diagonal(col))
            st.scores[l + 1] = col.sum(dim=0)[vis_start:vis_start + v].clone()
        st.entropy = ent
        st.ent_sum = ent_sum
        tok, margin = argmax_low(self._logits(x[n - 1:n])[0])
        st.pending = tok
        st.tap, st.tap_margin = self.select_tap(ent)
        self._last_hidden = x
        return st, tok, margin

    # ------------------------------------------------------------------ O3
    def select_tap(self, ent):
        """l* = argmin (or argmax) of AE over [tap_lo, tap_hi], ties to the lower layer."""
        c = self.cfg
        if c.tap_mode == TAP_FIXED:
            return c.tap_layer, float("inf")
        e = ent[c.tap_lo - 1:c.tap_hi].clone()
        if c.tap_mode == TAP_ENTROPY_MIN:
            e = -e
        i, margin = argmax_low(e)
        return c.tap_lo + i, margin

    # ------------------------------------------------------------------ O4 + O5
    def compress_visual(self, st, k, forced_idx=None):
        """Keep the k most important visual tokens and build the draft's context.

        Importance of visual token j = attention it receives from later tokens at
        layer l*, summed over heads (Section 3.3).  The compressed context C is the
        kept visual positions plus every text position, ascending.  Draft
        self-attention K/V rows come from the input embeddings at C with rotary
        angles of the original positions; cross-attention memory rows are
        S^{l*}_c W_K, S^{l*}_c W_V (Eq. 1, no norm on the memory side).
        Returns (kept indices ascending, scores, margin at the cut).
        """
        c, dw = self.cfg, self.dw
        sc = st.scores[st.tap]
        v = st.n_visual
        if forced_idx is None:
            vals, idx = topk_low(sc, k)
            margin = float("inf")
            if k < v:
                allv, _ = torch.sort(sc, descending=True, stable=True)
                margin = float(allv[k - 1] - allv[k])
            kept = torch.sort(idx).values
        else:
            kept, margin = torch.as_tensor(forced_idx, dtype=torch.long), float("inf")
        st.kept = kept
        n = st.n_prompt_total
        is_vis = torch.zeros(n, dtype=torch.bool)
        is_vis[st.vis_start:st.vis_start + v] = True
        keep = ~is_vis
        keep[st.vis_start + kept] = True
        C = torch.nonzero(keep).flatten()
        st.ctx_pos = C
        Hkv, hd, H = c.n_kv_heads, c.head_dim, c.n_heads
        a = rmsnorm(st.x0[C], dw["ln1"], c.rms_eps)
        qkv = linear(a, dw["wqkv"])
        kk = qkv[:, H * hd:(H + Hkv) * hd].reshape(-1, Hkv, hd)
        vv = qkv[:, (H + Hkv) * hd:].reshape(-1, Hkv, hd)
        st.dK, st.dV = rope(kk, C, c.rope_theta), vv
        M = torch.arange(n) if c.xattn_full_memory else C
        S = st.taps[st.tap][M]
        kv = linear(S, dw["xkv"])
        st.mK = kv[:, :Hkv * hd].reshape(-1, Hkv, hd)
        st.mV = kv[:, Hkv * hd:].reshape(-1, Hkv, hd)
        st.new_tokens, st.new_pos = [], []
        st.dpos, st.mpos = C.clone(), M.clone()
        if c.draft_blocks == 3:
            self._draft3_context(st)
        return kept, sc, margin

    # ------------------------------------------------------------------ O6
    def _draft_rows(self, st, toks, pos):
        """Draft self-attention q, k, v of tokens at given positions (from embeddings)."""
        c, dw = self.cfg, self.dw
        H, Hkv, hd = c.n_heads, c.n_kv_heads, c.head_dim
        x = self.embed_rows(toks)
        a = rmsnorm(x, dw["ln1"], c.rms_eps)
        qkv = linear(a, dw["wqkv"])
        p = torch.as_tensor(pos, dtype=torch.long)
        q = rope(qkv[:, :H * hd].reshape(-1, H, hd), p, c.rope_theta)
        k = rope(qkv[:, H * hd:(H + Hkv) * hd].reshape(-1, Hkv, hd), p, c.rope_theta)
        v = qkv[:, (H + Hkv) * hd:].reshape(-1, Hkv, hd)
        return x, q, k, v

    def _draft_catch_up(self, st):
        """Permanent draft rows of the tokens the last acceptance emitted (all but the pending one)."""
        if not st.new_tokens:
            return
        if self.cfg.draft_blocks == 3:
            self._draft3_rows(st, self.embed_rows(st.new_tokens), torch.as_tensor(st.new_pos, dtype=torch.long))
        else:
            _, _, k, v = self._draft_rows(st, st.new_tokens, st.new_pos)
            st.dK, st.dV = torch.cat([st.dK, k], 0), torch.cat([st.dV, v], 0)
        st.new_tokens, st.new_pos = [], []

    @staticmethod
    def _tree_mask(n_perm, n_tree, rows, anc, strict):
        """[rows, n_perm + n_tree]: every permanent row, and in the tree region the row's ancestors
        (and the row itself unless `strict`)."""
        mask = torch.zeros(len(rows), n_perm + n_tree, dtype=torch.bool)
        mask[:, :n_perm] = True
        for i, r in enumerate(rows):
            mask[i, [n_perm + a for a in anc[i] if not (strict and a == r)]] = True
        return mask

    def _draft_pass(self, st, tr, rows, toks, pos, anc):
        """One pass of the single-block draft over the input nodes `rows`: self-attention, Eq. 1,
        MLP.  Appends the rows' K/V and memory rows to the tree regions `tr`; returns e^M."""
        c, dw = self.cfg, self.dw
        H, Hkv, hd = c.n_heads, c.n_kv_heads, c.head_dim
        nK, nM = st.dK.shape[0], st.mK.shape[0]
        x, q, k, v = self._draft_rows(st, toks, pos)
        tr["K"], tr["V"] = torch.cat([tr["K"], k], 0), torch.cat([tr["V"], v], 0)
        # self-attention: all permanent rows, plus own ancestors and self in the tree region
        mask = self._tree_mask(nK, tr["K"].shape[0], rows, anc, strict=False)
        o, _ = attention(q, torch.cat([st.dK, tr["K"]], 0), torch.cat([st.dV, tr["V"]], 0), mask)
        h = x + linear(o, dw["wo"])
        # cross-attention: verified memory rows plus strict ancestors' draft features
        qx = linear(rmsnorm(h, dw["lnx"], c.rms_eps), dw["xq"]).reshape(-1, H, hd)
        mask = self._tree_mask(nM, tr["mK"].shape[0], rows, anc, strict=True)
        o, _ = attention(qx, torch.cat([st.mK, tr["mK"]], 0), torch.cat([st.mV, tr["mV"]], 0), mask)
        h = h + linear(o, dw["xo"])
        h = h + mlp(rmsnorm(h, dw["ln2"], c.rms_eps), dw["wgu"], dw["wd"], c.d_ff)
        # e^M: the draft's final feature joins the memory (raw, unnormalised)
        kv = linear(h, dw["xkv"])
        tr["mK"] = torch.cat([tr["mK"], kv[:, :Hkv * hd].reshape(-1, Hkv, hd)], 0)
        tr["mV"] = torch.cat([tr["mV"], kv[:, Hkv * hd:].reshape(-1, Hkv, hd)], 0)
        return h

    def draft_tree(self, st):
        """Expand the draft token tree from the pending token (Section 3.1, tree drafting).

        Returns a dict with tokens, parent, depth, mask (list of ancestor-or-self sets),
        cum (cumulative log-probability), and the decision margins met on the way.
        """
        c = self.cfg
        Hkv, hd, D, K = c.n_kv_heads, c.head_dim, c.tree_depth, c.tree_topk
        # tokens verified by the last accept get their permanent rows in the draft's caches
        self._draft_catch_up(st)
        P = st.P
        # input nodes of the draft: each has a row in the tree regions of the draft's caches
        in_tok, in_depth, in_anc, in_cum, in_cand = [st.pending], [0], [[0]], [0.0], [-1]
        empty = torch.empty(0, Hkv, hd, dtype=self.dtype)
        tr = {n: empty.clone() for n in ("K", "V", "mK", "mV", "fK", "fV")}   # tree regions
        cands = []            # (token, parent candidate index or -1 for the root, depth, cum)
        margins = []          # decision margins: top-K cut of a row, adjacent gaps, beam cut
        feats, logp_rows = [], []
        beam = [0]            # indices into in_* of the nodes this pass expands
        cand_to_in = {}       # candidate index -> input-node index, for candidates that were expanded
        for p in range(1, D + 1):
            rows = beam
            toks = [in_tok[r] for r in rows]
            pos = [P + in_depth[r] for r in rows]
            anc = [in_anc[r] for r in rows]
            h = (self._draft_pass3 if c.draft_blocks == 3 else self._draft_pass)(st, tr, rows, toks, pos, anc)
            logp = torch.log_softmax(self._logits(h), dim=-1)
            new = []
            for i, r in enumerate(rows):
                feats.append(h[i].clone())
                logp_rows.append(logp[i].clone())
                sv, si = torch.sort(logp[i], descending=True, stable=True)
                margins.append(float(sv[K - 1] - sv[K]))
                margins.extend(float(sv[j] - sv[j + 1]) for j in range(K - 1))
                for j in range(K):
                    cands.append((int(si[j]), in_cand[r], in_depth[r] + 1, in_cum[r] + float(sv[j])))
                    new.append(len(cands) - 1)
            if p == D:
                break
            # next beam: the `beam` best new candidates by cumulative score
            cs = torch.tensor([cands[i][3] for i in new], dtype=torch.float64)
            nb = min(c.tree_beam, len(new))
            sv, si = torch.sort(cs, descending=True, stable=True)
            if nb < len(new):
                margins.append(float(sv[nb - 1] - sv[nb]))
            margins.extend(float(sv[j] - sv[j + 1]) for j in range(nb - 1))
            beam = []
            for j in range(nb):
                ci = new[int(si[j])]
                tok, par, dep, cum = cands[ci]
                par_in = 0 if par < 0 else cand_to_in[par]
                in_tok.append(tok); in_depth.append(dep); in_cum.append(cum); in_cand.append(ci)
                in_anc.append(in_anc[par_in] + [len(in_tok) - 1])
                beam.append(len(in_tok) - 1)
                cand_to_in[ci] = len(in_tok) - 1
        # global re-rank: the N best candidates, kept in creation order, root first
        N = min(c.tree_max_nodes, len(cands))
        cs = torch.tensor([cd[3] for cd in cands], dtype=torch.float64)
        sv, si = torch.sort(cs, descending=True, stable=True)
        if N < len(cands):
            margins.append(float(sv[N - 1] - sv[N]))
        chosen = sorted(int(i) for i in si[:N])
        node_of = {ci: j + 1 for j, ci in enumerate(chosen)}
        tokens, parent, depth, cum = [st.pending], [-1], [0], [0.0]
        for ci in chosen:
            tok, par, dep, cm = cands[ci]
            tokens.append(tok); depth.append(dep); cum.append(cm)
            parent.append(0 if par < 0 else node_of[par])
        mask = [{0}]
        for i in range(1, len(tokens)):
            mask.append(mask[parent[i]] | {i})
        return dict(tokens=tokens, parent=parent, depth=depth, mask=mask, cum=cum,
                    margins=margins, min_margin=min(margins) if margins else float("inf"),
                    cands=cands, feats=feats, logp_rows=logp_rows, in_tok=in_tok, in_depth=in_depth,
                    in_anc=in_anc)

    # ------------------------------------------------------------------ three-block draft (Section 4)
    # Reading of "an initial decoder block, an intermediate cross-attention block, and a final decoder
    # block": each block is pre-norm with a gated MLP behind its attention; the initial and the final
    # block attend causally to the draft's own rows (rotary positions), the intermediate block is Eq. 1.
    # Weights: initial = ln1, wqkv, wo, i_ln2, i_wgu, i_wd; intermediate = lnx, xq, xkv, xo, ln2, wgu, wd;
    # final = f_ln1, f_wqkv, f_wo, f_ln2, f_wgu, f_wd.  A row at position p sees, in the self-attention
    # caches, every row of a position <= p that is on its own path, and in the memory every row of a
    # position < p on its path (a target feature s_p already encodes the prediction of token p + 1).
    def _self_block(self, x, pos, Kc, Vc, mask, names):
        """One decoder block of the draft on rows x; (Kc, Vc) cached rows, the new rows' K/V are
        appended behind them and mask [m, cached + m] covers both.  Returns (x, k, v)."""
        c, dw = self.cfg, self.dw
        ln1, wqkv, wo, ln2, wgu, wd = (dw[n] for n in names)
        H, Hkv, hd = c.n_heads, c.n_kv_heads, c.head_dim
        qkv = linear(rmsnorm(x, ln1, c.rms_eps), wqkv)
        p = torch.as_tensor(pos, dtype=torch.long)
        q = rope(qkv[:, :H * hd].reshape(-1, H, hd), p, c.rope_theta)
        k = rope(qkv[:, H * hd:(H + Hkv) * hd].reshape(-1, Hkv, hd), p, c.rope_theta)
        v = qkv[:, (H + Hkv) * hd:].reshape(-1, Hkv, hd)
        o, _ = attention(q, torch.cat([Kc, k], 0), torch.cat([Vc, v], 0), mask)
        x = x + linear(o, wo)
        x = x + mlp(rmsnorm(x, ln2, c.rms_eps), wgu, wd, c.d_ff)
        return x, k, v

    def _cross_block(self, x, MK, MV, mask):
        """The intermediate block: Eq. 1 over the memory rows the mask admits (a row that sees none
        gets no attention term), then the block's MLP."""
        c, dw = self.cfg, self.dw
        H, hd = c.n_heads, c.head_dim
        q = linear(rmsnorm(x, dw["lnx"], c.rms_eps), dw["xq"]).reshape(-1, H, hd)
        o = torch.zeros(x.shape[0], H * hd, dtype=x.dtype)
        live = mask.any(dim=1)
        if bool(live.any()):
            ol, _ = attention(q[live], MK, MV, mask[live])
            o[live] = ol
        x = x + linear(o, dw["xo"])
        return x + mlp(rmsnorm(x, dw["ln2"], c.rms_eps), dw["wgu"], dw["wd"], c.d_ff)

    def _draft3_rows(self, st, x, pos):
        """Permanent rows of the three-block draft for inputs x at ascending positions `pos` (the
        compressed context at set-up, then the tokens each acceptance emits): the initial block over
        its cache, Eq. 1 over the memory rows of an earlier position, the final block over its cache.
        Appends the K/V rows of both self-attention blocks."""
        m = x.shape[0]
        seen = torch.cat([torch.ones(m, st.dK.shape[0], dtype=torch.bool),
                          torch.ones(m, m, dtype=torch.bool).tril()], 1)
        h, k1, v1 = self._self_block(x, pos, st.dK, st.dV, seen, self.INITIAL)
        h = self._cross_block(h, st.mK, st.mV, st.mpos[None, :] < pos[:, None])
        _, k3, v3 = self._self_block(h, pos, st.fK, st.fV, seen, self.FINAL)
        st.dK, st.dV = torch.cat([st.dK, k1], 0), torch.cat([st.dV, v1], 0)
        st.fK, st.fV = torch.cat([st.fK, k3], 0), torch.cat([st.fV, v3], 0)
        st.dpos = torch.cat([st.dpos, pos])

    def _draft3_context(self, st):
        """Draft prefill over the compressed context C (Section 3.3: the draft works on the reduced
        sequence): every block's rows for the inputs at C, from empty caches."""
        c = self.cfg
        empty = torch.empty(0, c.n_kv_heads, c.head_dim, dtype=self.dtype)
        st.dK, st.dV, st.fK, st.fV = empty, empty.clone(), empty.clone(), empty.clone()
        st.dpos = torch.empty(0, dtype=torch.long)
        self._draft3_rows(st, st.x0[st.ctx_pos], st.ctx_pos)

    def _draft_pass3(self, st, tr, rows, toks, pos, anc):
        """One pass of the three-block draft over the input nodes `rows`; the tree regions of the
        two self-attention caches hold ancestors and self, that of the memory strict ancestors."""
        c, dw = self.cfg, self.dw
        Hkv, hd = c.n_kv_heads, c.head_dim
        x = self.embed_rows(toks)
        m, nt = len(rows), tr["K"].shape[0] + len(rows)
        mask = self._tree_mask(st.dK.shape[0], nt, rows, anc, strict=False)
        h, k, v = self._self_block(x, pos, torch.cat([st.dK, tr["K"]], 0), torch.cat([st.dV, tr["V"]], 0),
                                   mask, self.INITIAL)
        tr["K"], tr["V"] = torch.cat([tr["K"], k], 0), torch.cat([tr["V"], v], 0)
        mask = self._tree_mask(st.mK.shape[0], tr["mK"].shape[0], rows, anc, strict=True)
        h = self._cross_block(h, torch.cat([st.mK, tr["mK"]], 0), torch.cat([st.mV, tr["mV"]], 0), mask)
        mask = self._tree_mask(st.fK.shape[0], nt, rows, anc, strict=False)
        h, k, v = self._self_block(h, pos, torch.cat([st.fK, tr["fK"]], 0), torch.cat([st.fV, tr["fV"]], 0),
                                   mask, self.FINAL)
        tr["fK"], tr["fV"] = torch.cat([tr["fK"], k], 0), torch.cat([tr["fV"], v], 0)
        kv = linear(h, dw["xkv"])
        tr["mK"] = torch.cat([tr["mK"], kv[:, :Hkv * hd].reshape(-1, Hkv, hd)], 0)
        tr["mV"] = torch.cat([tr["mV"], kv[:, Hkv * hd:].reshape(-1, Hkv, hd)], 0)
        return h

    INITIAL = ("ln1", "wqkv", "wo", "i_ln2", "i_wgu", "i_wd")
    FINAL = ("f_ln1", "f_wqkv", "f_wo", "f_ln2", "f_wgu", "f_wd")

    # ------------------------------------------------------------------ O7
    def verify_tree(self, st, tree):
        """Run the T tree tokens through the target with the tree mask (Section 3.1).

        Node i sits at position P + depth_i, sees the verified prefix and the tail rows
        of its ancestors and itself.  Returns logits, argmax, margins, per-layer tail
        K/V and the tapped features of the tail.
        """
        c = self.cfg
        T, P = len(tree["tokens"]), st.P
        x = self.embed_rows(tree["tokens"])
        pos = torch.tensor([P + dd for dd in tree["depth"]])
        mask = torch.zeros(T, P + T, dtype=torch.bool)
        mask[:, :P] = True
        for i in range(T):
            mask[i, [P + j for j in tree["mask"][i]]] = True
        tailK, tailV, tap_rows, row_ent = [], [], None, []
        for l in range(c.n_layers):
            x, k, v, probs = self._block(x, l, pos, st.K[l][:P], st.V[l][:P], mask, want_probs=True)
            tailK.append(k); tailV.append(v)
            # entropy of each tree row's attention distribution, summed over heads: for a node on the
            # accepted path the distribution is the causal one of its position (it sees the prefix and
            # its ancestors, which are the accepted tokens before it)
            row_ent.append(row_entropy(probs).to(torch.float64).sum(dim=0))
            if l + 1 == st.tap:
                tap_rows = x.clone()
        logits = self._logits(x)
        am, mg = zip(*(argmax_low(logits[i]) for i in range(T)))
        return dict(logits=logits, argmax=list(am), margin=list(mg), tailK=tailK, tailV=tailV,
                    tap_rows=tap_rows, hidden=x, row_entropy=row_ent)

    # ------------------------------------------------------------------ O8
    @staticmethod
    def accept(tree, argmax):
        """Greedy acceptance: follow the child whose token equals the parent's argmax.

        Returns (A, out_tokens [A+1], path [A+1]) where path[0] = 0 is the root and the
        last emitted token is the target's own (bonus) token.
        """
        T = len(tree["tokens"])
        cur, path, out = 0, [0], []
        while True:
            g = argmax[cur]
            nxt = [i for i in range(T) if tree["parent"][i] == cur and tree["tokens"][i] == g]
            if not nxt:
                out.append(g)
                return len(path) - 1, out, path
            cur = nxt[0]
            path.append(cur)
            out.append(tree["tokens"][cur])

    # ------------------------------------------------------------------ O8, sampling form
    @staticmethod
    def accept_sample(tree, logits, temp, uniforms):
        """Stochastic acceptance at temperature `temp` > 0 (Section 2.1: a draft token d is kept
        with probability min(1, P_target(d) / P_draft(d)), which holds at any temperature;
        Section 4 evaluates Temp = 1).

        Reading for a tree whose children are the draft's top-K choices (no draw on the draft
        side): every child is a point-mass proposal, P_draft = 1, so child c of the current node
        is kept with probability p(token_c), p = softmax(logits[cur] / temp) with the tokens
        already refused at this node taken out and the rest renormalised (the residual
        max(p - P_draft, 0) of a point mass is p without that token).  Children are tried in
        node order.  When every child is refused, or the node has none, the emitted token is
        drawn from what is left of p by inverting its cumulative sum in token order.  The
        emitted token then follows p exactly, whatever the draft proposed.

        uniforms[j][r]: the number in [0, 1) used at path step j for the r-th child tried
        (r < K), uniforms[j][-1] for the final draw.  Returns (A, out_tokens, path, slack) with
        slack = the smallest distance of a used uniform from the threshold it was compared with.
        """
        T = len(tree["tokens"])
        lg = torch.as_tensor(logits, dtype=torch.float64)
        cur, path, out, slack, j = 0, [0], [], 1.0, 0
        while True:
            p = torch.softmax(lg[cur] / temp, 0)
            kids = [i for i in range(T) if tree["parent"][i] == cur]
            left, taken = 1.0, None
            for r, c in enumerate(kids):
                pc = float(p[tree["tokens"][c]]) / left
                u = float(uniforms[j][r])
                slack = min(slack, abs(u - pc))
                if u < pc:
                    taken = c
                    break
                left -= float(p[tree["tokens"][c]])
                p[tree["tokens"][c]] = 0.0
            if taken is None:
                cdf = torch.cumsum(p, 0)
                target = float(uniforms[j][-1]) * float(cdf[-1])
                g = int(torch.searchsorted(cdf, torch.tensor(target, dtype=torch.float64), right=True))
                g = min(g, len(p) - 1)
                while float(p[g]) == 0.0:        # a refused token or an underflowed tail entry
                    g -= 1
                lo = float(cdf[g - 1]) if g > 0 else 0.0
                slack = min(slack, (target - lo) / float(cdf[-1]), (float(cdf[g]) - target) / float(cdf[-1]))
                out.append(g)
                return len(path) - 1, out, path, slack
            cur = taken
            path.append(cur)
            out.append(tree["tokens"][cur])
            j += 1

    # ------------------------------------------------------------------ O9
    def commit(self, st, tree, ver, path, out_tokens):
        """Compact the target KV to the accepted path and extend the draft's caches."""
        c, dw = self.cfg, self.dw
        Hkv, hd = c.n_kv_heads, c.head_dim
        P, A1 = st.P, len(path)
        idx = torch.tensor(path)
        for l in range(c.n_layers):
            st.K[l] = torch.cat([st.K[l][:P], ver["tailK"][l][idx]], 0)
            st.V[l] = torch.cat([st.V[l][:P], ver["tailV"][l][idx]], 0)
        kv = linear(ver["tap_rows"][idx], dw["xkv"])
        st.mK = torch.cat([st.mK, kv[:, :Hkv * hd].reshape(-1, Hkv, hd)], 0)
        st.mV = torch.cat([st.mV, kv[:, Hkv * hd:].reshape(-1, Hkv, hd)], 0)
        st.new_tokens = [tree["tokens"][i] for i in path]
        st.new_pos = [P + j for j in range(A1)]
        if st.mpos is not None:
            st.mpos = torch.cat([st.mpos, torch.arange(P, P + A1)])
        if st.ent_sum is not None and "row_entropy" in ver:
            # Eq. 2 over the longer sequence: only the new rows' entropies are added (Section 3.2,
            # the selection "during each decoding step")
            st.ent_sum = st.ent_sum + torch.stack([re[idx].sum() for re in ver["row_entropy"]])
        st.P = P + A1
        st.pending = out_tokens[-1]
        return path

    def layer_entropy(self, st):
        """AE of Eq. 2 over the P rows verified so far, per layer, and the layer Section 3.2 would
        select from it now (the draft keeps the layer chosen at prefill: its memory holds that
        layer's features).  Returns (AE [L], layer, margin)."""
        ae = st.ent_sum / (self.cfg.n_heads * st.P)
        layer, margin = self.select_tap(ae)
        return ae, layer, margin

    def step(self, st, tree=None, temp=0.0, uniforms=None):
        """One draft + verify + accept + commit round; `tree` overrides the draft's tree.
        temp > 0 takes the sampling form of the acceptance with the given uniforms."""
        drafted = self.draft_tree(st)
        tree = drafted if tree is None else tree
        ver = self.verify_tree(st, tree)
        if temp > 0:
            A, out, path, _ = self.accept_sample(tree, ver["logits"], temp, uniforms)
        else:
            A, out, path = self.accept(tree, ver["argmax"])
        self.commit(st, tree, ver, path, out)
        return dict(tree=tree, drafted=drafted, ver=ver, A=A, out=out, path=path)

    # ------------------------------------------------------------------ O10
    def ar_decode(self, visual, vis_start, ids, n_new):
        """Plain greedy autoregressive decoding of the target with its own KV cache."""
        c = self.cfg
        st, tok, _ = self.prefill(visual, vis_start, ids)
        out, margins = [tok], []
        Ks, Vs = [k.clone() for k in st.K], [v.clone() for v in st.V]
        P = st.P
        while len(out) < n_new:
            x = self.embed_rows([out[-1]])
            pos = torch.tensor([P])
            for l in range(c.n_layers):
                mask = torch.ones(1, P + 1, dtype=torch.bool)
                x, k, v, _ = self._block(x, l, pos, Ks[l], Vs[l], mask)
                Ks[l], Vs[l] = torch.cat([Ks[l], k], 0), torch.cat([Vs[l], v], 0)
            P += 1
            t, m = argmax_low(self._logits(x)[0])
            out.append(t); margins.append(m)
        return out, margins


def make_tree(tokens, parent):
    """Build a tree dict (depth, ancestor sets) from tokens and parent indices; node 0 is the root."""
    depth, mask = [0], [{0}]
    for i in range(1, len(tokens)):
        depth.append(depth[parent[i]] + 1)
        mask.append(mask[parent[i]] | {i})
    return dict(tokens=list(tokens), parent=list(parent), depth=depth, mask=mask,
                cum=[0.0] * len(tokens))
