"""Thin ctypes binding of libdream.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/dream.h).  Torch
is used for device memory and streams; every step of the method runs in the library's CUDA
kernels.  There is no CPU or PyTorch fallback: if the library cannot be loaded, importing
`lib()` raises.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

DREAM_F32, DREAM_BF16 = 0, 1
MAX_DEPTH = 15

ERRORS = {0: "OK", -1: "E_ARG", -2: "E_STATE", -3: "E_NOMEM", -4: "E_CAPACITY", -5: "E_CUDA",
          -6: "E_DEVICE_TIMEOUT", -7: "E_UNSUPPORTED"}


class DreamError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"dream: {ERRORS.get(code, code)}: {msg}")
        self.code = code


class dream_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim",
                                          "d_ff", "vocab", "dtype")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("max_batch", "max_seq", "max_prompt", "max_visual", "page_tokens",
                                          "tree_depth", "tree_topk", "tree_beam", "tree_max_nodes",
                                          "tap_mode", "tap_layer", "tap_lo", "tap_hi",
                                          "score_include_self", "xattn_full_memory", "draft_blocks", "track_entropy")]


class dream_target_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("ln1", "wqkv", "wo", "ln2", "wgu", "wd")] + \
               [("ln_f", C.c_void_p), ("lm_head", C.c_void_p)]


DRAFT_TENSORS = ("ln1", "wqkv", "wo", "lnx", "xq", "xkv", "xo", "ln2", "wgu", "wd")
DRAFT_TENSORS_3 = ("i_ln2", "i_wgu", "i_wd", "f_ln1", "f_wqkv", "f_wo", "f_ln2", "f_wgu", "f_wd")   # draft_blocks = 3 only


class dream_draft_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in DRAFT_TENSORS + DRAFT_TENSORS_3]


class dream_tree(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("tokens", "parent", "depth", "mask", "cum_logp")]


def lib():
    """Load libdream.so from the package directory; fail loudly when it is missing."""
    global _LIB
    if _LIB is None:
        path = os.path.join(_HERE, "libdream.so")
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with `python -m paper_2505_19201_b200.build` "
                              "(there is no fallback path)")
        L = C.CDLL(path)
        vp, i32, i32p = C.c_void_p, C.c_int32, C.POINTER(C.c_int32)
        sig = {
            "dream_tree_nodes": [C.POINTER(dream_config), i32p],
            "dream_arena_bytes": [C.POINTER(dream_config), C.POINTER(C.c_size_t)],
            "dream_tree_from_parents": [i32p, i32, i32p, C.POINTER(C.c_uint32)],
            "dream_init": [C.POINTER(dream_config), C.POINTER(dream_target_weights), C.POINTER(dream_draft_weights),
                           vp, C.c_size_t, vp, C.POINTER(vp)],
            "dream_prefill": [vp, i32, vp, i32, i32, vp, i32, vp, vp, vp, vp],
            "dream_set_tap": [vp, i32, i32],
            "dream_compress_visual": [vp, i32, i32, vp, vp, vp],
            "dream_draft_tree": [vp, i32p, i32, C.POINTER(dream_tree)],
            "dream_verify_tree": [vp, i32p, i32, C.POINTER(dream_tree), vp, vp, vp],
            "dream_accept": [vp, i32p, i32, C.POINTER(dream_tree), vp, vp, vp, vp],
            "dream_accept_sample": [vp, i32p, i32, C.POINTER(dream_tree), vp, C.c_float, vp, vp, vp, vp],
            "dream_step_host": [vp, i32p, i32, vp, vp],
            "dream_seq_state": [vp, i32, i32p, i32p, i32p],
            "dream_layer_entropy": [vp, i32, vp, i32p],
            "dream_debug_read": [vp, i32, i32, i32, i32, vp],
            "dream_seq_reset": [vp, i32],
            "dream_debug_gemm": [vp, vp, vp, i32, i32, i32, i32, vp],
            "dream_gemm_counts": [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64)],
            "dream_gemm_timing": [vp, i32, C.POINTER(C.c_int64), C.POINTER(C.c_double), C.POINTER(C.c_double)],
            "dream_poll": [vp],
            "dream_trace": [vp, vp, C.c_int64],
            "dream_topk_lse_static": [vp, i32, i32, i32, vp, vp, vp, vp],
        }
        for name, args in sig.items():
            fn = getattr(L, name)
            fn.argtypes, fn.restype = args, i32
        L.dream_launch_count.argtypes, L.dream_launch_count.restype = [vp], C.c_int64
        L.dream_last_error.argtypes, L.dream_last_error.restype = [vp], C.c_char_p
        L.dream_free.argtypes, L.dream_free.restype = [vp], None
        L.dream_trace_name.argtypes, L.dream_trace_name.restype = [i32], C.c_char_p
        _LIB = L
    return _LIB


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def make_config(p, max_batch=None, max_seq=None, page_tokens=64):
    """dream_config from a preset dict (paper_2505_19201_b200.configs)."""
    c = dream_config()
    for k in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ff", "vocab", "tree_depth",
              "tree_topk", "tree_beam", "tree_max_nodes", "tap_mode", "tap_layer", "tap_lo", "tap_hi",
              "score_include_self", "xattn_full_memory"):
        setattr(c, k, int(p[k]))
    c.draft_blocks = int(p.get("draft_blocks", 1))
    c.track_entropy = int(p.get("track_entropy", 0))
    c.dtype = DREAM_BF16 if p["dtype"] == "bf16" else DREAM_F32
    c.rms_eps, c.rope_theta = p["rms_eps"], p["rope_theta"]
    n = p["n_visual"] + p["n_prompt"]
    c.max_batch = max_batch or p["batch"]
    c.max_prompt, c.max_visual, c.page_tokens = n, p["n_visual"], page_tokens
    T = dream_tree_nodes(c)
    c.max_seq = max_seq or (n + (p["decode_steps"] + 2) * (p["tree_depth"] + 1) + T)
    return c


def dream_tree_nodes(cfg):
    T = C.c_int32()
    _check(None, lib().dream_tree_nodes(C.byref(cfg), C.byref(T)))
    return T.value


def dream_arena_bytes(cfg):
    n = C.c_size_t()
    _check(None, lib().dream_arena_bytes(C.byref(cfg), C.byref(n)))
    return n.value


def _check(ctx, code):
    if code != 0:
        raise DreamError(code, lib().dream_last_error(ctx).decode())


def dream_topk_lse_static(logits, ktop, top_val, top_id, lse, stream=None):
    """Top-k and log-sum-exp of a device float32 matrix [rows][vocab] through the entry point that
    needs no arena (its scratch is built into the library).  Outputs are caller-allocated device
    tensors: top_val [rows][ktop] float32, top_id [rows][ktop] int32, lse [rows] float32."""
    rows, vocab = logits.shape
    st = stream or torch.cuda.current_stream(logits.device)
    with torch.cuda.device(logits.device):
        _check(None, lib().dream_topk_lse_static(_ptr(logits), rows, vocab, ktop, _ptr(top_val), _ptr(top_id), _ptr(lse),
                                                 C.c_void_p(st.cuda_stream)))


class Tree:
    """Device buffers of one token tree (capacity T nodes) plus the C struct that points at them."""

    def __init__(self, T, device):
        self.T = T
        self.tokens = torch.zeros(T, dtype=torch.int32, device=device)
        self.parent = torch.zeros(T, dtype=torch.int32, device=device)
        self.depth = torch.zeros(T, dtype=torch.int32, device=device)
        self.mask = torch.zeros(T, 4, dtype=torch.int32, device=device)
        self.cum_logp = torch.zeros(T, dtype=torch.float32, device=device)

    def struct(self):
        return dream_tree(*(t.data_ptr() for t in (self.tokens, self.parent, self.depth, self.mask, self.cum_logp)))

    def load(self, tokens, parent):
        """Fill from host lists (inject a tree); the library derives depths and masks
        (dream_tree_from_parents)."""
        T = self.T
        assert len(tokens) == T and len(parent) == T
        par = torch.tensor(parent, dtype=torch.int32)
        depth = torch.zeros(T, dtype=torch.int32)
        mask = torch.zeros(T, 4, dtype=torch.int32)
        _check(None, lib().dream_tree_from_parents(C.cast(par.data_ptr(), C.POINTER(C.c_int32)), T,
                                                   C.cast(depth.data_ptr(), C.POINTER(C.c_int32)),
                                                   C.cast(mask.data_ptr(), C.POINTER(C.c_uint32))))
        self.load_raw(tokens, par, depth, mask)

    def load_raw(self, tokens, parent, depth, mask):
        """Copy the four arrays to the device as they are (no checks: error-path tests use this)."""
        dev = self.tokens.device
        self.tokens.copy_(torch.as_tensor(tokens, dtype=torch.int32).to(dev))
        self.parent.copy_(torch.as_tensor(parent, dtype=torch.int32).to(dev))
        self.depth.copy_(torch.as_tensor(depth, dtype=torch.int32).to(dev))
        self.mask.copy_(torch.as_tensor(mask, dtype=torch.int32).reshape(self.T, 4).to(dev))

    def to_host(self):
        m = self.mask.cpu().to(torch.int64) & 0xFFFFFFFF
        sets = [{j for j in range(self.T) if (int(m[i, j >> 5]) >> (j & 31)) & 1} for i in range(self.T)]
        return dict(tokens=self.tokens.cpu().tolist(), parent=self.parent.cpu().tolist(),
                    depth=self.depth.cpu().tolist(), mask=sets, cum=self.cum_logp.cpu().tolist())


class Context:
    """Owns the arena tensor and the dream_ctx handle; methods carry the C entry points' names."""

    def __init__(self, cfg, tw, dw, device="cuda:0", stream=None):
        self.cfg, self.device = cfg, torch.device(device)
        self.tw, self.dw = tw, dw            # keep the borrowed weights alive
        L = cfg.n_layers
        self._arrs = {}
        t = dream_target_weights()
        t.embed, t.ln_f, t.lm_head = tw["embed"].data_ptr(), tw["ln_f"].data_ptr(), tw["lm_head"].data_ptr()
        for name in ("ln1", "wqkv", "wo", "ln2", "wgu", "wd"):
            arr = (C.c_void_p * L)(*(w.data_ptr() for w in tw[name]))
            self._arrs[name] = arr
            setattr(t, name, arr)
        d = dream_draft_weights(*(dw[n].data_ptr() for n in DRAFT_TENSORS),
                                *(dw[n].data_ptr() if n in dw else None for n in DRAFT_TENSORS_3))
        self.arena_bytes = dream_arena_bytes(cfg)
        self.arena = torch.empty(self.arena_bytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.arena.data_ptr() + 255) & ~255
        self.stream = stream or torch.cuda.current_stream(self.device)
        self.T = dream_tree_nodes(cfg)
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(None, lib().dream_init(C.byref(cfg), C.byref(t), C.byref(d), C.c_void_p(base), self.arena_bytes,
                                          C.c_void_p(self.stream.cuda_stream), C.byref(h)))
        self.h = h

    def close(self):
        if self.h:
            lib().dream_free(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def new_tree(self):
        return Tree(self.T, self.device)

    @staticmethod
    def _seqs(seqs):
        return (C.c_int32 * len(seqs))(*seqs), len(seqs)

    @staticmethod
    def _trees(trees):
        if trees is None:
            return None
        return (dream_tree * len(trees))(*(t.struct() for t in trees))

    def dream_prefill(self, seq, visual, vis_start, ids, first_token=None, first_margin=None, layer_entropy=None,
                      tap_layer=None):
        _check(self.h, lib().dream_prefill(self.h, seq, _ptr(visual), visual.shape[0] if visual is not None else 0,
                                           vis_start, _ptr(ids), ids.shape[0] if ids is not None else 0,
                                           _ptr(first_token), _ptr(first_margin), _ptr(layer_entropy), _ptr(tap_layer)))

    def dream_set_tap(self, seq, layer):
        _check(self.h, lib().dream_set_tap(self.h, seq, layer))

    def dream_compress_visual(self, seq, k, forced_idx=None, kept_idx=None, scores=None):
        _check(self.h, lib().dream_compress_visual(self.h, seq, k, _ptr(forced_idx), _ptr(kept_idx), _ptr(scores)))

    def dream_draft_tree(self, seqs, trees=None):
        a, n = self._seqs(seqs)
        _check(self.h, lib().dream_draft_tree(self.h, a, n, self._trees(trees)))

    def dream_verify_tree(self, seqs, trees, node_argmax, node_margin=None, logits=None):
        a, n = self._seqs(seqs)
        _check(self.h, lib().dream_verify_tree(self.h, a, n, self._trees(trees), _ptr(node_argmax), _ptr(node_margin),
                                               _ptr(logits)))

    def dream_accept(self, seqs, trees, node_argmax, accept_len, out_tokens, compaction_src=None):
        a, n = self._seqs(seqs)
        _check(self.h, lib().dream_accept(self.h, a, n, self._trees(trees), _ptr(node_argmax), _ptr(accept_len),
                                          _ptr(out_tokens), _ptr(compaction_src)))

    def dream_accept_sample(self, seqs, trees, logits, temperature, uniforms, accept_len, out_tokens, compaction_src=None):
        a, n = self._seqs(seqs)
        _check(self.h, lib().dream_accept_sample(self.h, a, n, self._trees(trees), _ptr(logits), float(temperature),
                                                 _ptr(uniforms), _ptr(accept_len), _ptr(out_tokens), _ptr(compaction_src)))

    def dream_step_host(self, seqs, accept_len_host, out_tokens_host):
        """accept_len_host / out_tokens_host: CPU int32 tensors (HOST buffers)."""
        a, n = self._seqs(seqs)
        _check(self.h, lib().dream_step_host(self.h, a, n, C.c_void_p(accept_len_host.data_ptr()),
                                             C.c_void_p(out_tokens_host.data_ptr())))

    def dream_seq_state(self, seq):
        P, t, tap = C.c_int32(), C.c_int32(), C.c_int32()
        _check(self.h, lib().dream_seq_state(self.h, seq, C.byref(P), C.byref(t), C.byref(tap)))
        return P.value, t.value, tap.value

    def dream_layer_entropy(self, seq):
        """(AE per layer over the rows verified so far [L] float32, the layer that would be selected now)."""
        ae = torch.empty(self.cfg.n_layers, dtype=torch.float32)
        layer = C.c_int32()
        _check(self.h, lib().dream_layer_entropy(self.h, seq, C.c_void_p(ae.data_ptr()), C.byref(layer)))
        return ae, layer.value

    def dream_debug_read(self, seq, what, layer, index):
        n = self.cfg.n_kv_heads * self.cfg.head_dim if what <= 5 or what >= 8 else self.cfg.d_model
        out = torch.empty(n, dtype=torch.float32)
        _check(self.h, lib().dream_debug_read(self.h, seq, what, layer, index, C.c_void_p(out.data_ptr())))
        return out

    def dream_debug_gemm(self, W, X, split=1):
        rows, K = X.shape
        N = W.shape[0]
        out = torch.empty(rows, N, dtype=torch.float32, device=self.device)
        _check(self.h, lib().dream_debug_gemm(self.h, _ptr(W), _ptr(X), rows, N, K, split, _ptr(out)))
        return out

    def dream_gemm_counts(self):
        a, b = C.c_int64(), C.c_int64()
        _check(self.h, lib().dream_gemm_counts(self.h, C.byref(a), C.byref(b)))
        return a.value, b.value

    def dream_gemm_timing(self, on):
        """on=True starts bracketing GEMM launches with events; on=False returns (launches, ms, bytes)."""
        n, ms, by = C.c_int64(), C.c_double(), C.c_double()
        _check(self.h, lib().dream_gemm_timing(self.h, 1 if on else 0, C.byref(n), C.byref(ms), C.byref(by)))
        return n.value, ms.value, by.value

    def dream_trace(self, capacity=0):
        """capacity > 0: start a timeline of this context's stream; 0: stop and return [(kernel, ns)]."""
        if capacity:
            self._trace = torch.zeros(2 + 2 * capacity, dtype=torch.int64, device=self.device)
            _check(self.h, lib().dream_trace(self.h, C.c_void_p(self._trace.data_ptr()), capacity))
            return None
        _check(self.h, lib().dream_trace(self.h, None, 0))
        t = self._trace.cpu().tolist()
        n = min(t[0], t[1])
        return [(lib().dream_trace_name(int(t[2 + 2 * i])).decode(), t[3 + 2 * i]) for i in range(n)]

    def dream_seq_reset(self, seq):
        _check(self.h, lib().dream_seq_reset(self.h, seq))

    def dream_poll(self):
        _check(self.h, lib().dream_poll(self.h))

    def dream_launch_count(self):
        return lib().dream_launch_count(self.h)
