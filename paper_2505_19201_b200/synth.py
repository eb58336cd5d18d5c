"""Seeded synthetic inputs: weights, visual embeddings, prompt ids.

The generator is counter based: element i of stream s is a pure function of
(s, i), built from 64-bit integer tensor operations only, then mapped through a
65536-entry table of standard-normal quantiles.  Integer tensor arithmetic and
a table lookup give the same bits on a CPU and on a GPU, so the CPU oracle and
the CUDA path can each materialise the same tensors on their own device without
a host<->device copy of gigabytes of weights.

This module holds none of the method's arithmetic; it only makes inputs.

Recipe (stands in for the paper's benchmark inputs, of which only the shape is
used): weight matrices ~ N(0, 0.02^2), norm gains 1, visual embeddings ~ N(0,1),
prompt ids uniform on [0, V); values rounded to the storage dtype.
"""
import math
import torch

_MASK32 = 0xFFFFFFFF
_CHUNK = 1 << 25


def _quantile_table():
    # z_j = Phi^-1((j + 0.5) / 65536), computed once in fp64 on the CPU
    u = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
    return math.sqrt(2.0) * torch.erfinv(2.0 * u - 1.0)


_TABLE64 = None
_TABLES = {}


def _table(device):
    global _TABLE64
    if _TABLE64 is None:
        _TABLE64 = _quantile_table()
    key = str(device)
    if key not in _TABLES:
        _TABLES[key] = _TABLE64.to(torch.float32).to(device)
    return _TABLES[key]


def stream_id(*parts):
    """Mix small non-negative integers into one 31-bit stream id."""
    s = 0x1234567
    for p in parts:
        s = (s * 1000003 + int(p) + 0x9E37) % 0x7FFFFFFF
    return s


def _hash32(idx, sid):
    """32-bit integer mix of (index, stream); int64 tensors, every product < 2^63."""
    x = (idx + sid * 0x9E3779B1) & _MASK32
    x = x ^ (x >> 16)
    x = (x * 0x7FEB352D) & _MASK32
    x = x ^ (x >> 15)
    x = (x * 0x2C1B3C6D) & _MASK32
    x = x ^ (x >> 16)
    x = (x * 0x297A2D39) & _MASK32
    x = x ^ (x >> 15)
    return x


def normal(shape, std, sid, dtype, device="cpu"):
    """Tensor of the given shape with entries std * z, z from the quantile table."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    tab = _table(device)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        h = _hash32(idx, sid)
        z = tab[(h >> 16)]
        out[lo:hi] = (z * std).to(dtype)
    return out.view(*shape)


def uniform_ids(n, vocab, sid, device="cpu"):
    idx = torch.arange(n, dtype=torch.int64, device=device)
    return (_hash32(idx, sid) % vocab).to(torch.int32)


def torch_dtype(name):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def target_weights(p, seed=0, device="cpu"):
    """Random-init target weights for preset p.  All matrices are [out, in] row-major.

    wqkv stacks the query, key and value projections by rows; wgu stacks the gate
    and up projections by rows.
    """
    dt = torch_dtype(p["dtype"])
    L, d, H, Hkv, hd, ff, V = (p[k] for k in ("n_layers", "d_model", "n_heads", "n_kv_heads",
                                              "head_dim", "d_ff", "vocab"))
    qkv = (H + 2 * Hkv) * hd
    w = {"embed": normal((V, d), 0.02, stream_id(seed, 1), dt, device),
         "lm_head": normal((V, d), 0.02, stream_id(seed, 2), dt, device),
         "ln_f": torch.ones(d, dtype=dt, device=device),
         "ln1": [], "wqkv": [], "wo": [], "ln2": [], "wgu": [], "wd": []}
    for l in range(L):
        w["ln1"].append(torch.ones(d, dtype=dt, device=device))
        w["ln2"].append(torch.ones(d, dtype=dt, device=device))
        w["wqkv"].append(normal((qkv, d), 0.02, stream_id(seed, 10, l, 0), dt, device))
        w["wo"].append(normal((d, H * hd), 0.02, stream_id(seed, 10, l, 1), dt, device))
        w["wgu"].append(normal((2 * ff, d), 0.02, stream_id(seed, 10, l, 2), dt, device))
        w["wd"].append(normal((d, ff), 0.02, stream_id(seed, 10, l, 3), dt, device))
    return w


def draft_weights(p, seed=0, device="cpu"):
    """Random-init weights of the draft: one layer (self-attention, cross-attention, MLP), or with
    draft_blocks = 3 the three blocks of Section 4."""
    dt = torch_dtype(p["dtype"])
    d, H, Hkv, hd, ff = (p[k] for k in ("d_model", "n_heads", "n_kv_heads", "head_dim", "d_ff"))
    one = lambda: torch.ones(d, dtype=dt, device=device)
    nrm = lambda shape, j: normal(shape, 0.02, stream_id(seed, 20, j), dt, device)
    w = {"ln1": one(), "wqkv": nrm(((H + 2 * Hkv) * hd, d), 0), "wo": nrm((d, H * hd), 1),
         "lnx": one(), "xq": nrm((H * hd, d), 2), "xkv": nrm((2 * Hkv * hd, d), 3),
         "xo": nrm((d, H * hd), 4),
         "ln2": one(), "wgu": nrm((2 * ff, d), 5), "wd": nrm((d, ff), 6)}
    if int(p.get("draft_blocks", 1)) == 3:
        # the paper's three blocks: the tensors above are the initial block's attention and the
        # intermediate (cross-attention) block; these are the initial block's MLP and the final block
        w.update({"i_ln2": one(), "i_wgu": nrm((2 * ff, d), 7), "i_wd": nrm((d, ff), 8),
                  "f_ln1": one(), "f_wqkv": nrm(((H + 2 * Hkv) * hd, d), 9), "f_wo": nrm((d, H * hd), 10),
                  "f_ln2": one(), "f_wgu": nrm((2 * ff, d), 11), "f_wd": nrm((d, ff), 12)})
    return w


def request_inputs(p, seq_seed=0, device="cpu"):
    """Visual embeddings [v, d] ~ N(0,1) and prompt ids [q] for one sequence."""
    dt = torch_dtype(p["dtype"])
    vis = normal((p["n_visual"], p["d_model"]), 1.0, stream_id(1000 + seq_seed, 1), dt, device)
    ids = uniform_ids(p["n_prompt"], p["vocab"], stream_id(1000 + seq_seed, 2), device)
    return vis, ids
