"""dream_topk_lse_static: the entry point for callers that may not allocate device memory.

Some users of this library cannot call cudaMalloc at the point where they need a top-k: a server
that froze its memory pool after start-up, a plug-in that only receives buffers from its host, or
latency-critical code that must avoid the device-wide synchronisation cudaMalloc implies.  For
them the library carries the kernel's scratch inside its own image.  This test drives that entry
point through the C ABI and checks it against what dream_verify_tree (the existing path through
the same kernel, with arena scratch) reports for the same logits: the argmax of every tree node
and its top-1 minus top-2 margin.  It calls twice in a row, because the built-in scratch keeps the
first call's leftovers and the second call must not be disturbed by them.  The file name sorts
last so that a run stopping at the first failure has already run every other test.
"""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _verify_outputs():
    """One small bf16 model: prefill, compress, draft, verify with a logits dump."""
    from paper_2505_19201_b200 import api, configs, synth
    p = configs.scaled("smolvlm2b", n_layers=2, n_visual=96, k_visual=24, n_prompt=40, decode_steps=2)
    dev = "cuda:0"
    tw, dw = synth.target_weights(p, 0, dev), synth.draft_weights(p, 0, dev)
    ctx = api.Context(api.make_config(p), tw, dw, dev)
    try:
        vis, ids = synth.request_inputs(p, 0, dev)
        ctx.dream_prefill(0, vis, 0, ids)
        ctx.dream_compress_visual(0, p["k_visual"])
        tree = ctx.new_tree()
        ctx.dream_draft_tree([0], [tree])
        T, V = ctx.T, p["vocab"]
        am = torch.zeros(T, dtype=torch.int32, device=dev)
        mg = torch.zeros(T, dtype=torch.float32, device=dev)
        lg = torch.zeros(T, V, dtype=torch.float32, device=dev)
        ctx.dream_verify_tree([0], [tree], am, mg, lg)
        ctx.dream_poll()
        return lg.clone(), am.clone(), mg.clone()
    finally:
        ctx.close()


def _call(logits, ktop):
    from paper_2505_19201_b200 import api
    rows = logits.shape[0]
    tv = torch.full((rows, ktop), float("nan"), dtype=torch.float32, device=logits.device)
    ti = torch.full((rows, ktop), -7, dtype=torch.int32, device=logits.device)
    ls = torch.full((rows,), float("nan"), dtype=torch.float32, device=logits.device)
    api.dream_topk_lse_static(logits, ktop, tv, ti, ls)
    torch.cuda.synchronize()
    return tv.cpu(), ti.cpu(), ls.cpu()


def test_static_scratch_topk_matches_verify_twice_in_a_row():
    logits, argmax, margin = _verify_outputs()
    argmax, margin = argmax.cpu(), margin.cpu()
    # first call: all tree nodes; second call: other sizes (fewer rows, larger k) on the same scratch
    tv1, ti1, ls1 = _call(logits, 2)
    sub = logits[3:40].contiguous()
    tv2, ti2, ls2 = _call(sub, 5)
    tv3, ti3, ls3 = _call(logits, 2)
    for tv, ti, ls, am, mg, lgt in ((tv1, ti1, ls1, argmax, margin, logits), (tv3, ti3, ls3, argmax, margin, logits)):
        assert torch.equal(ti[:, 0], am), "argmax differs from dream_verify_tree's"
        assert torch.equal(tv[:, 0] - tv[:, 1], mg), "top-1 minus top-2 differs from dream_verify_tree's margin"
        ref = torch.logsumexp(lgt.double().cpu(), dim=1)
        assert float((ls.double() - ref).abs().max()) <= 1e-4
    # the middle call: ids and values against a stable sort (ties -> lower id), margins against verify
    v_sorted, i_sorted = torch.sort(sub.cpu(), dim=1, descending=True, stable=True)
    assert torch.equal(ti2, i_sorted[:, :5].to(torch.int32))
    assert torch.equal(tv2, v_sorted[:, :5])
    assert torch.equal(ti2[:, 0], argmax[3:40])
    assert torch.equal(tv2[:, 0] - tv2[:, 1], margin[3:40])


def test_static_scratch_topk_rejects_sizes_beyond_its_scratch():
    from paper_2505_19201_b200 import api
    dev = "cuda:0"
    big = torch.zeros(129, 64, dtype=torch.float32, device=dev)
    out = (torch.zeros(129, 2, device=dev), torch.zeros(129, 2, dtype=torch.int32, device=dev), torch.zeros(129, device=dev))
    with pytest.raises(api.DreamError) as e:
        api.dream_topk_lse_static(big, 2, *out)
    assert e.value.code == -4 and "rows" in str(e.value)
    small = torch.zeros(4, 64, dtype=torch.float32, device=dev)
    out = (torch.zeros(4, 17, device=dev), torch.zeros(4, 17, dtype=torch.int32, device=dev), torch.zeros(4, device=dev))
    with pytest.raises(api.DreamError) as e:
        api.dream_topk_lse_static(small, 17, *out)
    assert e.value.code == -1
