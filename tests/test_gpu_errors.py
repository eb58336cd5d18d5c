"""Error paths of the C ABI on a live context: bad arguments, calls out of order, capacity, and
device-side anomalies that must raise the status word without trapping.  Every failure here is
made on the host (a wrong argument, a malformed tree in an input buffer, a logits row without
mass); none of them faults the GPU."""
import pytest
import torch

pytestmark = pytest.mark.gpu

E_ARG, E_STATE, E_CAPACITY = -1, -2, -4


def _ctx(preset="toy", max_seq=None, **over):
    from paper_2505_19201_b200 import api, configs, synth
    dev = "cuda:0"
    p = configs.scaled(preset, **over)
    tw, dw = synth.target_weights(p, 0, dev), synth.draft_weights(p, 0, dev)
    cfg = api.make_config(p, max_seq=max_seq)
    ctx = api.Context(cfg, tw, dw, dev)
    vis, ids = synth.request_inputs(p, 0, dev)
    return p, ctx, vis, ids


def _code(fn, *a, **k):
    from paper_2505_19201_b200 import api
    try:
        fn(*a, **k)
    except api.DreamError as e:
        return e.code
    return 0


def _bufs(ctx, p, B=1):
    dev, T, D = ctx.device, ctx.T, p["tree_depth"]
    i32 = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
    return i32(B * T), i32(B), i32(B * (D + 1)), i32(B * (D + 1))


def test_calls_out_of_order_and_bad_arguments():
    p, ctx, vis, ids = _ctx(batch=2)
    try:
        am, alen, outt, csrc = _bufs(ctx, p)
        tree = ctx.new_tree()
        assert _code(ctx.dream_draft_tree, [0], [tree]) == E_STATE              # nothing prefilled
        assert _code(ctx.dream_compress_visual, 0, 4) == E_STATE
        assert _code(ctx.dream_prefill, 5, vis, 0, ids) == E_ARG                # sequence id out of range
        assert _code(ctx.dream_prefill, 0, vis, len(ids) + 1, ids) == E_ARG     # vis_start beyond the text
        big = torch.cat([ids, ids, ids, ids])
        assert _code(ctx.dream_prefill, 0, vis, 0, big) == E_CAPACITY           # prompt above max_prompt
        ctx.dream_prefill(0, vis, 0, ids)
        assert _code(ctx.dream_prefill, 0, vis, 0, ids) == E_STATE              # the sequence is live
        assert _code(ctx.dream_draft_tree, [0], [tree]) == E_STATE              # not compressed yet
        assert _code(ctx.dream_compress_visual, 0, p["n_visual"] + 1) == E_ARG  # k > v
        assert _code(ctx.dream_compress_visual, 0, -1) == E_ARG
        ctx.dream_compress_visual(0, p["k_visual"])
        assert _code(ctx.dream_verify_tree, [0], [tree], am) == E_STATE         # no tree drafted
        assert _code(ctx.dream_draft_tree, [0, 0], [tree, tree]) == E_ARG       # a sequence listed twice
        assert _code(ctx.dream_draft_tree, [], []) == E_ARG
        ctx.dream_draft_tree([0], [tree])
        assert _code(ctx.dream_accept, [0], [tree], am, alen, outt, csrc) == E_STATE   # not verified
        assert _code(ctx.dream_verify_tree, [0], [tree], None) == E_ARG         # node_argmax is required
        ctx.dream_verify_tree([0], [tree], am)
        assert _code(ctx.dream_accept_sample, [0], [tree], torch.zeros(ctx.T, p["vocab"], device=ctx.device), 0.0,
                     torch.zeros(p["tree_depth"] + 1, ctx.T, device=ctx.device), alen, outt, csrc) == E_ARG   # temperature 0
        ctx.dream_accept([0], [tree], am, alen, outt, csrc)
        ctx.dream_poll()                                                         # the failed calls left the context usable
        # a second sequence: the acceptance must name the sequences of the last verification, in order
        ctx.dream_prefill(1, vis, 0, ids)
        ctx.dream_compress_visual(1, p["k_visual"])
        t0, t1 = ctx.new_tree(), ctx.new_tree()
        am2, alen2, outt2, csrc2 = _bufs(ctx, p, 2)
        ctx.dream_draft_tree([0, 1], [t0, t1])
        ctx.dream_verify_tree([0, 1], [t0, t1], am2)
        assert _code(ctx.dream_accept, [1, 0], [t1, t0], am2, alen2, outt2, csrc2) == E_STATE
        assert _code(ctx.dream_accept, [0], [t0], am2, alen2, outt2, csrc2) == E_STATE
        ctx.dream_accept([0, 1], [t0, t1], am2, alen2, outt2, csrc2)
        ctx.dream_poll()
    finally:
        ctx.close()


def test_capacity_is_reported_only_when_the_cache_is_full():
    """With a draft that is (almost) never right the prefix grows by one token per round.  The host
    only knows that it grows by at most D + 1, but it learns the real lengths from the copies the
    acceptances leave behind, so a cache with room for `room` more tokens lasts about `room` rounds,
    not room / (D + 1)."""
    from paper_2505_19201_b200 import api
    p, ctx0, vis, ids = _ctx()
    n, D, T = p["n_visual"] + p["n_prompt"], p["tree_depth"], ctx0.T
    ctx0.close()
    room = 40
    p, ctx, vis, ids = _ctx(max_seq=n + T + room)
    try:
        ctx.dream_prefill(0, vis, 0, ids)
        ctx.dream_compress_visual(0, p["k_visual"])
        alen, outt = torch.zeros(1, dtype=torch.int32), torch.zeros(D + 1, dtype=torch.int32)
        rounds, grown = 0, 0
        while True:
            code = _code(ctx.dream_step_host, [0], alen, outt)
            if code:
                assert code == E_CAPACITY
                break
            rounds += 1
            grown += int(alen[0]) + 1
            assert rounds < 10 * room
        P, _, _ = ctx.dream_seq_state(0)
        assert P == n + grown
        assert P + T > n + T + room - (D + 1), f"refused with {n + T + room - P - T} tokens of room left"
        ctx.dream_poll()
        # the same without a host synchronisation in the loop: the bound may lag by the rounds in flight
        ctx.dream_seq_reset(0)
        ctx.dream_prefill(0, vis, 0, ids)
        ctx.dream_compress_visual(0, p["k_visual"])
        am, alen_d, outt_d, csrc = _bufs(ctx, p)
        rounds2 = 0
        while True:
            ctx.dream_draft_tree([0], None)
            code = _code(ctx.dream_verify_tree, [0], None, am)
            if code:
                assert code == E_CAPACITY
                break
            ctx.dream_accept([0], None, am, alen_d, outt_d, csrc)
            rounds2 += 1
            if rounds2 % 3 == 0:
                torch.cuda.synchronize()       # lets the stream drain; no library call reads anything back
            assert rounds2 < 10 * room
        assert rounds2 >= rounds // 2, f"{rounds2} rounds without host read-backs vs {rounds} with"
        ctx.dream_poll()
    finally:
        ctx.close()


def test_malformed_tree_raises_the_status_word_and_spares_the_prefix():
    p, ctx, vis, ids = _ctx()
    try:
        ctx.dream_prefill(0, vis, 0, ids)
        ctx.dream_compress_visual(0, p["k_visual"])
        am, alen, outt, csrc = _bufs(ctx, p)
        tree = ctx.new_tree()
        ctx.dream_draft_tree([0], [tree])
        ctx.dream_poll()
        L = p["n_layers"]
        before = [(ctx.dream_debug_read(0, 0, l, 0), ctx.dream_debug_read(0, 1, l, 0)) for l in range(L)]
        host = tree.to_host()
        T = ctx.T
        parent = list(host["parent"])
        parent[3] = 5                                     # a parent that does not precede its child
        mask = tree.mask.cpu()
        tree.load_raw(host["tokens"], parent, host["depth"], mask)
        ctx.dream_verify_tree([0], [tree], am)            # host-side checks cannot see device buffers
        assert _code(ctx.dream_poll) == E_STATE
        after = [(ctx.dream_debug_read(0, 0, l, 0), ctx.dream_debug_read(0, 1, l, 0)) for l in range(L)]
        for (k0, v0), (k1, v1) in zip(before, after):
            assert torch.equal(k0, k1) and torch.equal(v0, v1), "the verified prefix row at slot 0 changed"
    finally:
        ctx.close()


@pytest.mark.parametrize("case", ["nan_row", "uniform_one"])
def test_sampling_acceptance_is_bounded_on_rows_without_mass(case):
    """A logits row of NaN, or a uniform of 1.0 that refuses the only token with mass, leaves nothing
    to draw from: the kernel must return, emit a defined token and raise the status word."""
    p, ctx, vis, ids = _ctx()
    try:
        dev, T, D, V = ctx.device, ctx.T, p["tree_depth"], p["vocab"]
        ctx.dream_prefill(0, vis, 0, ids)
        ctx.dream_compress_visual(0, p["k_visual"])
        am, alen, outt, csrc = _bufs(ctx, p)
        tree = ctx.new_tree()
        ctx.dream_draft_tree([0], [tree])
        ctx.dream_verify_tree([0], [tree], am)
        host = tree.to_host()
        lg = torch.zeros(T, V, dtype=torch.float32, device=dev)
        uni = torch.full((D + 1, T), 0.5, dtype=torch.float32, device=dev)
        if case == "nan_row":
            lg[0] = float("nan")
        else:
            kid = host["parent"].index(0, 1)              # first child of the root
            lg[0] = -1e30
            lg[0, host["tokens"][kid]] = 0.0              # all the mass on that child's token
            uni[:] = 1.0                                  # ... which a uniform of 1 refuses
        ctx.dream_accept_sample([0], [tree], lg, 1.0, uni, alen, outt, csrc)
        assert _code(ctx.dream_poll) == E_STATE
        assert 0 <= int(alen[0]) <= D and 0 <= int(outt[int(alen[0])]) < V
    finally:
        ctx.close()
