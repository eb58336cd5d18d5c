#!/usr/bin/env python
"""Benchmark of the DREAM draft+verify(+accept) step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one whole round of the hot path (draft tree, tree-masked verification, greedy
acceptance with KV compaction) for one batch of sequences on seeded synthetic inputs and
random-init weights.  The metric is verified tree-tokens per second: B*T tree tokens pass
the target per step.  With N > 1 every rank runs an independent replica (the path has no
exchange step); the timed region is bracketed by a barrier and the slowest rank counts.

One JSON line is printed by rank 0.  `--impl reference` times the CPU oracle instead.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_19201_b200 import configs, synth  # noqa: E402

# DRAM traffic of the dominant kernel from an ncu capture of the current k_gemm_tc
# (profiles/k_gemm_tc_llava7b_4layers_ncu_full.md): dram__bytes_read.sum + dram__bytes_write.sum
# over the four projections of one verify layer (wqkv, wo, wgu, wd), and their weight bytes.  The
# capture ran on the 4-layer cut of the workload (same layer shapes); traffic grows in proportion
# to the weight bytes, so a step's mean launch is scaled by this ratio.  None for workloads without
# a capture, and to be reset to None whenever the kernel changes.
TRAFFIC_RATIO = {"llava7b": (105.94 + 34.63 + 187.11 + 96.19) / (100.66 + 33.55 + 180.36 + 90.18)}

METRIC = "verified_tree_tokens_per_s"
UNIT = "tokens/s"


def step_bytes(p, T, P0):
    """Algorithmic bytes of one step (weights + KV read), bf16 storage; the draft is one layer, or
    with draft_blocks = 3 two decoder blocks around the cross-attention block (three caches)."""
    e = 2 if p["dtype"] == "bf16" else 4
    d, H, Hkv, hd, ff, V, L = (p[k] for k in ("d_model", "n_heads", "n_kv_heads", "head_dim", "d_ff", "vocab", "n_layers"))
    Hhd, kvw = H * hd, 2 * Hkv * hd
    layer = (Hhd + kvw) * d + d * Hhd + 3 * d * ff
    head = V * d
    three = int(p.get("draft_blocks", 1)) == 3
    draft_layer = layer + Hhd * d + kvw * d + d * Hhd      # + cross-attention q, kv, o
    if three:
        draft_layer += 3 * d * ff + layer                   # the initial block's MLP, the final block
    kv_tok = L * kvw
    B = p["batch"]
    verify = (L * layer + head) * e + B * P0 * kv_tok * e
    n_ctx = p["n_prompt"] + p["k_visual"]
    draft_pass = (draft_layer + head) * e + B * (3 if three else 2) * n_ctx * kvw * 4   # draft caches are fp32
    draft = p["tree_depth"] * draft_pass - kvw * d * e       # the last pass projects no memory rows (nothing reads them)
    accept = kvw * d * e
    return dict(verify=verify, draft=draft, accept=accept, total=verify + draft + accept,
                gemm_weights=(L * layer + head + p["tree_depth"] * (draft_layer + head)) * e)


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs: one nvidia-smi process
    started ahead of time that prints a line every 50 ms; mark() notes how far its output has got."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        import tempfile
        self.out = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(index), "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        self.marks = []

    def ready(self, timeout=5.0):
        """Waits until the first sample has been written."""
        t0 = time.time()
        while self.proc and time.time() - t0 < timeout and os.path.getsize(self.out.name) == 0:
            time.sleep(0.02)

    def mark(self):
        self.marks.append(os.path.getsize(self.out.name))

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        """Samples between the first and the last mark (plus the one in flight at each end)."""
        try:
            with open(self.out.name) as f:
                data = f.read()
            os.unlink(self.out.name)
        except Exception:
            data = ""
        lo = self.marks[0] if self.marks else 0
        hi = self.marks[-1] if len(self.marks) > 1 else len(data)
        lo = data.rfind("\n", 0, max(lo - 1, 0)) + 1            # include the sample before the first mark
        nxt = data.find("\n", hi)
        hi = len(data) if nxt < 0 else nxt + 1                   # and the one after the last
        rows = [[x.strip() for x in ln.split(",")] for ln in data[lo:hi].splitlines()]
        rows = [r for r in rows if len(r) >= 7]
        if not rows:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unsampled"])
        mhz = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].lower().startswith("active") for r in rows)]
        return dict(sm_mhz=statistics.median(mhz) if mhz else None, sm_max_mhz=float(rows[0][1]),
                    samples=len(rows), reasons=reasons)


def peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f), "measured"
    except Exception:
        return dict(hbm_gbs=6650.0, bf16_tflops=1590.0), "fallback"


def oracle_sample(p, twg, dwg, T, budget_s=12.0, max_steps=8):
    """Time one full draft+verify+accept step of the CPU oracle, as it stands, on this
    workload's shapes at the initial prefix length.  The sequence state is filled with
    random values instead of a CPU prefill (timing does not depend on values)."""
    from oracle.dream_oracle import DreamOracle, OracleConfig, SeqState
    dt = torch.float32 if p["dtype"] == "bf16" else torch.float64
    cpu = lambda w: [t.cpu() for t in w] if isinstance(w, list) else w.cpu()
    orc = DreamOracle(OracleConfig.from_preset(p), {k: cpu(v) for k, v in twg.items()},
                      {k: cpu(v) for k, v in dwg.items()}, dt,
                      kv_dtype=torch.bfloat16 if p["dtype"] == "bf16" else None)
    n = p["n_visual"] + p["n_prompt"]
    nc = p["n_prompt"] + p["k_visual"]
    Hkv, hd = p["n_kv_heads"], p["head_dim"]
    g = torch.Generator().manual_seed(0)
    rnd = lambda rows: torch.randn(rows, Hkv, hd, dtype=dt, generator=g)
    st = SeqState(P=n, pending=1, n_prompt_total=n, vis_start=0, n_visual=p["n_visual"], tap=max(1, p["n_layers"] // 2))
    st.K = [rnd(n) for _ in range(p["n_layers"])]
    st.V = [rnd(n) for _ in range(p["n_layers"])]
    st.dK, st.dV, st.mK, st.mV = rnd(nc), rnd(nc), rnd(nc), rnd(nc)
    if int(p.get("draft_blocks", 1)) == 3:
        st.fK, st.fV = rnd(nc), rnd(nc)
        st.dpos, st.mpos = torch.arange(nc), torch.arange(nc)
    t0 = time.perf_counter()
    done = 0
    while done < max_steps and (done == 0 or time.perf_counter() - t0 < budget_s):
        orc.step(st)
        done += 1
    dt_s = (time.perf_counter() - t0) / done
    return dict(value=T / dt_s, unit=UNIT, cores=torch.get_num_threads(), kind="oracle",
                sample=f"{done} full draft+verify+accept step(s) of 1 sequence, {p['name']} shapes, prefix {n} growing, "
                       f"state filled with random values (no CPU prefill); {dt_s:.1f} s per step", seconds=dt_s)


def slowest_rank(times_ms, world, device):
    """Element-wise maximum over the ranks of a list of durations (every rank calls this)."""
    ms = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    return [float(x) for x in ms]


def job_value(world, batch, tree_nodes, ms_per_step):
    """Whole-job throughput: every rank runs an independent replica of the same workload, so the
    job verifies world * batch * tree_nodes tree tokens per step of the slowest rank."""
    return world * batch * tree_nodes / (ms_per_step / 1e3)


def request_seed(seq, rank):
    """Input seed of sequence `seq` on rank `rank`: replicas decode different requests."""
    return seq + 100 * rank


def spawn_ranks(n):
    """`python bench.py --gpus N` without a launcher: start N ranks of this script on this node
    (one per GPU, rendezvous on 127.0.0.1) and pass their output through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def setup_flops(p):
    """Floating-point operations of one request's set-up (prefill): projections and MLP over the n
    prompt rows of every layer, causal attention (QK^T and PV over n (n + 1) / 2 pairs), LM head on one row."""
    d, H, Hkv, hd, ff, V, L = (p[k] for k in ("d_model", "n_heads", "n_kv_heads", "head_dim", "d_ff", "vocab", "n_layers"))
    n = p["n_visual"] + p["n_prompt"]
    layer_params = (H + 2 * Hkv) * hd * d + d * H * hd + 3 * d * ff
    attn = 2 * 2 * H * hd * n * (n + 1) / 2
    return L * (2 * layer_params * n + attn) + 2 * V * d


def run_reference(args, p):
    """The reference arm: the CPU oracle on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    twg, dwg = synth.target_weights(p, 0, dev), synth.draft_weights(p, 0, dev)
    from paper_2505_19201_b200 import api
    T = 1 + min(p["tree_max_nodes"], p["tree_topk"] + (p["tree_depth"] - 1) * min(p["tree_beam"], p["tree_topk"]) * p["tree_topk"])
    times = []
    for i in range(args.warmup + args.steps):
        r = oracle_sample(p, twg, dwg, T, budget_s=0.0, max_steps=1)
        if i >= args.warmup:
            times.append(r["seconds"])
        if sum(times) > 150:
            break
    ms = 1e3 * sum(times) / len(times)
    val = T / (ms / 1e3)
    line = dict(metric=METRIC, value=val, unit=UNIT, n_gpus=args.gpus, steps=len(times), warmup=args.warmup,
                ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f32" if p["dtype"] == "bf16" else "f64", data="synthetic", impl="reference",
                config=dict(workload=p["name"], batch=1, tree_nodes=T, note="CPU oracle, one sequence per step"),
                cpu_baseline=dict(value=val, unit=UNIT, cores=torch.get_num_threads(), kind="oracle", sample=r["sample"]),
                e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0,
                    help="timed steps; 0 = the workload's decode length (256 for the LLaVA-7B-shaped one), at most 256")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--workload", default="llava7b")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-gemm", type=int, default=1)
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: cut the target to this many layers (the line's workload name says so)")
    ap.add_argument("--keep", type=float, default=0.0,
                    help="sweep aid: fraction of the visual tokens the compression keeps (the preset's k otherwise)")
    ap.add_argument("--chain", action="store_true",
                    help="sweep aid: a chain-shaped draft (one child per node, depth D) instead of the tree")
    ap.add_argument("--batch", type=int, default=0, help="sweep aid: number of sequences per step")
    ap.add_argument("--track-entropy", action="store_true",
                    help="keep the layer entropies of Eq. 2 up to date while decoding (row entropies out of the "
                         "verify attention, added up by the acceptance)")
    ap.add_argument("--draft-blocks", type=int, default=1, choices=(1, 3),
                    help="3: the draft is an initial decoder block, a cross-attention block and a final decoder "
                         "block; 1: one layer of self-attention, cross-attention and MLP")
    ap.add_argument("--temp", type=float, default=0.0,
                    help="acceptance by the sampling rule at this temperature (greedy otherwise); the verify "
                         "call then also writes the logits")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        return spawn_ranks(args.gpus)
    p = dict(configs.PRESETS[args.workload])
    if args.steps <= 0:
        args.steps = min(256, int(p["decode_steps"]))
    if args.layers:
        p = configs.scaled(args.workload, n_layers=args.layers)
        p["name"] = "%s[n_layers=%d]" % (p["name"], args.layers)
    if args.keep:
        p["k_visual"] = max(1, min(p["n_visual"], int(p["n_visual"] * args.keep + 0.5)))
        p["name"] = "%s[k_visual=%d]" % (p["name"], p["k_visual"])
    if args.chain:
        p.update(tree_topk=1, tree_beam=1, tree_max_nodes=p["tree_depth"])
        p["name"] = "%s[chain]" % p["name"]
    if args.batch:
        p["batch"] = args.batch
        p["name"] = "%s[batch=%d]" % (p["name"], args.batch)
    if args.temp > 0:
        p["name"] = "%s[temp=%g]" % (p["name"], args.temp)
    if args.track_entropy:
        p["track_entropy"] = 1
        p["name"] = "%s[track_entropy]" % p["name"]
    if args.draft_blocks == 3:
        p["draft_blocks"] = 3
        p["name"] = "%s[draft_blocks=3]" % p["name"]
    if args.impl == "reference":
        return run_reference(args, p)

    from paper_2505_19201_b200 import api
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = f"cuda:{local}"
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))
    B = p["batch"]
    p["decode_steps"] = args.steps + args.warmup + 16 + 2 * args.steps   # room for every timed pass (the end-to-end pass and the profiled pass follow)
    twg, dwg = synth.target_weights(p, 0, dev), synth.draft_weights(p, 0, dev)
    cfg = api.make_config(p)
    ctx = api.Context(cfg, twg, dwg, dev)
    T = ctx.T
    seqs = list(range(B))
    setup_ms = []                      # per sequence: prefill (with entropy and tap choice) + compression
    for s in seqs:
        vis, ids = synth.request_inputs(p, request_seed(s, rank), dev)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(torch.cuda.current_stream(dev))
        ctx.dream_prefill(s, vis, 0, ids)
        ctx.dream_compress_visual(s, p["k_visual"])
        s1.record(torch.cuda.current_stream(dev))
        torch.cuda.synchronize(dev)
        setup_ms.append(s0.elapsed_time(s1))
    ctx.dream_poll()
    P0 = p["n_visual"] + p["n_prompt"]

    trees = None                              # the context's own tree buffers
    am = torch.zeros(B * T, dtype=torch.int32, device=dev)
    alen = torch.zeros(B, dtype=torch.int32, device=dev)
    outt = torch.zeros(B * (p["tree_depth"] + 1), dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream(dev)
    if args.temp > 0:
        lg = torch.zeros(B * T, p["vocab"], dtype=torch.float32, device=dev)
        uni = torch.rand(B, p["tree_depth"] + 1, T, dtype=torch.float32, device=dev,
                         generator=torch.Generator(dev).manual_seed(rank))

    def one_step(ev=None):
        if ev:
            ev[0].record(stream)
        ctx.dream_draft_tree(seqs, trees)
        if ev:
            ev[1].record(stream)
        ctx.dream_verify_tree(seqs, trees, am, None, lg if args.temp > 0 else None)
        if ev:
            ev[2].record(stream)
        if args.temp > 0:
            ctx.dream_accept_sample(seqs, trees, lg, args.temp, uni, alen, outt)
        else:
            ctx.dream_accept(seqs, trees, am, alen, outt)
        if ev:
            ev[3].record(stream)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    sampler = ClockSampler(local)
    for _ in range(args.warmup):
        one_step()
    barrier()
    sampler.ready()
    # ---- timed region: device-resident inputs, CUDA events on the launching stream
    sampler.mark()
    l0 = ctx.dream_launch_count()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(args.steps):
        one_step(evs[i])
    t_end.record(stream)
    barrier()
    sampler.mark()
    sampler.stop()
    launches = ctx.dream_launch_count() - l0
    total_ms = t_start.elapsed_time(t_end)
    draft_us = statistics.median(e[0].elapsed_time(e[1]) for e in evs) * 1e3
    verify_us = statistics.median(e[1].elapsed_time(e[2]) for e in evs) * 1e3
    accept_us = statistics.median(e[2].elapsed_time(e[3]) for e in evs) * 1e3
    per_step_ms = [e[0].elapsed_time(e[3]) for e in evs]
    srt = sorted(per_step_ms)
    pct = lambda q: srt[min(len(srt) - 1, int(q * len(srt)))]
    step_ms = dict(median=statistics.median(per_step_ms), p10=pct(0.10), p90=pct(0.90))
    k50 = min(50, len(per_step_ms))
    first_ms, last_ms = statistics.median(per_step_ms[:k50]), statistics.median(per_step_ms[-k50:])
    ctx.dream_poll()
    # ---- end to end: the serving call with host result buffers, synchronising every step
    alen_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    outt_h = torch.zeros(B * (p["tree_depth"] + 1), dtype=torch.int32).pin_memory()
    for _ in range(2):
        ctx.dream_step_host(seqs, alen_h, outt_h)
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        ctx.dream_step_host(seqs, alen_h, outt_h)
    e1.record(stream)
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3)
    # ---- dominant kernel: the weight-streaming GEMM, each launch bracketed by CUDA events on the
    # library's stream, in a pass of its own (the brackets keep its neighbours from overlapping it)
    gemm = None
    if args.profile_gemm:
        ctx.dream_gemm_timing(True)
        nprof = max(1, min(args.steps, 8))
        for _ in range(nprof):
            one_step()
        n_l, g_ms, g_bytes = ctx.dream_gemm_timing(False)
        if n_l and g_ms > 0:
            gemm = dict(kernel="k_gemm_tc", launches=n_l, launches_per_step=n_l / nprof, bytes_per_launch=g_bytes / n_l,
                        us_per_launch=1e3 * g_ms / n_l, gbs=g_bytes / g_ms / 1e6, ms_per_step=g_ms / nprof,
                        bytes_per_step=g_bytes / nprof)
    # ---- the same kernel inside the stream (no event between launches): the library's timeline stamps
    # every kernel when its predecessor has completed; a kernel's time on the critical path is the
    # distance to the next stamp, overlap with its neighbours included
    if gemm:
        n_tr = 4
        ctx.dream_trace(n_tr * (int(launches) // args.steps + 64))
        for _ in range(n_tr):
            one_step()
        tl = ctx.dream_trace(0)
        first = [i for i, (k, _) in enumerate(tl) if k == "k_draft_begin"]
        if len(first) >= 2:
            tl = tl[first[0]:first[-1] + 1]                      # whole steps only
            span = tl[-1][1] - tl[0][1]
            own = [tl[i + 1][1] - tl[i][1] for i in range(len(tl) - 1) if tl[i][0] == "k_gemm_tc"]
            if own and span > 0:
                us = sum(own) / len(own) / 1e3
                gemm["in_stream"] = dict(us_per_launch=us, gbs=gemm["bytes_per_launch"] / us / 1e3,
                                         share_of_step=sum(own) / span, steps=len(first) - 1)
    total_ms, e2e_ms = slowest_rank([total_ms, e2e_ms], world, dev)
    if rank != 0:
        return
    pk, pk_src = peaks()
    sb = step_bytes(p, T, P0)
    ms_step = total_ms / args.steps
    value = job_value(world, B, T, ms_step)
    step_gbs = sb["total"] / (ms_step / 1e3) / 1e9
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16" if p["dtype"] == "bf16" else "f32", data="synthetic",
                config=dict(workload=p["name"], batch=B, tree_nodes=T, prefix=P0, parallelism=f"replicas{world}",
                            l2="step working set (weights, %.1f GB) exceeds the 126 MB L2" % (sb["gemm_weights"] / 1e9)),
                draft_us=draft_us, verify_us=verify_us, accept_us=accept_us,
                step_ms=step_ms, first_steps_ms=first_ms, last_steps_ms=last_ms,
                setup_ms_per_sequence=statistics.median(setup_ms),
                setup_tflops=setup_flops(p) / (statistics.median(setup_ms) / 1e3) / 1e12,
                setup_frac_of_bf16_sustained=(setup_flops(p) / (statistics.median(setup_ms) / 1e3) / 1e12 / pk["bf16_tflops_sustained"]
                                              if pk.get("bf16_tflops_sustained") else None),
                step_bytes=sb["total"], step_gbs=step_gbs,
                step_roofline_frac=step_gbs / pk["hbm_gbs"], step_roofline_frac_nominal_8tbs=step_gbs / 8000.0,
                step_bytes_note="weights of every GEMM of the step + prefix KV of the verify + the draft's two caches (4 B per element)",
                clocks=sampler.summary(), gpu_launches=int(launches),
                e2e=dict(value=job_value(world, B, T, e2e_ms / args.steps), unit=UNIT,
                         h2d_bytes_per_step=4 * B, d2h_bytes_per_step=4 * B * (p["tree_depth"] + 2)))
    if gemm:
        line["roofline"] = dict(bound="hbm", achieved=gemm["gbs"], peak=pk["hbm_gbs"], unit="GB/s",
                                frac=gemm["gbs"] / pk["hbm_gbs"], traffic=(TRAFFIC_RATIO[p["name"]] * gemm["bytes_per_launch"] if p["name"] in TRAFFIC_RATIO else None), peak_source=pk_src,
                                kernel=gemm["kernel"], launches_per_step=gemm["launches_per_step"],
                                bytes_per_launch=gemm["bytes_per_launch"], us_per_launch=gemm["us_per_launch"],
                                bytes_per_step=gemm["bytes_per_step"], ms_per_step=gemm["ms_per_step"],
                                in_stream=(dict(gemm["in_stream"], frac=gemm["in_stream"]["gbs"] / pk["hbm_gbs"],
                                                note="the same launches timed inside the stream by the library's timeline stamps "
                                                     "(dependency resolved to next kernel's dependency resolved); `frac` above is the bracketed, serialised figure")
                                           if "in_stream" in gemm else None),
                                note="algorithmic bytes = weight bytes of each launch; duration = CUDA events around each launch; "
                                     "traffic = ncu DRAM bytes of one layer's four projections on the 4-layer cut, scaled by weight bytes")
    else:
        line["roofline"] = dict(bound="hbm", achieved=step_gbs, peak=pk["hbm_gbs"], unit="GB/s",
                                frac=step_gbs / pk["hbm_gbs"], traffic=None, peak_source=pk_src, kernel="whole step")
    if not args.no_cpu_baseline and world == 1:
        cb = oracle_sample(p, twg, dwg, T)
        cb.pop("seconds")
        line["cpu_baseline"] = cb
    print(json.dumps(line))
    ctx.close()


if __name__ == "__main__":
    main()
