#!/usr/bin/env python
"""Benchmark of the tree-verify step (attention + acceptance + KV compaction).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole hot path over one synthetic input set, made
through the library's one-call form (attention beside acceptance, then
compaction).  The input sets are rotated over enough copies that the bytes each
timed function touches before it returns to a set exceed twice the L2 capacity,
and L2 is flushed between replays, so every step reads its inputs from HBM.
Every quantity is timed as several replays of a CUDA graph holding K calls;
median and minimum are reported.  Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2408_15562_b200 import synth  # noqa: E402

METRIC = "tree_verify_step_latency"
UNIT = "us/step"
L2_BYTES = 126 * 1024 * 1024
REPLAYS = 10                       # timed graph replays per quantity (median and minimum are reported)
SET_MEMORY_CAP = 40e9              # bytes of device memory the rotated input sets may take


def workload_config(w: synth.Workload, n_layers: int, L_mean: float):
    """What both arms print as `config` (the workload, nothing about how it was run)."""
    return {"workload": w.name, "batch": w.batch, "n_nodes": w.n_nodes, "prefix_len_mean": L_mean, "vocab": w.vocab,
            "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads, "layers_compacted": n_layers,
            "temperatures": sorted(set(float(t) for t in w.temperatures))}


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes per launch of `kernel` from the ncu capture recorded under profiles/, or None when there
    is no record or a source file of the kernel has changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "%s_%s.json" % (kernel, workload))
    if not os.path.exists(path):
        return None, "no ncu record for this kernel and workload"
    with open(path) as f:
        rec = json.load(f)
    for rel, digest in rec.get("source_sha256", {}).items():
        src = os.path.join(ROOT, rel)
        if not os.path.exists(src) or hashlib.sha256(open(src, "rb").read()).hexdigest() != digest:
            return None, "kernel source changed since the ncu capture in profiles/%s" % os.path.basename(path)
    return int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"]), "dram__bytes_read+write per launch, profiles/%s" % os.path.basename(path)


def algorithmic_bytes(w: synth.Workload, L_mean: float, n_acc_rows: float):
    """Bytes a verify step must move (inputs read once, outputs written once)."""
    N, d = w.n_nodes, w.head_dim
    attn = 2 * 2 * w.n_kv_heads * d * (L_mean + N) + 2 * 2 * N * w.n_q_heads * d
    sampling = sum(1 for t in w.temperatures if t > 0)
    accept_rows = 4 * N * w.vocab * w.batch                 # every node's logits row
    accept_all = accept_rows + 4 * N * w.vocab * sampling   # + every draft row (the all-rows definition)
    compact = 2 * w.n_layers * 2 * w.n_kv_heads * n_acc_rows * 2 * d
    return {"attention": attn * w.batch, "accept_logits": accept_rows, "accept_all_rows": accept_all,
            "compaction": compact * w.batch}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peak():
    """Dense bf16 TFLOP/s (burst figure: the attention call is timed alone)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    return 1590.0, "fallback"


def attention_report(w, L_mean, attn_us, attn_bytes, hbm_peak):
    """The attention call (range kernel + merge kernel) against both of its roofs: bytes of Q, K, V and
    the output once, and the dense-tile flops 4 * N * Hq * d * (L + N) of the two products."""
    flops = 4.0 * w.n_nodes * w.n_q_heads * w.head_dim * (L_mean + w.n_nodes) * w.batch
    tpeak, tkind = tensor_peak()
    gbs, tfl = attn_bytes / (attn_us * 1e-6) / 1e9, flops / (attn_us * 1e-6) / 1e12
    g = w.n_q_heads // w.n_kv_heads
    return {"us": attn_us, "algorithmic_bytes": attn_bytes, "gbs": gbs, "frac_of_hbm_peak": gbs / hbm_peak,
            "dense_tile_flops": flops, "tflops": tfl, "frac_of_bf16_peak": tfl / tpeak, "bf16_peak_tflops": tpeak,
            "bf16_peak_kind": tkind, "flop_per_byte": w.n_nodes * g,
            "bound": "hbm" if w.n_nodes * g < 200 else ("tensor" if w.n_nodes * g > 300 else "ridge")}


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) > 2 + i and r[2 + i].startswith("Active") for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def time_oracle(inp: synth.VerifyInputs, steps: int, threads=None):
    """The CPU oracle as it stands, timed on whole verify steps of this workload, on `threads`
    OpenMP threads (default: every host core)."""
    import oracle
    oracle.build()
    cache = synth.make_cache(inp, 1)
    threads = threads or (os.cpu_count() or 1)
    oracle.set_threads(threads)
    times = []
    for _ in range(steps):
        c = cache.copy()
        t0 = time.perf_counter()
        oracle.tree_attn(inp.q, inp.k_cache, inp.v_cache, inp.tree_k, inp.tree_v, inp.parent, inp.prefix_len)
        r = oracle.tree_accept(inp.target_logits, inp.draft_probs, inp.draft_tokens, inp.parent,
                               inp.temperature, inp.uniforms if inp.draft_probs is not None else None)
        oracle.kv_compact(c, r["accepted_path"], r["n_accepted"], inp.prefix_len)
        times.append(time.perf_counter() - t0)
    return statistics.median(times) * 1e6, threads


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = synth.generate(w, 0)
    steps = max(1, min(args.steps, 5))
    for _ in range(min(args.warmup, 1)):
        time_oracle(inp, 1)
    us, threads = time_oracle(inp, steps)
    us1, _ = time_oracle(inp, 1, threads=1)
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": us / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, w.n_layers, float(inp.prefix_len.mean())),
            "cpu_baseline": {"value": us, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "value_one_thread": us1,
                             "sample": "%d whole verify steps of %s (layer-0 cache only; a bounded sample: the oracle is capped "
                                       "at 5 steps whatever --steps says)" % (steps, w.name)},
            "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="llama3_8b_2k", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-verify", action="store_true", help="skip the oracle check of the timed step")
    ap.add_argument("--no-lm-head", action="store_true", help="skip the LM-head leg (a vocabulary matrix of 2*H*V bytes)")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        return run_reference(args, w)
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import torch.distributed as dist
    from paper_2408_15562_b200 import binding

    from paper_2408_15562_b200 import dist_util
    rank, world, local = dist_util.rank_info()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # ---- inputs: R rotated sets, each a full verify step (replicas: every rank its own copy) ----
    inp = synth.generate(w, 0)
    B, N = inp.parent.shape
    L_mean = float(inp.prefix_len.mean())
    n_layers = w.n_layers
    step_bytes = algorithmic_bytes(w, L_mean, 0)
    # Bytes each timed function is sure to read per call (the walk reads only the draft rows of the realised
    # path, so draft rows are not counted): the rotation is sized for the function that touches the least.
    touched = {"step": step_bytes["attention"] + step_bytes["accept_logits"], "tree_attn": step_bytes["attention"],
               "tree_accept": step_bytes["accept_logits"], "accept_stats_kernel": step_bytes["accept_logits"]}
    cache_host = synth.make_cache(inp, n_layers)
    set_bytes = cache_host.nbytes + 2 * inp.q.nbytes + 2 * inp.tree_k.nbytes + inp.target_logits.nbytes * \
        (2 if inp.draft_probs is not None else 1)
    R = max(2, int(np.ceil(2 * L2_BYTES / min(touched.values()))))
    R = max(2, min(R, int(SET_MEMORY_CAP // set_bytes)))
    bf = binding.bf16_tensor
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()  # noqa: E731
    sets = []
    cache0 = bf(cache_host)                            # [layers][2][B][Hkv][max_len][d]
    for r in range(R):
        s = {"cache": cache0.clone(), "q": bf(inp.q).clone(), "tree_k": bf(inp.tree_k), "tree_v": bf(inp.tree_v),
             "logits": dev(inp.target_logits), "draft": dev(inp.draft_probs) if inp.draft_probs is not None else None}
        sets.append(s)
    parent, prefix = dev(inp.parent), dev(inp.prefix_len)
    tokens, temp = dev(inp.draft_tokens), dev(inp.temperature)
    unif = dev(inp.uniforms) if inp.draft_probs is not None else None
    ctx = binding.Context(w.n_q_heads, w.n_kv_heads, w.vocab, inp.max_len, max_nodes=N, n_layers=n_layers,
                          max_batch=B)
    out = torch.empty_like(sets[0]["q"])
    path = torch.empty((B, N), dtype=torch.int32, device="cuda")
    n_acc = torch.empty((B,), dtype=torch.int32, device="cuda")
    bonus = torch.empty((B,), dtype=torch.int32, device="cuda")
    new_len = torch.empty((B,), dtype=torch.int32, device="cuda")
    flush_buf = torch.empty(3 * L2_BYTES, dtype=torch.uint8, device="cuda")

    def attn(s):
        ctx.tree_attn(s["q"], s["cache"][0, 0], s["cache"][0, 1], s["tree_k"], s["tree_v"], parent, prefix, out=out)

    def accept(s):
        ctx.tree_accept(s["logits"], s["draft"], tokens, parent, temp, unif, path, n_acc, bonus)

    def compact(s):
        ctx.kv_compact(s["cache"], path, n_acc, prefix, new_len)

    def step(i):
        """The verify step as a user makes it: one call of the library."""
        s = sets[i % R]
        ctx.verify_step(s["cache"], s["q"], s["tree_k"], s["tree_v"], parent, prefix, s["logits"], s["draft"], tokens,
                        temp, unif, out, path, n_acc, bonus, new_len)

    def step_three_calls(i):
        s = sets[i % R]
        attn(s)
        accept(s)
        compact(s)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # compaction is in place: it is idempotent on the same path only after the first call, so the
    # tree rows of every set are restored (untimed) before each timed pass
    tree_rows = [torch.stack([s["cache"][:, :, b, :, int(inp.prefix_len[b]):int(inp.prefix_len[b]) + N].clone()
                              for b in range(B)]) for s in sets]

    def restore():
        for s, t in zip(sets, tree_rows):
            for b in range(B):
                Lb = int(inp.prefix_len[b])
                s["cache"][:, :, b, :, Lb:Lb + N] = t[b]
        flush_buf.fill_(1)                               # nothing of the inputs is left in L2
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    ctx.check()

    def timed(fn, steps, graph=True, replays=REPLAYS):
        """(median, minimum) us per call of fn.  `steps` calls are captured once into a CUDA graph (the
        library only enqueues kernels and events on the given stream), replayed once untimed, and then
        timed `replays` times: each timed region is exactly one replay = `steps` calls, bracketed by
        events on that stream, after the tree rows were restored and L2 was flushed."""
        restore()
        g = None
        if graph:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(steps):
                    fn(i)
            g.replay()
        samples = []
        for _ in range(replays):
            restore()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            if g is not None:
                g.replay()
            else:
                for i in range(steps):
                    fn(i)
            e1.record()
            barrier()
            samples.append(e0.elapsed_time(e1) * 1e3 / steps)          # us per call
        return statistics.median(samples), min(samples)

    sampler = ClockSampler(local)
    sampler.start()
    launches0 = ctx.launch_count()
    step_us, step_min = timed(step, args.steps)
    launches = (ctx.launch_count() - launches0)          # kernels enqueued into the graph = kernels per replay
    # per-call breakdown and the dominant kernel alone (same rotated inputs, same stream)
    three_us, three_min = timed(step_three_calls, args.steps)
    attn_us, attn_min = timed(lambda i: attn(sets[i % R]), args.steps)
    accept_us, accept_min = timed(lambda i: accept(sets[i % R]), args.steps)
    compact_us, _ = timed(lambda i: compact(sets[i % R]), args.steps)
    # the same rows written from a tree K/V array held outside the cache (fspad_kv_append)
    gen = torch.Generator(device="cuda").manual_seed(24081556200)
    tree_kv = torch.randn((n_layers, 2, B, w.n_kv_heads, N, 128), dtype=torch.float32, device="cuda", generator=gen).to(torch.bfloat16)
    append_us, _ = timed(lambda i: ctx.kv_append(sets[i % R]["cache"], tree_kv, path, n_acc, prefix, new_len), args.steps)
    del tree_kv
    lg2d = [s["logits"].view(B * N, w.vocab) for s in sets]
    st_out = (torch.empty(B * N, dtype=torch.float32, device="cuda"), torch.empty(B * N, dtype=torch.float64, device="cuda"),
              torch.empty(B * N, dtype=torch.int32, device="cuda"))
    stats_us, stats_min = timed(lambda i: ctx.accept_stats(lg2d[i % R], temp, N, out="scan_only"), args.steps)
    stats_merge_us, _ = timed(lambda i: ctx.accept_stats(lg2d[i % R], temp, N, out=st_out), args.steps)
    eager_us, _ = timed(step, args.steps, graph=False, replays=3)
    # the step before the verify step (not part of `value`): candidates of a top-10, five-level draft
    # phase -> the flattened tree of N nodes; verified against the oracle, oracle timed beside it
    cpa, cta, lpa, rta = synth.tree_candidates(w.cfg, B)
    dcand = [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in (cpa, cta, lpa, rta)]
    tb_out = tuple(torch.empty((B, N), dtype=torch.int32, device="cuda") for _ in range(3)) + \
        (torch.empty((B,), dtype=torch.int32, device="cuda"),)
    tree_build_us, _ = timed(lambda i: ctx.tree_build(*dcand, N, out=tb_out), args.steps, replays=3)
    # one draft step of that phase: ten frontier rows of log-probabilities -> top-10 each, joint values, next frontier
    DF, DK = 10, 10
    dlp_host = synth.draft_logprob_rows(w.cfg, B, DF, w.vocab)
    dlp = [torch.from_numpy(dlp_host).cuda() for _ in range(max(2, min(R, 1 + int(3e8 // dlp_host.nbytes))))]
    dfl = torch.zeros((B, DF), dtype=torch.float32, device="cuda")
    dfc = torch.full((B, DF), -1, dtype=torch.int32, device="cuda")
    dx_arr = (torch.zeros((B, DF * DK), dtype=torch.int32, device="cuda"), torch.zeros((B, DF * DK), dtype=torch.int32, device="cuda"),
              torch.zeros((B, DF * DK), dtype=torch.float32, device="cuda"))
    dx_next = (torch.empty((B, DK), dtype=torch.int32, device="cuda"), torch.empty((B, DK), dtype=torch.float32, device="cuda"))
    draft_expand_us, _ = timed(lambda i: ctx.draft_expand(dlp[i % len(dlp)], dfl, dfc, DK, DK, 0, *dx_arr, next_cand=dx_next[0],
                                                          next_logp=dx_next[1]), args.steps, replays=3)
    # the step in front of the acceptance (not part of `value`): the LM-head product with the scan as its
    # epilogue, alone and with the acceptance walk behind it; the vocabulary matrix is far larger than L2
    lm_H = w.n_q_heads * w.head_dim
    lm = None
    if not args.no_lm_head:
        hid_host, wgt_host = synth.lm_head_inputs(w.cfg, B * N, lm_H, w.vocab)
        d_hid, d_wgt = bf(hid_host).view(B, N, lm_H), bf(wgt_host)
        lm_logits = torch.empty((B, N, w.vocab), dtype=torch.float32, device="cuda") if inp.draft_probs is not None else None
        lm_out = (torch.empty(B * N, dtype=torch.float32, device="cuda"), torch.empty(B * N, dtype=torch.float64, device="cuda"),
                  torch.empty(B * N, dtype=torch.int32, device="cuda"))
        lm_path, lm_nacc, lm_bonus = torch.empty_like(path), torch.empty_like(n_acc), torch.empty_like(bonus)
        lm_steps = max(2, min(args.steps, 10))
        lm_stats_us, lm_stats_min = timed(lambda i: ctx.lm_head_stats(d_hid.view(B * N, lm_H), d_wgt, temp, N, out=lm_out),
                                          lm_steps, replays=5)
        lm_accept_us, lm_accept_min = timed(
            lambda i: ctx.lm_head_accept(d_hid, d_wgt, sets[i % R]["draft"], tokens, parent, temp, unif, logits=lm_logits,
                                         accepted_path=lm_path, n_accepted=lm_nacc, bonus_token=lm_bonus), lm_steps, replays=5)
        lm = {"stats_us": lm_stats_us, "stats_us_min": lm_stats_min, "accept_us": lm_accept_us, "accept_us_min": lm_accept_min}
    # the draft side's Feature Sampler on a frontier of ten rows (intermediate size 3.5 x hidden, as in the
    # LLaMA-3 family); not part of `value`
    fs = None
    if not args.no_lm_head:
        fs_rows, fs_I = 10, int(3.5 * lm_H)
        fs_host = synth.feature_sampler_inputs(w.cfg, fs_rows, lm_H, fs_I)
        fs_dev = [bf(x) for x in fs_host]
        fs_inter = torch.empty((fs_rows, fs_I), dtype=torch.bfloat16, device="cuda")
        fs_eta = torch.empty((fs_rows, lm_H), dtype=torch.bfloat16, device="cuda")
        fs_ws = torch.empty((binding.load().fspad_feature_sampler_workspace_bytes(fs_rows, lm_H, fs_I),), dtype=torch.uint8,
                            device="cuda")
        fs_us, fs_min = timed(lambda i: ctx.feature_sampler(*fs_dev, inter=fs_inter, eta=fs_eta, workspace=fs_ws),
                              max(2, min(args.steps, 10)), replays=5)
        fs = {"us": fs_us, "us_min": fs_min, "rows": fs_rows, "hidden": lm_H, "intermediate": fs_I,
              "weight_bytes": 6.0 * lm_H * fs_I, "gbs": 6.0 * lm_H * fs_I / (fs_us * 1e-6) / 1e9}
    clocks = sampler.stop()
    ctx.check()

    # ---- correctness of what was timed: compare the last step with the oracle on rank 0 ----
    n_acc_host = n_acc.cpu().numpy()
    verified = None
    tree_build_ok, tree_build_cpu_us = None, None
    draft_expand_ok, draft_expand_cpu_us = None, None
    if rank == 0 and not args.no_verify:
        import oracle
        restore()
        step(0)
        torch.cuda.synchronize()
        ref = oracle.tree_accept(inp.target_logits, inp.draft_probs, inp.draft_tokens, inp.parent, inp.temperature,
                                 inp.uniforms if inp.draft_probs is not None else None)
        k = ref["n_accepted"]
        ok_acc = (np.array_equal(n_acc.cpu().numpy(), k) and np.array_equal(bonus.cpu().numpy(), ref["bonus_token"])
                  and all(np.array_equal(path[b_, :k[b_]].cpu().numpy(), ref["accepted_path"][b_, :k[b_]]) for b_ in range(B)))
        ref_o = oracle.tree_attn(inp.q, inp.k_cache, inp.v_cache, inp.tree_k, inp.tree_v, inp.parent, inp.prefix_len)
        err = np.abs(out.float().cpu().numpy() - ref_o)
        t0 = time.perf_counter()
        tb_ref = oracle.tree_build(cpa, cta, lpa, rta, N)
        tree_build_cpu_us = (time.perf_counter() - t0) * 1e6
        tree_build_ok = all(np.array_equal(tb_out[j].cpu().numpy(), tb_ref[k_])
                            for j, k_ in enumerate(("parent", "token", "cand", "n_out")))
        dx_ref = [np.zeros((B, DF * DK), np.int32), np.zeros((B, DF * DK), np.int32), np.zeros((B, DF * DK), np.float32)]
        t0 = time.perf_counter()
        nc_ref, nl_ref = oracle.draft_expand(dlp_host, np.zeros((B, DF), np.float32), np.full((B, DF), -1, np.int32), DK, DK, 0,
                                             *dx_ref)
        draft_expand_cpu_us = (time.perf_counter() - t0) * 1e6
        draft_expand_ok = (all(np.array_equal(dx_arr[j].cpu().numpy(), dx_ref[j]) for j in range(3))
                           and np.array_equal(dx_next[0].cpu().numpy(), nc_ref) and np.array_equal(dx_next[1].cpu().numpy(), nl_ref))
        if lm is not None:
            # two rows of the LM-head statistics against the fp64 product over the whole vocabulary
            pick = sorted({0, B * N - 1})
            ctx.lm_head_stats(d_hid.view(B * N, lm_H), d_wgt, temp, N, out=lm_out)
            torch.cuda.synchronize()
            lm_ok = True
            for i_ in pick:
                T_ = float(inp.temperature[i_ // N]) or 1.0
                r_ = oracle.lm_head_stats(np.ascontiguousarray(hid_host[i_:i_ + 1]), wgt_host, T_)
                lm_ok &= abs(float(lm_out[0][i_]) - r_["max"][0]) <= 1e-3 and abs(float(lm_out[1][i_]) / r_["sum"][0] - 1) <= 3e-3 \
                    and (r_["gap"][0] <= 2e-3 or int(lm_out[2][i_]) == int(r_["arg"][0]))
            lm["rows_checked_against_oracle"] = pick
            lm["ok"] = bool(lm_ok)
        if fs is not None:
            ctx.feature_sampler(*fs_dev, inter=fs_inter, eta=fs_eta, workspace=fs_ws)
            torch.cuda.synchronize()
            fs_err = np.abs(fs_eta.float().cpu().numpy() - oracle.feature_sampler(*fs_host))
            fs["max_abs_err_vs_oracle"], fs["mean_abs_err_vs_oracle"] = float(fs_err.max()), float(fs_err.mean())
            fs["ok"] = bool(fs_err.max() <= 2.5e-2 and fs_err.mean() <= 3e-3)
        verified = {"accept_bit_exact": bool(ok_acc), "attn_max_abs_err": float(err.max()),
                    "attn_mean_abs_err": float(err.mean()),
                    "ok": bool(ok_acc and err.max() <= 1e-2 and err.mean() <= 1e-3)}

    # ---- end to end through the host entry point (pinned host buffers, copies inside the timed region) ----
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()  # noqa: E731
    hq = binding.bf16_tensor(inp.q, "cpu").pin_memory()
    htk = binding.bf16_tensor(inp.tree_k, "cpu").pin_memory()
    htv = binding.bf16_tensor(inp.tree_v, "cpu").pin_memory()
    hpar, hpre, htok, htemp = pin(inp.parent), pin(inp.prefix_len), pin(inp.draft_tokens), pin(inp.temperature)
    hlg = pin(inp.target_logits)
    hdp = pin(inp.draft_probs) if inp.draft_probs is not None else None
    hun = pin(inp.uniforms) if inp.draft_probs is not None else None
    hout = torch.empty_like(hq).pin_memory()
    hpath = torch.empty((B, N), dtype=torch.int32).pin_memory()
    hn, hb, hl = (torch.empty((B,), dtype=torch.int32).pin_memory() for _ in range(3))

    def e2e_step(i):
        ctx.verify_step_host(sets[i % R]["cache"], hq, htk, htv, hpar, hpre, hlg, hdp, htok, htemp, hun, hout,
                             hpath, hn, hb, hl)

    e2e_steps = max(3, min(args.steps, 20))
    for i in range(3):
        e2e_step(i)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        e2e_step(i)
    barrier()
    e2e_us = (time.perf_counter() - t0) * 1e6 / e2e_steps
    h2d = sum(t.numel() * t.element_size() for t in (hq, htk, htv, hpar, hpre, htok, htemp, hlg) if t is not None)
    h2d += sum(t.numel() * t.element_size() for t in (hdp, hun) if t is not None)
    d2h = sum(t.numel() * t.element_size() for t in (hout, hpath, hn, hb, hl))

    # max over ranks
    (step_us, step_min, three_us, three_min, attn_us, attn_min, accept_us, accept_min, compact_us, stats_us, stats_min, e2e_us,
     eager_us, stats_merge_us) = dist_util.max_over_ranks(
        [step_us, step_min, three_us, three_min, attn_us, attn_min, accept_us, accept_min, compact_us, stats_us, stats_min,
         e2e_us, eager_us, stats_merge_us], device="cuda")

    if rank == 0:
        peak, peak_kind = peaks()
        bytes_real = algorithmic_bytes(w, L_mean, float(n_acc_host.mean()))
        stats_bytes = bytes_real["accept_logits"]
        step_all = bytes_real["attention"] + bytes_real["accept_all_rows"] + bytes_real["compaction"]
        achieved = stats_bytes / (stats_us * 1e-6) / 1e9
        traffic, traffic_note = recorded_traffic("accept_stats_kernel", w.name)
        cfg = workload_config(w, n_layers, L_mean)
        cfg.update({"launch": "K calls of fspad_verify_step captured in one CUDA graph; %d replays timed one by one, "
                              "value = median" % REPLAYS,
                    "l2": "inputs rotated over %d sets; bytes touched before a set is reused: step %.0f MB, tree_attn %.0f MB, "
                          "tree_accept and the scan kernel alone %.0f MB (L2: %.0f MB); L2 flushed between replays"
                          % (R, R * touched["step"] / 1e6, R * touched["tree_attn"] / 1e6,
                             R * touched["tree_accept"] / 1e6, L2_BYTES / 1e6),
                    "multi_gpu": "independent replicas, no collective"})
        line = {
            "metric": METRIC, "value": step_us, "value_median": step_us, "value_min": step_min, "replays": REPLAYS,
            "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_us / 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": cfg,
            "steps_per_s_all_gpus": dist_util.aggregate_replicas(step_us, world),
            "step_hbm_gbs_all_rows_definition": step_all / (step_us * 1e-6) / 1e9,
            "step_frac_of_hbm_peak": step_all / (step_us * 1e-6) / 1e9 / peak,
            "step_algorithmic_bytes": step_all,
            "breakdown_us": {"three_calls_on_one_stream": three_us, "three_calls_on_one_stream_min": three_min,
                             "tree_attn": attn_us, "tree_attn_min": attn_min, "tree_accept": accept_us,
                             "tree_accept_min": accept_min, "kv_compact_warm_l2": compact_us, "kv_append_warm_l2": append_us,
                             "accept_stats_kernel_alone": stats_us, "accept_stats_kernel_alone_min": stats_min,
                             "accept_stats_with_merge": stats_merge_us,
                             "whole_step_eager_python_launches": eager_us},
            "verified_against_oracle": verified,
            "mean_accepted_len": float(n_acc_host.mean()),
            "roofline": {"kernel": "accept_stats_kernel", "bound": "hbm", "achieved": achieved, "peak": peak,
                         "peak_kind": "%s copy bandwidth (burst, kernel timed alone)" % peak_kind, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": traffic, "traffic_note": traffic_note,
                         "algorithmic_bytes_per_launch": stats_bytes, "launch_us_median": stats_us, "launch_us_min": stats_min},
            "tree_attn_call": attention_report(w, L_mean, attn_us, bytes_real["attention"], peak),
            "tree_build_call": {"us": tree_build_us, "candidates_per_sequence": int(cpa.shape[1]), "n_nodes": N,
                                "batch": B, "bit_exact_vs_oracle": tree_build_ok,
                                "oracle_us_one_thread": tree_build_cpu_us,
                                "note": "step before the verify step; not part of value"},
            "draft_expand_call": {"us": draft_expand_us, "rows": B * DF, "top_k": DK, "width": DK,
                                  "algorithmic_bytes": int(dlp_host.nbytes),
                                  "gbs": dlp_host.nbytes / (draft_expand_us * 1e-6) / 1e9,
                                  "frac_of_hbm_peak": dlp_host.nbytes / (draft_expand_us * 1e-6) / 1e9 / peak,
                                  "bit_exact_vs_oracle": draft_expand_ok, "oracle_us_one_thread": draft_expand_cpu_us,
                                  "note": "one level of the draft phase (three kernels); not part of value"},
            "lm_head_call": None if lm is None else dict(lm, **{
                "rows": B * N, "hidden": lm_H, "vocab": w.vocab, "weight_bytes": 2.0 * lm_H * w.vocab,
                "slabs_of_128_rows": (B * N + 127) // 128,
                "stats_gbs": 2.0 * lm_H * w.vocab * ((B * N + 127) // 128) / (lm["stats_us"] * 1e-6) / 1e9,
                "stats_frac_of_hbm_peak": 2.0 * lm_H * w.vocab * ((B * N + 127) // 128) / (lm["stats_us"] * 1e-6) / 1e9 / peak,
                "note": "LM head with the scan as its epilogue (stats) and with the walk behind it (accept); weights are "
                        "streamed once per slab; not part of value"}),
            "feature_sampler_call": None if fs is None else dict(fs, **{
                "frac_of_hbm_peak": fs["gbs"] / peak,
                "note": "draft side: eta = Wdown(silu(Wgate e) * Wup f) + f on the frontier rows; three matrices streamed once; "
                        "not part of value"}),
            "e2e": {"value": e2e_us, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "note": "fspad_verify_step_host: pinned host inputs, device-resident KV cache"},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            us, threads = time_oracle(inp, 3)
            us1, _ = time_oracle(inp, 1, threads=1)
            line["cpu_baseline"] = {"value": us, "unit": UNIT, "cores": threads, "kind": "oracle",
                                    "value_one_thread": us1,
                                    "sample": "3 whole verify steps of %s (layer-0 cache only) on all cores, median; "
                                              "one step on one thread" % w.name}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
