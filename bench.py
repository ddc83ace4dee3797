#!/usr/bin/env python
"""Verify-step benchmark: one step = as_plan + as_verify_attn + as_accept + as_kv_commit over one
synthetic Qwen3-8B-shaped batch (batch 64, lognormal contexts, k ~ U{0..8}, greedy acceptance).

Prints ONE JSON line.  `value` is verified draft tokens per second (sum of k_i over the batch divided
by the step time) with inputs resident in HBM; `e2e` is the same metric with the step's inputs (Q,
new K/V rows, logits, draft tokens) copied from pinned host memory and the results copied back inside
the timed region; `roofline` is the attention kernel's KV-read rate against the measured HBM peak;
`cpu_baseline` is the fp64 oracle on this machine's host cores.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

With N > 1 (under torchrun) every rank runs its own replica of the workload (different seed): the
path has no exchange step, so there is no collective on the data path; timing is the max over ranks.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_24004_b200 import workloads  # noqa: E402

METRIC = "verified draft tokens/s per verify step"
UNIT = "draft tokens/s"
# DRAM bytes moved per algorithmic KV byte by the tensor-core attention kernels, from the ncu captures summarised in
# profiles/ (batch-16 slices): traffic grows in proportion to the KV bytes, so the ratio is scaled to the launch timed here.
#   head_dim 128 (attn_tc_kernel), attn_tc_qwen3_8b_batch16_ncu_full.md: (721.05 MB read + 4.21 MB written) / 719.79 MB
#   head_dim 64 (attn_rows_kernel), attn_rows_gpt_oss_20b_batch16_ncu_full.md: 1.017 for requests of up to 128 query rows;
#     a request with more is walked once per block of rows ((2375.1 + 15.7) / 1185.4 = 2.017 with every request at 136)
ATTN_TC_DRAM_BYTES_PER_KV_BYTE = {128: 1.0076, 64: 1.017}


def extra_walks_share(b, kind):
    """Share of the layer's KV bytes that is read a second (third) time: requests whose query rows exceed what one launch
    item holds are walked once per row block (head_dim 64: blocks of 128 rows; head_dim 128: blocks of at most 96 rows for
    requests above 112 rows)."""
    G = b.num_q_heads // b.num_kv_heads
    rows = G * (b.draft_lens.astype(np.int64) + 1)
    if b.head_dim == 64:
        blocks = -(-rows // 128)
    else:
        blocks = np.where(rows > 112, -(-rows // 96), 1)
    W = b.kinds[kind].window
    vis = np.minimum(b.seq_lens.astype(np.int64) + b.draft_lens + 1, W + b.draft_lens if W > 0 else 1 << 60)
    return float(((blocks - 1) * vis).sum() / max(vis.sum(), 1))


HBM_NOMINAL_GBS = 8000.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# hidden sizes of the models the workloads are shaped after
HIDDEN_DIM = {"qwen3_8b": 4096, "r1_distill_llama_8b": 4096, "gpt_oss_20b": 2880, "gpt_oss_20b_all_k16": 2880, "tiny": 512}


def lm_head_leg(bnd, vs, b, workload, steps):
    """as_accept_lm_head on this batch's rows: seeded hidden states [total_q, H] and weights [V, H] (bf16, logits ~ N(0, 2)),
    CUDA events around the call (memset + projection/argmax kernel + finish + decision), against the measured bf16 GEMM peak
    and, when few rows make the single pass over the weights the bound, against the measured copy bandwidth."""
    H = HIDDEN_DIM.get(workload, 4096) // 64 * 64
    V = b.vocab
    g = torch.Generator(device="cuda").manual_seed(77)
    hidden = torch.randn((b.total_q, H), generator=g, device="cuda").to(torch.bfloat16)
    weight = torch.empty((V, H), dtype=torch.bfloat16, device="cuda")
    for at in range(0, V, 16384):
        weight[at:at + 16384] = (torch.randn((min(16384, V - at), H), generator=g, device="cuda") * (2.0 / H ** 0.5)).to(torch.bfloat16)
    vs.plan_step()
    call = lambda: bnd.as_accept_lm_head(vs.plan, hidden, weight, vs.draft_tokens, vs.accept_len, vs.out_tokens)
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    bnd.as_plan_check(vs.plan)
    tf = 2.0 * b.total_q * H * V / (ms * 1e-3) / 1e12
    tf_padded = 2.0 * (-(-b.total_q // 128) * 128) * H * V / (ms * 1e-3) / 1e12
    peak_tf = 1590.0
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            peak_tf = float(json.load(f)["bf16_tflops"])
    hbm, _ = measured_peaks()
    return ({"rows": b.total_q, "hidden_dim": H, "vocab": V, "ms": ms, "tflops": tf, "tflops_incl_row_padding": tf_padded,
             "peak_tflops": peak_tf, "frac_of_peak": tf / peak_tf, "weight_gbs": V * H * 2 / (ms * 1e-3) / 1e9,
             "weight_frac_of_hbm_peak": V * H * 2 / (ms * 1e-3) / 1e9 / hbm, "logits_bytes_not_materialised": b.total_q * V * 4},
            hidden, weight)


def roofline_of(bnd, b, vs, kind, attn_ms):
    """KV bytes every (request, kv-head) must read once, over the measured duration of the attention launch(es) of layer
    kind `kind` (CUDA events recorded by the library around them), against the measured copy bandwidth."""
    peak, peak_kind = measured_peaks()
    kv_bytes = b.kv_bytes(kind)
    achieved = kv_bytes / (attn_ms * 1e-3) / 1e9
    stats = bnd.as_plan_stats(vs.plan, kind)
    tc_kernel = "attn_tc" if b.head_dim == 128 else "attn_rows"
    roofline = {"bound": "hbm", "kernel": tc_kernel if stats["impl"] == bnd.AS_ATTN_TC else "attn_simt",
                "achieved": achieved, "peak": peak, "peak_source": f"{peak_kind} copy bandwidth", "unit": "GB/s",
                "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / HBM_NOMINAL_GBS, "traffic": None,
                "algorithmic_bytes_per_launch": kv_bytes, "avg_launch_ms": attn_ms,
                "ctas": stats["num_ctas"], "items": stats["num_items"], "merged_pairs": stats["num_merges"]}
    if roofline["kernel"] != "attn_simt":
        roofline["traffic"] = (ATTN_TC_DRAM_BYTES_PER_KV_BYTE[b.head_dim] + extra_walks_share(b, kind)) * kv_bytes
        roofline["traffic_note"] = ("dram__bytes_read.sum + dram__bytes_write.sum of one launch on a batch-16 slice (ncu), "
                                    "divided by that launch's algorithmic KV bytes, times this batch's KV bytes")
    return roofline


def other_workload(bnd, label, b, dev, steps, target_ms=250.0):
    """One more named workload under the same clock: whole steps (plan + attention of every layer kind + acceptance +
    commit) timed with CUDA events over a region of about target_ms, and per layer kind the attention launch's own
    duration and roofline, computed exactly like the headline's."""
    vs = bnd.VerifyStep(b, device=dev)
    n_kinds = len(b.kinds)
    bt0, seq0 = vs.block_table.clone(), vs.seq_lens.clone()

    def run(n, pairs=None):
        for i in range(n):
            vs.block_table.copy_(bt0); vs.seq_lens.copy_(seq0)
            vs.plan_step()
            for kind in range(n_kinds):
                if pairs is not None:
                    bnd.as_plan_set_profile_events(vs.plan, *pairs[i][kind])
                vs.attn(kind)
            vs.accept()
            vs.commit(kind=n_kinds - 1)
    run(3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); run(3); e1.record()
    torch.cuda.synchronize()
    n = int(min(2000, max(steps, round(target_ms / max(e0.elapsed_time(e1) / 3, 1e-3)))))
    pairs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_kinds)] for _ in range(n)]
    for row in pairs:
        for a, c in row:
            a.record(); c.record()
    e0.record(); run(n, pairs); e1.record()
    torch.cuda.synchronize()
    bnd.as_plan_set_profile_events(vs.plan, None, None)
    assert bnd.as_plan_check(vs.plan) == 0
    ms_step = e0.elapsed_time(e1) / n
    entry = {"config": dict(workload_config(b, b.name), label=label), "timed_steps": n, "ms_per_step": ms_step,
             "value": b.total_d / (ms_step * 1e-3), "unit": UNIT, "layers": []}
    for kind in range(n_kinds):
        attn_ms = statistics.mean(row[kind][0].elapsed_time(row[kind][1]) for row in pairs)
        entry["layers"].append({"kind": kind, "window": int(b.kinds[kind].window), "roofline": roofline_of(bnd, b, vs, kind, attn_ms)})
    entry["roofline"] = entry["layers"][-1]["roofline"]
    if b.temperature is not None:
        # the same step with the hidden states as the acceptance input (as_accept_lm_head_sampled): the [rows, vocab]
        # logits and what reads them are replaced by the projection itself, two passes over the weights (every row for
        # the accept test, then one row per request for the recovery draw).  Seeded random hidden states and weights:
        # the drafts of this workload were drawn from its own logits, so nearly every request rejects its first draft
        # here; the work of the call does not depend on that.
        H = HIDDEN_DIM.get(b.name, 4096) // 64 * 64
        g = torch.Generator(device="cuda").manual_seed(78)
        hidden = torch.randn((b.total_q, H), generator=g, device="cuda").to(torch.bfloat16)
        weight = torch.empty((b.vocab, H), dtype=torch.bfloat16, device="cuda")
        for at in range(0, b.vocab, 16384):
            weight[at:at + 16384] = (torch.randn((min(16384, b.vocab - at), H), generator=g, device="cuda") * (2.0 / H ** 0.5)).to(torch.bfloat16)
        scratch = torch.empty(bnd.as_accept_lm_head_scratch_bytes(vs.plan, H, b.vocab), dtype=torch.uint8, device="cuda")
        acc_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(10)]

        def run_lm(n, ev=None):
            for i in range(n):
                vs.block_table.copy_(bt0); vs.seq_lens.copy_(seq0)
                vs.plan_step()
                for kind in range(n_kinds):
                    vs.attn(kind)
                if ev is not None:
                    ev[i][0].record()
                bnd.as_accept_lm_head_sampled(vs.plan, hidden, weight, vs.draft_tokens, vs.draft_probs, vs.temperature, vs.u, vs.w,
                                              None, scratch, vs.accept_len, vs.out_tokens)
                if ev is not None:
                    ev[i][1].record()
                vs.commit(kind=n_kinds - 1)
        run_lm(3)
        e0.record(); run_lm(10, acc_ev); e1.record()
        torch.cuda.synchronize()
        assert bnd.as_plan_check(vs.plan) == 0
        acc_ms = statistics.mean(a.elapsed_time(c) for a, c in acc_ev)
        flops = 2.0 * (b.total_q + b.batch) * H * b.vocab
        entry["from_hidden_states"] = {"ms_per_step": e0.elapsed_time(e1) / 10, "accept_call_ms": acc_ms, "rows": b.total_q,
                                       "recovery_rows": b.batch, "hidden_dim": H, "vocab": b.vocab,
                                       "tflops": flops / (acc_ms * 1e-3) / 1e12,
                                       "logits_bytes_not_materialised": b.total_q * b.vocab * 4}
    return entry


def other_workloads(bnd, dev, headline, steps):
    """The named workloads other than the headline's, one after the other (each is freed before the next is built)."""
    makers = [
        ("gpt_oss_20b: window-128 layer + full layer, batch 128", "gpt_oss_20b", lambda: workloads.gpt_oss_20b(device=dev, seed=3000)),
        ("gpt_oss_20b with every request at k = 16 (136 query rows per KV head)", "gpt_oss_20b_all_k16",
         lambda: workloads.gpt_oss_20b(device=dev, seed=3000, all_max=True)),
        ("r1_distill_llama_8b: batch 256, k = 6, sampled acceptance", "r1_distill_llama_8b",
         lambda: workloads.r1_distill_llama_8b(device=dev, seed=4000)),
        ("qwen3_8b, only the requests with n >= 8192", "qwen3_8b_min_context_8192",
         lambda: workloads.qwen3_8b(device=dev, seed=2000, min_context=8192)),
        ("r1_distill_llama_8b, only the requests with n >= 8192", "r1_distill_llama_8b_min_context_8192",
         lambda: workloads.r1_distill_llama_8b(device=dev, seed=4000, min_context=8192)),
        ("qwen3_8b: batch 64 (the headline workload of the default run)", "qwen3_8b", lambda: workloads.qwen3_8b(device=dev, seed=2000)),
    ]
    out = []
    for label, key, make in makers:
        if key == headline:
            continue
        b = make()
        out.append(other_workload(bnd, label, b, dev, steps))
        out[-1]["config"]["workload"] = key
        del b
        torch.cuda.empty_cache()
    return out


def make_workload(name, device, seed_offset=0, batch=None, min_context=0):
    over = {"batch": batch} if batch else {}
    if name == "qwen3_8b":
        return workloads.qwen3_8b(device=device, seed=2000 + seed_offset, min_context=min_context, **over)
    if name == "tiny":
        return workloads.tiny(device=device)
    if name == "r1_distill_llama_8b":
        return workloads.r1_distill_llama_8b(device=device, seed=4000 + seed_offset, min_context=min_context, **over)
    if name == "gpt_oss_20b":
        return workloads.gpt_oss_20b(device=device, seed=3000 + seed_offset, **over)
    if name == "gpt_oss_20b_all_k16":
        return workloads.gpt_oss_20b(device=device, seed=3000 + seed_offset, all_max=True, **over)
    raise SystemExit(f"unknown workload {name}")


def workload_config(b, name):
    return {"workload": name, "batch": b.batch, "num_q_heads": b.num_q_heads, "num_kv_heads": b.num_kv_heads,
            "head_dim": b.head_dim, "block_size": b.block_size, "vocab": b.vocab,
            "sum_context": int(b.seq_lens.sum()), "max_context": int(b.seq_lens.max()),
            "draft_tokens": b.total_d, "query_rows": b.total_q, "layers_per_step": len(b.kinds),
            "kv_bytes_per_layer": [b.kv_bytes(k) for k in range(len(b.kinds))],
            "logits_bytes": b.total_q * b.vocab * 4,
            "l2": "inputs larger than L2 (KV read per step >> 126 MB)" if b.kv_bytes(len(b.kinds) - 1) > 4 * 126e6
            else "L2-resident working set"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (read-only)."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_time(b, req_ids, threads):
    """Seconds the oracle needs for attention (every layer kind) + acceptance + commit of the
    requests req_ids, as it stands, on `threads` host threads."""
    import oracle
    np_bits = oracle.bf16_bits
    sb, rows = workloads.sub_batch(b, req_ids)
    cu_q = np.concatenate([[0], np.cumsum(b.draft_lens + 1)])
    cu_d = np.concatenate([[0], np.cumsum(b.draft_lens)])
    drows = np.concatenate([np.arange(cu_d[i], cu_d[i + 1]) for i in req_ids]).astype(np.int64)
    logits = b.logits[torch.as_tensor(rows, device=b.logits.device)].cpu().numpy()
    drafts = b.draft_tokens[drows]
    dp = None if b.draft_probs is None else b.draft_probs[torch.as_tensor(drows, device=b.logits.device)].cpu().numpy()
    temp = None if b.temperature is None else b.temperature[req_ids]
    u = None if b.u is None else b.u[drows]
    w = None if b.w is None else b.w[rows]
    t0 = time.perf_counter()
    for kind in range(len(sb.kinds)):
        L, K = sb.layers[kind], sb.kinds[kind]
        oracle.verify_attn(sb.seq_lens, sb.draft_lens, np_bits(L.q), np_bits(L.k_new), np_bits(L.v_new),
                           np_bits(L.k_pool), np_bits(L.v_pool), sb.block_table, num_q_heads=b.num_q_heads,
                           num_kv_heads=b.num_kv_heads, head_dim=b.head_dim, block_size=b.block_size,
                           window=K.window, sinks=None if K.sinks is None else K.sinks.double().numpy(),
                           threads=threads)
    acc = oracle.accept(sb.draft_lens, logits, b.vocab, drafts, k_max=b.k_max, draft_probs=dp, temperature=temp,
                        u=u, w=w, threads=threads)
    L = sb.layers[-1]
    oracle.kv_commit(sb.seq_lens, sb.draft_lens, acc["accept_len"], sb.block_table, np_bits(L.k_new), np_bits(L.v_new),
                     np_bits(L.k_pool), np_bits(L.v_pool), num_kv_heads=b.num_kv_heads, head_dim=b.head_dim,
                     block_size=b.block_size)
    return time.perf_counter() - t0, int(b.draft_lens[req_ids].sum())


def run_reference(args, rank):
    """The oracle as the reference arm: every step runs a bounded sample of the workload on the host."""
    if rank != 0:
        return
    import oracle
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    b = make_workload(args.workload, dev)
    threads = oracle.hardware_threads()
    sample = list(range(min(16, b.batch)))
    for _ in range(args.warmup):
        oracle_time(b, sample[:2], threads)
    t, drafts = 0.0, 0
    for _ in range(args.steps):
        dt, d = oracle_time(b, sample, threads)
        t += dt; drafts += d
    val = drafts / t
    cfg = workload_config(b, args.workload)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"requests 0..{len(sample) - 1} of {b.batch} per step (attention + accept + commit)"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_sweep(args):
    """Scaling sweep on the Qwen3-8B shape: batch x draft length x context.  Per point: attention-launch
    time (CUDA events around the kernel), whole-step time, KV GB/s, fraction of the measured and nominal HBM
    peaks, and cost relative to the k = 0 point of the same (batch, context).  Writes one JSON line per
    point to stdout and a markdown table to --sweep-out."""
    from paper_2608_24004_b200 import build as as_build
    as_build.build_library()
    from paper_2608_24004_b200 import binding as bnd
    peak, _ = measured_peaks()
    free_bytes = torch.cuda.mem_get_info()[0]
    rows = []
    for B in (1, 8, 32, 128, 512):
        for ctx in (1024, 8192, 32768, 131072):
            base = {}
            for k in (0, 1, 4, 8, 16):
                pool_bytes = 2 * B * (ctx + 64) * 8 * 128 * 2
                logit_bytes = B * (k + 1) * 151936 * 4
                if pool_bytes + logit_bytes > 0.8 * free_bytes:
                    rows.append(dict(batch=B, k=k, ctx=ctx, skipped="does not fit in HBM"))
                    continue
                b = workloads.sweep_point(B, k, ctx, device="cuda", with_logits=True)
                vs = bnd.VerifyStep(b)
                bt0, seq0 = vs.block_table.clone(), vs.seq_lens.clone()
                small = b.kv_bytes(0) < 4 * 126e6            # working set near L2 size: flush between launches
                flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if small else None

                def step():
                    vs.block_table.copy_(bt0); vs.seq_lens.copy_(seq0)
                    if flush is not None:
                        flush.zero_()
                    vs.plan_step(); vs.attn(0); vs.accept(); vs.commit()
                for _ in range(3):
                    step()
                n = 5
                ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
                sv = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
                for a, c in ev:
                    a.record(); c.record()
                for (a, c), (s0, s1) in zip(ev, sv):
                    vs.block_table.copy_(bt0); vs.seq_lens.copy_(seq0)
                    if flush is not None:
                        flush.zero_()
                    bnd.as_plan_set_profile_events(vs.plan, a, c)
                    s0.record()
                    vs.plan_step(); vs.attn(0); vs.accept(); vs.commit()
                    s1.record()
                torch.cuda.synchronize()
                assert bnd.as_plan_check(vs.plan) == 0
                t_attn = statistics.median(a.elapsed_time(c) for a, c in ev)
                t_step = statistics.median(a.elapsed_time(c) for a, c in sv)
                kv = b.kv_bytes(0)
                r = dict(batch=B, k=k, ctx=ctx, attn_us=1e3 * t_attn, step_us=1e3 * t_step, kv_gb=kv / 1e9,
                         kv_gbs=kv / t_attn / 1e6, frac_measured=kv / t_attn / 1e6 / peak,
                         frac_nominal=kv / t_attn / 1e6 / HBM_NOMINAL_GBS, l2_flush=bool(small),
                         draft_tokens=b.total_d)
                # the same step with fixed launches, its three device calls replayed from a CUDA graph: what a
                # serving loop pays at small batches, where the calls above are bound by launch overhead
                if B <= 32 and kv < 2e9:
                    del vs
                    vs = bnd.VerifyStep(b)
                    bnd.as_plan_set_fixed_launch(vs.plan, True)
                    vs.plan_step(); vs.attn(0); vs.accept(); vs.commit()
                    torch.cuda.synchronize()
                    vs.block_table.copy_(bt0); vs.seq_lens.copy_(seq0); vs.plan_step()
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph):
                        vs.attn(0); vs.accept(); vs.commit()
                    gv = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n + 3)]
                    for s0, s1 in gv:
                        vs.block_table.copy_(bt0); vs.seq_lens.copy_(seq0)
                        if flush is not None:
                            flush.zero_()
                        s0.record()
                        vs.plan_step(); graph.replay()
                        s1.record()
                    torch.cuda.synchronize()
                    assert bnd.as_plan_check(vs.plan) == 0
                    r["replayed_step_us"] = 1e3 * statistics.median(a.elapsed_time(c) for a, c in gv[3:])
                    del graph
                if k == 0:
                    base = dict(attn=t_attn, step=t_step)
                if base:
                    r["attn_vs_k0"] = t_attn / base["attn"]
                    r["step_vs_k0"] = t_step / base["step"]
                rows.append(r)
                print(json.dumps(r), flush=True)
                del vs, b, flush
                torch.cuda.empty_cache()
    if args.sweep_out:
        with open(args.sweep_out, "w") as f:
            f.write("| batch | ctx | k | attention us | step us | replayed step us | KV GB | KV GB/s | of measured | of 8 TB/s | attn vs k=0 | step vs k=0 |\n")
            f.write("|---|---|---|---|---|---|---|---|---|---|---|---|\n")
            for r in rows:
                if "skipped" in r:
                    f.write(f"| {r['batch']} | {r['ctx']} | {r['k']} | skipped: {r['skipped']} | | | | | | | | |\n")
                else:
                    f.write(f"| {r['batch']} | {r['ctx']} | {r['k']} | {r['attn_us']:.1f} | {r['step_us']:.1f} | "
                            f"{('%.1f' % r['replayed_step_us']) if 'replayed_step_us' in r else ''} | {r['kv_gb']:.3f} | "
                            f"{r['kv_gbs']:.0f} | {100 * r['frac_measured']:.1f} % | {100 * r['frac_nominal']:.1f} % | "
                            f"{r.get('attn_vs_k0', float('nan')):.2f} | {r.get('step_vs_k0', float('nan')):.2f} |\n")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3_8b")
    ap.add_argument("--attn", default="auto", choices=["auto", "simt", "tc"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch size (profiling only)")
    ap.add_argument("--min-context", type=int, default=0,
                    help="keep only the workload's requests with at least this committed length (profiling only)")
    ap.add_argument("--lm-head", action="store_true", help="(the default now: kept so that old command lines still parse)")
    ap.add_argument("--no-lm-head", action="store_true",
                    help="skip as_accept_lm_head (output projection fused with greedy acceptance) on this batch's rows")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the other named workloads (GPT-OSS-shaped pair, its all-k=16 variant, R1-shaped batch, n >= 8k subsets)")
    ap.add_argument("--repeats", type=int, default=0, help="blocks of --steps steps inside the timed region (0: about --target-ms)")
    ap.add_argument("--target-ms", type=float, default=1000.0, help="length of the timed region the repeats aim for")
    ap.add_argument("--sweep", action="store_true", help="run the batch x draft-length x context sweep instead")
    ap.add_argument("--sweep-out", default=None, help="markdown table of the sweep")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verify path has no CPU fallback")
    if args.sweep:
        torch.cuda.set_device(local_rank)
        run_sweep(args)
        return
    from paper_2608_24004_b200 import build as as_build
    as_build.build_library()
    from paper_2608_24004_b200 import binding as bnd
    from paper_2608_24004_b200 import replicas

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = f"cuda:{local_rank}"
    b = make_workload(args.workload, dev, seed_offset=100 * rank, batch=args.batch, min_context=args.min_context)
    impl = {"auto": bnd.AS_ATTN_AUTO, "simt": bnd.AS_ATTN_SIMT, "tc": bnd.AS_ATTN_TC}[args.attn]
    vs = bnd.VerifyStep(b, device=dev, attn_impl=impl)
    n_kinds = len(b.kinds)
    bt0, seq0 = vs.block_table.clone(), vs.seq_lens.clone()
    stream = torch.cuda.current_stream()

    def restore():
        vs.block_table.copy_(bt0); vs.seq_lens.copy_(seq0)

    def step():
        vs.plan_step()
        for kind in range(n_kinds):
            vs.attn(kind)
        vs.accept()
        vs.commit(kind=n_kinds - 1)

    def barrier():
        replicas.barrier(dev)

    def max_over_ranks(ms):
        return replicas.max_over_ranks(ms, dev)

    # ---- device-resident timing -------------------------------------------------------------
    # K = --steps steps form one block; the block is repeated R times back to back inside the timed region so that the
    # region lasts about a second (the clock sampler then sees ten or more samples, and one slow step does not
    # decide the number).  ms_per_step is the mean over all K * R steps; the per-block means give min / median / max.
    for _ in range(args.warmup):
        restore(); step()
    assert bnd.as_plan_check(vs.plan) == 0
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0.record()
    for _ in range(3):
        restore(); step()
    w1.record()
    torch.cuda.synchronize()
    est_ms = max(w0.elapsed_time(w1) / 3, 1e-3)
    repeats = args.repeats if args.repeats > 0 else int(min(400, max(1, round(args.target_ms / (est_ms * args.steps)))))
    repeats = int(replicas.max_over_ranks(float(repeats), dev))
    n_timed = args.steps * repeats
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_timed)]
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    for a, c in pairs:
        a.record(); c.record()
    sampler = ClockSampler(local_rank)
    l0 = bnd.as_plan_launch_count(vs.plan)
    barrier()
    sampler.start()
    marks[0].record()
    for r in range(repeats):
        for a, c in pairs[r * args.steps:(r + 1) * args.steps]:
            restore()
            bnd.as_plan_set_profile_events(vs.plan, a, c)      # last layer kind of the step is the one kept
            step()
        marks[r + 1].record()
    barrier()
    clocks = sampler.stop()
    bnd.as_plan_set_profile_events(vs.plan, None, None)
    launches = bnd.as_plan_launch_count(vs.plan) - l0
    ms_total = max_over_ranks(marks[0].elapsed_time(marks[-1]))
    ms_step = ms_total / n_timed
    block_ms = [marks[r].elapsed_time(marks[r + 1]) / args.steps for r in range(repeats)]
    attn_all = [a.elapsed_time(c) for a, c in pairs]
    attn_ms = statistics.mean(attn_all)
    assert bnd.as_plan_check(vs.plan) == 0
    total_drafts = replicas.sum_over_ranks(float(b.total_d), dev)
    value = total_drafts / (ms_step * 1e-3)

    # ---- end to end: host buffers in, results out, inside the timed region ----------------------
    L = vs.layers[n_kinds - 1]
    host_in = {"q": [l.q for l in vs.layers], "k_new": [l.k_new for l in vs.layers], "v_new": [l.v_new for l in vs.layers]}
    pinned = {k: [t.cpu().pin_memory() for t in v] for k, v in host_in.items()}
    pin_logits = vs.logits.cpu().pin_memory()
    pin_drafts = vs.draft_tokens.cpu().pin_memory() if vs.draft_tokens is not None and b.total_d else None
    pin_dp = vs.draft_probs.cpu().pin_memory() if vs.draft_probs is not None else None
    h_acc = torch.empty_like(vs.accept_len, device="cpu").pin_memory()
    h_tok = torch.empty_like(vs.out_tokens, device="cpu").pin_memory()
    h_freed = torch.empty_like(vs.freed, device="cpu").pin_memory()
    h_nf = torch.empty_like(vs.freed_count, device="cpu").pin_memory()
    h2d = sum(t.numel() * t.element_size() for v in pinned.values() for t in v) + pin_logits.numel() * 4 \
        + (pin_drafts.numel() * 4 if pin_drafts is not None else 0) + (pin_dp.numel() * 4 if pin_dp is not None else 0)
    d2h = sum(t.numel() * t.element_size() for t in (h_acc, h_tok, h_freed, h_nf))

    # The logits (and dense draft probabilities) are by far the largest input and only acceptance reads them,
    # so their copy runs on a second stream beside plan + attention; acceptance waits for it.
    side = torch.cuda.Stream()

    def e2e_step():
        main = torch.cuda.current_stream()
        # small inputs and the plan's metadata first: copies of one direction share a copy engine in issue order
        for kind in range(n_kinds):
            vs.layers[kind].q.copy_(pinned["q"][kind], non_blocking=True)
            vs.layers[kind].k_new.copy_(pinned["k_new"][kind], non_blocking=True)
            vs.layers[kind].v_new.copy_(pinned["v_new"][kind], non_blocking=True)
        if pin_drafts is not None:
            vs.draft_tokens.copy_(pin_drafts, non_blocking=True)
        vs.plan_step()
        side.wait_stream(main)                             # the previous step's acceptance has read the old logits
        with torch.cuda.stream(side):
            vs.logits.copy_(pin_logits, non_blocking=True)
            if pin_dp is not None:
                vs.draft_probs.copy_(pin_dp, non_blocking=True)
        for kind in range(n_kinds):
            vs.attn(kind)
        main.wait_stream(side)
        vs.accept()
        vs.commit(kind=n_kinds - 1)
        h_acc.copy_(vs.accept_len, non_blocking=True); h_tok.copy_(vs.out_tokens, non_blocking=True)
        h_freed.copy_(vs.freed, non_blocking=True); h_nf.copy_(vs.freed_count, non_blocking=True)
        main.synchronize()                                 # the caller reads the accepted tokens every step

    e2e_steps = max(3, min(args.steps, 10))
    restore(); e2e_step()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(e2e_steps):
        restore(); e2e_step()
    f1.record()
    barrier()
    e2e_ms = max_over_ranks(f0.elapsed_time(f1)) / e2e_steps
    assert int(h_acc.sum()) == int(vs.accept_len.sum())

    # ---- roofline of the dominant kernel (attention of the last layer kind) ----------------------
    roofline = roofline_of(bnd, b, vs, n_kinds - 1, attn_ms)

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "repeats": repeats, "timed_steps": n_timed, "timed_region_ms": ms_total,
           "ms_per_step_blocks": {"min": min(block_ms), "median": statistics.median(block_ms), "max": max(block_ms)},
           "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
           "data": "synthetic", "config": workload_config(b, args.workload), "clocks": clocks,
           "e2e": {"value": total_drafts / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                   "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
           "gpu_launches": int(launches), "roofline": roofline,
           "query_rows_per_s": b.total_q * world / (ms_step * 1e-3)}
    if not args.no_lm_head and rank == 0 and world == 1:
        lm, hidden, weight = lm_head_leg(bnd, vs, b, args.workload, max(3, min(args.steps, 10)))
        # the same end-to-end step with the hidden states as the step's input instead of the logits they project to
        # (the weights stay resident like the KV pools; greedy acceptance, whatever the workload's own mode)
        pin_hidden = hidden.cpu().pin_memory()

        def e2e_lm_step():
            main = torch.cuda.current_stream()
            for kind in range(n_kinds):
                vs.layers[kind].q.copy_(pinned["q"][kind], non_blocking=True)
                vs.layers[kind].k_new.copy_(pinned["k_new"][kind], non_blocking=True)
                vs.layers[kind].v_new.copy_(pinned["v_new"][kind], non_blocking=True)
            if pin_drafts is not None:
                vs.draft_tokens.copy_(pin_drafts, non_blocking=True)
            hidden.copy_(pin_hidden, non_blocking=True)
            vs.plan_step()
            for kind in range(n_kinds):
                vs.attn(kind)
            bnd.as_accept_lm_head(vs.plan, hidden, weight, vs.draft_tokens, vs.accept_len, vs.out_tokens)
            vs.commit(kind=n_kinds - 1)
            h_acc.copy_(vs.accept_len, non_blocking=True); h_tok.copy_(vs.out_tokens, non_blocking=True)
            h_freed.copy_(vs.freed, non_blocking=True); h_nf.copy_(vs.freed_count, non_blocking=True)
            main.synchronize()

        restore(); e2e_lm_step()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(e2e_steps):
            restore(); e2e_lm_step()
        g1.record()
        torch.cuda.synchronize()
        lm["e2e_ms_per_step_from_hidden_states"] = g0.elapsed_time(g1) / e2e_steps
        lm["e2e_h2d_bytes_per_step_from_hidden_states"] = h2d - pin_logits.numel() * 4 - (pin_dp.numel() * 4 if pin_dp is not None else 0) \
            + pin_hidden.numel() * 2
        assert bnd.as_plan_check(vs.plan) == 0
        out["lm_head"] = lm
    if rank == 0 and world == 1 and not args.no_other_workloads and not args.batch and not args.min_context:
        del vs
        if not args.no_lm_head:
            del hidden, weight
        torch.cuda.empty_cache()
        out["other_workloads"] = other_workloads(bnd, dev, args.workload, max(3, min(args.steps, 10)))
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        threads = oracle.hardware_threads()
        sample = list(range(b.batch))
        # bound the sample to roughly 10-30 s of host work (the oracle runs ~10 GFLOP/s on 8 cores)
        flops = 4.0 * ((b.seq_lens + b.draft_lens + 1.0) * (b.draft_lens + 1)) * b.num_q_heads * b.head_dim * n_kinds
        budget, acc_f, keep = 2.0e11, 0.0, []
        for i in sample:
            if acc_f + flops[i] > budget and keep:
                break
            keep.append(i); acc_f += flops[i]
        dt, d = oracle_time(b, keep, threads)
        out["cpu_baseline"] = {"value": d / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                               "sample": f"requests 0..{len(keep) - 1} of {b.batch} (attention + accept + commit), once"}
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
