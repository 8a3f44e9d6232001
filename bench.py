#!/usr/bin/env python
"""Benchmark of the block-diffusion decode hot path (one JSON line on stdout).

A "step" of this bench is one whole pass of the hot path over one block: block_begin, the denoise
steps of the workload's schedule (each = decoder forward in denoise mode + LM head + confidence +
unmask selection) and commit_block (causal forward with KV-cache update).  The metric is batch-1
decode tokens/s = block tokens / time, whole job over all GPUs (independent replicas, one request
per GPU: the path has no data-path collective).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

`--impl reference` times the CPU oracle (as it stands) on the host cores instead.
"""
from __future__ import annotations

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

from paper_2604_06832_b200 import inputs as I  # noqa: E402

DEFAULT_WORKLOAD = "cfg2_3b_bf16_p1024_b32_top8"
METRIC = "batch-1 decode tok/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.t.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def config_of(wl: I.Workload, block: int, world: int) -> dict:
    """The workload description both arms print."""
    return {"workload": wl.name, "block": block, "prefix": wl.n_embeds + wl.n_tokens,
            "denoise_steps_per_block": schedule(wl, block), "rule": wl.rule,
            "cache_flush": "inputs (gigabytes of weights per forward) larger than L2", "parallelism": f"replicas x{world}"}


def schedule(wl: I.Workload, block: int):
    """Denoise steps per block on a random-init model: top-k gives ceil(B/k) steps; threshold 0.9 never
    fires on near-uniform confidences, so the at-least-one rule gives B steps."""
    return (block + wl.k - 1) // wl.k if wl.rule == "topk" else block


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (the reported cpu_baseline, and the whole of --impl reference)
# ------------------------------------------------------------------------------------------------
def make_oracle_at_prefix(wl: I.Workload, weights_cpu: dict):
    """The oracle with a cache of the workload's prefix length.  The prefill is outside the metric and would take the
    oracle minutes at these lengths, so the cache is filled with N(0, 1) values of the right shape instead: the time of
    a denoise or commit forward depends on the cache's length, not on its contents."""
    import numpy as np
    from oracle import fdvlm_oracle as orc
    shape = wl.shape
    o = orc.Oracle(shape, I.weights_to_numpy(weights_cpu), act_fp8=(shape.dtype == I.W8A8))
    L0 = wl.n_embeds + wl.n_tokens
    rng = np.random.default_rng(wl.prefix_seed)
    for l in range(shape.n_layers):
        o.K[l] = rng.standard_normal((L0, shape.n_kv_heads, shape.head_dim))
        o.V[l] = rng.standard_normal((L0, shape.n_kv_heads, shape.head_dim))
    o.cache_len = L0
    return o


def oracle_forward_seconds(o, wl: I.Workload, block: int, commit: bool):
    """One timed oracle forward of a block at the current cache length: a denoise step, or the causal commit (whose
    cache growth is undone afterwards so that every sample sees the same length)."""
    import numpy as np
    from oracle import fdvlm_oracle as orc
    rule = orc.TOPK if wl.rule == "topk" else orc.THRESHOLD
    L0 = o.cache_len
    o.block_begin(block)
    if not commit:
        t0 = time.perf_counter()
        o.block_step(rule, wl.threshold, wl.k)
        return time.perf_counter() - t0
    o.block_tokens[:] = np.arange(block) % (wl.shape.vocab - 1)
    o.masked[:] = False
    t0 = time.perf_counter()
    o.commit_block(want_logits=False)
    dt = time.perf_counter() - t0
    o.truncate(L0)
    return dt


def oracle_tok_s(wl, block, t_step, t_commit):
    return block / (schedule(wl, block) * t_step + t_commit)


def run_reference(args, wl, block):
    from paper_2604_06832_b200 import replicas as R
    if not R.prints_result(int(os.environ.get("RANK", "0"))):
        return
    shape = wl.shape
    weights = I.make_weights(shape, wl.weight_seed)
    cores = torch.get_num_threads()
    o = make_oracle_at_prefix(wl, weights)
    L0 = o.cache_len
    n_steps = schedule(wl, block)
    # A bench step is one block = n_steps denoise forwards + 1 commit forward.  One oracle forward of the 3B shape takes
    # ~13 s, so each timed "step" of this arm is a bounded sample of the block: ONE denoise forward (the commit forward
    # is timed once, before the loop); tokens/s extrapolates the block from them.  The loop stops after ~3 minutes and
    # `steps` reports what was really run.
    t_commit = oracle_forward_seconds(o, wl, block, commit=True)
    t_all0 = time.perf_counter()
    for _ in range(max(0, args.warmup)):
        if time.perf_counter() - t_all0 > 45.0:
            break
        oracle_forward_seconds(o, wl, block, commit=False)
    t_loop0 = time.perf_counter()
    t_steps = []
    for _ in range(max(1, args.steps)):
        t_steps.append(oracle_forward_seconds(o, wl, block, commit=False))
        if time.perf_counter() - t_loop0 > 170.0:
            break
    wall = time.perf_counter() - t_all0
    t_step = statistics.median(t_steps)
    value = oracle_tok_s(wl, block, t_step, t_commit)
    sample = (f"each timed step = one denoise forward of a {block}-token block at cache length {L0} (median {t_step:.1f} s over "
              f"{len(t_steps)} forwards); the commit forward was timed once ({t_commit:.1f} s); tokens/s = {block} / "
              f"({n_steps} x step + commit); the cache holds N(0,1) values (the prefill is outside the metric)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tok/s", "n_gpus": args.gpus,
            "steps": len(t_steps), "steps_requested": args.steps, "warmup": args.warmup,
            "ms_per_step": 1000.0 * t_step, "ms_per_block_extrapolated": 1000.0 * block / value, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, block, 1),
            "cpu_baseline": {"value": value, "unit": "tok/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": wall}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# the CUDA path
# ------------------------------------------------------------------------------------------------
def run_ours(args, wl, block):
    from paper_2604_06832_b200 import binding as B
    from paper_2604_06832_b200 import build as build_mod
    from paper_2604_06832_b200 import replicas as R
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build_mod.build()
    if dist is not None:
        dist.barrier()
    shape = wl.shape
    n_steps = schedule(wl, block)
    K, W = args.steps, args.warmup
    L0 = wl.n_embeds + wl.n_tokens
    max_seq = L0 + (2 * (K + W) + 2) * block + (2 * K + 4) * block + 64 + 8 * (K + 2) + 64
    weights = I.make_weights(shape, wl.weight_seed, device="cuda")
    stream = torch.cuda.Stream()
    # the 7B configuration prescribes a bf16 KV cache; the others leave the cache's element type open
    kv_dtype = B.KV_BF16 if shape.dtype in (I.FP8, I.W8A8) else B.KV_F16
    # top-k schedules: the commit of block t rides in the forward of block t+1's first step (one forward over 2 x block rows)
    fused_commit = 2 * block <= 64 and not args.separate_commit
    handle = B.Handle(shape, weights, max_seq=max_seq, max_block=max(2 * block if fused_commit else block, 32), stream=stream,
                      kv_dtype=kv_dtype)
    emb, toks = I.make_prefix(shape, wl.n_embeds, wl.n_tokens, wl.prefix_seed)
    emb_d, toks_d = emb.cuda(), toks.cuda()
    rule = B.RULE_TOPK if wl.rule == "topk" else B.RULE_THRESHOLD
    ev = lambda: torch.cuda.Event(enable_timing=True)
    tensor_core_path = shape.dtype != I.F32
    device_loop = tensor_core_path and os.environ.get("FDVLM_NO_GRAPH", "0") != "1"

    with torch.cuda.stream(stream):
        t0, t1 = ev(), ev()
        t0.record(stream)
        handle.prefill(emb_d, toks_d)
        t1.record(stream)
        stream.synchronize()
        prefill_ms = t0.elapsed_time(t1)

        launches = [0]
        fused_device = fused_commit and (wl.rule == "topk" or device_loop)    # (the stepwise exact path commits separately)
        open_block = [False]          # fused_commit: the block decoded by the previous call, not yet committed

        def close_open_block():
            if open_block[0]:
                handle.commit_block()
                open_block[0] = False

        def one_block_device():
            if fused_device:
                # no host round trip between the steps (top-k: fixed schedule enqueued back to back; threshold: the loop
                # runs on the device); the previous call's block is committed by this call's first forward.  Per call: one
                # block committed, one block decoded.
                if wl.rule == "topk":
                    info = handle.commit_decode_block_topk(block, wl.k)
                else:
                    info = handle.commit_decode_block(block, rule, wl.threshold, wl.k)
                launches[0] += handle.last_launch_count()
                open_block[0] = True
                return info.step_index
            close_open_block()
            if wl.rule == "topk":
                info = handle.decode_block_topk(block, wl.k)
                launches[0] += handle.last_launch_count()
                handle.commit_block()
                launches[0] += handle.last_launch_count()
                return info.step_index
            if device_loop:
                # threshold rule: the step count depends on the confidences, so the loop itself runs on the device
                info = handle.decode_block(block, rule, wl.threshold, wl.k)
                launches[0] += handle.last_launch_count()
                handle.commit_block()
                launches[0] += handle.last_launch_count()
                return info.step_index
            handle.block_begin(block)       # (exact fp32 path, or graphs switched off: one host read-back per step)
            n = 0
            while True:
                info = handle.block_step(rule, wl.threshold, wl.k)
                launches[0] += handle.last_launch_count()
                n += 1
                if info.n_remaining == 0:
                    break
            handle.commit_block()
            launches[0] += handle.last_launch_count()
            return n

        conf_h = torch.empty(block, dtype=torch.float32).pin_memory()
        pred_h = torch.empty(block, dtype=torch.int32).pin_memory()
        um_h = torch.empty(block, dtype=torch.uint8).pin_memory()
        tok_h = torch.empty(block, dtype=torch.int32).pin_memory()
        init_h = torch.full((block,), shape.mask_id, dtype=torch.int32).pin_memory()

        def one_block_host():
            if fused_commit:
                if open_block[0]:
                    info = handle.commit_begin_step_host(block, rule, wl.threshold, wl.k, next_init_tokens=init_h, conf=conf_h,
                                                         pred=pred_h, unmask=um_h, block_tokens=tok_h)
                else:
                    handle.block_begin_host(block, init_h)
                    info = handle.block_step_host(rule, wl.threshold, wl.k, conf=conf_h, pred=pred_h, unmask=um_h, block_tokens=tok_h)
                while info.n_remaining:
                    info = handle.block_step_host(rule, wl.threshold, wl.k, conf=conf_h, pred=pred_h, unmask=um_h, block_tokens=tok_h)
                open_block[0] = True
                return
            handle.block_begin_host(block, init_h)
            while True:
                info = handle.block_step_host(rule, wl.threshold, wl.k, conf=conf_h, pred=pred_h, unmask=um_h, block_tokens=tok_h)
                if info.n_remaining == 0:
                    break
            handle.commit_block()

        def timed(fn, k):
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record(stream)
            for _ in range(k):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return R.max_over_ranks_ms(a.elapsed_time(b), dist, torch.device("cuda", local))

        for _ in range(W):
            steps_seen = one_block_device()
        sampler = ClockSampler(local)
        sampler.start()
        launches[0] = 0
        ms_dev = timed(one_block_device, K)
        n_launch = launches[0]
        clocks = sampler.stop()
        # end to end: host buffers through the C ABI (H2D of the block's init tokens, D2H of every step's results)
        one_block_host()
        ms_e2e = timed(one_block_host, K)
        close_open_block()

        # (1) the projection launches timed one by one with CUDA events (kernels launched singly: no overlap)
        handle.profile_enable(1)
        handle.block_begin(block)
        for _ in range(n_steps):
            handle.block_step(rule, wl.threshold, wl.k)
        prof = handle.profile_read()
        handle.profile_enable(0)
        handle.commit_block()
        # (2) in-chain timing: the production launch sequence (graph replay, dependent launches), every kernel stamping the
        # GPU's global timer.  The timeline of a forward is cut at the kernels' end times: kernel i owns the interval
        # (end of kernel i-1, end of kernel i], so the shares add up to the forward's duration.
        chain_us, chain_total, chain_n = {}, [], 0
        if tensor_core_path:
            handle.profile_enable(2)
        handle.block_begin(block)
        handle.block_step(rule, wl.threshold, wl.k)        # the stamped graph's first use (capture)
        while handle.last_info_remaining() > 0:
            handle.block_step(rule, wl.threshold, wl.k)
            if not tensor_core_path:
                continue
            recs = handle.profile_read_chain()
            prev = recs[0]["start_us"]
            for r in recs:
                end = max(r["end_us"], prev)
                chain_us[r["kind"]] = chain_us.get(r["kind"], 0.0) + (end - prev)
                prev = end
            chain_total.append(prev - recs[0]["start_us"])
            chain_n += 1
        handle.profile_enable(0)
        handle.commit_block()
        chain_us = {k_: v / max(chain_n, 1) for k_, v in chain_us.items()}
        # (3) unprofiled per-step latency
        handle.block_begin(block)
        L_step = handle.cache_len()
        lat = []
        for _ in range(n_steps):
            a, b = ev(), ev()
            a.record(stream)
            handle.block_step(rule, wl.threshold, wl.k)
            b.record(stream)
            stream.synchronize()
            lat.append(a.elapsed_time(b))
        handle.commit_block()

        # The paper's own decoding conventions on the same workload (reported beside the headline, not in it):
        # (a) blocks seeded by the causal pass and denoised under shift-by-one (Sec. 3.4 "causal context decoding"),
        # (b) linear self-speculative decoding (Appendix B, Alg. 1).  On random-init weights drafts almost never
        # agree with the verifier, so (b) shows the cost of an iteration (two passes), not the paper's acceptance:
        # `tok_s_if_all_accepted` is the same iteration time at the other end of the range (B tokens per iteration).
        # (c) quadratic self-speculative decoding (Appendix B, Alg. 2) at block size 5: one 30-row forward per iteration.
        modes = None
        if block > 1:
            row_pred = torch.empty(block, dtype=torch.int32, device="cuda")
            init_d = torch.full((block,), shape.mask_id, dtype=torch.int32, device="cuda")
            handle.block_begin(block)
            handle.block_step(B.RULE_THRESHOLD, -1.0, 0)
            handle.commit_block_verify(row_pred)

            def one_block_seeded():
                init_d[0:1].copy_(row_pred[block - 1:block])      # the previous commit's last-row argmax
                handle.block_begin(block, init_d)
                n = 0
                while True:
                    info = handle.block_step(rule, wl.threshold, wl.k, pred_shift=1)
                    n += 1
                    if info.n_remaining == 0:
                        break
                handle.commit_block_verify(row_pred)
                return n

            seeded_steps = one_block_seeded()
            ms_seeded = timed(one_block_seeded, K)
            stream.synchronize()
            state = {"seed": int(row_pred[block - 1].item()), "accepted": 0}

            def one_spec_iteration():
                info = handle.spec_block(block, state["seed"])
                state["seed"] = info.next_token
                state["accepted"] += info.accepted

            one_spec_iteration()
            state["accepted"] = 0
            ms_spec = timed(one_spec_iteration, K)
            modes = {"seeded_shift_by_one": {"tok_s": K * block * world / (ms_seeded / 1000.0), "denoise_steps_per_block": seeded_steps},
                     "self_speculative_linear": {"tok_s": state["accepted"] * world / (ms_spec / 1000.0), "ms_per_iteration": ms_spec / K,
                                                 "accepted_per_iteration": state["accepted"] / K,
                                                 "tok_s_if_all_accepted": block * world / (ms_spec / K / 1000.0)}}
            QB = 5
            if QB * (QB + 1) <= max(block, 32):
                handle.quad_begin(QB, state["seed"])
                qstate = {"accepted": 0}

                def one_quad_iteration():
                    qstate["accepted"] += handle.quad_step().accepted

                one_quad_iteration()
                qstate["accepted"] = 0
                ms_quad = timed(one_quad_iteration, K)
                handle.quad_end()
                modes["self_speculative_quadratic"] = {"block": QB, "rows_per_forward": QB * (QB + 1),
                                                       "tok_s": qstate["accepted"] * world / (ms_quad / 1000.0),
                                                       "ms_per_iteration": ms_quad / K,
                                                       "accepted_per_iteration": qstate["accepted"] / K,
                                                       "tok_s_if_all_accepted": QB * world / (ms_quad / K / 1000.0)}

    value = R.whole_job_rate(K * block, world, ms_dev)
    e2e_value = R.whole_job_rate(K * block, world, ms_e2e)
    peak, peak_kind = measured_peaks()
    wbytes = shape.weight_bytes()
    gemm_ms_isolated = prof["ms_linear"] / n_steps
    gemm_kinds = ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_lm_head")
    gemm_us_chain = sum(chain_us.get(k_, 0.0) for k_ in gemm_kinds)
    if gemm_us_chain <= 0:          # exact fp32 path: no in-chain stamps, the one-by-one figure stands in
        gemm_us_chain = gemm_ms_isolated * 1000.0
    gemm_gbs = wbytes / (gemm_us_chain * 1e-6) / 1e9
    kv_bytes = shape.kv_bytes_per_token() * L_step
    attn_us_chain = chain_us.get("attention", 0.0) + chain_us.get("attn_merge", 0.0)
    # DRAM bytes of the same launches: dram read + write over algorithmic bytes of the layer projections, from the ncu
    # capture summarised in profiles/ncu_traffic.json (taken on the 4-layer cut of the shape; traffic grows in
    # proportion to the weight bytes).  Null when there is no capture of the kernel as it stands.
    traffic, traffic_note = None, None
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            cap = json.load(f).get("gemm_tc", {}).get(shape.dtype)
        if cap and block == cap.get("block"):
            traffic = wbytes * cap["dram_bytes"] / cap["algorithmic_bytes"]
            traffic_note = cap.get("note")
    except (OSError, ValueError, KeyError):
        pass
    step_bytes = wbytes + kv_bytes
    step_med = statistics.median(lat)
    lat_sorted = sorted(lat)
    pct = lambda q: lat_sorted[min(len(lat_sorted) - 1, max(0, int(round(q * (len(lat_sorted) - 1)))))]
    # a second denominator beside the copy bandwidth: what a plain read-only streaming kernel of the library reaches on this
    # GPU, on a 2 GiB buffer (larger than L2), median of 5 after 3 warm-up launches
    with torch.cuda.stream(stream):
        rbuf = torch.empty(2 << 30, dtype=torch.uint8, device="cuda")
        rsink = torch.zeros(1, dtype=torch.int32, device="cuda")
        rt = []
        for i in range(8):
            a, b = ev(), ev()
            a.record(stream)
            B.util_stream_read(rbuf, rsink, stream)
            b.record(stream)
            stream.synchronize()
            if i >= 3:
                rt.append(a.elapsed_time(b))
        read_peak = rbuf.numel() / (statistics.median(rt) / 1000.0) / 1e9
        del rbuf
    line = {
        "metric": METRIC, "value": value, "unit": "tok/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_dev / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {"f32": "f32", "bf16": "bf16", "fp8": "f16 x e4m3 weights", "w8a8": "e4m3 x e4m3 (per-token activation scales)"}[shape.dtype], "data": "synthetic",
        "config": config_of(wl, block, world),
        "kv_dtype": "bf16" if kv_dtype == B.KV_BF16 else "f16",
        # per block: n denoise steps + one causal commit; with fused_commit the commit of block t and the first step of
        # block t+1 are one forward over 2 x block rows (same results, every weight byte streamed once for both)
        "forwards_per_block": (n_steps if fused_device else n_steps + 1), "fused_commit": fused_device,
        "e2e_fused_commit": fused_commit,
        "e2e": {"value": e2e_value, "unit": "tok/s", "h2d_bytes_per_step": block * 4,
                "d2h_bytes_per_step": n_steps * (block * 13 + 32)},
        "gpu_launches": n_launch,
        "clocks": clocks,
        # dominant kernel: the projection GEMMs.  achieved = every linear weight byte of one forward / the time those
        # launches own in the production chain (in-chain timing, see above); frac x peak x that time = the bytes.
        "roofline": {"bound": "hbm", "achieved": gemm_gbs, "peak": peak, "unit": "GB/s", "frac": gemm_gbs / peak,
                     "traffic": traffic, "traffic_note": traffic_note, "peak_kind": peak_kind,
                     "kernel": "gemm_tc_kernel: all projection launches of one denoise forward, in-chain",
                     "algorithmic_bytes_per_forward": wbytes, "in_chain_ms_per_forward": gemm_us_chain / 1000.0,
                     "forward_ms_in_chain_timing": statistics.median(chain_total) / 1000.0 if chain_total else None,
                     "isolated": {"ms_per_forward": gemm_ms_isolated, "achieved": wbytes / (gemm_ms_isolated / 1000.0) / 1e9,
                                  "note": "the same launches timed one by one with CUDA events, without the chain's overlap"}},
        "attention": {"kernel": "attn_mma_kernel + attn_combine_kernel, in-chain", "kv_bytes_per_forward": kv_bytes,
                      "in_chain_ms_per_forward": attn_us_chain / 1000.0,
                      "achieved_gbs": kv_bytes / (attn_us_chain * 1e-6) / 1e9 if attn_us_chain > 0 else None},
        "chain_us_per_forward": {k_: round(v, 2) for k_, v in sorted(chain_us.items())},
        "step": {"latency_ms_median": step_med, "latency_ms_p10": pct(0.1), "latency_ms_p90": pct(0.9), "latency_ms_all": lat,
                 "cache_len": L_step, "bytes": step_bytes,
                 "gbs": step_bytes / (step_med / 1000.0) / 1e9, "frac_of_peak": step_bytes / (step_med / 1000.0) / 1e9 / peak,
                 "frac_of_8tbs": step_bytes / (step_med / 1000.0) / 1e9 / 8000.0,
                 "read_only_stream_gbs": read_peak, "frac_of_read_only_stream": step_bytes / (step_med / 1000.0) / 1e9 / read_peak},
        "prefill_ms": prefill_ms,
        "modes": modes,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        wcpu = {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in weights.items() if k != "layers"}
        wcpu["layers"] = [{k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in lw.items()} for lw in weights["layers"]]
        o = make_oracle_at_prefix(wl, wcpu)
        ts = oracle_forward_seconds(o, wl, block, commit=False)
        tc = oracle_forward_seconds(o, wl, block, commit=True)
        line["cpu_baseline"] = {"value": oracle_tok_s(wl, block, ts, tc), "unit": "tok/s", "cores": torch.get_num_threads(),
                                "kind": "oracle",
                                "sample": f"one denoise forward ({ts:.1f} s) + one commit forward ({tc:.1f} s) of a {block}-token block "
                                          f"at cache length {o.cache_len} (cache filled with N(0,1) values: the prefill is outside the "
                                          f"metric), extrapolated over {n_steps} denoise steps + 1 commit per block"}
    handle.close()
    if R.prints_result(rank):
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(I.WORKLOADS))
    ap.add_argument("--block", type=int, default=0, help="block size (default: the workload's last listed size)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--separate-commit", action="store_true",
                    help="commit every block by a forward of its own instead of inside the next block's first step")
    args = ap.parse_args()
    wl = I.WORKLOADS[args.workload]
    block = args.block or (32 if 32 in wl.block_sizes else wl.block_sizes[-1])
    if args.impl == "reference":
        run_reference(args, wl, block)
    else:
        run_ours(args, wl, block)


if __name__ == "__main__":
    main()
