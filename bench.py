#!/usr/bin/env python
"""Benchmark of the draft / verify MoE hot path on DeepSeek-V2-Lite-shaped synthetic layers.

One *step* is one pass of the whole hot path over one block on one MoE layer:
    moe_draft_step (1 token, Eq. 5)  ->  moe_verify_block (K tokens, Eq. 4 grouped by the expert union)
    ->  spec_accept (greedy verification over the vocabulary).
Steps rotate over independently seeded layers (default 8 x 1.16 GB of bf16 experts) so that no weight is
ever re-read from L2 between timed iterations.

Prints ONE JSON line (keys: metric, value, roofline, e2e, cpu_baseline, clocks, ...).  ``--impl reference`` times the CPU checker
(``oracle/``) on the host cores on the same configuration instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2607_24434_b200 import synth

METRIC = "verify_block_moe_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + write) per launch of the grouped-SwiGLU kernel from the ncu capture summarised in
# profiles/hot_kernels_v2lite_k4_ncu_full.txt: 259.63 MB read + 3.56 MB written at 259.59 MB algorithmic
# (|U| = 13).  The capture runs a 2-layer case; traffic grows with the units streamed, so a launch's traffic is
# that ratio x its bytes.
NCU_TRAFFIC_RATIO = (259.635 + 3.561) / 259.59
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.idx = device_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.idx}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def build_workload(binding, ctx, shape, n_layers, K, V, seed0, device, q4=False):
    """Packed layers, hidden blocks, LM head and draft tokens, all resident on the GPU."""
    layers, blocks, hosts = [], [], []
    for i in range(n_layers):
        w = synth.make_layer(shape, seed0 + i, device, zipf=True)
        if q4:
            w = synth.quantize_layer(w)      # experts 4-bit block-quantised, resident in that form
        L = binding.Layer.from_weights(ctx, w)
        torch.cuda.synchronize()
        del w
        layers.append(L)
        blocks.append(synth.hidden_block(K, shape.hidden, seed0 + 100 + i, 0.0, device))
    torch.cuda.empty_cache()
    W_lm = synth.lm_head(V, shape.hidden, seed0 + 999, torch.bfloat16, device)
    return layers, blocks, W_lm


def run_gpu(args):
    from paper_2607_24434_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    shape = synth.shape_v2lite()
    if args.wide:
        import dataclasses
        shape = dataclasses.replace(shape, weight_dtype=synth.DTYPE_BF16_WIDE)
    K, V, NL = args.block, args.vocab, args.layers
    ctx = binding.Context(local)
    if args.launch_overlap is not None:
        ctx.set_launch_overlap(args.launch_overlap)
    if args.accept_l2_mb is not None:
        ctx.set_accept_l2_keep(int(args.accept_l2_mb * 1e6))
    layers, blocks, W_lm = build_workload(binding, ctx, shape, NL, K, V, 1000 + 50 * rank, device, args.q4_resident)
    H = shape.hidden
    stream = torch.cuda.current_stream()

    # persistent output buffers (one set per layer so results can be inspected afterwards)
    rb = [binding._routing_buffers(shape, K, device) for _ in range(NL)]
    ys = [torch.empty((K, H), device=device) for _ in range(NL)]
    yd = torch.empty((1, H), device=device)
    dbuf = {"topk_ids": torch.empty((shape.top_k,), dtype=torch.int32, device=device),
            "topk_w": torch.empty((shape.top_k,), dtype=torch.float32, device=device)}
    abuf = {"target": torch.empty((K,), dtype=torch.int32, device=device),
            "n_accept": torch.empty((1,), dtype=torch.int32, device=device),
            "next_token": torch.empty((1,), dtype=torch.int32, device=device)}
    draft_tok = torch.zeros((K,), dtype=torch.int32, device=device)

    def step(i):
        li = i % NL
        binding.moe_draft_step(layers[li], blocks[li][:1], yd, dbuf)
        binding.moe_verify_block(layers[li], blocks[li], ys[li], rb[li])
        binding.spec_accept(ctx, ys[li], W_lm, draft_tok, True, abuf)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # draft tokens that agree with the target for a geometric(0.85) prefix (per layer 0's block)
    step(0)
    torch.cuda.synchronize()
    tgt = abuf["target"].cpu().numpy()
    draft_tok.copy_(torch.from_numpy(synth.draft_tokens_from_target(tgt, V, 7)).to(device))

    for i in range(args.warmup):
        step(i)
    barrier()
    launches_per_step = 5
    graph = rem_graph = None
    n_full, n_rem = divmod(args.steps, NL)
    if not args.no_graph:
        # one CUDA graph holding a step on each of the NL layers, replayed steps // NL times, and a second graph with
        # the remaining steps % NL steps: exactly --steps steps are timed
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            for i in range(NL):
                step(i)
        stream.wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        l0 = ctx.kernel_launches()
        with torch.cuda.graph(graph, stream=side):
            for i in range(NL):
                step(i)
        launches_per_step = (ctx.kernel_launches() - l0) // NL
        if n_rem:
            rem_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(rem_graph, stream=side):
                for i in range(n_rem):
                    step(i)
            rem_graph.replay()
        for _ in range(2):
            graph.replay()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ctx.kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    if graph is not None:
        for _ in range(n_full):
            graph.replay()
        if rem_graph is not None:
            rem_graph.replay()
    else:
        for i in range(args.steps):
            step(i)
    e1.record(stream)
    barrier()
    launches = (ctx.kernel_launches() - launches0) if graph is None else launches_per_step * args.steps
    total_ms = e0.elapsed_time(e1)

    def check_status(where):
        code = ctx.device_status()
        if code != 0:
            raise RuntimeError(f"device status word {code} set during {where}")

    check_status("the timed steps")

    # ---- per-kernel timings.  All of them use a fixed number of launches, whatever --steps is.
    ev = lambda: torch.cuda.Event(enable_timing=True)
    N_ISOLATED, N_BACK_TO_BACK = 200, 50          # event pairs around single launches; repetitions over the NL layers
    exp_bytes = binding.expert_blob_bytes(layers[0].shape, shape.inter)   # bytes of one expert as it is streamed

    def graph_ms(fn, reps=200):
        """fn(i) for the NL layers captured into one CUDA graph and replayed back to back: ms per call."""
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            for i in range(NL):
                fn(i)
        stream.wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for i in range(NL):
                fn(i)
        g.replay()
        torch.cuda.synchronize()
        x0, x1 = ev(), ev()
        x0.record(stream)
        for _ in range(reps):
            g.replay()
        x1.record(stream)
        torch.cuda.synchronize()
        return x0.elapsed_time(x1) / (reps * NL)

    # every layer gets a second handle under its own context (own work list), so that back-to-back launches of the
    # expert kernel alone never wait for another layer's routing
    ctxs = [binding.Context(local) for _ in range(NL)]
    twins = [layers[i].share(ctxs[i]) for i in range(NL)]

    def measure_block(Kb, blocks_b, ys_b, rb_b):
        """The grouped-SwiGLU kernel of a verify block of Kb rows, timed three ways (same bytes, same kernel):
        pipelined  -- events around N_BACK_TO_BACK x NL back-to-back launches of the kernel alone over the rotating
                      layers: the next launch's prologue overlaps the previous launch's tail;
        isolated   -- an event pair around every single launch (launch gap and an empty pipeline included);
        as_called  -- moe_verify_block (routing + experts, overlapped) replayed from a CUDA graph: what a caller
                      gets, with the router's bytes added to the algorithmic bytes."""
        iso = []
        for i in range(N_ISOLATED):
            li = i % NL
            binding.moe_verify_route(layers[li], blocks_b[li], ys_b[li], rb_b[li])
            c, d = ev(), ev()
            c.record(stream)
            binding.moe_verify_experts(layers[li], blocks_b[li], ys_b[li])
            d.record(stream)
            iso.append((c, d))
        torch.cuda.synchronize()
        union_b = [int(rb_b[li]["union_count"].item()) for li in range(NL)]
        alg = float(np.mean([(u + shape.n_shared) * exp_bytes + 2 * Kb * H * 4 for u in union_b]))
        iso_ms = float(np.mean([x.elapsed_time(y) for x, y in iso]))
        for i in range(NL):
            binding.moe_verify_route(twins[i], blocks_b[i], ys_b[i], rb_b[i])
        for i in range(NL):
            binding.moe_verify_experts(twins[i], blocks_b[i], ys_b[i])
        torch.cuda.synchronize()
        x0, x1 = ev(), ev()
        x0.record(stream)
        for _ in range(N_BACK_TO_BACK):
            for i in range(NL):
                binding.moe_verify_experts(twins[i], blocks_b[i], ys_b[i])
        x1.record(stream)
        torch.cuda.synchronize()
        pipe_ms = x0.elapsed_time(x1) / (N_BACK_TO_BACK * NL)
        res = {"K": Kb, "union_sizes": union_b, "algorithmic_bytes_per_launch": alg,
               "launches_timed": {"pipelined": N_BACK_TO_BACK * NL, "isolated": N_ISOLATED},
               "pipelined_ms": pipe_ms, "pipelined_gbs": alg / (pipe_ms * 1e-3) / 1e9,
               "isolated_ms": iso_ms, "isolated_gbs": alg / (iso_ms * 1e-3) / 1e9}
        if not args.no_graph:
            blk_ms = graph_ms(lambda i: binding.moe_verify_block(layers[i], blocks_b[i], ys_b[i], rb_b[i]))
            blk_alg = alg - 2 * Kb * H * 4 + shape.n_experts * H * 2
            res.update({"as_called_ms": blk_ms, "as_called_gbs": blk_alg / (blk_ms * 1e-3) / 1e9,
                        "as_called_tokens_per_s": Kb / (blk_ms * 1e-3)})
        return res

    blk = measure_block(K, blocks, ys, rb)
    union = blk["union_sizes"]
    # the other end of the block-length range the target is stated for
    K8 = 8
    blk8 = None
    if K != K8 and not args.no_k8:
        blocks8 = [synth.hidden_block(K8, H, 1000 + 50 * rank + 300 + i, 0.0, device) for i in range(NL)]
        rb8 = [binding._routing_buffers(shape, K8, device) for _ in range(NL)]
        ys8 = [torch.empty((K8, H), device=device) for _ in range(NL)]
        blk8 = measure_block(K8, blocks8, ys8, rb8)
    for t in twins:
        t.close()
    for c in ctxs:
        c.close()

    # the step's kernels one by one with an event pair around each call (launch gaps included)
    t_route, t_draft, t_acc = [], [], []
    for i in range(N_ISOLATED):
        li = i % NL
        a, b, c, d, e = ev(), ev(), ev(), ev(), ev()
        a.record(stream)
        binding.moe_draft_step(layers[li], blocks[li][:1], yd, dbuf)
        b.record(stream)
        binding.moe_verify_route(layers[li], blocks[li], ys[li], rb[li])
        c.record(stream)
        binding.moe_verify_experts(layers[li], blocks[li], ys[li])
        d.record(stream)
        binding.spec_accept(ctx, ys[li], W_lm, draft_tok, True, abuf)
        e.record(stream)
        t_route.append((b, c)); t_draft.append((a, b)); t_acc.append((d, e))
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    exp_alg = [blk["algorithmic_bytes_per_launch"]]
    exp_ms = [blk["pipelined_ms"]]
    verify_gbs = blk["pipelined_gbs"]
    draft_ms = float(np.mean([x.elapsed_time(y) for x, y in t_draft]))
    route_ms = float(np.mean([x.elapsed_time(y) for x, y in t_route]))
    acc_ms = float(np.mean([x.elapsed_time(y) for x, y in t_acc]))

    # ---- each component replayed back to back from its own CUDA graph (no launch gaps, routing overlapped)
    comp = {}
    if not args.no_graph:
        comp["verify_block_ms"] = blk["as_called_ms"]
        comp["draft_step_ms"] = graph_ms(lambda i: binding.moe_draft_step(layers[i], blocks[i][:1], yd, dbuf))
        comp["accept_ms"] = graph_ms(lambda i: binding.spec_accept(ctx, ys[i], W_lm, draft_tok, True, abuf))
        comp["verify_block_gbs"] = blk["as_called_gbs"]
        comp["verify_block_frac_of_8TBs"] = comp["verify_block_gbs"] / NOMINAL_HBM_GBS
        comp["verify_block_tokens_per_s"] = K / (comp["verify_block_ms"] * 1e-3)
        comp["draft_step_gbs"] = ((shape.n_shared + 2) * exp_bytes + shape.n_experts * H * 2) / (
            comp["draft_step_ms"] * 1e-3) / 1e9
        comp["accept_gbs"] = V * H * 2 / (comp["accept_ms"] * 1e-3) / 1e9
        if args.accept_l2_mb is None:
            # the same step with the head of the LM head kept in L2 from step to step (dx_set_accept_l2_keep, off by
            # default and not part of the line's headline): reported beside it
            ctx.set_accept_l2_keep(64 * 1000 * 1000)
            graph_ms(step, reps=100)        # (what L2 holds settles over a few hundred steps)
            comp["step_ms_with_64MB_of_lm_head_kept_in_l2"] = graph_ms(step, reps=100)
            ctx.set_accept_l2_keep(0)
    draft_bytes = (shape.n_shared + 2) * exp_bytes + shape.n_experts * H * 2
    acc_bytes = V * H * 2

    # ---- end to end through the binding with host buffers (pinned), transfers inside the timed region.  Inputs (block
    # and draft tokens) sit in one pinned buffer and go to one device buffer with dx_stage_block (a kernel that reads
    # the pinned buffer through its device mapping: a copy-engine node for 32 KB costs 13 us of set-up in front of the
    # step, this 4 us).  The step's result for the host -- target tokens, accepted length, next token -- is written by
    # the accept kernel straight into a pinned host buffer; the block's output rows stay on the device, where the next
    # layer would read them.
    in_bytes, out_bytes = K * H * 4 + K * 4, K * 4 + 8
    in_host = [torch.empty((in_bytes,), dtype=torch.uint8).pin_memory() for _ in range(NL)]
    for li in range(NL):
        in_host[li][:K * H * 4].view(torch.float32).copy_(blocks[li].cpu().reshape(-1))
        in_host[li][K * H * 4:].view(torch.int32).copy_(draft_tok.cpu())
    res_host = torch.zeros((K + 2,), dtype=torch.int32).pin_memory()
    in_dev = torch.empty((in_bytes,), dtype=torch.uint8, device=device)
    h_dev = in_dev[:K * H * 4].view(torch.float32).view(K, H)
    d_dev = in_dev[K * H * 4:].view(torch.int32)
    y_e2e = torch.empty((K, H), device=device)
    abuf_e2e = {"target": res_host[:K], "n_accept": res_host[K:K + 1], "next_token": res_host[K + 1:K + 2]}

    def e2e_body(li):
        binding.stage_block(ctx, in_dev, in_host[li])
        binding.moe_draft_step(layers[li], h_dev[:1], yd, dbuf)
        binding.moe_verify_block(layers[li], h_dev, y_e2e, rb[li])
        binding.spec_accept(ctx, y_e2e, W_lm, d_dev, True, abuf_e2e)

    # one graph per layer: the host -> device transfer of the step's inputs (from fixed pinned buffers a caller would
    # fill) and the five kernels, the last of which writes the results to the host; a step = one graph launch + one sync
    e2e_graphs = None
    if not args.no_graph:
        side2 = torch.cuda.Stream(device=device)
        side2.wait_stream(stream)
        with torch.cuda.stream(side2):
            for li in range(NL):
                e2e_body(li)
        stream.wait_stream(side2)
        torch.cuda.synchronize()
        e2e_graphs = []
        for li in range(NL):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side2):
                e2e_body(li)
            e2e_graphs.append(g)

    def e2e_step(i):
        li = i % NL
        if e2e_graphs is not None:
            e2e_graphs[li].replay()
        else:
            e2e_body(li)
        stream.synchronize()

    for i in range(max(3, args.warmup)):
        e2e_step(i)
    barrier()
    g0, g1 = ev(), ev()
    g0.record(stream)
    for i in range(args.steps):
        e2e_step(i)
    g1.record(stream)
    barrier()
    e2e_ms = g0.elapsed_time(g1)
    check_status("the component timings or the end-to-end steps")
    # what came back over the link must be what the device-resident loop produced for the same layer
    li_last = (args.steps - 1) % NL
    got_y = y_e2e.cpu()
    got_t, got_n, got_next = res_host[:K].clone(), int(res_host[K]), int(res_host[K + 1])
    binding.moe_verify_block(layers[li_last], blocks[li_last], ys[li_last], rb[li_last])
    binding.spec_accept(ctx, ys[li_last], W_lm, draft_tok, True, abuf)
    torch.cuda.synchronize()
    if not torch.equal(got_t, abuf["target"].cpu()) or got_n != int(abuf["n_accept"].item()) or \
            got_next != int(abuf["next_token"].item()) or \
            (got_y - ys[li_last].cpu()).abs().max().item() > 1e-4 * ys[li_last].abs().max().item():
        raise RuntimeError("end-to-end results differ from the device-resident run")

    from paper_2607_24434_b200 import multi
    agg = multi.aggregate({"step": total_ms, "e2e": e2e_ms}, units=K * args.steps, launches=launches, device=device)
    total_ms, e2e_ms, launches = agg["step"], agg["e2e"], int(agg["launches"])
    units_all = agg["units"]

    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return
    peak, peak_kind = measured_peaks()
    value = multi.throughput(units_all, total_ms)
    # the drafter through the rotating layers chained as a stack (Eq. 5 per layer, pre-norm residual form) in one
    # persistent launch: the "draft step us per token" figure, per layer
    # (a stack as deep as the model, 26 MoE sub-layers, cycling over the rotating layers: 8 x 69 MB of drafter weights
    # are more than L2 holds, so a layer that comes round again is read from HBM again)
    NSTACK = 26
    dstack = binding.DraftStack(ctx, [layers[i % NL] for i in range(NSTACK)]) if not (args.q4_resident or args.wide) else None
    h_stack = torch.empty((1, H), device=device)

    def stack_once():
        binding.moe_draft_stack(dstack, blocks[0][:1], h_stack)

    stack_us = None
    if dstack is not None:
        side3 = torch.cuda.Stream(device=device)
        side3.wait_stream(stream)
        with torch.cuda.stream(side3):
            stack_once()
        stream.wait_stream(side3)
        torch.cuda.synchronize()
        gs = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gs, stream=side3):
            stack_once()
        for _ in range(3):
            gs.replay()
        torch.cuda.synchronize()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for _ in range(50):
            gs.replay()
        s1.record(stream)
        torch.cuda.synchronize()
        stack_us = s0.elapsed_time(s1) * 1e3 / 50
        dev_status = ctx.device_status()
        if dev_status != 0:
            raise RuntimeError(f"device status word {dev_status} set during the run (draft stack last)")
        dstack.close()

    def fractions(b):
        """The same kernel's three timings as fractions of the measured copy peak and of the nominal 8 TB/s."""
        res = {}
        for name in ("pipelined", "isolated", "as_called"):
            if name + "_gbs" in b:
                res[name] = {"ms": b[name + "_ms"], "gbs": b[name + "_gbs"], "of_peak": b[name + "_gbs"] / peak,
                             "of_nominal_8TBs": b[name + "_gbs"] / NOMINAL_HBM_GBS}
        return res

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("4-bit block-quantised experts (fp16 scale per 32 weights) de-quantised in the kernel, bf16 router "
                  "and LM head, fp32 accumulate") if args.q4_resident else (
                      "bf16 weights, activations as bf16 tensor-core operands, fp32 accumulate"),
        "data": "synthetic",
        "config": workload_config(shape, K, V, NL, exp_bytes, world, args.q4_resident),
        "launch": "CUDA graph replay" if graph is not None else "eager launches",
        "gpu_launches": launches,
        "e2e": {"value": multi.throughput(units_all, e2e_ms), "unit": UNIT,
                "h2d_bytes_per_step": K * H * 4 + K * 4, "d2h_bytes_per_step": K * 4 + 8,
                "ms_per_step": e2e_ms / args.steps,
                "transfers": "inputs (block rows, draft tokens): pinned host buffer -> device by dx_stage_block; result "
                             "(target tokens, accepted length, next token): written by the accept kernel into a pinned "
                             "host buffer; the block's output rows stay on the device",
                "launch": ("one CUDA graph launch (input transfer, five kernels) and one stream "
                           "synchronisation per step") if e2e_graphs is not None else
                          "eager calls and one stream synchronisation per step"},
        "roofline": {"kernel": ("dx_experts_wide_kernel (grouped SwiGLU of the verify block, tcgen05)" if args.wide else
                                "dx_experts_bf16_kernel (grouped SwiGLU of the verify block)"), "bound": "hbm",
                     "achieved": verify_gbs, "peak": peak, "unit": "GB/s", "frac": verify_gbs / peak,
                     "frac_is": "pipelined: the kernel alone, back-to-back launches (see `fractions` for the other two "
                                "ways of timing the same kernel; this is the most favourable of the three)",
                     "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": verify_gbs / NOMINAL_HBM_GBS,
                     "fractions": fractions(blk),
                     "traffic": args.traffic if args.traffic is not None else (
                         None if (args.q4_resident or args.wide) else NCU_TRAFFIC_RATIO * float(np.mean(exp_alg))),
                     "traffic_source": "ncu capture of a 2-layer case scaled by algorithmic bytes (see profiles/)",
                     "ms_per_launch": blk["pipelined_ms"],
                     "ms_per_launch_isolated": blk["isolated_ms"],
                     "launches_timed": blk["launches_timed"],
                     "timing": "CUDA events on the launch stream; a fixed number of launches whatever --steps is.  "
                               "pipelined: events around back-to-back launches of the kernel alone over the rotating "
                               "layers (the next launch's prologue overlaps the previous one's tail); isolated: an "
                               "event pair around every single launch (launch gap included); as_called: "
                               "moe_verify_block (routing + experts) replayed from a CUDA graph, router bytes added",
                     "algorithmic_bytes_per_launch": float(np.mean(exp_alg)), "union_sizes": union,
                     "k8": None if blk8 is None else dict(blk8, fractions=fractions(blk8)),
                     # the other kernels of the step, each timed back to back from its own graph, same peak
                     "others": {
                         "dx_accept_ring_kernel (greedy accept, LM head streamed once)": {
                             "ms_per_launch": comp.get("accept_ms", acc_ms),
                             "achieved": acc_bytes / (comp.get("accept_ms", acc_ms) * 1e-3) / 1e9,
                             "frac": acc_bytes / (comp.get("accept_ms", acc_ms) * 1e-3) / 1e9 / peak},
                         "draft step (routing + expert kernel, one token)": {
                             "ms_per_launch": comp.get("draft_step_ms", draft_ms),
                             "achieved": draft_bytes / (comp.get("draft_step_ms", draft_ms) * 1e-3) / 1e9,
                             "frac": draft_bytes / (comp.get("draft_step_ms", draft_ms) * 1e-3) / 1e9 / peak}}},
        "kernels": {"verify_experts_ms": float(np.mean(exp_ms)), "verify_route_ms": route_ms,
                    "verify_tokens_per_s": K / ((float(np.mean(exp_ms)) + route_ms) * 1e-3),
                    "draft_step_us": draft_ms * 1e3, "draft_gbs": draft_bytes / (draft_ms * 1e-3) / 1e9,
                    "draft_frac_of_peak": draft_bytes / (draft_ms * 1e-3) / 1e9 / peak,
                    "accept_ms": acc_ms, "accept_gbs": acc_bytes / (acc_ms * 1e-3) / 1e9,
                    "accept_frac_of_peak": acc_bytes / (acc_ms * 1e-3) / 1e9 / peak},
        "graph_components": comp,
        "draft_stack": None if stack_us is None else {
            "layers": NSTACK, "us_per_token": stack_us, "us_per_layer": stack_us / NSTACK,
            "gbs": NSTACK * draft_bytes / (stack_us * 1e-6) / 1e9,
            "frac_of_nominal_8TBs": NSTACK * draft_bytes / (stack_us * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
            "path": f"moe_draft_stack: {NSTACK} sub-layers (the model's depth) cycling over the {NL} rotating layers, "
                    "one persistent cooperative launch per token (CUDA graph replay, 50 tokens)"},
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline and not args.q4_resident:
        out["cpu_baseline"] = cpu_baseline(shape, K, V)
    print(json.dumps(out))
    if world > 1:
        torch.distributed.destroy_process_group()


def run_stack(args):
    """configs[2] / configs[3]: a stack of MoE sub-layers (attention stubbed out, pre-norm residual form) with all
    experts resident.  The draft stack is timed per token; the verify stack (routing + grouped SwiGLU per layer,
    then greedy accept on the normalised final rows) is timed for K in {1, 2, 4, 8, 16} with block rows that follow
    an AR(1) process (rho 0.9), and the union sizes per layer are reported with the bytes they imply."""
    from paper_2607_24434_b200 import binding
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    shape = synth.shape_moonlight() if args.moonlight else synth.shape_v2lite()
    if args.wide:
        import dataclasses
        shape = dataclasses.replace(shape, weight_dtype=synth.DTYPE_BF16_WIDE)
    V = 163840 if args.moonlight else args.vocab
    NLAY, H = args.stack_layers, shape.hidden
    ctx = binding.Context(0)
    layers = []
    for l in range(NLAY):
        w = synth.make_layer(shape, 7000 + l, device, zipf=args.zipf)
        if args.q4_resident:
            w = synth.quantize_layer(w)
        layers.append(binding.Layer.from_weights(ctx, w))
        torch.cuda.synchronize()
        del w
    torch.cuda.empty_cache()
    W_lm = synth.lm_head(V, H, 7999, torch.bfloat16, device)
    exp_bytes = binding.expert_blob_bytes(layers[0].shape, shape.inter)   # as streamed (bf16 or 4-bit units)
    peak, peak_kind = measured_peaks()
    stream = torch.cuda.current_stream()

    def timed_graph(body, reps):
        side = torch.cuda.Stream(device=device)
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            body()
        stream.wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            body()
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    # ---- draft stack: one token through all layers
    hd = [torch.empty((1, H), device=device) for _ in range(NLAY + 1)]
    hd[0].copy_(synth.hidden_block(1, H, 7100, 0.0, device))
    db = [{"topk_ids": torch.empty((shape.top_k,), dtype=torch.int32, device=device),
           "topk_w": torch.empty((shape.top_k,), dtype=torch.float32, device=device)} for _ in range(NLAY)]

    def draft_body():
        for l in range(NLAY):
            binding.moe_draft_step_residual(layers[l], hd[l], hd[l + 1], db[l])

    chain_ms = timed_graph(draft_body, args.stack_reps)
    # ... and the same chain as one persistent launch (streaming blob layout only)
    if args.wide:
        draft_ms, same_ids, drift = chain_ms, True, 0.0
    else:
        dstack = binding.DraftStack(ctx, layers)
        sb = {"topk_ids": torch.empty((NLAY, shape.top_k), dtype=torch.int32, device=device),
              "topk_w": torch.empty((NLAY, shape.top_k), dtype=torch.float32, device=device)}
        h_stack = torch.empty((1, H), device=device)

        def stack_body():
            binding.moe_draft_stack(dstack, hd[0], h_stack, sb)

        draft_ms = timed_graph(stack_body, args.stack_reps)
        if ctx.device_status() != 0:
            raise RuntimeError("device status word set during the draft stack")
        same_ids = all(torch.equal(sb["topk_ids"][l], db[l]["topk_ids"]) for l in range(NLAY))
        drift = float(((h_stack - hd[NLAY]).norm() / hd[NLAY].norm()).item())
    draft_bytes = NLAY * ((shape.n_shared + 2) * exp_bytes + shape.n_experts * H * 2)
    out = {"metric": "draft_stack_us_per_token", "value": draft_ms * 1e3, "unit": "us/token", "n_gpus": 1,
           "higher_is_better": False, "data": "synthetic",
           "dtype": "4-bit block-quantised experts, fp32 accumulate" if args.q4_resident else
                    "bf16 weights, fp32 accumulate",
           "config": {"workload": f"{'configs[3] Moonlight' if args.moonlight else 'configs[2] DeepSeek-V2-Lite'}-shaped "
                                  f"stack of {NLAY} MoE sub-layers, experts resident "
                                  f"({NLAY * (shape.n_experts + shape.n_shared + 1) * exp_bytes / 1e9:.1f} GB), "
                                  f"AR(1) block rows (rho 0.9), Zipf router bias {'on' if args.zipf else 'off'}, "
                                  f"vocab {V}; CUDA graph replay, {args.stack_reps} timed replays per point",
                      "layers": NLAY},
           "draft_gbs": draft_bytes / (draft_ms * 1e-3) / 1e9,
           "draft_frac_of_8TBs": draft_bytes / (draft_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
           "draft_us_per_layer": draft_ms * 1e3 / NLAY,
           "draft_path": "per-layer launch chain (wide blob layout)" if args.wide else
                         "one persistent cooperative launch for the whole stack",
           "per_layer_launch_chain_us_per_token": chain_ms * 1e3,
           "chain_agreement": {"same_selection": bool(same_ids), "rel_l2_diff": drift}, "peak_gbs": peak, "peak_kind": peak_kind, "verify": []}
    # ---- the comparison axes of the paper's draft-side table on these synthetic weights: the training-free
    # shared + top-r self-drafters (r = 1, 2, 3) and the fixed-footprint drafter, a block of 4 draft tokens each:
    # unique routed (layer, expert) pairs the drafter reads, and its time per token relative to shared + top-1
    if args.drafters:
        KD = 4
        rows = synth.hidden_block(KD, H, 7300, 0.9, device)     # consecutive tokens' inputs: AR(1), rho 0.9
        variants = [("shared + top-1", 1, False), ("shared + top-2", 2, False), ("shared + top-3", 3, False),
                    ("DraftExpert (shared + top-1 + draft expert)", 1, True)]
        table = []
        for name, r_top, use_draft in variants:
            hx = [torch.empty((1, H), device=device) for _ in range(NLAY + 1)]

            def body():
                for l in range(NLAY):
                    binding.moe_draft_step_topr_residual(layers[l], hx[l], hx[l + 1], r_top, use_draft, db[l])

            touched = set()
            for t in range(KD):
                hx[0].copy_(rows[t:t + 1])
                body()
                torch.cuda.synchronize()
                for l in range(NLAY):
                    touched |= {(l, int(e)) for e in db[l]["topk_ids"][:r_top].tolist()}
            ms = timed_graph(body, args.stack_reps)
            table.append({"drafter": name, "unique_layer_experts": len(touched), "max_possible": KD * NLAY * r_top,
                          "us_per_token": ms * 1e3})
        base = table[0]["us_per_token"]
        for row in table:
            row["cost_vs_shared_top1"] = row["us_per_token"] / base
        out["drafters"] = {"block_tokens": KD, "layers": NLAY, "rows": table,
                           "paper_context": "Table 3 (trained draft experts, real text, K = 4, 26 MoE layers): unique "
                                            "layer-experts 84 / 183 / 244 / 88, draft cost 1.00 / - / - / 1.05-1.08 for "
                                            "top-1 / top-2 / top-3 / DraftExpert; context only, other weights and data",
                           "note": "synthetic weights and AR(1) inputs; the AR baseline is the K = 1 entry of `verify`"}
        if ctx.device_status() != 0:
            raise RuntimeError("device status word set during the drafter comparison")
    # ---- verify stack for every block length
    for K in (1, 2, 4, 8, 16):
        hs = [torch.empty((K, H), device=device) for _ in range(NLAY + 1)]
        hs[0].copy_(synth.hidden_block(K, H, 7200 + K, 0.9, device))
        rb = [binding._routing_buffers(shape, K, device) for _ in range(NLAY)]
        draft_tok = torch.zeros((K,), dtype=torch.int32, device=device)
        abuf = {"target": torch.empty((K,), dtype=torch.int32, device=device),
                "n_accept": torch.empty((1,), dtype=torch.int32, device=device),
                "next_token": torch.empty((1,), dtype=torch.int32, device=device)}

        def layers_body():
            for l in range(NLAY):
                binding.moe_verify_block_residual(layers[l], hs[l], hs[l + 1], rb[l])

        def accept_body():
            binding.spec_accept(ctx, hs[NLAY], W_lm, draft_tok, True, abuf)

        ms_layers = timed_graph(layers_body, args.stack_reps)
        ms_accept = timed_graph(accept_body, args.stack_reps)
        if ctx.device_status() != 0:
            raise RuntimeError("device status word set during the stack run")
        unions = [int(rb[l]["union_count"].item()) for l in range(NLAY)]
        vbytes = sum((u + shape.n_shared) * exp_bytes + shape.n_experts * H * 2 for u in unions)
        out["verify"].append({
            "K": K, "stack_ms": ms_layers, "accept_ms": ms_accept,
            "tokens_per_s": K / ((ms_layers + ms_accept) * 1e-3),
            "union_mean": float(np.mean(unions)), "union_min": min(unions), "union_max": max(unions),
            "layers_gbs": vbytes / (ms_layers * 1e-3) / 1e9,
            "layers_frac_of_8TBs": vbytes / (ms_layers * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            "layers_frac_of_measured": vbytes / (ms_layers * 1e-3) / 1e9 / peak,
            "accept_gbs": V * H * 2 / (ms_accept * 1e-3) / 1e9})
        del hs, rb
    print(json.dumps(out))


def run_offload(args):
    """configs[4]: offloaded V2-Lite-shaped stack, one exact DraftExpert decode step per iteration (Algorithm 1).
    Routed experts live in pinned host memory; each layer has an HBM cache of 16 slots with LRU eviction; shared and
    draft experts are resident.  Per step: draft tokens go one by one through the drafter's stack (chained residual
    stream, top-1 expert staged on demand), each is scored by the draft LM head, the confidence-expansion controller
    decides whether to keep it, and the newly predicted verifier experts are prefetched on the side stream; then the
    block is verified through the target stack (route, read the union on the host, wait for useful transfers, load
    misses on demand, waves if the union exceeds the slots) and greedily accepted.  The drafter's hidden states
    differ from the verifier's from the second layer on, so its router's predictions can miss.  Two acceptance
    modes: scripted geometric(0.85) (the draft experts are random, not trained) and closed-loop (the comparison's
    own accepted length).  The routing decisions are read on the host (one sync per layer), which is the
    serialisation on-demand loading inherently has; the workload is bound by the host link by construction."""
    from paper_2607_24434_b200 import binding, decode
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    shape = synth.shape_v2lite()
    NLAY, S, V, H = args.offload_layers, args.slots, args.vocab, shape.hidden
    ctx = binding.Context(0)
    nbytes = binding.expert_blob_bytes(shape, shape.inter)
    pool_bytes = binding.q4_expert_bytes(shape, shape.inter) if args.q4 else nbytes
    # the host pool first: if the box cannot pin it all, fewer layers are used (and reported)
    pools = []
    for l in range(NLAY):
        try:
            pools.append(torch.empty((shape.n_experts, pool_bytes), dtype=torch.uint8).pin_memory())
        except RuntimeError:
            break
    if len(pools) < NLAY:
        sys.stderr.write(f"could pin only {len(pools)} of {NLAY} layers' experts; running with that many\n")
        NLAY = len(pools)
    cache = binding.ExpertCache(ctx, NLAY, shape.n_experts, S, nbytes)
    if args.q4:
        cache.set_q4(shape)      # host pool of 4-bit block-quantised experts, expanded into the slots after each copy
    layers = []
    for l in range(NLAY):
        w = synth.make_layer(shape, 3000 + l, device, zipf=True)
        L = binding.Layer.from_weights(ctx, w, routed_resident=False)
        torch.cuda.synchronize()
        if args.q4:
            Wg, Wu, Wd = w["experts"]
            for e in range(shape.n_experts):
                pools[l][e].copy_(synth.q4_expert_blob(Wg[e].float().cpu(), Wu[e].float().cpu(), Wd[e].float().cpu()))
        else:
            pools[l].copy_(L.blobs)
        L.blobs = None
        del w
        for e in range(shape.n_experts):
            cache.register(l, e, pools[l][e])
        cache.attach(L, l)
        layers.append(L)
    torch.cuda.empty_cache()
    emb = synth.embedding_table(V, H, 3998, device)
    W_lm = synth.lm_head(V, H, 3999, torch.bfloat16, device)
    dec = decode.OffloadedDecoder(ctx, layers, cache, emb, W_lm, k_max=args.k_max, tau=args.tau,
                                  budget="cache" if args.budget < 0 else args.budget, native=not args.python_loop)
    rng = np.random.default_rng(11)

    def scripted():
        n = 0
        while n < args.k_max and rng.random() < 0.85:
            n += 1
        return n

    closed = args.acceptance == "closed-loop"
    t0_tok = 1
    for i in range(args.warmup):
        t0_tok = dec.step(t0_tok, scripted_accept=None if closed else scripted())["next"]
    torch.cuda.synchronize()
    st0 = cache.stats()
    t0 = time.perf_counter()
    accepted = emitted = drafted = rows = 0
    union_sum = np.zeros(NLAY)
    for i in range(args.offload_steps):
        r = dec.step(t0_tok, scripted_accept=None if closed else scripted())
        t0_tok = r["next"]
        union_sum += np.asarray(r["union_sizes"])
        accepted += r["n_accept"]; emitted += len(r["emitted"]); drafted += len(r["drafted"]); rows += r["block_rows"]
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    if ctx.device_status() != 0:
        raise RuntimeError("device status word set during the offload run")
    st1 = cache.stats()
    d = {k: st1[k] - st0[k] for k in st1}
    steps = args.offload_steps
    print(json.dumps({
        "metric": "offload_accepted_tokens_per_s", "value": accepted / dt, "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": args.warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "data": "synthetic",
        "dtype": "bf16 weights, fp32 accumulate",
        "config": {"workload": f"configs[4]: offloaded V2-Lite-shaped stack, {NLAY} MoE layers, experts in pinned host "
                               f"memory ({NLAY * shape.n_experts * pool_bytes / 1e9:.1f} GB, "
                               f"{'4-bit block-quantised, expanded to bf16 after each copy' if args.q4 else 'bf16 blobs'}), "
                               f"{S} HBM slots per layer (LRU); per step: draft up to {args.k_max} tokens through the "
                               f"drafter's stack (chained residual stream), confidence-expansion controller "
                               f"(tau {args.tau}, budget {'= free cache pairs' if args.budget < 0 else args.budget}), "
                               f"prefetch of the newly predicted top-{shape.top_k} experts, verify through the target "
                               f"stack in waves, greedy accept over vocab {V}",
                   "layers": NLAY, "layers_requested": args.offload_layers, "k_max": args.k_max,
                   "acceptance": "closed-loop (token chain through a seeded embedding table; random draft experts)"
                                 if closed else "scripted geometric(0.85) prefix (stand-in for trained draft experts)"},
        "emitted_tokens_per_s": emitted / dt,
        "drafted_per_step": drafted / steps, "block_rows_per_step": rows / steps,
        "acceptance_rate": accepted / max(1, drafted),
        "cache_hit_rate": d["hits"] / max(1, d["lookups"]),
        "prefetch_hit": d["prefetch_used"] / max(1, d["prefetch_issued"]),
        "prefetch_waste": d["prefetch_wasted"] / max(1, d["prefetch_issued"]),
        "prefetch_note": "used / wasted are counted when they happen; experts prefetched in the last step and still "
                         "pending are in neither",
        "h2d_gbs": d["bytes_h2d"] / dt / 1e9, "waited_copies_per_step": d["waited_copies"] / steps,
        "stream_wait_for_copies_ms_per_step": d["stream_stall_ns"] / steps / 1e6, "cache": d,
        "union_size_per_layer_mean": [round(float(u) / steps, 2) for u in union_sum],
    }))
    dec.close()


def _blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def oracle_step(O, ref, h_np, W_np, draft, K):
    """The same step on the CPU checker, as it stands: draft step, verify block, greedy accept."""
    O.moe_draft(h_np[:1], ref)
    y = O.moe_target(h_np, ref)[0]
    return O.greedy_accept_fast(O.rmsnorm(y), W_np, draft)


def cpu_baseline(shape, K, V, budget_s=12.0):
    """Times the CPU checker, as it stands, on a bounded sample of the workload: whole steps (draft step + verify
    block + greedy accept over the full vocabulary) on one layer, repeated for about ``budget_s`` seconds."""
    from oracle import moe_oracle as O
    layer = synth.make_layer(shape, 4242, "cpu", zipf=True)
    ref = synth.layer_to_numpy(layer)
    del layer
    h_np = synth.hidden_block(K, shape.hidden, 4243, 0.0).numpy().astype(np.float64)
    W_np = synth.to_numpy_f32(synth.lm_head(V, shape.hidden, 4244, torch.bfloat16)).astype(np.float64)
    draft = np.zeros(K, np.int32)
    oracle_step(O, ref, h_np, W_np, draft, K)          # untimed first touch
    n, t0 = 0, time.perf_counter()
    while True:
        oracle_step(O, ref, h_np, W_np, draft, K)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or n >= 200:
            break
    return {"value": K * n / dt, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle", "dtype": "f64",
            "seconds": dt, "steps": n,
            "sample": f"{n} whole steps on one layer of the {shape.n_experts}-expert shape: draft step + verify block "
                      f"K={K} + greedy accept over all {V} vocabulary rows (the checker's default fp64 numpy "
                      f"arithmetic, {dt:.1f} s of CPU work)"}


def workload_config(shape, K, V, NL, exp_bytes, world=1, q4=False):
    """The `config` object of the JSON line: the same for the GPU arm and the reference arm."""
    return {"workload": "configs[1]: DeepSeek-V2-Lite-shaped MoE layer (H 2048, 64 experts x 1408, top-6, "
                        "2 shared + 1 draft expert, Zipf(1.1) router bias); step = draft step (1 token) + "
                        f"verify block K={K} + greedy accept over vocab {V}"
                        + ("; experts resident in HBM as 4-bit blocks" if q4 else ""),
            "block_tokens": K, "vocab": V, "layers_rotated": NL,
            "l2": f"inputs larger than L2: steps rotate over {NL} independently seeded layers "
                  f"({NL * (shape.n_experts + shape.n_shared + 1) * exp_bytes / 1e9:.1f} GB of weights)",
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def run_reference(args):
    """The reference arm: the CPU checker, as it stands, on the host cores (rank 0 only), on the GPU arm's
    configuration: the same seeded layers rotated in the same order, the same block length, the full vocabulary."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import moe_oracle as O
    shape = synth.shape_v2lite()
    K, V, n_layers = args.block, args.vocab, args.layers
    refs, hs = [], []
    for i in range(n_layers):
        layer = synth.make_layer(shape, 1000 + i, "cpu", zipf=True)
        refs.append(synth.layer_to_numpy(layer))
        del layer
        hs.append(synth.hidden_block(K, shape.hidden, 1100 + i, 0.0).numpy().astype(np.float64))
    W_np = synth.to_numpy_f32(synth.lm_head(V, shape.hidden, 1999, torch.bfloat16)).astype(np.float64)
    draft = np.zeros(K, np.int32)
    # bounded: the checker is slow by design, so at most ~2 minutes of it are timed
    budget_s, t_w = 120.0, time.perf_counter()
    n_warm = max(1, min(args.warmup, n_layers))
    for i in range(n_warm):
        oracle_step(O, refs[i % n_layers], hs[i % n_layers], W_np, draft, K)
    per_step = (time.perf_counter() - t_w) / n_warm
    timed = max(1, min(args.steps, int(budget_s / max(per_step, 1e-3))))
    t0 = time.perf_counter()
    for i in range(timed):
        oracle_step(O, refs[i % n_layers], hs[i % n_layers], W_np, draft, K)
    dt = time.perf_counter() - t0
    value = K * timed / dt
    sample = (f"each step: draft step + verify block K={K} on one of {n_layers} rotating layers + greedy accept over "
              f"all {V} vocabulary rows (the checker's default fp64 numpy arithmetic)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get(
            "WORLD_SIZE", "1")), "steps": args.steps, "steps_timed": timed, "warmup": args.warmup, "ms_per_step": dt / timed * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(shape, K, V, n_layers, shape.expert_bytes()),
        "launch": "host cores (numpy)",
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle", "dtype": "f64",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def spawn_replicas(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this script (one per GPU, replicas only)
    under torch.distributed.run on this node and hand back its exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1,
                    help="GPUs of this node, one replica each; under torchrun the ranks come from the environment, "
                         "without a launcher N > 1 ranks are spawned here")
    ap.add_argument("--steps", type=int, default=8000)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--block", type=int, default=4, help="verify block length K")
    ap.add_argument("--vocab", type=int, default=102400)
    ap.add_argument("--layers", type=int, default=8, help="independently seeded layers to rotate over")
    ap.add_argument("--no-k8", action="store_true", help="skip the K = 8 figures of the dominant kernel")
    ap.add_argument("--launch-overlap", type=int, default=None,
                    help="dx_set_launch_overlap mask (bit 0 routing, 1 experts, 2 greedy accept; library default 3)")
    ap.add_argument("--accept-l2-mb", type=float, default=None,
                    help="dx_set_accept_l2_keep: MB at the head of the LM head kept in L2 between steps (library default 0)")
    ap.add_argument("--wide", action="store_true",
                    help="layer / stack workloads: experts in the wide blob layout (tcgen05 kernel, any block length)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of a CUDA graph replay")
    ap.add_argument("--stack-layers", type=int, default=26)
    ap.add_argument("--stack-reps", type=int, default=20)
    ap.add_argument("--moonlight", action="store_true", help="stack workload: Moonlight shapes (sigmoid router, vocab 163840)")
    ap.add_argument("--zipf", action="store_true", help="stack workload: Zipf(1.1) router bias")
    ap.add_argument("--drafters", action="store_true",
                    help="stack workload: shared + top-r self-drafters against the fixed-footprint drafter")
    ap.add_argument("--workload", default="layer", choices=["layer", "offload", "stack"],
                    help="layer: configs[1] (default, the driver's line); offload: configs[4] expert-cache workload; "
                         "stack: configs[2] / configs[3] layer stacks, K sweep and draft us per token")
    ap.add_argument("--offload-layers", type=int, default=26)
    ap.add_argument("--k-max", type=int, default=8, help="offload workload: most tokens drafted per step")
    ap.add_argument("--tau", type=float, default=1.0, help="offload workload: confidence threshold of the stop rule")
    ap.add_argument("--budget", type=int, default=-1,
                    help="offload workload: layer-expert budget of the stop rule (-1: what is left of the cache)")
    ap.add_argument("--acceptance", default="scripted", choices=["scripted", "closed-loop"])
    ap.add_argument("--q4", action="store_true",
                    help="offload workload: keep the host pool 4-bit block-quantised (Q4_0 blocks)")
    ap.add_argument("--q4-resident", action="store_true",
                    help="layer workload: experts resident in HBM as 4-bit blocks, de-quantised in the expert kernel")
    ap.add_argument("--offload-steps", type=int, default=64)
    ap.add_argument("--slots", type=int, default=16, help="offload workload: HBM cache slots per layer")
    ap.add_argument("--python-loop", action="store_true",
                    help="offload workload: the decode step's host loop in Python (decode.py) instead of dx_decoder_step")
    ap.add_argument("--traffic", type=float, default=None,
                    help="ncu DRAM bytes per launch of the dominant kernel, if known")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus > 1 and "RANK" not in os.environ and args.impl != "reference":
        sys.exit(spawn_replicas(args.gpus))
    if args.workload == "offload" and args.impl != "reference":
        run_offload(args)
    elif args.workload == "stack" and args.impl != "reference":
        run_stack(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
