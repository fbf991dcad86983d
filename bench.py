#!/usr/bin/env python
"""Benchmark of the mixed-format (FP8 + TQ3) paged decode path on B200.

One step = one decode step of the whole hot path over the batch, for every layer of the workload:
Append of the new token's K/V into the Recent FP8 page, Demote (FP8 -> TQ3, publish) of the page
that leaves the Recent window when one does, and
mkv_decode_attention (table walk, query rotation, FP8 and TQ3 page scans, split partials, merge).
Default workload: 2 requests x 59,008 tokens, 16 layers each with its own pool, d = 256,
4 KV x 6 query heads, first 256 tokens Anchor, last 2,048 Recent, the rest TQ3.

Prints ONE JSON line (rank 0).  `value` is decode tokens/s with everything resident in HBM;
`e2e` is the same metric with the step's inputs copied from pinned host memory and its outputs read
back inside the timed region; `roofline` is achieved KV GB/s of the decode kernel against the
measured HBM copy bandwidth; `cpu_baseline` is the fp64 CPU oracle timed on a bounded sample.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 0..4]
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import mkv_workloads as W  # noqa: E402

METRIC = "decode attention tokens/s and achieved KV HBM GB/s (% of B200 peak) at 1 GPU"
UNIT = "tokens/s"
# DRAM traffic of the decode kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture) is kept
# as data beside the profile summaries; the line reports it only for the workload and format it was taken on.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")
FALLBACK_HBM_GBS = 6650.0
STAGE_PAGES = 512


def traffic_per_launch(workload_key, layers_per_launch):
    """DRAM bytes of one decode launch from the recorded capture (per layer, scaled to the layers of a launch:
    the scan reads every page once, so traffic grows in proportion), or None when no capture covers the workload."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(workload_key)
    except (OSError, ValueError):
        return None
    if not rec:
        return None
    return int((rec["dram_read_bytes_per_layer"] + rec["dram_write_bytes_per_layer"]) * layers_per_launch)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()          # the exact child started above
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self):
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(values, device=None):
    """MAX over the ranks of every entry (the step time of a multi-replica run is the slowest replica's)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_value(batch_per_replica, steps, ms, world):
    """Whole-job tokens/s of `world` independent replicas that each decode `batch_per_replica` tokens per step."""
    return world * batch_per_replica * steps / (ms * 1e-3)


# --------------------------------------------------------------------------------------------- ours
class LayerState:
    pass


def build_layers(spec, steps_total, device, M, torch, spec_format=1):
    """Pools of every layer filled through the library's own Append and Demote kernels from seeded
    synthetic bf16 K/V, plus the tables, slots and retier plan of every timed step."""
    B, d, hkv, hq = spec.batch, spec.head_dim, spec.n_kv_heads, spec.n_q_heads
    T = spec.page_tokens                      # 16, or 16 M for the paper-scale pages
    stage_pages = max(1, STAGE_PAGES * 16 // T)
    final_lens = [n + steps_total for n in spec.seq_lens]
    max_pages = max((n + T - 1) // T for n in final_lens) + 1
    tab0 = W.tables(spec)
    n_fp8_0, n_tq3_0 = tab0.fp8_pages, tab0.tq3_pages
    extra_pages = sum((fl + T - 1) // T - (n + T - 1) // T for fl, n in zip(final_lens, spec.seq_lens))
    demotes_per_req = steps_total // T + 2
    fp8_cap = n_fp8_0 + extra_pages + stage_pages + 8
    tq3_cap = n_tq3_0 + B * demotes_per_req + 8

    # host plan shared by all layers: table, tags, per-step slots and retier events
    bt = np.full((B, max_pages), -1, np.int32)
    tg = np.zeros((B, max_pages), np.uint8)
    bt[:, :tab0.block_table.shape[1]] = tab0.block_table
    tg[:, :tab0.tier_tag.shape[1]] = tab0.tier_tag
    next_fp8, next_tq3 = n_fp8_0, n_tq3_0
    lens = np.array(spec.seq_lens, np.int64)
    n_pages = (lens + T - 1) // T
    slots = np.zeros((steps_total, B), np.int32)
    lens_steps = np.zeros((steps_total, B), np.int32)
    events = []              # per step: list of (b, logical page, src fp8 id, dst tq3 id)
    recent = spec.recent_tokens if spec.stale_fraction is None else int(round((1 - spec.stale_fraction) * lens[0]))
    for st in range(steps_total):
        ev = []
        for b in range(B):
            if lens[b] % T == 0:                        # Append opens a Recent page
                bt[b, n_pages[b]] = next_fp8
                tg[b, n_pages[b]] = W.TAG_RECENT
                next_fp8 += 1
                n_pages[b] += 1
            slots[st, b] = bt[b, lens[b] // T] * T + lens[b] % T
            lens[b] += 1
            lens_steps[st, b] = lens[b]
            # age: a full Recent page wholly before the window is demoted (tags tracked on the host too)
            first_recent = max(0, lens[b] - recent) // T
            for lp in range(max(0, first_recent - 2), first_recent):
                if tg[b, lp] == W.TAG_RECENT:
                    ev.append((b, lp, int(bt[b, lp]), next_tq3))
                    tg[b, lp] = W.TAG_STALE
                    bt[b, lp] = next_tq3
                    next_tq3 += 1
        events.append(ev)
    assert next_fp8 <= fp8_cap - stage_pages and next_tq3 <= tq3_cap

    layers = []
    gen = torch.Generator(device=device)
    for layer in range(spec.n_layers):
        L = LayerState()
        sigma = W.rotation_signs(spec, layer)
        L.pool = M.Pool(d, hkv, hq, fp8_cap, tq3_cap, sigma, max_batch=B, device=device, page_tokens=T,
                        tq3_format=spec_format)
        gen.manual_seed(1000 * spec.seed + layer)
        k_out = torch.from_numpy(W.outlier_channels(spec, layer, 0)).to(device)
        v_out = torch.from_numpy(W.outlier_channels(spec, layer, 1)).to(device)

        def synth(n_tok):
            k = torch.randn((n_tok, hkv, d), generator=gen, device=device, dtype=torch.float32)
            v = torch.randn((n_tok, hkv, d), generator=gen, device=device, dtype=torch.float32)
            k[:, :, k_out] *= 8.0
            v[:, :, v_out] *= 8.0
            return k.to(torch.bfloat16).contiguous(), v.to(torch.bfloat16).contiguous()

        stage0 = fp8_cap - stage_pages
        for b in range(B):
            npg = (spec.seq_lens[b] + T - 1) // T
            tags_b, ids_b = tab0.tier_tag[b, :npg], tab0.block_table[b, :npg]
            fp8_lp = np.nonzero(tags_b != W.TAG_STALE)[0]
            # Recent/Anchor pages: append straight into their pages
            tok = np.concatenate([np.arange(lp * T, min(lp * T + T, spec.seq_lens[b])) for lp in fp8_lp]) \
                if len(fp8_lp) else np.zeros(0, np.int64)
            if len(tok):
                sm = (ids_b[tok // T].astype(np.int64) * T + tok % T).astype(np.int32)
                k, v = synth(len(tok))
                L.pool.append(k, v, torch.from_numpy(sm).to(device))
            # Stale pages: append into staging FP8 pages, demote into their TQ3 pages, reuse the staging pages
            st_lp = np.nonzero(tags_b == W.TAG_STALE)[0]
            for c0 in range(0, len(st_lp), stage_pages):
                chunk = st_lp[c0:c0 + stage_pages]
                n = len(chunk)
                sm = ((stage0 + np.arange(n))[:, None] * T + np.arange(T)[None, :]).reshape(-1).astype(np.int32)
                k, v = synth(T * n)
                L.pool.append(k, v, torch.from_numpy(sm).to(device))
                src = torch.arange(stage0, stage0 + n, dtype=torch.int32, device=device)
                dst = torch.from_numpy(ids_b[chunk].astype(np.int32)).to(device)
                L.pool.demote(src, dst)
        torch.cuda.synchronize(device)
        if L.pool.status() != M.OK:
            raise RuntimeError("pool status after fill")
        # future Recent pages are already named in the table (decode reads only ceil(len/16) entries)
        L.bt = torch.from_numpy(initial_table(tab0, bt)).to(device)
        L.tags = torch.from_numpy(initial_tags(tab0, tg)).to(device)
        L.q = torch.randn((B, hq, d), generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
        L.k_new, L.v_new = synth(B)
        L.out = torch.empty((B, hq, d), dtype=torch.float32, device=device)
        layers.append(L)
    plan = {
        "slots": torch.from_numpy(slots).to(device), "lens": torch.from_numpy(lens_steps).to(device),
        "events": events, "max_pages": max_pages, "lens_host": lens_steps, "slots_host": slots,
    }
    # device-side arguments of every retier event
    plan["ev_dev"] = []
    for ev in events:
        if not ev:
            plan["ev_dev"].append(None)
            continue
        src = torch.tensor([e[2] for e in ev], dtype=torch.int32, device=device)
        dst = torch.tensor([e[3] for e in ev], dtype=torch.int32, device=device)
        ent = torch.tensor([e[0] * max_pages + e[1] for e in ev], dtype=torch.int64, device=device)
        plan["ev_dev"].append((src, dst, ent, [e[0] * max_pages + e[1] + 1 for e in ev]))
    return layers, plan, tab0


def initial_table(tab0, bt_final):
    """Table at time zero: the initial mapping, plus the ids of pages that Append will open later;
    entries that Demote will rewrite keep their initial FP8 ids."""
    out = bt_final.copy()
    w = tab0.block_table.shape[1]
    used = tab0.block_table >= 0
    out[:, :w][used] = tab0.block_table[used]
    return out


def initial_tags(tab0, tg_final):
    out = tg_final.copy()
    w = tab0.tier_tag.shape[1]
    used = tab0.block_table >= 0
    out[:, :w][used] = tab0.tier_tag[used]
    return out


def kv_bytes_at(spec, tags_host_rows, lens_row):
    """Algorithmic KV bytes of one decode launch: 2d per valid FP8 token + M (12d + 32) + 4d per Stale page of
    16 M tokens (16d + 32 at M = 1), per KV head."""
    d, total, T, Mt = spec.head_dim, 0, spec.page_tokens, spec.tiles_per_page
    for b, ln in enumerate(lens_row):
        npg = (int(ln) + T - 1) // T
        stale = int((tags_host_rows[b, :npg] == W.TAG_STALE).sum())
        total += spec.n_kv_heads * ((int(ln) - T * stale) * 2 * d + stale * (Mt * (12 * d + 32) + 4 * d))
    return total


def run_ours(args):
    import torch
    import paper_2608_23834_b200 as M

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    device = torch.device(f"cuda:{local}")
    torch.cuda.set_device(device)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    M.lib()
    spec = workload_spec(args)
    K, Wm = args.steps, args.warmup
    total = 3 * (K + Wm)                       # eager run (per-launch events), graph run (timed), end-to-end run
    fmt = 2 if args.format == "v2" else 1
    layers, plan, tab0 = build_layers(spec, total, device, M, torch, fmt)
    for L in layers:
        L.pool.set_decode_variant({"scalar": M.DECODE_SCALAR, "tmem": M.DECODE_TMEM}.get(args.variant, M.DECODE_TENSOR))
    B, d, hq, hkv = spec.batch, spec.head_dim, spec.n_q_heads, spec.n_kv_heads
    stream = torch.cuda.current_stream()
    launches = [0]
    decode_launches = 2 if args.variant == "scalar" else 1    # tensor: one scan launch; scalar: scan + merge
    # host mirror of the tags, advanced with the retier events, for the byte count of each step
    tags_host = initial_tags(tab0, np.zeros((B, plan["max_pages"]), np.uint8))
    ev_pairs = []

    def retier(L, ev):
        src, dst, ent, _ = ev
        L.pool.demote(src, dst, L.bt, L.tags, ent)
        launches[0] += 1

    def mark_retired(i):
        if plan["ev_dev"][i] is not None:
            for (b, lp, _, _) in plan["events"][i]:
                tags_host[b, lp] = W.TAG_STALE

    # The library's batched calls take all layers of the step in one launch each (append, decode); they serve
    # the tensor-core kernel.  Other variants go layer by layer.
    batched = (not args.per_layer) and args.variant == "tensor" and len(layers) <= M.MAX_LAYERS_PER_CALL
    pools = [L.pool for L in layers]
    layers_per_decode_launch = len(layers) if batched else 1

    def calls(slots_t, lens_t, qs, ks, vs, outs, timed_events=None):
        """The append and decode calls of one step for all layers."""
        if batched:
            M.append_layers(pools, ks, vs, slots_t)
            if timed_events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            M.decode_attention_layers(pools, qs, [L.bt for L in layers], [L.tags for L in layers], lens_t, spec.scale, outs)
            if timed_events is not None:
                e1.record(stream)
                timed_events.append((e0, e1))
            return 2
        for li, L in enumerate(layers):
            L.pool.append(ks[li], vs[li], slots_t)
            if timed_events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            L.pool.decode_attention(qs[li], L.bt, L.tags, lens_t, spec.scale, out=outs[li])
            if timed_events is not None:
                e1.record(stream)
                timed_events.append((e0, e1))
        return len(layers) * (1 + decode_launches)

    all_q, all_k, all_v, all_out = ([L.q for L in layers], [L.k_new for L in layers], [L.v_new for L in layers],
                                    [L.out for L in layers])

    def step(i, timed_events=None):
        """One step, every call issued from Python: demote where a page leaves the window, append, decode."""
        ev = plan["ev_dev"][i]
        if ev is not None:
            for L in layers:
                retier(L, ev)
        launches[0] += calls(plan["slots"][i], plan["lens"][i], all_q, all_k, all_v, all_out, timed_events)
        mark_retired(i)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(device)

    # ---- eager run: one CUDA-event pair around every decode launch (the roofline's launch time) ---
    for i in range(Wm):
        step(i)
    barrier()
    bytes_per_launch = []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for i in range(Wm, Wm + K):
        bytes_per_launch.append(kv_bytes_at(spec, tags_host, plan["lens_host"][i]))
        step(i, ev_pairs)
    t1.record(stream)
    barrier()
    eager_ms = t0.elapsed_time(t1)
    kern_ms = [a.elapsed_time(b) for a, b in ev_pairs]

    # ---- graph run (the timed region of `value`): the step's append + decode calls of all layers are
    # captured once into a CUDA graph that reads the step's slots and lengths from two fixed device
    # buffers; a step = two small copies into those buffers, the retier calls where one falls due
    # (a demoted page is never the page the step appends to, so they commute with the appends), one replay
    cur_slots = torch.empty_like(plan["slots"][0])
    cur_lens = torch.empty_like(plan["lens"][0])
    base_g = Wm + K

    per_step_launches = [0]

    def layer_calls():
        per_step_launches[0] = calls(cur_slots, cur_lens, all_q, all_k, all_v, all_out)

    def step_graph(i, graph):
        ev = plan["ev_dev"][i]
        cur_slots.copy_(plan["slots"][i], non_blocking=True)
        cur_lens.copy_(plan["lens"][i], non_blocking=True)
        if ev is not None:
            for L in layers:
                retier(L, ev)
        graph.replay()
        launches[0] += per_step_launches[0]
        mark_retired(i)

    graph = torch.cuda.CUDAGraph()
    cur_slots.copy_(plan["slots"][base_g])
    cur_lens.copy_(plan["lens"][base_g])
    torch.cuda.synchronize(device)
    with torch.cuda.graph(graph):
        layer_calls()                             # captured, not run: the pools are untouched
    for i in range(Wm):
        step_graph(base_g + i, graph)
    barrier()
    launches[0] = 0
    with ClockSampler(local) as clocks:
        t0.record(stream)
        for i in range(K):
            step_graph(base_g + Wm + i, graph)
        t1.record(stream)
        barrier()
    ms = t0.elapsed_time(t1)
    n_launch = launches[0]
    for L in layers:
        if L.pool.status() != M.OK:
            raise RuntimeError("device status word set during the timed region")

    # ---- end-to-end run: host buffers in, host buffers out, through the same calls --------------
    # A step's inputs (q, new K, new V of every layer, then slots and lengths) sit in ONE pinned host
    # buffer and arrive with one copy; the layers' device tensors are views of the device-side image of
    # that buffer, the outputs of all layers views of one device buffer that goes back with one copy.
    n_q, n_kv = B * hq * d, B * hkv * d
    per_layer = n_q + 2 * n_kv                                       # bf16 elements
    tail = 2 * B                                                     # int32 slots + lengths
    in_bytes = len(layers) * per_layer * 2 + tail * 4
    h_in = torch.empty(in_bytes, dtype=torch.uint8).pin_memory()
    d_in = torch.empty(in_bytes, dtype=torch.uint8, device=device)
    h_bf = h_in[:len(layers) * per_layer * 2].view(torch.bfloat16)
    d_bf = d_in[:len(layers) * per_layer * 2].view(torch.bfloat16)
    h_tail = h_in[len(layers) * per_layer * 2:].view(torch.int32)
    d_tail = d_in[len(layers) * per_layer * 2:].view(torch.int32)
    d_slots, d_lens = d_tail[:B], d_tail[B:]
    views = []
    for li, L in enumerate(layers):
        o = li * per_layer
        h_bf[o:o + n_q].copy_(L.q.reshape(-1).cpu())
        h_bf[o + n_q:o + n_q + n_kv].copy_(L.k_new.reshape(-1).cpu())
        h_bf[o + n_q + n_kv:o + per_layer].copy_(L.v_new.reshape(-1).cpu())
        views.append((d_bf[o:o + n_q].view(B, hq, d), d_bf[o + n_q:o + n_q + n_kv].view(B, hkv, d),
                      d_bf[o + n_q + n_kv:o + per_layer].view(B, hkv, d)))
    d_out = torch.empty((len(layers), B, hq, d), dtype=torch.float32, device=device)
    h_out = torch.empty((len(layers), B, hq, d), dtype=torch.float32).pin_memory()
    h_slots = torch.from_numpy(plan["slots_host"])
    h_lens = torch.from_numpy(plan["lens_host"])
    h2d = in_bytes
    d2h = h_out.numel() * 4

    # The graph of the end-to-end step holds the copies too: the inputs arrive first (one copy), and every
    # layer's output leaves for the host on a second stream as soon as its decode has finished, under the
    # later layers' kernels.
    copy_stream = torch.cuda.Stream(device=device)

    def layer_calls_e2e():
        main = torch.cuda.current_stream()
        d_in.copy_(h_in, non_blocking=True)          # host -> device: the step's inputs (one copy; per-layer copies
        if batched:                                  # on a second stream measured slower)
            calls(d_slots, d_lens, [v_[0] for v_ in views], [v_[1] for v_ in views], [v_[2] for v_ in views],
                  [d_out[li] for li in range(len(layers))])
            h_out.copy_(d_out, non_blocking=True)    # device -> host: the outputs of all layers
            return
        for li, L in enumerate(layers):
            qv, kv_, vv = views[li]
            L.pool.append(kv_, vv, d_slots)
            L.pool.decode_attention(qv, L.bt, L.tags, d_lens, spec.scale, out=d_out[li])
            done = torch.cuda.Event()
            done.record(main)
            copy_stream.wait_event(done)
            with torch.cuda.stream(copy_stream):
                h_out[li].copy_(d_out[li], non_blocking=True)    # device -> host: this layer's output
        main.wait_stream(copy_stream)

    d_in.copy_(h_in)
    torch.cuda.synchronize(device)
    graph_e2e = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph_e2e):
        layer_calls_e2e()

    def step_e2e(i):
        ev = plan["ev_dev"][i]
        h_tail[:B].copy_(h_slots[i])                 # this step's slots and lengths join the host image
        h_tail[B:].copy_(h_lens[i])
        if ev is not None:
            for L in layers:
                retier(L, ev)
        graph_e2e.replay()                           # inputs in, 16 x (append + decode), outputs out
        torch.cuda.synchronize(device)               # the step's result is on the host

    base = 2 * (Wm + K)
    for i in range(Wm):
        step_e2e(base + i)
    barrier()
    w0 = time.perf_counter()
    t0.record(stream)
    for i in range(K):
        step_e2e(base + Wm + i)
    t1.record(stream)
    barrier()
    e2e_ms = max(t0.elapsed_time(t1), (time.perf_counter() - w0) * 1e3)
    if not bool(torch.isfinite(h_out).all()) or not bool(h_out.any()) or any(L.pool.status() != M.OK for L in layers):
        raise RuntimeError("end-to-end run produced no valid output")

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], device)

    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])
    avg_kernel_ms = sum(kern_ms) / len(kern_ms)
    # bytes_per_launch holds one layer's algorithmic bytes per step; a launch covers layers_per_decode_launch layers
    avg_bytes = sum(bytes_per_launch) / len(bytes_per_launch) * layers_per_decode_launch
    achieved = avg_bytes / (avg_kernel_ms * 1e-3) / 1e9
    step_bytes = avg_bytes / layers_per_decode_launch * spec.n_layers
    result = {
        "metric": METRIC, "value": aggregate_value(B, K, ms, world), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": Wm, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("u8 codes (e4m3 / 3-bit TQ3); Stale key products s8 x s8 -> s32, other products f16 x f16 -> f32" if fmt == 2 else
                  "u8 codes (e4m3 / 3-bit TQ3) -> f16 tensor-core operands, f32 accumulate"), "data": "synthetic",
        "config": config_dict(spec, args, world, step_bytes, batched, layers_per_decode_launch),
        "eager_ms_per_step": eager_ms / K,
        "kv_gbs_whole_step": step_bytes / (ms / K * 1e-3) / 1e9,
        "roofline": {"bound": "hbm", "kernel": {"tensor": "decode_tensor_kernel", "tmem": "decode_tmem_kernel"}.get(args.variant, "decode_scalar_kernel + merge"), "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_kind + " copy bandwidth",
                     "frac_of_nominal_8000": achieved / 8000.0, "traffic": traffic_per_launch("cfg2_%s_%s" % (args.variant, args.format), layers_per_decode_launch)
                     if (args.config == 2 and args.ctx == 0 and args.page_tokens == 0) else None,
                     "algorithmic_bytes_per_launch": avg_bytes, "avg_launch_ms": avg_kernel_ms,
                     "median_launch_ms": statistics.median(kern_ms), "min_launch_ms": min(kern_ms)},
        "e2e": {"value": aggregate_value(B, K, e2e_ms, world), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / K},
        "gpu_launches": n_launch,
        "clocks": clocks.summary(),
    }
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            result["cpu_baseline"] = cpu_baseline(spec, fmt)
        print(json.dumps(result))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


# ------------------------------------------------------------------------------- lifecycle kernels
def run_lifecycle(args):
    """`--lifecycle`: bulk throughput of Append, Demote and Promote (Algorithm 1's state changes) for the
    head geometry of the chosen config, each timed alone with CUDA events over data larger than L2.
    Prints its own JSON line; the decode benchmark above is the contract's line."""
    import torch
    import paper_2608_23834_b200 as M

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    device = torch.device("cuda:%d" % int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    M.lib()
    spec = workload_spec(args)
    d, hkv, hq = spec.head_dim, spec.n_kv_heads, spec.n_q_heads
    Tp, Mt = spec.page_tokens, spec.tiles_per_page
    fp8_page, tq3_page = Mt * 32 * d * hkv, (Mt * (12 * d + 32) + 4 * d) * hkv
    P = max(1024 // Mt, (384 << 20) // fp8_page)         # FP8 pages converted per call: 384 MB, 3 x L2
    fmt = 2 if args.format == "v2" else 1
    pool = M.Pool(d, hkv, hq, 2 * P + 8, P + 8, W.rotation_signs(spec, 0), max_batch=1, device=device, page_tokens=Tp,
                  tq3_format=fmt)
    gen = torch.Generator(device=device)
    gen.manual_seed(spec.seed)
    T = Tp * P
    k = torch.randn((T, hkv, d), generator=gen, device=device, dtype=torch.float32)
    k[:, :, torch.from_numpy(W.outlier_channels(spec, 0, 0)).to(device)] *= 8.0
    k = k.to(torch.bfloat16)
    v = torch.randn((T, hkv, d), generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
    slots = torch.arange(T, dtype=torch.int32, device=device)
    ids = torch.arange(P, dtype=torch.int32, device=device)
    ids_hi = ids + P
    stream = torch.cuda.current_stream()
    reps, warm = max(3, min(args.steps, 10)), 3
    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])

    def timed(fn):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize(device)
        evs = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize(device)
        return statistics.median(x.elapsed_time(y) for x, y in evs)

    def line(ms, units, unit_name, bytes_moved):
        gbs = bytes_moved / (ms * 1e-3) / 1e9
        return {"ms_per_call": ms, unit_name + "_per_s": units / (ms * 1e-3), "GB_per_s_in_plus_out": gbs,
                "frac_of_%s_copy_bandwidth" % peak_kind: gbs / peak}

    with ClockSampler(device.index or 0) as clocks:
        ms_append = timed(lambda: pool.append(k, v, slots))                       # bf16 K,V in; e4m3 records out
        ms_demote = timed(lambda: pool.demote(ids, ids))                          # FP8 pages in; TQ3 pages out
        ms_promote = timed(lambda: pool.promote(ids, ids_hi))                     # TQ3 pages in; FP8 pages out
    if pool.status() != M.OK:
        raise RuntimeError("device status word set during the lifecycle run")
    new = [torch.randn((spec.batch, hkv, d), generator=gen, device=device).to(torch.bfloat16) for _ in range(2)]
    step_slots = (torch.arange(spec.batch, dtype=torch.int32, device=device) * Tp + 5)
    ms_step_append = timed(lambda: pool.append(new[0], new[1], step_slots))
    src1, dst1 = ids[:spec.batch].contiguous(), ids[:spec.batch].contiguous()
    ms_step_demote = timed(lambda: pool.demote(src1, dst1))
    print(json.dumps({
        "mode": "lifecycle", "data": "synthetic", "n_gpus": 1,
        "config": {"workload": "Append / Demote / Promote alone, head geometry of " + workload_name(spec),
                   "tq3_record_format": fmt,
                   "head_dim": d, "kv_heads": hkv, "page_tokens": Tp, "pages_per_call": P, "tokens_per_append_call": T,
                   "fp8_page_bytes": fp8_page, "tq3_page_bytes": tq3_page, "repetitions": reps,
                   "l2": "every call moves more than 3 x L2"},
        "append": line(ms_append, T, "tokens", T * hkv * d * (4 + 2)),
        "demote": line(ms_demote, P, "pages", P * (fp8_page + tq3_page)),
        "promote": line(ms_promote, P, "pages", P * (fp8_page + tq3_page)),
        "decode_step_calls": {"append_%d_tokens_ms" % spec.batch: ms_step_append,
                              "demote_%d_pages_ms" % spec.batch: ms_step_demote,
                              "note": "launch-bound sizes of one decode step, event-timed from Python"},
        "peak": peak, "peak_source": peak_kind + " copy bandwidth", "clocks": clocks.summary(),
    }))


# ------------------------------------------------------------------------------- lifecycle sweep
def run_sweep(args):
    """`--config 4 --sweep`: the 27 cells batch {1, 8, 32} x context {4K, 32K, 128K} x Stale fraction {0, 0.5, 0.95}
    (head_dim 128, 8 KV x 4 query heads, 16-token pages).  Per cell, each on its own and summed: Append of one
    token per request, Demote of the page that leaves the Recent window of every request (FP8 -> TQ3 encode),
    decode attention.  Every repetition starts from a flushed L2 (a 256 MB buffer is rewritten before it) and is
    timed with a CUDA-event pair on the launching stream; the median is reported with its roofline fraction
    (bytes the step must move / time / measured copy bandwidth)."""
    import torch
    import paper_2608_23834_b200 as M

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    device = torch.device("cuda:%d" % int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    M.lib()
    fmt = 2 if args.format == "v2" else 1
    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    reps = max(5, min(args.steps, 20))

    def timed(fn):
        for _ in range(3):
            fn()
        evs = []
        for _ in range(reps):
            flush.zero_()                               # L2 (126 MB) holds nothing of the pool afterwards
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize(device)
        return statistics.median(x.elapsed_time(y) for x, y in evs) * 1e3        # microseconds

    def entry(us, nbytes, **extra):
        gbs = nbytes / (us * 1e-6) / 1e9
        out = {"us": us, "bytes": nbytes, "GB_per_s": gbs, "frac_of_%s_copy_bandwidth" % peak_kind: gbs / peak}
        out.update(extra)
        return out

    cells = []
    with ClockSampler(device.index or 0) as clocks:
        for B in (1, 8, 32):
            for ctx in (4096, 32768, 131072):
                for f in (0.0, 0.5, 0.95):
                    spec = W.config(4, batch=B, ctx=ctx, stale_fraction=f)
                    d, hkv, T = spec.head_dim, spec.n_kv_heads, spec.page_tokens
                    layers, plan, tab0 = build_layers(spec, 4, device, M, torch, fmt)
                    L = layers[0]
                    tags_host = initial_tags(tab0, np.zeros((B, plan["max_pages"]), np.uint8))
                    n_stale = int((tags_host[0] == W.TAG_STALE).sum())
                    # Demote: the oldest FP8 page of every request into spare TQ3 pages (not published: the table
                    # stays as it is, so every repetition converts the same pages)
                    src = torch.from_numpy(np.ascontiguousarray(tab0.block_table[:, n_stale]).astype(np.int32)).to(device)
                    dst = torch.arange(tab0.tq3_pages, tab0.tq3_pages + B, dtype=torch.int32, device=device)
                    us_append = timed(lambda: L.pool.append(L.k_new, L.v_new, plan["slots"][0]))
                    us_demote = timed(lambda: L.pool.demote(src, dst))
                    us_decode = timed(lambda: L.pool.decode_attention(L.q, L.bt, L.tags, plan["lens"][0], spec.scale, out=L.out))
                    if L.pool.status() != M.OK:
                        raise RuntimeError("device status word set in cell %s" % spec.name)
                    kv = kv_bytes_at(spec, tags_host, plan["lens_host"][0])
                    cell = {
                        "mode": "sweep_cell", "cell": {"batch": B, "context_tokens": ctx, "stale_fraction": f},
                        "tq3_record_format": fmt,
                        "append": entry(us_append, B * hkv * d * (4 + 2), tokens=B),
                        "demote": entry(us_demote, B * hkv * (32 * d + 16 * d + 32), pages=B,
                                        pages_per_s=B / (us_demote * 1e-6)),
                        "decode": entry(us_decode, kv, tokens_per_s=B / (us_decode * 1e-6)),
                        "sum_us": us_append + us_demote + us_decode,
                        "tokens_per_s_whole_cell": B / ((us_append + us_demote + us_decode) * 1e-6),
                    }
                    cells.append(cell)
                    print(json.dumps(cell), flush=True)
                    del layers, L, plan
                    torch.cuda.empty_cache()
    summary = {"mode": "sweep", "metric": METRIC, "data": "synthetic", "n_gpus": 1, "repetitions": reps,
               "config": {"workload": "configs[4]: lifecycle sweep, 27 cells, head_dim 128, 8 KV x 4 q heads, 16-token pages",
                          "tq3_record_format": fmt, "l2": "L2 flushed (256 MB rewritten) before every timed repetition"},
               "peak": peak, "peak_source": peak_kind + " copy bandwidth", "clocks": clocks.summary(), "cells": cells}
    if args.out:
        with open(args.out, "w") as fh:
            json.dump(summary, fh, indent=1)
    print(json.dumps({k: v for k, v in summary.items() if k != "cells"}))


# ---------------------------------------------------------------------------------------- oracle arm
def workload_spec(args):
    over = {"n_layers": args.layers} if args.layers > 0 else {}
    if args.page_tokens > 0:
        over["page_tokens"] = args.page_tokens
    if args.ctx > 0 and args.config != 4:
        over["seq_lens"] = (args.ctx,) * W.config(args.config).batch
    if args.config == 4:
        return W.config(4, batch=args.batch or 8, ctx=args.ctx or 32768, stale_fraction=args.stale, **over)
    if args.config == 5 and args.layers <= 0:
        over["n_layers"] = 16                      # the canary's 16 full-attention layers
    return W.config(args.config, **over)


def workload_name(spec):
    if spec.page_tokens != 16 and spec.name != "cfg5_canary_blocks_1792":
        return "%s with pages of %d tokens" % (spec.name, spec.page_tokens)
    return {"cfg2_canary_59k": "configs[2]: 2 x 59,008 tokens, 16 layers, d=256, 4 KV x 6 q heads, ~96% TQ3 pages",
            "cfg5_canary_blocks_1792": "the configs[2] shape with pages of 1,792 tokens (paper-scale blocks): 2 x 59,008 "
                                       "tokens, d=256, 4 KV x 6 q heads, 10 FP8 + 23 TQ3 pages per request"}.get(
        spec.name, spec.name)


def config_dict(spec, args, world, step_bytes=None, batched=None, layers_per_launch=None):
    """The `config` object of the JSON line; both arms print the same workload keys."""
    fmt = 2 if args.format == "v2" else 1
    cfg = {"workload": workload_name(spec), "batch": spec.batch, "context_tokens": list(spec.seq_lens)[:4],
           "tq3_record_format": fmt, "layers": spec.n_layers, "head_dim": spec.head_dim, "kv_heads": spec.n_kv_heads,
           "q_heads": spec.n_q_heads, "page_tokens": spec.page_tokens,
           "parallelism": "replicas only" if world > 1 else "single GPU"}
    if step_bytes is not None:
        cfg["l2"] = "inputs larger than L2 (%.0f MB of KV per step)" % (step_bytes / 1e6)
        cfg["step"] = "append + demote at its natural cadence + decode attention, every layer"
        cfg["launch"] = ("one CUDA graph per step holding mkv_append_layers and mkv_decode_attention_layers (all layers in "
                         "one launch each); retier calls issued directly") if batched else \
                        "one CUDA graph per step (append + decode of every layer); retier calls issued directly"
        cfg["layers_per_decode_launch"] = layers_per_launch
    return cfg


def oracle_sample(spec, seconds_hint=20.0):
    """One layer of the workload prepared for the oracle (bounded: at most 4 requests)."""
    import oracle
    from oracle.harness import build_layer
    reqs = list(range(min(spec.batch, 4)))
    sub = W.config(0, seq_lens=[spec.seq_lens[b] for b in reqs], head_dim=spec.head_dim, n_kv_heads=spec.n_kv_heads,
                   group=spec.group, anchor_prefix=spec.anchor_prefix, anchor_spans=max(spec.anchor_spans, 0),
                   anchor_span_tokens=spec.anchor_span_tokens, recent_tokens=spec.recent_tokens,
                   n_outlier=spec.n_outlier, seed=spec.seed, stale_fraction=spec.stale_fraction,
                   page_tokens=spec.page_tokens)
    tab = W.tables(sub)
    L = build_layer(sub, tab)
    return oracle, sub, tab, L


def time_oracle(spec, reps=3):
    oracle, sub, tab, L = oracle_sample(spec)
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        oracle.decode_attention(L.fp8_arena, L.tq3_arena, sub.head_dim, sub.n_kv_heads, sub.group, L.sigma, L.q_bits,
                                tab.block_table, tab.tier_tag, tab.seq_lens, sub.scale, page_tokens=sub.page_tokens)
        times.append(time.perf_counter() - t0)
    layer_s = sum(times) / len(times)
    # one decode step = all layers over the whole batch; the sample covers one layer of `sub.batch` requests
    step_s = layer_s * spec.n_layers * spec.batch / sub.batch
    cores = min(os.cpu_count() or 1, sub.batch * sub.n_kv_heads)
    return {"value": spec.batch / step_s, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "fp64 dequantise-then-attend of 1 of %d layers, %d of %d requests, %d repetitions (%.2f s each on %d "
                      "threads, scaled to a whole step)" % (spec.n_layers, sub.batch, spec.batch, reps, layer_s, cores),
            "kv_gbs": W.kv_bytes(sub, tab) / layer_s / 1e9}


def time_oracle_lifecycle(spec, seconds=3.0):
    """The oracle's own Append (bf16 -> e4m3 record) and Demote (FP8 record -> TQ3 record) per page and KV head,
    single-threaded as the oracle is written, on seeded data of the workload's head geometry."""
    import oracle
    d = spec.head_dim
    rng = np.random.default_rng(spec.seed)
    k = rng.standard_normal((16, d)).astype(np.float32)
    v = rng.standard_normal((16, d)).astype(np.float32)
    sigma = W.rotation_signs(spec, 0)
    out = {}
    for name, fn in (("append", lambda: oracle.fp8_pack_record(k, v)),
                     ("demote", None)):
        if name == "demote":
            rec8 = oracle.fp8_pack_record(k, v)
            fn = lambda: oracle.demote_record(rec8, d, sigma)
        n, t0 = 0, time.perf_counter()
        while time.perf_counter() - t0 < seconds:
            fn()
            n += 1
        dt = time.perf_counter() - t0
        out[name + "_page_heads_per_s"] = n / dt
    out["append_tokens_per_s_all_heads"] = out["append_page_heads_per_s"] * 16 / spec.n_kv_heads
    out["demote_pages_per_s_all_heads"] = out["demote_page_heads_per_s"] / spec.n_kv_heads
    out["threads"] = 1
    return out


def cpu_baseline(spec, fmt=1):
    import oracle
    with oracle.record_format(fmt):
        res = time_oracle(spec)
        res["lifecycle"] = time_oracle_lifecycle(spec)
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = workload_spec(args)
    import oracle as _o
    _o.set_format(2 if args.format == "v2" else 1)
    oracle, sub, tab, L = oracle_sample(spec)
    K, Wm = args.steps, args.warmup

    def one():
        t0 = time.perf_counter()
        oracle.decode_attention(L.fp8_arena, L.tq3_arena, sub.head_dim, sub.n_kv_heads, sub.group, L.sigma, L.q_bits,
                                tab.block_table, tab.tier_tag, tab.seq_lens, sub.scale, page_tokens=sub.page_tokens)
        return time.perf_counter() - t0
    for _ in range(Wm):
        one()
    layer_s = sum(one() for _ in range(K)) / K
    step_s = layer_s * spec.n_layers * spec.batch / sub.batch
    cores = min(os.cpu_count() or 1, sub.batch * sub.n_kv_heads)
    val = spec.batch / step_s
    sample = ("each step = fp64 dequantise-then-attend of 1 of %d layers, %d of %d requests, scaled to a whole step"
              % (spec.n_layers, sub.batch, spec.batch))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": K, "warmup": Wm,
        "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_dict(spec, args, 1),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling on a small case)")
    ap.add_argument("--variant", default="tensor", choices=["tensor", "scalar", "tmem"],
                    help="decode kernel: the tensor-core product kernel, or the CUDA-core comparison kernel")
    ap.add_argument("--ctx", type=int, default=0, help="override the context length of every request (profiling)")
    ap.add_argument("--batch", type=int, default=0, help="config 4 only: requests of the lifecycle cell (default 8)")
    ap.add_argument("--stale", type=float, default=0.5, help="config 4 only: Stale fraction of the lifecycle cell")
    ap.add_argument("--page-tokens", type=int, default=0,
                    help="override the page size (a multiple of 16; 1792 and 832 are the paper's block sizes)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--format", default="v2", choices=["v1", "v2"],
                    help="TQ3 record format of the pools (v2: key codebook of exact small integers, integer key products)")
    ap.add_argument("--per-layer", action="store_true",
                    help="issue mkv_append / mkv_decode_attention layer by layer instead of the batched calls")
    ap.add_argument("--sweep", action="store_true",
                    help="config 4 only: all 27 cells (batch x context x Stale fraction), each timing Append, Demote and "
                         "decode separately; one JSON line per cell and a summary, also written to --out")
    ap.add_argument("--out", default="", help="--sweep: file that receives the results as JSON")
    ap.add_argument("--lifecycle", action="store_true",
                    help="time Append, Demote and Promote alone (bulk throughput) instead of the decode step")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    # --gpus N: N independent replicas, one process per GPU.  Under torchrun WORLD_SIZE must agree with N; started
    # plainly with N > 1 the script re-launches itself under torch.distributed.run on this node.
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is not None and int(world_env) != args.gpus:
        sys.stderr.write("bench.py: --gpus %d but WORLD_SIZE=%s; launch with --nproc-per-node equal to --gpus\n"
                         % (args.gpus, world_env))
        sys.exit(2)
    if world_env is None and args.gpus > 1 and not args.lifecycle and not args.sweep:
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        os.execv(sys.executable, cmd)
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    elif args.lifecycle:
        run_lifecycle(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
