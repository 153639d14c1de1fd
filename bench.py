#!/usr/bin/env python
"""Benchmark of the HPD decode step on B200: branch-tokens/s per decode step at 96 branches/prompt.

One "step" = the whole hot path on one layer: hpd_build_meta -> hpd_rope -> hpd_kv_append ->
hpd_attn_decode over the main workload (Llama-3-8B attention geometry, 64 prompts x 4 documents
x 512 prefix tokens x 24 branches, depths uniform in [0,16)).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload main|long]

N > 1: one rank per GPU, started by torchrun or, when no rank environment is present, by this script
itself.  Prompts are independent, so the global prompt list (N x the single-GPU batch) is split into
contiguous shards, every rank decodes its own shard, and nothing crosses NVLink on the data path (weak
scaling); only the timing scalars are reduced.
``--impl reference`` times the CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_26209_b200 import synth  # noqa: E402

METRIC = "branch_tokens_per_s_per_decode_step"
UNIT = "branch-tokens/s"


def workload_prompts(workload: str) -> int:
    """Prompts of the single-GPU batch of a workload."""
    if workload == "main":
        return 64
    if workload == "long":
        return 32
    if workload.startswith("main_p"):
        return int(workload[6:])
    if workload.startswith("long_p"):
        return int(workload[6:])
    if workload.startswith("posorder_p"):
        return int(workload[10:])
    raise SystemExit(f"unknown workload {workload}")


def rank_structure(workload: str, world: int, rank: int):
    """The shard of the global prompt list that rank ``rank`` of ``world`` decodes (no GPU needed).

    The global batch has ``world`` x the single-GPU prompts; ``synth.shard_prompts`` gives each rank a contiguous
    range of prompt indices; the rank's structure is drawn with the index of its first prompt as seed, so rank 0 of
    a one-rank run is the single-GPU workload itself.  Returns (structure, range of global prompt indices)."""
    per_gpu = workload_prompts(workload)
    mine = synth.shard_prompts(per_gpu * world, world, rank)
    if workload.startswith("long"):
        s = synth.config_long(n_prompts=len(mine), seed=mine.start)
    elif workload.startswith("posorder_p"):
        # the mask the paper runs (Sec. 4.3.2): every prompt is ONE group -- 4 stacked documents of 512 tokens as the
        # prompt, then the skeleton of its 96 attribute keys -- shared by all of its 96 branches; K_max = 16
        s = _posorder_structure(len(mine), mine.start)
        s.n_prompts, s.docs_per_prompt = len(mine), 4
    else:
        s = synth.config_main(n_prompts=len(mine), seed=mine.start)
    return s, mine


def _posorder_structure(n_prompts: int, seed: int):
    g = synth.LLAMA3_8B
    return synth.config_skeleton(f"posorder_p{n_prompts}", g["Hq"], g["Hkv"], g["D"], g["rope_theta"], 16,
                                 [2048] * n_prompts, [96] * n_prompts, key_len_hi=4, seed=seed)


def algorithmic_bytes(s) -> dict:
    """Bytes one step must move (per layer): each live document's prefix K+V once, each live branch's
    cached tokens (new token included) once, q in and o out; rope and append add their own traffic."""
    g = s.geom
    row = g.Hkv * g.D * 2 * 2                                   # K+V bytes of one token
    alive = s.slot_alive.astype(bool)
    docs_live = np.unique(s.slot_doc()[alive])
    prefix = int(s.doc_prefix_len[docs_live].astype(np.int64).sum()) * row
    suffix = int((s.slot_depth[alive].astype(np.int64) + 1).sum()) * row
    if s.slot_vis is not None:
        # position-order mode: a group's cached tokens -- of retired slots too -- are read once for the rows behind them
        sd = s.slot_doc()
        last_live = np.full(s.n_docs, -1, np.int64)
        np.maximum.at(last_live, sd[alive], np.nonzero(alive)[0])
        seen = np.arange(s.n_slots) <= last_live[sd]
        suffix = int((s.slot_depth[seen].astype(np.int64) + alive[seen]).sum()) * row
    n = int(alive.sum())
    qo = n * g.Hq * g.D * 2 * 2
    rope = 2 * n * (g.Hq + g.Hkv) * g.D * 2
    append = 2 * 2 * n * g.Hkv * g.D * 2
    keys = int((s.doc_prefix_len[s.slot_doc()[alive]].astype(np.int64) + s.slot_depth[alive] + 1).sum())
    if s.slot_vis is not None:
        # keys a row sees: the prefix up to its attribute key, every cached token of the group's slots up to its own
        tok = s.slot_depth.astype(np.int64) + alive
        cum = np.cumsum(tok)
        first = np.concatenate([[0], np.cumsum(s.doc_branch_cnt)])[s.slot_doc()]
        before_group = np.where(first > 0, cum[np.maximum(first - 1, 0)], 0)
        keys = int((s.slot_vis.astype(np.int64) + cum - before_group)[alive].sum())
    return dict(attn=prefix + suffix + qo, prefix=prefix, suffix=suffix, qo=qo, rope=rope, append=append,
                flops=4 * g.D * g.Hq * keys, n_active=n)


def measured_peaks() -> dict:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


class ClockSampler:
    """nvidia-smi clock/throttle samples (read-only query), time-stamped so that only those taken inside the timed
    regions are summarised."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 50):
        self.index, self.period_ms, self.lines, self.proc, self.windows = index, period_ms, [], None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", str(self.period_ms)],
                                         stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def window(self, t0: float, t1: float):
        """Mark [t0, t1] (time.time()) as a timed region."""
        self.windows.append((t0, t1))

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(2 * self.period_ms * 1e-3)
        self.proc.terminate()
        sm, mx, pw, reasons, n_all = [], [], [], set(), 0
        for ts, ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            n_all += 1
            if self.windows and not any(t0 <= ts <= t1 + self.period_ms * 1e-3 for t0, t1 in self.windows):
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "samples_total": n_all,
                "power_w_max": max(pw) if pw else None,
                "note": "samples taken inside the timed regions (graph replay, direct calls, end to end)"}


def time_oracle_sample(s, tb, budget_rows: int, n_threads: int = 0):
    """The CPU oracle, as it stands, on a sample of the workload's rows.  Returns (tokens/s, threads, rows)."""
    from oracle import capi
    g = s.geom
    f = {k: synth.bf16_bits_to_f32(v) for k, v in tb.items()}
    meta = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, g.suffix_cap, s.pos_gap)
    act = meta.active_slot[: meta.n_active]
    rows = np.linspace(0, meta.n_active - 1, num=min(budget_rows, meta.n_active)).astype(np.int64)
    q, k, v = f["q"][act], f["k_new"][act], f["v_new"][act]
    t0 = time.perf_counter()
    out = capi.decode_step(g, meta, s.doc_prefix_len, q, k, v, f["prefix_k"], f["prefix_v"], f["suffix_k"],
                           f["suffix_v"], n_threads=n_threads, rows=rows)
    dt = time.perf_counter() - t0
    return len(rows) / dt, out.threads, len(rows), dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    s, _ = rank_structure(args.workload, 1, 0)
    tb = synth.make_tensors(s)
    rows_per_step = 256
    for _ in range(args.warmup):
        time_oracle_sample(s, tb, 32)
    tot_rows, tot_t, threads = 0, 0.0, 0
    for _ in range(args.steps):
        _, threads, n, dt = time_oracle_sample(s, tb, rows_per_step)
        tot_rows += n
        tot_t += dt
    val = tot_rows / tot_t
    sample = f"{rows_per_step} evenly spaced rows of the {s.n_active}-row step per timed step (oracle/hpd_oracle.c, fp64, OpenMP)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": s.name, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def block_stats(ms) -> dict:
    a = np.asarray(ms, dtype=np.float64)
    return {"blocks": int(a.size), "median_ms": float(np.median(a)), "min_ms": float(a.min()), "max_ms": float(a.max()),
            "p10_ms": float(np.percentile(a, 10)), "p90_ms": float(np.percentile(a, 90))}


def agree_block_count(first_block_ms: float, target_ms: float, reduce_max) -> int:
    """How many K-step blocks to time so that about ``target_ms`` of device time is covered; every rank gets the
    same count (the slowest rank's first block decides)."""
    t = max(reduce_max(first_block_ms), 1e-3)
    return int(min(max(np.ceil(target_ms / t), 3), 5000))


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2604_26209_b200 import runtime, binding
    from paper_2604_26209_b200.dist import reduce_timing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    binding.load()

    s, my_prompts = rank_structure(args.workload, world, rank)      # this rank's shard of the global prompt list
    tb = synth.make_tensors(s)
    db = runtime.DeviceBatch(s, tb)
    db.build_meta()
    torch.cuda.synchronize()
    tabs = db.tables()
    n = tabs["n_active"]
    act = tabs["active_slot"][:n]
    db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    ab = algorithmic_bytes(s)
    assert ab["n_active"] == n

    stream = torch.cuda.current_stream()
    K = args.steps

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_max(x: float) -> float:
        return reduce_timing([x], 0, device="cuda")[0][0]

    def time_block(fn) -> float:
        """Exactly K steps between two events, a barrier and a synchronize on both sides."""
        barrier()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(K):
            fn()
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)

    # ---- direct C-ABI calls, one per operation, CUDA events between them: per-kernel breakdown --------------------
    for _ in range(args.warmup):
        db.step(with_meta=True, fused=not args.unfused)

    def direct_block():
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
        barrier()
        for i in range(K):
            ev[i][0].record(stream)
            db.build_meta()
            if args.unfused:
                db.rope(); db.kv_append()
            else:
                db.rope_append()
            ev[i][1].record(stream)
            db.attn(True)
            ev[i][2].record(stream)
        barrier()
        return (ev[0][0].elapsed_time(ev[-1][2]), float(np.mean([e[1].elapsed_time(e[2]) for e in ev])),
                float(np.mean([e[0].elapsed_time(e[1]) for e in ev])))

    first = direct_block()
    n_direct = agree_block_count(first[0], args.min_ms * 0.4, reduce_max)
    t_w0 = time.time()
    direct = [direct_block() for _ in range(n_direct)]
    sampler.window(t_w0, time.time())
    ms_total_blocks = [d[0] for d in direct]
    ms_attn = float(np.median([d[1] for d in direct]))
    ms_pre = float(np.median([d[2] for d in direct]))
    attn_stats = block_stats([d[1] for d in direct])
    status = db.status()

    # ---- the same step replayed from a CUDA graph: the headline ----------------------------------------------------
    graph_blocks = None
    if not args.no_graph:
        barrier()
        g = db.capture_step(with_meta=True, fused=not args.unfused)
        for _ in range(3):
            g.replay()
        first_g = time_block(g.replay)
        n_graph = agree_block_count(first_g, args.min_ms, reduce_max)
        t_w0 = time.time()
        graph_blocks = [time_block(g.replay) for _ in range(n_graph)]
        sampler.window(t_w0, time.time())
        if db.status() != 0:
            status = db.status()

    # ---- end to end: host buffers in, host result out, through the same calls ------------------------------------
    # Every step copies its inputs from pinned host memory and reads its result back.  Two buffer sets and three streams:
    # the copy-in of step i+1 and the copy-out of step i-1 run while step i computes (the host link is full duplex).
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
    hq, hk, hv = pin(tb["q"][act]), pin(tb["k_new"][act]), pin(tb["v_new"][act])
    h_depth = torch.from_numpy(s.slot_depth.copy()).pin_memory()
    h_alive = torch.from_numpy(s.slot_alive.copy()).pin_memory()
    h_o = [torch.empty((n, s.geom.Hq, s.geom.D), dtype=torch.int16).pin_memory() for _ in range(2)]
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, h_depth, h_alive))
    d2h = h_o[0].numel() * h_o[0].element_size()
    dbs = [db, runtime.DeviceBatch(s, tb)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]; ev_done = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]
    for e in ev_done + ev_out:
        e.record(stream)
    e2e_i = [0]

    def e2e_step():
        i = e2e_i[0] & 1
        e2e_i[0] += 1
        d = dbs[i]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_done[i])                  # the step that last used this buffer set has read its inputs
            d.slot_depth.copy_(h_depth, non_blocking=True)
            d.slot_alive.copy_(h_alive, non_blocking=True)
            d.q[:n].view(torch.int16).copy_(hq, non_blocking=True)
            d.k_new[:n].view(torch.int16).copy_(hk, non_blocking=True)
            d.v_new[:n].view(torch.int16).copy_(hv, non_blocking=True)
            ev_in[i].record(s_in)
        stream.wait_event(ev_in[i])
        stream.wait_event(ev_out[i])                     # its previous result has left the device
        d.step(with_meta=True, fused=not args.unfused)
        ev_done[i].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[i])
            h_o[i].copy_(d.o[:n].view(torch.int16), non_blocking=True)
            ev_out[i].record(s_out)

    def e2e_block() -> float:
        barrier()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(K):
            e2e_step()
        stream.wait_event(ev_out[0]); stream.wait_event(ev_out[1])      # the last results are on the host
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    for _ in range(4):
        e2e_step()
    first_e = e2e_block()
    n_e2e = agree_block_count(first_e, args.min_ms * 0.3, reduce_max)
    t_w0 = time.time()
    e2e_blocks = [e2e_block() for _ in range(n_e2e)]
    sampler.window(t_w0, time.time())
    if dbs[1].status() != 0:
        status = dbs[1].status()
    clocks = sampler.stop() if rank == 0 else None

    # ---- max over ranks of every block time, sum over ranks of the rows -------------------------------------------
    head_blocks = graph_blocks if graph_blocks is not None else ms_total_blocks
    head_max, tok_all = reduce_timing(head_blocks, n, device="cuda")
    direct_max, _ = reduce_timing(ms_total_blocks, 0, device="cuda")
    e2e_max, _ = reduce_timing(e2e_blocks, 0, device="cuda")
    (ms_attn_max,), _ = reduce_timing([ms_attn], 0, device="cuda")

    if rank == 0:
        peaks = measured_peaks()
        # Headline: K steps replayed from a CUDA graph (the same kernels per step, launched back to back by the GPU
        # instead of one host call each), median over the timed K-step blocks of the slowest rank's time.
        hs, ds, es = block_stats(head_max), block_stats(direct_max), block_stats(e2e_max)
        ms_head = hs["median_ms"]
        value = tok_all * K / (ms_head * 1e-3)
        value_direct = tok_all * K / (ds["median_ms"] * 1e-3)
        e2e_val = tok_all * K / (es["median_ms"] * 1e-3)
        ach = ab["attn"] / (ms_attn * 1e-3) / 1e9
        tflops = ab["flops"] / (ms_attn * 1e-3) / 1e12
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            rows_done, t_cpu, thr = 0, 0.0, 0
            while t_cpu < args.cpu_seconds:
                _, thr, rows, dt = time_oracle_sample(s, tb, args.cpu_rows)
                rows_done += rows
                t_cpu += dt
            cpu = {"value": rows_done / t_cpu, "unit": UNIT, "cores": thr, "kind": "oracle",
                   "sample": f"{rows_done} rows ({args.cpu_rows} evenly spaced rows of the {n}-row step per pass), "
                             f"{t_cpu:.1f} s of oracle time"}
        comparison = None
        if world == 1 and not args.no_comparison and s.slot_vis is None:
            # the in-repo comparison: every branch with a private physical copy of [prefix ; branch tokens]
            free_b, _ = torch.cuda.mem_get_info()
            row_b = s.geom.Hkv * s.geom.D * 2 * 2
            need = int((s.doc_prefix_len[s.slot_doc()[s.slot_alive.astype(bool)]].astype(np.int64)
                        + s.slot_depth[s.slot_alive.astype(bool)] + 1).sum()) * row_b
            rows_std = n if need < 0.6 * free_b else max(1, int(n * 0.6 * free_b / need))
            dup = runtime.DupBatch(db, include_new=True, rows=rows_std)
            for _ in range(3):
                dup.attn(db.q)
            reps, t_std = 5, []
            for _ in range(7):
                c0 = torch.cuda.Event(enable_timing=True); c1 = torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                c0.record(stream)
                for _ in range(reps):
                    dup.attn(db.q)
                c1.record(stream)
                torch.cuda.synchronize()
                t_std.append(c0.elapsed_time(c1) / reps)
            ms_std = float(np.median(t_std)) * (n / dup.n)          # linear in rows: no sharing between sequences
            std_bytes = dup.total_tokens * row_b * (n / dup.n) + ab["qo"]
            comparison = {"kernel": "std_attn_decode (duplicated prefix)", "ms_per_launch": ms_std,
                          "rows_timed": dup.n, "rows_total": n,
                          "hbm_frac_of_measured": std_bytes / (ms_std * 1e-3) / 1e9 / peaks["hbm_gbs"],
                          "algorithmic_bytes": int(std_bytes), "bytes_ratio_std_over_hpd": std_bytes / ab["attn"],
                          "speedup_hpd_over_std": ms_std / ms_attn,
                          "note": "the speedup is bounded by the byte ratio; both kernels stream at their own fraction of HBM"}
            del dup
        traffic = None
        tp = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(tp):
            traffic = json.load(open(tp)).get(f"hpd_attn_decode:{s.name}")
        launches_per_step = 1 + (2 if args.unfused else 1) + 2      # table kernel, rope/append, attention + merge
        n_steps_timed = K * (len(head_blocks) + len(ms_total_blocks) + len(e2e_blocks))
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_head / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": s.name, "mask": "position order (Sec. 4.3.2)" if s.slot_vis is not None else "branch-local (Eq. 5-6)",
                       "prompts_per_gpu": s.n_prompts, "global_prompts": s.n_prompts * world,
                       "branches_per_prompt": 96, "docs_per_prompt": s.docs_per_prompt, "n_active_per_gpu": n,
                       "geometry": "Hq32/Hkv8/D128", "layers": 1,
                       "l2": f"inputs larger than L2 ({ab['attn'] / 1e6:.0f} MB touched per step vs 126 MB L2); no flush",
                       "rope_append": "two launches" if args.unfused else "one launch (hpd_rope_append)"},
            "timing": {"what": f"blocks of exactly {K} steps, each between a barrier + synchronize; value = median block",
                       "headline": hs, "direct_calls": ds, "e2e": es, "attn_launch_ms_per_block_mean": attn_stats},
            "clocks": clocks,
            "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "ms_per_step": es["median_ms"] / K, "steps": K,
                    "how": "per step: pinned host q/k/v and slot tables copied in, the step's four kernels, o copied out; "
                           "two buffer sets, copies of neighbouring steps overlap the compute"},
            "gpu_launches": launches_per_step * K,
            "gpu_launches_all_timed_regions": launches_per_step * n_steps_timed,
            "roofline": {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": ach / peaks["hbm_gbs"], "traffic": traffic, "kernel": "hpd_attn_decode",
                         "peak_source": peaks["source"], "ms_per_launch": ms_attn, "algorithmic_bytes": ab["attn"],
                         "frac_of_nominal_8TBs": ach / 8000.0, "tensor_tflops_algorithmic": tflops,
                         "tensor_frac_of_measured_bf16": tflops / peaks["bf16_tflops"]},
            "breakdown_ms": {"meta_rope_append": ms_pre, "attn": ms_attn},
            "launch": ("cuda graph replay of the step (captured once from the C-ABI calls)" if graph_blocks is not None
                       else "one C-ABI call per kernel group"),
            "direct_calls": {"ms_per_step": ds["median_ms"] / K, "value": value_direct, "unit": UNIT,
                             "note": "the same K steps as one C-ABI call per operation with CUDA events between them; "
                                     "source of breakdown_ms and of the roofline's launch time"},
            "cpu_baseline": cpu, "comparison": comparison, "dev_status": status,
        }
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_shared3(args):
    """Three sharing levels (Sec. 4.3.5): the main workload with the first ``--block-tokens`` tokens of every document's
    512-token prefix moved into ONE block shared by all documents (instruction and attribute definitions).  A step =
    tables of both levels, rope + append, document/branch attention, block attention, log-sum-exp merge."""
    import torch
    from paper_2604_26209_b200 import runtime, binding
    torch.cuda.set_device(0)
    binding.load()
    P, LB = int(args.workload.split("_p")[1]), args.block_tokens
    s = synth.config_main(n_prompts=P, seed=0)
    s.doc_prefix_len[:] = 512 - LB
    s.name = f"shared3_p{P}_block{LB}"
    tb = synth.make_tensors(s)
    rng = np.random.default_rng(123)
    bk = synth.randn_bf16(rng, (LB, s.geom.Hkv, s.geom.D)); bv = synth.randn_bf16(rng, (LB, s.geom.Hkv, s.geom.D))
    sb = runtime.SharedBlockBatch(s, tb, np.zeros(s.n_docs, np.int32), np.array([LB], np.int32), bk, bv)
    sb.build_meta()
    torch.cuda.synchronize()
    n = sb.db.tables()["n_active"]
    sb.db.set_step_inputs(tb["q"][:n], tb["k_new"][:n], tb["v_new"][:n])
    s.name += "_two_pass" if args.two_pass else ""
    for _ in range(args.warmup):
        sb.step(args.two_pass)
    g = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        sb.step(args.two_pass)
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(0); sampler.start(); time.sleep(0.2)
    blocks, t_w0 = [], time.time()
    while sum(blocks) < args.min_ms or len(blocks) < 3:
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        blocks.append(e0.elapsed_time(e1))
    sampler.window(t_w0, time.time())
    # the attention part alone (three launches groups), direct calls
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    att = []
    for _ in range(20):
        ev[0].record(stream); (sb.attn_two_pass() if args.two_pass else sb.attn()); ev[1].record(stream); torch.cuda.synchronize()
        att.append(ev[0].elapsed_time(ev[1]))
    ab = algorithmic_bytes(s)
    row = s.geom.Hkv * s.geom.D * 4
    bytes_attn = ab["attn"] + LB * row + (2 * ab["qo"] if args.two_pass else 0)   # + the block once (+ the merge pass's traffic)
    hs = block_stats(blocks)
    peaks = measured_peaks()
    ms_att = float(np.median(att))
    print(json.dumps({
        "metric": METRIC, "value": n * args.steps / (hs["median_ms"] * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": hs["median_ms"] / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": s.name, "block_tokens": LB, "doc_tokens": 512 - LB, "prompts": P, "n_active": n,
                   "launch": "cuda graph replay of the step"},
        "timing": {"headline": hs}, "clocks": sampler.stop(), "gpu_launches": (9 if args.two_pass else 4) * args.steps,
        "roofline": {"bound": "hbm", "achieved": bytes_attn / (ms_att * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": bytes_attn / (ms_att * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                     "kernel": "hpd_attn_decode x2 + hpd_merge_lse" if args.two_pass else "hpd_attn_decode_shared", "ms_per_launch": ms_att, "algorithmic_bytes": int(bytes_attn)},
        "dev_status": sb.db.status(),
    }), flush=True)


def run_prefill(args):
    """First inference step (Sec. 4.3.2): causal attention of every prompt token of P prompts (2048 prompt tokens + the
    skeleton of 96 attribute keys each) with Algorithm 2's position IDs.  A step = hpd_rope over all prompt tokens (keys
    rotated in place in the prefix cache) + hpd_prefill_attn; the tables are built once.  Compute-bound: the roofline is
    the measured dense bf16 rate."""
    import torch
    from paper_2604_26209_b200 import binding as B
    torch.cuda.set_device(0)
    B.load()
    P = int(args.workload.split("_p")[1])
    s = _posorder_structure(P, 0)
    s.name = f"prefill_p{P}"
    g, dev, T = s.geom, "cuda", s.total_prefix
    gen = torch.Generator(device=dev); gen.manual_seed(0)
    rnd = lambda *shape: torch.randn(*shape, device=dev, dtype=torch.float32, generator=gen).to(torch.bfloat16)
    q0, k0, pv = rnd(T, g.Hq, g.D), rnd(T, g.Hkv, g.D), rnd(T, g.Hkv, g.D)
    q, pk = q0.clone(), k0.clone()
    o = torch.zeros_like(q)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    L, cnt, vis = i32(s.doc_prefix_len), i32(s.doc_branch_cnt), i32(s.slot_vis)
    t = B.PrefillTables.alloc(g, s.n_docs, T, dev)
    B.hpd_prefill_meta(g, s.n_docs, s.n_slots, T, L, cnt, vis, s.pos_gap, t)
    stream = torch.cuda.current_stream()

    def step():
        B.hpd_rope(g, T, t.n_tokens, t.tok_pos, q, pk)          # (rotating again and again changes values, not the work)
        B.hpd_prefill_attn(g, s.n_docs, T, q, pk, pv, L, t, o, None)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(0); sampler.start(); time.sleep(0.2)
    K = max(1, min(args.steps, 5))
    blocks, att, t_w0 = [], [], time.time()
    while sum(blocks) < args.min_ms or len(blocks) < 3:
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * K + 1)]
        torch.cuda.synchronize()
        ev[0].record(stream)
        for i in range(K):
            B.hpd_rope(g, T, t.n_tokens, t.tok_pos, q, pk); ev[2 * i + 1].record(stream)
            B.hpd_prefill_attn(g, s.n_docs, T, q, pk, pv, L, t, o, None); ev[2 * i + 2].record(stream)
        torch.cuda.synchronize()
        blocks.append(ev[0].elapsed_time(ev[2 * K]))
        att.append(float(np.mean([ev[2 * i + 1].elapsed_time(ev[2 * i + 2]) for i in range(K)])))
    sampler.window(t_w0, time.time())
    Ld = s.doc_prefix_len.astype(np.int64)
    flops = 4 * g.D * g.Hq * int((Ld * (Ld + 1) // 2).sum())          # causal: token t sees t + 1 keys
    hs = block_stats(blocks)
    ms_att = float(np.median(att))
    peaks = measured_peaks()
    tf = flops / (ms_att * 1e-3) / 1e12
    print(json.dumps({
        "metric": "prompt_tokens_per_s_first_inference_step", "value": T * K / (hs["median_ms"] * 1e-3), "unit": "prompt-tokens/s",
        "n_gpus": 1, "steps": K, "warmup": args.warmup, "ms_per_step": hs["median_ms"] / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": s.name, "prompts": P, "tokens": T, "tokens_per_prompt": int(Ld.mean()), "geometry": "Hq32/Hkv8/D128",
                   "launch": "direct calls (rope, attention)"},
        "timing": {"headline": hs}, "clocks": sampler.stop(), "gpu_launches": 3 * K,
        "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"],
                     "traffic": None, "kernel": "hpd_prefill_attn", "ms_per_launch": ms_att, "algorithmic_flops": flops,
                     "peak_source": peaks["source"]},
        "dev_status": int(t.dev_status.item()),
    }), flush=True)


def spawn_ranks(args) -> int:
    """``--gpus N`` without a rank environment: start one process per GPU (the environment torchrun would give them),
    wait for all, pass rank 0's JSON line through."""
    import socket
    import torch
    have = torch.cuda.device_count()
    world = min(args.gpus, have) if have > 0 else 0
    if world < 1:
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    if world < args.gpus:
        sys.stderr.write(f"bench.py: {args.gpus} GPUs asked for, {have} visible: running {world} ranks\n")
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world), LOCAL_WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *sys.argv[1:]], env=env))
    rc = 0
    for p in procs:
        rc = max(rc, p.wait())
    return rc


def run_loop(args):
    """Decode loop: 32 layers x up to 32 steps over the main structure with ragged retirement (end-of-value lengths
    min(Geom(1/8), 32)).  Per step: hpd_build_meta once, then per layer hpd_rope_append -> hpd_attn_decode
    on that layer's own prefix and branch caches.  Caches are filled on the device (torch.randn, seeded): 43 GB."""
    import torch
    from paper_2604_26209_b200 import binding as B
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("--workload loop is a single-GPU workload")
    torch.cuda.set_device(0)
    B.load()
    s = synth.config_loop(n_prompts=args.loop_prompts, seed=0)
    g, dev, L = s.geom, "cuda", args.layers
    gen = torch.Generator(device=dev); gen.manual_seed(0)
    rnd = lambda *shape: torch.randn(*shape, device=dev, dtype=torch.float32, generator=gen).to(torch.bfloat16)
    kv = g.Hkv * g.D
    pre_k = [rnd(s.total_prefix, kv) for _ in range(L)]; pre_v = [rnd(s.total_prefix, kv) for _ in range(L)]
    suf_k = [torch.zeros(s.n_slots * g.suffix_cap, kv, dtype=torch.bfloat16, device=dev) for _ in range(L)]
    suf_v = [torch.zeros_like(suf_k[0]) for _ in range(L)]
    q = [rnd(s.n_slots, g.Hq * g.D) for _ in range(2)]
    kn = [rnd(s.n_slots, kv) for _ in range(2)]; vn = [rnd(s.n_slots, kv) for _ in range(2)]
    o = torch.zeros(s.n_slots, g.Hq * g.D, dtype=torch.bfloat16, device=dev)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    L_d, cnt, eos = i32(s.doc_prefix_len), i32(s.doc_branch_cnt), i32(s.eos_len)
    depth = torch.zeros(s.n_slots, dtype=torch.int32, device=dev)
    alive = torch.ones(s.n_slots, dtype=torch.uint8, device=dev)
    meta = B.MetaTables.alloc(g, s.n_docs, s.n_slots, s.total_prefix, dev)
    steps = int(s.eos_len.max())
    n_act = [int((s.eos_len > t).sum()) for t in range(steps)]
    stream = torch.cuda.current_stream()

    t_dev = torch.zeros((), dtype=torch.int32, device=dev)      # step counter on the device (the graph advances it)

    def one_step(t):
        # caller-side state of the loop (which branches are still decoding, how deep they are); t: host int or t_dev
        torch.minimum(eos, t_dev if t is None else torch.full_like(eos, t), out=depth)
        alive.copy_((eos > (t_dev if t is None else t)).to(torch.uint8))
        B.hpd_build_meta(g, s.n_docs, s.n_slots, L_d, cnt, depth, alive, 0, meta)
        for l in range(L):
            b = l & 1
            B.hpd_rope_append(g, s.n_slots, s.n_slots, meta.n_active, meta.pos_id, meta.suffix_off, meta.suffix_len, q[b], kn[b],
                              vn[b], suf_k[l], suf_v[l], meta.dev_status)
            B.hpd_attn_decode(g, s.n_docs, s.n_slots, s.n_slots, s.total_prefix, q[b], pre_k[l], pre_v[l], suf_k[l],
                              suf_v[l], L_d, meta, True, o, None)

    for t in range(min(3, steps)):
        one_step(t)
    torch.cuda.synchronize()
    sampler = ClockSampler(0); sampler.start(); time.sleep(0.3)
    graph = None
    if not args.no_graph:
        # one decode step (table build + all layers) captured once; the step counter lives on the device
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            one_step(None)
            t_dev.add_(1)
        t_dev.zero_()
        torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record(stream)
    for t in range(steps):
        if graph is not None:
            graph.replay()
        else:
            one_step(t)
        ev[t + 1].record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = [ev[t].elapsed_time(ev[t + 1]) for t in range(steps)]
    total_ms = ev[0].elapsed_time(ev[steps])
    tokens = sum(n_act)
    print(json.dumps({
        "metric": METRIC, "value": tokens / (total_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": 3,
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": {"workload": f"{s.name}_L{L}", "layers": L, "prompts": s.n_prompts,
                                        "branches_per_prompt": 96, "suffix_cap": g.suffix_cap,
                                        "l2": "inputs larger than L2 (every layer has its own caches); no flush",
                                        "launch": "cuda graph replay of one decode step" if graph is not None else "direct calls"},
        "clocks": clocks, "gpu_launches": steps * (1 + 3 * L), "dev_status": int(meta.dev_status.item()),
        "per_layer_branch_tokens_per_s": tokens * L / (total_ms * 1e-3),
        "series": [{"step": t, "n_active": n_act[t], "ms": ms[t]} for t in range(steps)],
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="main")
    ap.add_argument("--cpu-rows", type=int, default=2048)
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-comparison", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay leg")
    ap.add_argument("--unfused", action="store_true", help="hpd_rope and hpd_kv_append as two launches instead of hpd_rope_append")
    ap.add_argument("--min-ms", type=float, default=1000.0, help="device time to cover with timed K-step blocks")
    ap.add_argument("--block-tokens", type=int, default=128, help="shared3 workloads: tokens of the block common to all documents")
    ap.add_argument("--two-pass", action="store_true", help="shared3 workloads: block attention as a second launch + hpd_merge_lse")
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--loop-prompts", type=int, default=64)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.workload == "loop" and args.impl != "reference":
        run_loop(args)
    elif args.workload.startswith("shared3_p") and args.impl != "reference":
        run_shared3(args)
    elif args.workload.startswith("prefill_p") and args.impl != "reference":
        run_prefill(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
