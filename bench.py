#!/usr/bin/env python
"""Benchmark of the BLoad packing path on B200.

One step = one pass of the whole path over one epoch of a synthetic workload: plan (validate,
scan, keys, sort, fill rule, inverse tables), per-slot metadata, pack of all blocks, unpack of a
per-frame output of all blocks, statistics.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With N > 1 (under torchrun) every rank runs an independent replica of the same workload on its own
GPU ("replicas only": the path has no exchange step); time is the maximum over ranks.
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
from types import SimpleNamespace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "pack+unpack GB/s (algorithmic bytes of the pack and unpack copies / time of the whole step)"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
POLICY = 0  # fill policy of this run (set from --policy)
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------------------------
def algorithmic_bytes(sum_t: int, n_blocks: int, t_block: int, fb: int, ofb: int) -> dict:
    """pack reads every frame once and writes every slot (padding included); unpack reads and
    writes every frame once (pad slots are not read); metadata writes 10 bytes per slot."""
    return dict(pack=sum_t * fb + n_blocks * t_block * fb, unpack=2 * sum_t * ofb, meta=10 * n_blocks * t_block)


def measured_peak() -> tuple[float, str]:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([time.monotonic()] + [x.strip() for x in line.split(",")])

    def mark(self):
        """Start of the timed region: only samples taken after this moment are reported."""
        self.t_mark = time.monotonic()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons, pw = [], [], set(), []
        t_mark = getattr(self, "t_mark", 0.0)
        rows = [r[1:] for r in self.rows if r[0] >= t_mark] or [r[1:] for r in self.rows[-1:]]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def host_memory_available() -> float:
    """Bytes of host memory that can still be allocated (MemAvailable of /proc/meminfo; +inf if unknown)."""
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return float(line.split()[1]) * 1024.0
    except Exception:
        pass
    return float("inf")


def dist_max(x: float, device=None) -> float:
    """Maximum of a per-rank scalar over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Whole-job throughput of `world` independent replicas: all units / slowest rank's time."""
    return units_per_rank * world / seconds_max


# ----------------------------------------------------------------------------------------------
class CpuOracleSample:
    """The CPU oracle, as it stands, on a bounded sample of the workload: the full plan, then
    metadata + pack + unpack of `target_blocks` consecutive blocks (0 = all), single thread.
    Buffers are set up once; run() times one pass."""

    def __init__(self, w, target_blocks: int):
        import numpy as np
        from oracle import bload_oracle as O
        from paper_2310_10879_b200 import workloads as W
        self.O, self.w = O, w
        self.T = W.lengths(w)
        op = self.plan()
        fb, ofb, tb = w.frame_bytes, w.out_frame_bytes, w.t_block
        self.cnt = cnt = min(target_blocks, op.n_blocks) if target_blocks > 0 else op.n_blocks
        self.b0 = b0 = (op.n_blocks - cnt) // 2
        # host store: only the frames of the sampled blocks' sequences are touched (the rest stays untouched
        # virtual memory); the output pages are faulted in before timing
        self.store = np.empty(op.sum_t * fb, np.uint8)
        self.ragged_out = np.empty(op.sum_t * ofb, np.uint8)
        self.frames = 0
        for k in range(op.block_seg_begin[b0], op.block_seg_begin[b0 + cnt]):
            s = int(op.seg_seq[k]); lo, hi = int(op.offsets[s]), int(op.offsets[s + 1])
            self.store[lo * fb:hi * fb] = (s * 37 + 11) & 255
            self.ragged_out[lo * ofb:hi * ofb] = 0
            self.frames += hi - lo
        self.dense_out = np.ones(cnt * tb * ofb, np.uint8)
        self.bytes = dict(pack=self.frames * fb + cnt * tb * fb, unpack=2 * self.frames * ofb)

    def plan(self):
        t0 = time.perf_counter()
        self.op = self.O.plan(self.T, self.w.t_block, self.w.seed, POLICY)
        self.t_plan = time.perf_counter() - t0
        return self.op

    def run_threaded(self, threads: int) -> dict:
        """The same sample with its blocks spread over `threads` host threads (contiguous block ranges; the oracle's C
        functions run outside the interpreter lock).  The plan is sequential and is not repeated here."""
        from concurrent.futures import ThreadPoolExecutor
        O, w, op = self.O, self.w, self.op
        fb, ofb = w.frame_bytes, w.out_frame_bytes
        threads = max(1, min(threads, self.cnt))
        cuts = [self.b0 + self.cnt * i // threads for i in range(threads + 1)]
        parts = [(cuts[i], cuts[i + 1] - cuts[i]) for i in range(threads) if cuts[i + 1] > cuts[i]]
        tbb = w.t_block * ofb

        def do_pack(part):
            O.pack(op, self.store, fb, part[0], part[1], 0)

        def do_unpack(part):
            lo = (part[0] - self.b0) * tbb
            O.unpack(op, self.dense_out[lo:lo + part[1] * tbb], ofb, part[0], part[1], self.ragged_out)

        with ThreadPoolExecutor(max_workers=len(parts)) as pool:
            t0 = time.perf_counter(); list(pool.map(do_pack, parts)); t_pack = time.perf_counter() - t0
            t0 = time.perf_counter(); list(pool.map(do_unpack, parts)); t_unpack = time.perf_counter() - t0
        by = self.bytes
        return {"cores": len(parts), "pack_GB/s": by["pack"] / t_pack / 1e9, "unpack_GB/s": by["unpack"] / t_unpack / 1e9,
                "value": (by["pack"] + by["unpack"]) / (t_pack + t_unpack) / 1e9, "unit": UNIT,
                "what": "pack + unpack of the same blocks spread over host threads (plan and metadata not included)"}

    def run(self) -> dict:
        O, w, op = self.O, self.w, self.plan()
        fb, ofb = w.frame_bytes, w.out_frame_bytes
        t0 = time.perf_counter(); O.metadata(op, self.b0, self.cnt); t_meta = time.perf_counter() - t0
        t0 = time.perf_counter(); O.pack(op, self.store, fb, self.b0, self.cnt, 0); t_pack = time.perf_counter() - t0
        t0 = time.perf_counter(); O.unpack(op, self.dense_out, ofb, self.b0, self.cnt, self.ragged_out)
        t_unpack = time.perf_counter() - t0
        by = self.bytes
        t_total = self.t_plan * self.cnt / op.n_blocks + t_meta + t_pack + t_unpack
        return dict(value=(by["pack"] + by["unpack"]) / t_total / 1e9, unit=UNIT, cores=1, kind="oracle",
                    sample="full plan (N=%d, %.3f s, charged pro rata) + metadata/pack/unpack of %d of %d blocks "
                           "(%d frames); pack %.2f GB/s, unpack %.2f GB/s, single thread"
                           % (op.n, self.t_plan, self.cnt, op.n_blocks, self.frames, by["pack"] / t_pack / 1e9,
                              by["unpack"] / t_unpack / 1e9),
                    seconds=self.t_plan + t_meta + t_pack + t_unpack, frames_per_s=self.frames / t_total,
                    plan_s=self.t_plan, pack_GBs=by["pack"] / t_pack / 1e9, unpack_GBs=by["unpack"] / t_unpack / 1e9,
                    _bytes=by["pack"] + by["unpack"], _t=t_total)


def run_reference(args, w) -> dict:
    """The reference arm: the CPU oracle on this machine's host cores, a bounded sample per step.  The
    sample (blocks per step) is sized from a 2-block calibration so that the whole run of
    warmup + steps stays near two minutes."""
    blocks = args.ref_blocks
    if blocks <= 0:
        cal = CpuOracleSample(w, 2).run()
        per_block = max(cal["seconds"] - cal["plan_s"], 1e-3) / 2
        seconds_per_step = 100.0 / max(1, args.warmup + args.steps) - cal["plan_s"]
        blocks = int(max(1, min(seconds_per_step / per_block, 64)))
    sample = CpuOracleSample(w, blocks)
    times, last = [], None
    for i in range(args.warmup + args.steps):
        r = sample.run()
        if i >= args.warmup:
            times.append(r["_t"])
        last = r
    t = sum(times) / len(times)
    value = last["_bytes"] / t / 1e9
    cb = {k: v for k, v in last.items() if not k.startswith("_")}
    cb["value"] = value
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": config_of(w, None), "cpu_baseline": cb,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def config_of(w, extra) -> dict:
    which = "configs[%d]" % w.index if 0 <= w.index <= 4 else "extra workload (not an evaluation configuration)"
    c = {"workload": "%s %s: N=%d, lengths %s, frame %d B (%s), T_block=%d, unpack of %d B/frame outputs; "
                     "one whole-epoch call per direction" % (which, w.name, w.n, w.dist, w.frame_bytes, w.payload,
                                                             w.t_block, w.out_frame_bytes),
         "batch_blocks": w.batch_blocks, "l2": "inputs larger than L2 (no flush needed)", "seed": w.seed,
         "policy": POLICY}
    if extra:
        c.update(extra)
    return c


# ----------------------------------------------------------------------------------------------
# ---- the same work as a two-stage pipeline: the plan of epoch e+1 runs on a side stream (one warp of one SM)
# under the metadata/pack/unpack traffic of epoch e; and eight plans side by side on eight streams
def _time_pipelined(c):
    torch, B, W, args, w, T, fb, ofb, tb, d_len, sizes, plan_buf, work, plan, nb, sum_t, by, store, dense, seq_id, pos, reset, valid, dense_out, ragged_out, ev, barrier, world, dev = (c.torch, c.B, c.W, c.args, c.w, c.T, c.fb, c.ofb, c.tb, c.d_len, c.sizes, c.plan_buf, c.work, c.plan, c.nb, c.sum_t, c.by, c.store, c.dense, c.seq_id, c.pos, c.reset, c.valid, c.dense_out, c.ragged_out, c.ev, c.barrier, c.world, c.dev)
    pipelined = None
    if not args.no_pipeline:
        side = torch.cuda.Stream(priority=-1)   # the planner's small kernels go ahead of queued copy CTAs
        main = torch.cuda.current_stream()
        bufs = [torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=dev) for _ in range(2)]
        work2 = torch.empty(sizes.work_bytes, dtype=torch.uint8, device=dev)

        def pipeline(steps):
            side.wait_stream(main)
            B.bload_plan_async(d_len, tb, w.seed, policy=args.policy, stream=side, work=work2, plan_buf=bufs[0])
            p = B.bload_plan_finish(bufs[0], sizes, stream=side)
            done = [None, None]
            for i in range(steps):
                nxt = (i + 1) % 2
                if done[nxt] is not None:
                    side.wait_event(done[nxt])          # the copies that read this plan buffer have finished
                B.bload_plan_async(d_len, tb, w.seed, policy=args.policy, stream=side, work=work2, plan_buf=bufs[nxt])
                B.bload_pack(p, None, fb, 0, nb, seq_id=seq_id, pos=pos, reset=reset, valid=valid)
                B.bload_pack(p, store, fb, 0, nb, dense=dense)
                B.bload_unpack(p, dense_out, ofb, 0, nb, ragged_out)
                done[i % 2] = main.record_event()
                p = B.bload_plan_finish(bufs[nxt], sizes, stream=side)   # the host waits for the plan only
                B.bload_stats(p.info)
            main.wait_stream(side)

        pipeline(3)
        torch.cuda.synchronize()
        psteps = max(10, min(args.steps, 100))
        a, b_ = ev(), ev()
        a.record(); pipeline(psteps); b_.record()
        torch.cuda.synchronize()
        pms = a.elapsed_time(b_) / psteps
        streams8 = [torch.cuda.Stream() for _ in range(8)]
        jobs8 = [(torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=dev),
                  torch.empty(sizes.work_bytes, dtype=torch.uint8, device=dev)) for _ in range(8)]

        def eight():
            for e, (st8, (pb, wk)) in enumerate(zip(streams8, jobs8)):
                st8.wait_stream(main)
                B.bload_plan_async(d_len, tb, w.seed + e, policy=args.policy, stream=st8, work=wk, plan_buf=pb)
            for st8, (pb, wk) in zip(streams8, jobs8):
                B.bload_plan_finish(pb, sizes, stream=st8)
        eight()
        torch.cuda.synchronize()
        t0 = time.perf_counter(); eight(); torch.cuda.synchronize(); t8 = (time.perf_counter() - t0) * 1e3
        pipelined = {"ms_per_step": pms, "value": (by["pack"] + by["unpack"]) / pms / 1e6, "unit": UNIT, "steps": psteps,
                     "what": "plan of epoch e+1 on a side stream under metadata+pack+unpack of epoch e (every step still "
                             "plans, packs and unpacks one whole epoch)",
                     "eight_plans_side_by_side_ms": t8, "plans_per_s": 8e3 / t8}
        del bufs, work2, jobs8
    return pipelined


# ---- the whole step as ONE call (bload_epoch): the fill rule in chunks on this stream, tables, metadata, pack and
# unpack of the blocks each chunk has closed on a side stream under the next chunk
def _time_fused_epoch(c):
    torch, B, W, args, w, T, fb, ofb, tb, d_len, sizes, plan_buf, work, plan, nb, sum_t, by, store, dense, seq_id, pos, reset, valid, dense_out, ragged_out, ev, barrier, world, dev = (c.torch, c.B, c.W, c.args, c.w, c.T, c.fb, c.ofb, c.tb, c.d_len, c.sizes, c.plan_buf, c.work, c.plan, c.nb, c.sum_t, c.by, c.store, c.dense, c.seq_id, c.pos, c.reset, c.valid, c.dense_out, c.ragged_out, c.ev, c.barrier, c.world, c.dev)
    fused = None
    if not args.no_fused:
        side2 = torch.cuda.Stream()
        chain = torch.cuda.Stream(priority=-1)  # the chain's single CTA goes ahead of queued copy CTAs

        def fused_step():
            chain.wait_stream(torch.cuda.current_stream())
            p = B.bload_epoch(d_len, tb, w.seed, nb, store=store, frame_bytes=fb, dense=dense, seq_id=seq_id, pos=pos,
                              reset=reset, valid=valid, dense_out=dense_out, out_frame_bytes=ofb, ragged_out=ragged_out,
                              stream=chain, side_stream=side2, work=work, plan_buf=plan_buf)
            return B.bload_stats(p.info)
        for _ in range(max(3, args.warmup)):
            fused_step()
        barrier()
        a, b_ = ev(), ev()
        a.record()
        for _ in range(args.steps):
            fused_step()
        b_.record()
        barrier()
        f_s = dist_max(a.elapsed_time(b_) / 1e3, dev) / args.steps
        B.bload_set_plan_timing(True)
        fused_step()
        st_ms = B.bload_epoch_stage_times()
        B.bload_set_plan_timing(False)
        fused = {"ms_per_step": f_s * 1e3, "value": aggregate(by["pack"] + by["unpack"], world, f_s) / 1e9, "unit": UNIT,
                 "steps": args.steps,
                 "what": "bload_epoch: one call per step = plan + metadata + pack + unpack of the whole epoch, copies of "
                         "finished blocks on a side stream while the fill rule is still running",
                 "stage_ms_summed_over_chunks": {"fill": st_ms[0], "tables": st_ms[1], "metadata": st_ms[2],
                                                 "pack": st_ms[3], "unpack": st_ms[4]}}
    return fused


# ---- batch-by-batch use: one pack call (metadata + dense) per training batch of w.batch_blocks blocks,
# the last batch rounded up with filler blocks; the output buffers of one batch are reused
def _time_per_batch(c):
    torch, B, W, args, w, T, fb, ofb, tb, d_len, sizes, plan_buf, work, plan, nb, sum_t, by, store, dense, seq_id, pos, reset, valid, dense_out, ragged_out, ev, barrier, world, dev = (c.torch, c.B, c.W, c.args, c.w, c.T, c.fb, c.ofb, c.tb, c.d_len, c.sizes, c.plan_buf, c.work, c.plan, c.nb, c.sum_t, c.by, c.store, c.dense, c.seq_id, c.pos, c.reset, c.valid, c.dense_out, c.ragged_out, c.ev, c.barrier, c.world, c.dev)
    bb = w.batch_blocks
    n_batches = (nb + bb - 1) // bb
    per_batch = None
    if not args.no_batch and n_batches * bb * tb * fb <= dense.numel() + bb * tb * fb:
        b_dense = torch.empty(bb * tb * fb, dtype=torch.uint8, device=dev)
        b_meta = [torch.empty(bb * tb, dtype=d, device=dev) for d in (torch.int32, torch.int32, torch.uint8, torch.uint8)]
        reps = max(1, min(n_batches, 4000))

        def batch_loop():
            for i in range(reps):
                B.bload_pack(plan, store, fb, i * bb, bb, dense=b_dense, seq_id=b_meta[0], pos=b_meta[1],
                             reset=b_meta[2], valid=b_meta[3])
        batch_loop()
        torch.cuda.synchronize()
        l0 = B.bload_kernel_launches()
        a, b_ = ev(), ev()
        a.record(); batch_loop(); b_.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b_)
        per_batch = {"batch_blocks": bb, "batches_timed": reps, "us_per_call": ms * 1e3 / reps,
                     "GB/s": (2 * bb * tb * fb) * reps / ms / 1e6,
                     "launches_per_call": (B.bload_kernel_launches() - l0) / reps, "kernel": B.bload_last_copy_kernel("pack")}
        # the same loop captured once in a CUDA graph and replayed (the calls are asynchronous and allocate nothing)
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    batch_loop()
            torch.cuda.current_stream().wait_stream(side)
            graph.replay()
            torch.cuda.synchronize()
            a, b_ = ev(), ev()
            a.record(); graph.replay(); b_.record()
            torch.cuda.synchronize()
            gms = a.elapsed_time(b_)
            per_batch["graph_us_per_call"] = gms * 1e3 / reps
            per_batch["graph_GB/s"] = (2 * bb * tb * fb) * reps / gms / 1e6
            del graph
        except Exception as exc:  # capture is an optimisation of the measurement, not part of the path
            per_batch["graph_us_per_call"] = None
            per_batch["graph_error"] = str(exc)[:200]
        del b_dense, b_meta
    return per_batch


# ---- consumer side of the start table (not part of the step): the shifted copy over the whole epoch, the
# masked sum of a per-slot loss, and the per-slot state reset of a batch
def _time_consumer(c):
    torch, B, W, args, w, T, fb, ofb, tb, d_len, sizes, plan_buf, work, plan, nb, sum_t, by, store, dense, seq_id, pos, reset, valid, dense_out, ragged_out, ev, barrier, world, dev = (c.torch, c.B, c.W, c.args, c.w, c.T, c.fb, c.ofb, c.tb, c.d_len, c.sizes, c.plan_buf, c.work, c.plan, c.nb, c.sum_t, c.by, c.store, c.dense, c.seq_id, c.pos, c.reset, c.valid, c.dense_out, c.ragged_out, c.ev, c.barrier, c.world, c.dev)
    consumer = None
    if not args.no_consumer:
        def timed(fn, reps):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            a, b_ = ev(), ev()
            a.record()
            for _ in range(reps):
                fn()
            b_.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b_) / reps
        prev = torch.empty_like(dense)
        ms = timed(lambda: B.bload_carry_prev(plan, dense, fb, 0, nb, prev), 20)
        cp_bytes = (sum_t - T.size) * fb + nb * tb * fb
        del prev
        vals = torch.empty(nb * tb, dtype=torch.float32, device=dev).normal_()
        bsum = torch.empty(nb, dtype=torch.float64, device=dev)
        tot = torch.empty(2, dtype=torch.float64, device=dev)
        ms_sum = timed(lambda: B.bload_valid_sum(plan, vals, 0, nb, bsum, tot), 20)
        bb = min(w.batch_blocks, nb)
        state = torch.zeros(bb * 4096, dtype=torch.uint8, device=dev)
        ms_reset = timed(lambda: B.bload_reset_state(plan, 0, bb, tb // 2, state, 4096), 200)
        # per-sample frame sizes: the same lengths, frame sizes drawn from {1/4, 1/2, 3/4, 1} of the workload's frame
        var = None
        if fb >= 64:
            import numpy as np
            rngv = np.random.Generator(np.random.PCG64(w.seed + 77))
            Fv = (rngv.integers(1, 5, size=T.size) * (fb // 4)).astype(np.int32)
            d_Fv = torch.from_numpy(Fv).to(dev)
            boff, vinfo = B.bload_var_offsets(d_len, d_Fv)
            vstore = torch.empty(vinfo.total_bytes, dtype=torch.uint8, device=dev)
            vstore.view(torch.int32)[:].random_() if vinfo.total_bytes % 4 == 0 else vstore.random_()
            vback = torch.empty_like(vstore)
            ms_p = timed(lambda: B.bload_pack_var(plan, vstore, d_Fv, boff, fb, 0, nb, dense), 10)
            ms_u = timed(lambda: B.bload_unpack_var(plan, dense, d_Fv, boff, fb, 0, nb, vback), 10)
            ok = bool(torch.equal(vback, vstore))
            var = {"frame_bytes": "uniform over {1/4, 1/2, 3/4, 1} x %d" % fb, "slot_bytes": fb,
                   "store_bytes": int(vinfo.total_bytes),
                   "pack_ms": ms_p, "pack_GB/s": (vinfo.total_bytes + nb * tb * fb) / ms_p / 1e6,
                   "unpack_ms": ms_u, "unpack_GB/s": 2 * vinfo.total_bytes / ms_u / 1e6, "round_trip_ok": ok}
            del vstore, vback, boff
        consumer = {"carry_prev": {"ms": ms, "GB/s": cp_bytes / ms / 1e6, "algorithmic_bytes": cp_bytes,
                                   "what": "prev[q,s] = dense[q,s-1] inside sequences, fill elsewhere, all blocks; "
                                           "bytes = (sum_t - n) frames read + n_blocks*t_block frames written"},
                    "valid_sum": {"ms": ms_sum, "GB/s": 4 * sum_t / ms_sum / 1e6, "slots": nb * tb,
                                  "what": "fp32 per-slot values, frames only, per-block and total sums in double; "
                                          "bytes = 4 per frame read"},
                    "reset_state": {"us_per_call": ms_reset * 1e3, "batch_blocks": bb, "state_bytes": 4096},
                    "var_frames": var}
        del vals, bsum, tot, state
    return consumer


# ---- end to end through the same calls with HOST buffers (pinned), copies inside the timed region
def _time_end_to_end(c):
    torch, B, W, args, w, T, fb, ofb, tb, d_len, sizes, plan_buf, work, plan, nb, sum_t, by, store, dense, seq_id, pos, reset, valid, dense_out, ragged_out, ev, barrier, world, dev = (c.torch, c.B, c.W, c.args, c.w, c.T, c.fb, c.ofb, c.tb, c.d_len, c.sizes, c.plan_buf, c.work, c.plan, c.nb, c.sum_t, c.by, c.store, c.dense, c.seq_id, c.pos, c.reset, c.valid, c.dense_out, c.ragged_out, c.ev, c.barrier, c.world, c.dev)
    e2e = None
    e2e_need = T.size * 4 + store.numel() + dense_out.numel() + dense.numel() + 10 * nb * tb + ragged_out.numel()
    e2e_second_set = 1.05 * (store.numel() + dense_out.numel() + dense.numel() + 10 * nb * tb + ragged_out.numel())
    if not args.no_e2e and torch.cuda.mem_get_info()[0] < e2e_second_set:
        e2e = {"value": None, "unit": UNIT, "skipped": "not enough free device memory for the second buffer set"}
    elif not args.no_e2e and host_memory_available() < 1.3 * e2e_need * max(1, int(os.environ.get("LOCAL_WORLD_SIZE", world))):
        e2e = {"value": None, "unit": UNIT, "skipped": "not enough free host memory for the pinned buffers of all local ranks"}
    elif not args.no_e2e:
        h_len = torch.from_numpy(T).pin_memory()
        h_store = torch.empty(store.numel(), dtype=torch.uint8, pin_memory=True); h_store.copy_(store)
        h_dense = torch.empty(dense.numel(), dtype=torch.uint8, pin_memory=True)
        h_meta = [torch.empty(x.numel(), dtype=x.dtype, pin_memory=True) for x in (seq_id, pos, reset, valid)]
        h_dense_out = torch.empty(dense_out.numel(), dtype=torch.uint8, pin_memory=True); h_dense_out.copy_(dense_out)
        h_ragged_out = torch.empty(ragged_out.numel(), dtype=torch.uint8, pin_memory=True)
        h2d = h_len.numel() * 4 + h_store.numel() + h_dense_out.numel()
        d2h = h_dense.numel() + sum(x.numel() * x.element_size() for x in h_meta) + h_ragged_out.numel()

        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        # two sets of device buffers, used in turn, so that consecutive steps overlap: the uploads of step i+1 run
        # while step i is still downloading its results (PCIe is full duplex); every step still uploads all of its
        # inputs and downloads all of its outputs inside the timed region
        sets = [dict(d_len=d_len, store=store, dense=dense, meta=(seq_id, pos, reset, valid), dense_out=dense_out,
                     ragged_out=ragged_out, plan_buf=plan_buf)]
        sets.append(dict(d_len=torch.empty_like(d_len), store=torch.empty_like(store), dense=torch.empty_like(dense),
                         meta=tuple(torch.empty_like(x) for x in (seq_id, pos, reset, valid)),
                         dense_out=torch.empty_like(dense_out), ragged_out=torch.empty_like(ragged_out),
                         plan_buf=torch.empty_like(plan_buf)))
        for st_ in sets:
            st_["kernels_done"] = None   # event: the kernels of the step that last used this set have finished
            st_["dense_read"] = None     # event: its dense/metadata download has finished
            st_["ragged_read"] = None    # event: its ragged download has finished
        counter = [0]

        def e2e_step():
            # three streams: host->device copies, the library's kernels, device->host copies.  The plan needs only
            # the lengths, so it runs while the store is still arriving; the dense batches leave while the per-frame
            # outputs arrive.
            cur = torch.cuda.current_stream()
            S = sets[counter[0] & 1]
            counter[0] += 1
            with torch.cuda.stream(s_in):
                if S["kernels_done"] is not None:
                    s_in.wait_event(S["kernels_done"])
                S["d_len"].copy_(h_len, non_blocking=True)
                ev_len = s_in.record_event()
                S["store"].copy_(h_store, non_blocking=True)
                ev_store = s_in.record_event()
                S["dense_out"].copy_(h_dense_out, non_blocking=True)
                ev_outputs = s_in.record_event()
            cur.wait_event(ev_len)
            p = B.bload_plan(S["d_len"], tb, w.seed, policy=args.policy, work=work, plan_buf=S["plan_buf"])
            cur.wait_event(ev_store)
            if S["dense_read"] is not None:
                cur.wait_event(S["dense_read"])
            m = S["meta"]
            B.bload_pack(p, S["store"], fb, 0, nb, dense=S["dense"], seq_id=m[0], pos=m[1], reset=m[2], valid=m[3])
            ev_packed = cur.record_event()
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_packed)
                h_dense.copy_(S["dense"], non_blocking=True)
                for h, d in zip(h_meta, m):
                    h.copy_(d, non_blocking=True)
                S["dense_read"] = s_out.record_event()
            cur.wait_event(ev_outputs)
            if S["ragged_read"] is not None:
                cur.wait_event(S["ragged_read"])
            B.bload_unpack(p, S["dense_out"], ofb, 0, nb, S["ragged_out"])
            S["kernels_done"] = cur.record_event()
            with torch.cuda.stream(s_out):
                s_out.wait_event(S["kernels_done"])
                h_ragged_out.copy_(S["ragged_out"], non_blocking=True)
                S["ragged_read"] = s_out.record_event()
            return B.bload_stats(p.info)

        def e2e_drain():
            torch.cuda.current_stream().wait_stream(s_out)
            torch.cuda.current_stream().wait_stream(s_in)

        e2e_step(); e2e_step()
        e2e_drain()
        barrier()
        a, b_ = ev(), ev()
        a.record()
        s_in.wait_stream(torch.cuda.current_stream()); s_out.wait_stream(torch.cuda.current_stream())
        for _ in range(args.e2e_steps):
            e2e_step()
        e2e_drain()
        b_.record()
        barrier()
        e2e_s = dist_max(a.elapsed_time(b_) / 1e3, dev) / args.e2e_steps
        # one more step on its own (nothing to overlap with): the latency of a single step
        a, b_ = ev(), ev()
        a.record()
        s_in.wait_stream(torch.cuda.current_stream()); s_out.wait_stream(torch.cuda.current_stream())
        e2e_step()
        e2e_drain()
        b_.record()
        barrier()
        e2e = {"value": aggregate(by["pack"] + by["unpack"], world, e2e_s) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s * 1e3,
               "steps": args.e2e_steps, "single_step_ms": a.elapsed_time(b_),
               "how": "pinned host buffers; every step uploads lengths, store and per-frame outputs and downloads dense, "
                      "metadata and the ragged result; two device buffer sets used in turn, so the uploads of step i+1 "
                      "overlap the downloads of step i; timed from the first upload to the last download of the last step"}
        del sets
        del h_store, h_dense, h_dense_out, h_ragged_out
    return e2e


def run_gpu(args, w) -> dict:
    import torch
    import torch.distributed as dist

    import paper_2310_10879_b200 as B
    from paper_2310_10879_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback of the packing path")
    B.load()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=dev)

    T = W.lengths(w)
    fb, ofb, tb = w.frame_bytes, w.out_frame_bytes, w.t_block
    d_len = torch.from_numpy(T).to(dev)
    sizes = B.bload_plan_sizes(T.size, tb)
    plan_buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=dev)
    work = torch.empty(sizes.work_bytes, dtype=torch.uint8, device=dev)
    plan = B.bload_plan(d_len, tb, w.seed, policy=args.policy, work=work, plan_buf=plan_buf)
    nb, sum_t = plan.n_blocks, plan.sum_t
    by = algorithmic_bytes(sum_t, nb, tb, fb, ofb)

    store = W.payload_torch(w, sum_t, dev).view(torch.uint8).reshape(-1)
    dense = torch.empty(nb * tb * fb, dtype=torch.uint8, device=dev)
    seq_id = torch.empty(nb * tb, dtype=torch.int32, device=dev)
    pos = torch.empty(nb * tb, dtype=torch.int32, device=dev)
    reset = torch.empty(nb * tb, dtype=torch.uint8, device=dev)
    valid = torch.empty(nb * tb, dtype=torch.uint8, device=dev)
    dense_out = W.payload_torch(w, nb * tb, dev, out=True).view(torch.uint8).reshape(-1)
    ragged_out = torch.empty(sum_t * ofb, dtype=torch.uint8, device=dev)

    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(rec=None):
        e = [ev() for _ in range(5)] if rec is not None else None
        if e: e[0].record()
        p = B.bload_plan(d_len, tb, w.seed, policy=args.policy, work=work, plan_buf=plan_buf)
        if e: e[1].record()
        B.bload_pack(p, None, fb, 0, nb, seq_id=seq_id, pos=pos, reset=reset, valid=valid)
        if e: e[2].record()
        B.bload_pack(p, store, fb, 0, nb, dense=dense)
        if e: e[3].record()
        B.bload_unpack(p, dense_out, ofb, 0, nb, ragged_out)
        if e: e[4].record()
        st = B.bload_stats(p.info)
        if rec is not None:
            rec.append((e, st))
        return st

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    launches0 = B.bload_kernel_launches()
    rec = []
    t_begin, t_end = ev(), ev()
    barrier()
    sampler.mark()
    t_begin.record()
    for _ in range(args.steps):
        stats = step(rec)
    t_end.record()
    barrier()
    launches = B.bload_kernel_launches() - launches0
    # planner stage times from a few extra, untimed plans (the library's stage events stay out of the timed steps)
    B.bload_set_plan_timing(True)
    stage_runs = []
    for _ in range(5):
        B.bload_plan(d_len, tb, w.seed, policy=args.policy, work=work, plan_buf=plan_buf)
        stage_runs.append(B.bload_plan_stage_times())
    B.bload_set_plan_timing(False)
    seconds = dist_max(t_begin.elapsed_time(t_end) / 1e3, dev)
    clocks = sampler.stop()

    def avg(i):
        return sum(r[0][i].elapsed_time(r[0][i + 1]) for r in rec) / len(rec)
    plan_ms, meta_ms, pack_ms, unpack_ms = avg(0), avg(1), avg(2), avg(3)
    stage = [sum(r[i] for r in stage_runs) / len(stage_runs) for i in range(4)]
    step_s = seconds / args.steps
    value = aggregate(by["pack"] + by["unpack"], world, step_s) / 1e9

    c = SimpleNamespace(torch=torch, B=B, W=W, args=args, w=w, T=T, fb=fb, ofb=ofb, tb=tb, d_len=d_len, sizes=sizes,
                        plan_buf=plan_buf, work=work, plan=plan, nb=nb, sum_t=sum_t, by=by, store=store, dense=dense,
                        seq_id=seq_id, pos=pos, reset=reset, valid=valid, dense_out=dense_out, ragged_out=ragged_out,
                        ev=ev, barrier=barrier, world=world, dev=dev)
    pipelined = _time_pipelined(c)
    fused = _time_fused_epoch(c)
    per_batch = _time_per_batch(c)
    consumer = _time_consumer(c)

    def timed_launch(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b_ = ev(), ev()
        a.record()
        for _ in range(reps):
            fn()
        b_.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b_) / reps
    rank_share = rank_share_figures(c, timed_launch) if not args.no_consumer else None
    e2e = _time_end_to_end(c)
    if rank != 0:
        return {}

    peak, peak_kind = measured_peak()
    # the names of the copy kernels are the library's own answer for the calls of the timed steps
    k_pack, k_unpack = B.bload_last_copy_kernel("pack"), B.bload_last_copy_kernel("unpack")
    kernels = {k_unpack: (unpack_ms, by["unpack"]), k_pack: (pack_ms, by["pack"]), "k4_fill": (stage[2], None)}
    dom = max((k_unpack, k_pack), key=lambda k: kernels[k][0])
    d_ms, d_bytes = kernels[dom]
    achieved = d_bytes / (d_ms / 1e3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": "of " + peak_kind, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "traffic": TRAFFIC.get((w.name, dom)) if not (args.n or args.frame_bytes or args.policy) else None,
                "note": "largest HBM-bound kernel of the step; the planner's fill rule (k4_fill, %.2f ms) is a latency-bound "
                        "chain of dependent draws on one warp and is reported in kernels.plan as time and draws/s" % stage[2], "launch_ms": d_ms, "algorithmic_bytes_per_launch": d_bytes}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "u8", "data": "synthetic", "config": config_of(w, {"parallelism": "replicas only"}),
           "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
           "frames_per_s": aggregate(sum_t, world, step_s), "per_batch_pack": per_batch, "pipelined": pipelined, "fused_epoch": fused, "consumer": consumer,
           "one_rank_of_eight": rank_share,
           "kernels": {
               "pack_copy": {"kernel": k_pack, "ms": pack_ms, "GB/s": by["pack"] / pack_ms / 1e6, "frac_measured": by["pack"] / pack_ms / 1e6 / peak,
                             "frac_nominal": by["pack"] / pack_ms / 1e6 / NOMINAL_HBM_GBS, "frames_per_s": sum_t / pack_ms * 1e3},
               "unpack_copy": {"kernel": k_unpack, "ms": unpack_ms, "GB/s": by["unpack"] / unpack_ms / 1e6,
                               "frac_measured": by["unpack"] / unpack_ms / 1e6 / peak,
                               "frac_nominal": by["unpack"] / unpack_ms / 1e6 / NOMINAL_HBM_GBS,
                               "frames_per_s": sum_t / unpack_ms * 1e3},
               "metadata": {"ms": meta_ms, "GB/s": by["meta"] / meta_ms / 1e6},
               "plan": plan_figures(plan_ms, stage, T.size, clocks)},
           "padding": {"n": stats["n"], "sum_t": stats["sum_t"], "t_max": stats["t_max"], "n_blocks": stats["n_blocks"],
                       "min_blocks": stats["min_blocks"], "frac_packed": stats["frac_packed"],
                       "frac_naive_tmax": stats["frac_naive_tmax"], "frac_naive_tblock": stats["frac_naive_tblock"],
                       "reduction_vs_tmax": stats["reduction_vs_tmax"],
                       "chunking_strategy": chunk_strategy_figures(B, torch, d_len, tb)}}
    if not args.no_cpu and world == 1:
        blocks = args.ref_blocks
        need = (fb + ofb) * (sum_t + nb * tb) * 1.3          # host arrays of a whole-workload sample
        if blocks <= 0 and host_memory_available() < need:
            blocks = max(1, int(nb * host_memory_available() / need / 1.5))
        sample = CpuOracleSample(w, blocks)
        cb = sample.run()
        out["cpu_baseline"] = {k: v for k, v in cb.items() if not k.startswith("_")}
        out["cpu_baseline"]["all_cores"] = sample.run_threaded(host_cores())
        del sample
    else:
        out["cpu_baseline"] = None
    if not args.no_by_config and world == 1 and not (args.n or args.frame_bytes):
        # the other large configurations, one after the other, with the buffers of this one released first
        del c, store, dense, seq_id, pos, reset, valid, dense_out, ragged_out, plan, plan_buf, work
        torch.cuda.empty_cache()
        out["by_config"] = {name: measure_config(args, W.WORKLOADS[name], dev, peak, clocks)
                            for name in BY_CONFIG if name != w.name}
    return out


BY_CONFIG = ("raw_frames", "tokens")


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def chunk_strategy_figures(B, torch, d_len, t_block) -> dict:
    """The chunking strategy the paper compares with, as a planner on the same lengths (context for the padding figures):
    chunks of an eighth of the block length, tails kept and tails dropped; device time of count + plan per variant."""
    out = {}
    c = max(1, t_block // 8)
    for name, tail in (("keep_tail", 0), ("drop_tail", 1)):
        try:
            B.bload_plan_chunks(d_len, c, tail)                      # warm-up
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            plan, ci, _, _ = B.bload_plan_chunks(d_len, c, tail)
            b_.record(); torch.cuda.synchronize()
            out[name] = {"t_chunk": c, "n_chunks": int(ci.n_chunks), "pad_frames": int(ci.pad_frames),
                         "frames_deleted": int(ci.frames_deleted), "frac_padding": ci.pad_frames / max(1, ci.n_chunks * c),
                         "frac_deleted": ci.frames_deleted / max(1, ci.sum_t), "count_and_plan_ms": a.elapsed_time(b_)}
            del plan
        except Exception as exc:                                     # e.g. nothing is kept when every sequence is shorter
            out[name] = {"t_chunk": c, "error": str(exc)[:120]}
    return out


def rank_share_figures(c, timed) -> dict:
    """What ONE of eight data-parallel ranks does per epoch (the paper's setting; every rank computes the same plan and
    takes its own contiguous block range, bload_rank_range): pack and unpack of that range, whole-range launches."""
    B, torch = c.B, c.torch
    b0, cnt = B.bload_rank_range(c.nb, 8, 3, c.w.batch_blocks)
    real = max(0, min(c.nb, b0 + cnt) - b0)
    fill = int(c.plan.tables()["block_fill"][b0:b0 + real].to(torch.int64).sum().item())
    bb = c.tb * c.fb
    dense = c.dense[:min(cnt, c.nb) * bb] if cnt * bb <= c.dense.numel() else torch.empty(cnt * bb, dtype=torch.uint8, device=c.dev)
    ms_p = timed(lambda: B.bload_pack(c.plan, c.store, c.fb, b0, cnt, dense=dense))
    k_p = B.bload_last_copy_kernel("pack")
    obb = c.tb * c.ofb
    dout = c.dense_out[:cnt * obb] if cnt * obb <= c.dense_out.numel() else torch.empty(cnt * obb, dtype=torch.uint8, device=c.dev)
    ms_u = timed(lambda: B.bload_unpack(c.plan, dout, c.ofb, b0, cnt, c.ragged_out))
    k_u = B.bload_last_copy_kernel("unpack")
    return {"world": 8, "rank": 3, "block_begin": b0, "block_count": cnt, "frames": fill,
            "pack": {"kernel": k_p, "ms": ms_p, "GB/s": (fill * c.fb + cnt * bb) / ms_p / 1e6},
            "unpack": {"kernel": k_u, "ms": ms_u, "GB/s": 2 * fill * c.ofb / ms_u / 1e6}}


def plan_figures(plan_ms, stage, n, clocks) -> dict:
    """Stage times of the planner; the fill rule (a chain of n dependent draws on one warp) also as time and SM
    cycles per draw, the cycles from the median SM clock sampled while the timed region ran."""
    fill_ns = stage[2] * 1e6 / n if n else None
    mhz = clocks.get("sm_mhz") if clocks else None
    return {"ms": plan_ms, "scan_keys_ms": stage[0], "sort_ms": stage[1], "fill_ms": stage[2], "tables_ms": stage[3],
            "draws_per_s": n / stage[2] * 1e3 if stage[2] > 0 else None, "ns_per_draw": fill_ns,
            "cycles_per_draw": fill_ns * mhz / 1e3 if fill_ns and mhz else None, "sm_mhz_used": mhz}


def measure_config(args, w, dev, peak, clocks) -> dict:
    """Whole-epoch kernel times of one more workload (context beside the headline): every launch bracketed by CUDA
    events on the launching stream, the kernel names as the library reports them, planner stages, per-batch calls, and
    the CPU oracle on a bounded sample of the same workload (one thread and all host cores)."""
    import torch

    import paper_2310_10879_b200 as B
    from paper_2310_10879_b200 import workloads as W

    T = W.lengths(w)
    fb, ofb, tb = w.frame_bytes, w.out_frame_bytes, w.t_block
    d_len = torch.from_numpy(T).to(dev)
    sizes = B.bload_plan_sizes(T.size, tb)
    plan_buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=dev)
    work = torch.empty(sizes.work_bytes, dtype=torch.uint8, device=dev)
    plan = B.bload_plan(d_len, tb, w.seed, policy=args.policy, work=work, plan_buf=plan_buf)
    nb, sum_t = plan.n_blocks, plan.sum_t
    by = algorithmic_bytes(sum_t, nb, tb, fb, ofb)
    store = W.payload_torch(w, sum_t, dev).view(torch.uint8).reshape(-1)
    dense = torch.empty(nb * tb * fb, dtype=torch.uint8, device=dev)
    seq_id = torch.empty(nb * tb, dtype=torch.int32, device=dev)
    pos = torch.empty(nb * tb, dtype=torch.int32, device=dev)
    reset = torch.empty(nb * tb, dtype=torch.uint8, device=dev)
    valid = torch.empty(nb * tb, dtype=torch.uint8, device=dev)
    dense_out = W.payload_torch(w, nb * tb, dev, out=True).view(torch.uint8).reshape(-1)
    ragged_out = torch.empty(sum_t * ofb, dtype=torch.uint8, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        pairs = []
        for _ in range(reps):   # inputs and outputs are far larger than L2, so back-to-back launches start cold
            a, b_ = ev(), ev()
            a.record(); fn(); b_.record()
            pairs.append((a, b_))
        torch.cuda.synchronize()
        ms = sorted(a.elapsed_time(b_) for a, b_ in pairs)
        return ms[len(ms) // 2]

    meta_ms = timed(lambda: B.bload_pack(plan, None, fb, 0, nb, seq_id=seq_id, pos=pos, reset=reset, valid=valid))
    pack_ms = timed(lambda: B.bload_pack(plan, store, fb, 0, nb, dense=dense))
    k_pack = B.bload_last_copy_kernel("pack")
    unpack_ms = timed(lambda: B.bload_unpack(plan, dense_out, ofb, 0, nb, ragged_out))
    k_unpack = B.bload_last_copy_kernel("unpack")
    prev = torch.empty_like(dense)
    carry_ms = timed(lambda: B.bload_carry_prev(plan, dense, fb, 0, nb, prev))
    k_carry = B.bload_last_copy_kernel("carry_prev")
    del prev
    cp_bytes = (sum_t - T.size) * fb + nb * tb * fb
    B.bload_set_plan_timing(True)
    stage_runs = []
    t_plan = []
    for _ in range(3):
        a, b_ = ev(), ev()
        a.record()
        B.bload_plan(d_len, tb, w.seed, policy=args.policy, work=work, plan_buf=plan_buf)
        b_.record(); torch.cuda.synchronize()
        t_plan.append(a.elapsed_time(b_))
        stage_runs.append(B.bload_plan_stage_times())
    B.bload_set_plan_timing(False)
    stage = [sum(r[i] for r in stage_runs) / len(stage_runs) for i in range(4)]
    st = B.bload_stats(plan.info)

    def rate(nbytes, ms):
        g = nbytes / ms / 1e6
        return {"ms": ms, "GB/s": g, "frac_measured": g / peak, "frac_nominal": g / NOMINAL_HBM_GBS,
                "algorithmic_bytes": nbytes}
    c = SimpleNamespace(torch=torch, B=B, W=W, args=args, w=w, T=T, fb=fb, ofb=ofb, tb=tb, d_len=d_len, sizes=sizes,
                        plan_buf=plan_buf, work=work, plan=plan, nb=nb, sum_t=sum_t, by=by, store=store, dense=dense,
                        seq_id=seq_id, pos=pos, reset=reset, valid=valid, dense_out=dense_out, ragged_out=ragged_out,
                        ev=ev, barrier=torch.cuda.synchronize, world=1, dev=dev)
    out = {"workload": config_of(w, None)["workload"], "n_blocks": nb, "sum_t": sum_t,
           "kernels": {"pack_copy": dict(rate(by["pack"], pack_ms), kernel=k_pack, frames_per_s=sum_t / pack_ms * 1e3),
                       "unpack_copy": dict(rate(by["unpack"], unpack_ms), kernel=k_unpack, frames_per_s=sum_t / unpack_ms * 1e3),
                       "metadata": dict(rate(by["meta"], meta_ms), kernel="k6_metadata"),
                       "carry_prev": dict(rate(cp_bytes, carry_ms), kernel=k_carry),
                       "plan": plan_figures(sum(t_plan) / len(t_plan), stage, T.size, clocks)},
           "per_batch_pack": _time_per_batch(c),
           "one_rank_of_eight": rank_share_figures(c, timed),
           "padding": {"n_blocks": st["n_blocks"], "min_blocks": st["min_blocks"], "frac_packed": st["frac_packed"],
                       "frac_naive_tmax": st["frac_naive_tmax"], "reduction_vs_tmax": st["reduction_vs_tmax"],
                       "chunking_strategy": chunk_strategy_figures(B, torch, d_len, tb)}}
    del c, store, dense, seq_id, pos, reset, valid, dense_out, ragged_out, plan, plan_buf, work
    torch.cuda.empty_cache()
    if not args.no_cpu:
        # bounded sample: about 2 GB of dense blocks from the middle of the epoch
        blocks = max(1, min(nb, (2 << 30) // max(1, tb * (fb + ofb))))
        sample = CpuOracleSample(w, blocks)
        cb = sample.run()
        out["cpu_baseline"] = {k: v for k, v in cb.items() if not k.startswith("_")}
        out["cpu_baseline"]["all_cores"] = sample.run_threaded(host_cores())
        del sample
    return out


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of one whole-epoch launch, keyed by workload and
# by the kernel name the library reports; taken once from an ncu capture of a 1,500-sequence case of the same workload
# and scaled by frames (traffic grows in proportion to the frames moved).  Reads equal the algorithmic bytes, writes are
# slightly below them (the tail of the output is still in L2 when the kernel ends).  An entry is removed when its
# kernel changes; a missing entry reports null.
def frame_sweep(args) -> dict:
    """Pack, whole-plan unpack and sub-range unpack across frame sizes and three shapes of length distribution (token
    lengths, the heavy-tailed lengths, the clip lengths of the paper's dataset), about 1.5 GB per direction and case: which
    kernel the library chooses and what it reaches.  Not a step of the benchmark; printed as its own JSON line."""
    import torch
    import paper_2310_10879_b200 as B
    from paper_2310_10879_b200 import workloads as W
    dev = torch.device("cuda:0")
    peak, _ = measured_peak()
    mean_len = {"tokens": 868.0, "heavy_tail_bf16": 57.8, "video_dataset_shape": 22.3}
    sizes = [int(x) for x in args.frame_sweep.split(",")] if args.frame_sweep != "default" else \
        [1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 48, 64, 100, 128, 250, 256, 512, 1024, 4096, 4100, 12288, 150528]

    def timed(fn, reps=5):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    rows = []
    for name in ("tokens", "heavy_tail_bf16", "video_dataset_shape"):
        base = W.WORKLOADS[name]
        for fb in sizes:
            n = int(min(2_000_000, max(16, 1.5e9 / (mean_len[name] * fb))))
            w = W.scaled(base, n)
            T = W.lengths(w)
            tb = w.t_block
            if int(T.sum()) * fb < 2.5e8:  # below twice the L2 size the figures say little about HBM
                continue
            plan = B.bload_plan(torch.from_numpy(T).to(dev), tb, w.seed)
            nb, st = plan.n_blocks, plan.sum_t
            g = torch.Generator(device=dev)
            g.manual_seed(fb)
            store = torch.randint(0, 256, (st * fb,), dtype=torch.uint8, device=dev, generator=g)
            dense = torch.empty(nb * tb * fb, dtype=torch.uint8, device=dev)
            back = torch.zeros_like(store)
            ms_p = timed(lambda: B.bload_pack(plan, store, fb, 0, nb, dense=dense))
            k_p = B.bload_last_copy_kernel("pack")
            ms_u = timed(lambda: B.bload_unpack(plan, dense, fb, 0, nb, back))
            k_u = B.bload_last_copy_kernel("unpack")
            row = {"lengths": name, "frame_bytes": fb, "n": n, "n_blocks": nb, "mean_run_bytes": round(st * fb / n),
                   "store_MB": round(st * fb / 1e6), "round_trip_ok": bool(torch.equal(back, store)),
                   "pack": {"kernel": k_p, "GB/s": round((st * fb + nb * tb * fb) / ms_p / 1e6), "frac_measured": round((st * fb + nb * tb * fb) / ms_p / 1e6 / peak, 3)},
                   "unpack": {"kernel": k_u, "GB/s": round(2 * st * fb / ms_u / 1e6), "frac_measured": round(2 * st * fb / ms_u / 1e6 / peak, 3)}}
            if nb > 2 and (tb * fb) % 16 == 0:  # all blocks but the first (the buffer of a sub-range is 16-byte aligned)
                ms_s = timed(lambda: B.bload_unpack(plan, dense[tb * fb:], fb, 1, nb - 1, back))
                gbs = 2 * st * fb * (nb - 1) / nb / ms_s / 1e6
                row["unpack_sub_range"] = {"kernel": B.bload_last_copy_kernel("unpack"), "GB/s": round(gbs), "frac_measured": round(gbs / peak, 3)}
            # the consumer-side shifted copy over the same blocks, and the per-slot metadata of the call
            prev = back = None
            prev = torch.empty_like(dense)
            ms_c = timed(lambda: B.bload_carry_prev(plan, dense, fb, 0, nb, prev, 0))
            gbs = ((st - n) * fb + nb * tb * fb) / ms_c / 1e6
            row["carry_prev"] = {"kernel": B.bload_last_copy_kernel("carry_prev"), "GB/s": round(gbs), "frac_measured": round(gbs / peak, 3)}
            del prev
            if nb * tb >= 1 << 22:  # (smaller calls are bound by the launch, not by the 10 bytes per slot)
                ids = [torch.empty(nb * tb, dtype=torch.int32, device=dev) for _ in range(2)]   # (each array 16-byte aligned)
                flags = [torch.empty(nb * tb, dtype=torch.uint8, device=dev) for _ in range(2)]
                ms_m = timed(lambda: B.bload_pack(plan, None, fb, 0, nb, seq_id=ids[0], pos=ids[1], reset=flags[0], valid=flags[1]))
                row["metadata"] = {"GB/s": round(nb * tb * 10 / ms_m / 1e6), "frac_measured": round(nb * tb * 10 / ms_m / 1e6 / peak, 3),
                                   "slots": nb * tb, "t_block": tb}
                del ids, flags
            rows.append(row)
            del store, dense, back, plan
            torch.cuda.empty_cache()
    return {"frame_sweep": rows, "peak_GB/s": peak,
            "unit": "GB/s of algorithmic bytes (pack: frames read + blocks written; unpack: frames read + written; carry_prev: "
                    "frames but the first of every sequence read + blocks written; metadata: 10 bytes per slot written)"}


TRAFFIC: dict = {
    ("heavy_tail_bf16", "k7_copy<unpack>"): 18.27e9,
    ("heavy_tail_bf16", "k7_copy<pack>"): 9.09e9,
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="bload", choices=["bload", "reference"])
    ap.add_argument("--workload", default="heavy_tail_bf16")
    ap.add_argument("--n", type=int, default=0, help="override the number of sequences (small profiling cases)")
    ap.add_argument("--policy", type=int, default=0, help="fill policy: 0 uniform over sequences, 1 uniform over lengths")
    ap.add_argument("--frame-bytes", type=int, default=0, help="override the frame size of the workload (experiments)")
    ap.add_argument("--e2e-steps", type=int, default=12,
                    help="steps of the end-to-end leg (the pipeline over PCIe fills and drains once: about 200 ms that "
                         "are shared by these steps)")
    ap.add_argument("--ref-blocks", type=int, default=0,
                    help="blocks in the CPU oracle's sample (0 = all blocks for the CPU baseline; sized from a "
                         "calibration run for --impl reference)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-pipeline", action="store_true")
    ap.add_argument("--no-batch", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-consumer", action="store_true")
    ap.add_argument("--no-fused", action="store_true")
    ap.add_argument("--no-by-config", action="store_true", help="skip the extra measurements of the other large workloads")
    ap.add_argument("--frame-sweep", default="", metavar="SIZES",
                    help="instead of the benchmark: pack / unpack throughput and the kernel chosen across frame sizes "
                         "('default' or a comma-separated list of bytes) and three length distributions; one JSON line")
    args = ap.parse_args()
    if args.frame_sweep:
        print(json.dumps(frame_sweep(args)), flush=True)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "bload" else args.warmup

    global POLICY
    POLICY = args.policy
    from paper_2310_10879_b200 import workloads as W
    w = W.WORKLOADS[args.workload]
    if args.n:
        w = W.scaled(w, args.n)
    if args.frame_bytes:
        from dataclasses import replace
        w = replace(w, frame_bytes=args.frame_bytes, out_frame_bytes=args.frame_bytes, payload="u8")

    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            print(json.dumps(run_reference(args, w)), flush=True)
        return
    out = run_gpu(args, w)
    if out:
        print(json.dumps(out), flush=True)
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
