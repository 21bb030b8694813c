"""Benchmark of the frame-pruned CTC prefix beam search library.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python bench.py --report FILE     # all five workloads, written as a markdown table

One step = one pass of the whole hot path (prune, extend, merge, select, trie
append, readback) over one synthetic wav2vec2-shaped batch: B=64 utterances,
T uniform in [250, 1750], V=32, beam 50, R=1e-3.  The same input is also
decoded at R=0 (no pruning) and both are reported.  The emissions are 14 MB,
far below L2, so a buffer larger than L2 is written between timed steps.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

# fltop_decode_host runs a batch as up to 16 groups on as many streams; with CUDA's default of 8
# hardware connections streams share queues and wait on one another's work.  Read by the
# driver when the process creates its CUDA context.
os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "frames/sec decoded (batch 64, beam 50, r=1e-3 vs r=0); % HBM roofline"
UNIT = "frames/s"
BATCH, BEAM, R_PRUNED = 64, 50, 1e-3
L2_FLUSH_BYTES = 256 << 20
NODE_BYTES, SURVIVOR_BYTES = 8, 8
# ncu's DRAM byte count of one launch of the dominant kernel on the default workload is kept
# beside its profile summary, together with a hash of the kernel's sources: the bench reports
# it as `roofline.traffic` only while the sources still are the ones that were profiled
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "decode_rows_kernel_wav2vec2_B64_K50_full.txt")
KERNEL_SOURCES = ("fltop_decode_rows.cu", "fltop_device.cuh", "fltop_internal.h")


def kernel_source_hash():
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2510_09085_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic():
    """DRAM bytes per launch from the profile summary, or None if the kernel changed since."""
    try:
        text = open(TRAFFIC_RECORD).read()
    except OSError:
        return None
    rec = dict(line.split(":", 1) for line in text.splitlines()
               if line.startswith(("dram_bytes_per_launch:", "kernel_source_hash:")))
    if rec.get("kernel_source_hash", "").strip() != kernel_source_hash():
        return None
    try:
        return float(rec["dram_bytes_per_launch"])
    except (KeyError, ValueError):
        return None


def _algorithmic_bytes(V, st, out_bytes, fused, esize=4):
    """(prune kernel, decode kernel) HBM bytes that one call has to move.

    Two kernels: the prune kernel reads every emission row and writes a count and the survivor
    list per frame, the decode kernel reads those back.  One kernel (it prunes its own rows):
    the emission rows are the decode kernel's input and no survivor list exists.  Either way
    the decode kernel writes one 8-byte trie record per prefix that enters the beam and the
    hypotheses at the end.  ``esize``: bytes per stored emission (4, or 2 for fp16 / bf16)."""
    trie = NODE_BYTES * st["trie_nodes_created"]
    if fused:
        return 0, st["frames"] * esize * V + trie + out_bytes
    prune = st["frames"] * (esize * V + 4) + st["survivors"] * SURVIVOR_BYTES
    return prune, st["frames"] * 4 + st["survivors"] * SURVIVOR_BYTES + trie + out_bytes


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(gpu_index), "-lms", "50"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def _workload(rank: int, world: int = 1, args=None):
    """This rank's share of the job's workload, and the number of utterances of the whole job.

    The job decodes ONE batch of 64 utterances per GPU (wav2vec2-shaped, K=50, unless --workload
    / --batch say otherwise).  It is split over the ranks by total frames, longest utterance
    first (paper_2510_09085_b200/sharding.py); no data crosses ranks.  With --independent
    every rank draws a batch of its own instead."""
    import dataclasses
    from paper_2510_09085_b200 import sharding, workloads
    subword = args is not None and args.workload == "subword"
    per_gpu = (args.batch if args is not None and args.batch else (256 if subword else BATCH))
    independent = args is not None and args.independent

    def draw(seed, batch):
        if subword:
            return workloads.workload_subword(seed=seed, batch=batch)
        return workloads.workload_wav2vec2(seed=seed, batch=batch, beam_width=BEAM)
    if world == 1 or independent:
        return draw((2 if subword else 1) + 1000 * rank, per_gpu), per_gpu * world
    whole = draw(2 if subword else 1, per_gpu * world)
    mine = sharding.shard_of_rank(whole.lengths, rank, world)
    T = max(1, int(whole.lengths[mine].max())) if len(mine) else 1
    part = dataclasses.replace(whole, emissions=np.ascontiguousarray(whole.emissions[mine, :T]),
                               lengths=np.ascontiguousarray(whole.lengths[mine]))
    return part, per_gpu * world


def _oracle_frames_per_s(wl, r, utterances):
    """The CPU oracle, as it stands, single thread, on a subset of the utterances."""
    import oracle
    em, ln = wl.emissions[utterances], wl.lengths[utterances]
    t0 = time.perf_counter()
    oracle.decode(em, ln, wl.blank_id, wl.beam_width, r)
    dt = time.perf_counter() - t0
    return float(ln.sum()) / dt, dt


def run_reference(args):
    """The CPU oracle as the reference arm: each step decodes a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl, _ = _workload(0)
    order = np.argsort(wl.lengths)
    sample = [int(i) for i in order[::8]]          # 8 utterances spread over the length range
    for _ in range(args.warmup):
        _oracle_frames_per_s(wl, R_PRUNED, sample[:1])
    frames, total = 0.0, 0.0
    for _ in range(args.steps):
        fps, dt = _oracle_frames_per_s(wl, R_PRUNED, sample)
        frames += fps * dt
        total += dt
    value = frames / total
    desc = f"{len(sample)} of {BATCH} utterances per step, r=1e-3, K={BEAM}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "batch": BATCH, "beam": BEAM, "r": R_PRUNED,
                   "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def all_reduce_scalar(x, op, dist, device):
    """max / sum of one scalar over the ranks (identity when there is one rank)."""
    if dist is None:
        return x
    import torch
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(local_frames, local_ms_total, steps, dist, device):
    """frames/s of the whole job: frames of all ranks over the slowest rank's time."""
    total_frames = all_reduce_scalar(float(local_frames), "sum", dist, device)
    ms_per_step = all_reduce_scalar(float(local_ms_total), "max", dist, device) / steps
    return total_frames / (ms_per_step * 1e-3), ms_per_step


def run_ours(args):
    import torch
    from paper_2510_09085_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torch.distributed.run")
    if not torch.cuda.is_available():
        raise SystemExit("no CUDA device: this benchmark has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wl, n_global = _workload(rank, world, args)
    BEAM = wl.beam_width
    B, T, V = wl.emissions.shape
    n_frames = int(wl.lengths.sum())
    host_em = torch.from_numpy(wl.emissions).pin_memory()
    host_ln = torch.from_numpy(wl.lengths).pin_memory()
    dev_em = host_em.cuda()
    dev_ln = host_ln.cuda()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()

    def make(r):
        # trie capacity: half the worst case of one new prefix per beam slot and frame (the
        # workload creates 0.36 per slot and frame; running out would be reported per utterance
        # and is asserted not to happen below)
        d = binding.Decoder(V, wl.blank_id, BEAM, r, B, T, device=local_rank,
                            max_trie_nodes=max(1024, BEAM * T // 2))
        d.set_profiling(True)
        if args.no_fusion:
            d.set_fusion(0)
        return d

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(dec, steps, warmup, e2e=False):
        """Per-step device times (ms) of `steps` decodes; warm-up steps are not timed."""
        if e2e:  # host buffers in, host buffers out, through the library's host call
            dec.enable_host_io()
        step_ms, prune_ms, decode_ms = [], [], []
        launches0 = 0
        with torch.cuda.stream(stream):
            for i in range(warmup + steps):
                if i == warmup:
                    barrier()
                    launches0 = dec.launch_count
                flush.fill_(i & 0xff)                      # evict the inputs from L2
                t0, t1 = torch.cuda.Event(True), torch.cuda.Event(True)
                t0.record(stream)
                if e2e:
                    dec.decode_host(host_em, host_ln, stream=stream)
                else:
                    dec.decode(dev_em, dev_ln, stream=stream)
                t1.record(stream)
                t1.synchronize()
                if i >= warmup:
                    step_ms.append(t0.elapsed_time(t1))
                    pk, dk = (0.0, 0.0) if e2e else dec.last_kernel_ms()
                    prune_ms.append(pk)
                    decode_ms.append(dk)
            barrier()
        return step_ms, prune_ms, decode_ms, dec.launch_count - launches0

    dec_p, dec_0 = make(R_PRUNED), make(0.0)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms_p, prune_p, decode_p, launches = timed(dec_p, args.steps, args.warmup)
    clocks = sampler.stop() if sampler else None
    ms_0, prune_0, decode_0, _ = timed(dec_0, args.steps, args.warmup)
    ms_e, _, _, _ = timed(dec_p, args.steps, args.warmup, e2e=True)

    value_p, t_p = whole_job_throughput(n_frames, sum(ms_p), args.steps, dist, "cuda")
    value_0, t_0 = whole_job_throughput(n_frames, sum(ms_0), args.steps, dist, "cuda")
    value_e, t_e = whole_job_throughput(n_frames, sum(ms_e), args.steps, dist, "cuda")
    stats_p = dec_p.last_call_stats()
    stats_0 = dec_0.last_call_stats()
    assert int((dec_p.status != 0).sum()) == 0 and int((dec_0.status != 0).sum()) == 0

    def kernel_bytes(dec, st):
        """Algorithmic HBM bytes of one launch of each kernel (inputs of this rank)."""
        out_bytes = 4 * int(dec.lens.sum()) + 8 * int(dec.nhyp.sum()) + 8 * B
        return _algorithmic_bytes(V, st, out_bytes, fused=(launches_per_step == 1))

    peak, peak_kind = _peaks()
    launches_per_step = launches // max(1, args.steps)
    pb, db = kernel_bytes(dec_p, stats_p)
    pb0, db0 = kernel_bytes(dec_0, stats_0)
    dk_ms = statistics.mean(decode_p)
    achieved = db / (dk_ms * 1e-3) / 1e9
    h2d, d2h = dec_p.host_io_bytes()  # counted by the library from the copies it issued
    # (scores and counts only: which of two exactly tied hypotheses comes first is not unique)
    e2e_same = all(torch.equal(d.cpu(), h) for d, h in ((dec_p.scores, dec_p.h_scores),
                                                        (dec_p.nhyp, dec_p.h_nhyp)))
    assert e2e_same, "host-buffer decode and device-buffer decode disagree"

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        order = np.argsort(wl.lengths)
        if args.workload == "wav2vec2":
            main_sample, r0_sample = list(range(B)), [int(i) for i in order[::8]]
        else:  # large vocabularies are slow on the oracle: a few short utterances
            main_sample, r0_sample = [int(i) for i in order[:4]], [int(order[0])]
        fps, dt = _oracle_frames_per_s(wl, R_PRUNED, main_sample)
        fps0, dt0 = _oracle_frames_per_s(wl, 0.0, r0_sample)
        cpu = {"value": fps, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"{len(main_sample)} of {B} utterances of the workload at r=1e-3 ({dt:.1f} s); "
                         f"r=0 on {len(r0_sample)} utterances: {fps0:.0f} frames/s ({dt0:.1f} s)",
               "value_r0": fps0, "host_cores_available": len(os.sched_getaffinity(0))}

    line = {
        "metric": METRIC, "value": value_p, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_p,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": wl.name if world == 1 else f"{wl.name} (rank 0's share)",
                   "utterances": n_global, "utterances_rank0": B, "beam": BEAM, "r": R_PRUNED,
                   "vocab": V, "frames_per_step_rank0": n_frames, "max_frames": int(T),
                   "l2": f"flushed: {L2_FLUSH_BYTES >> 20} MiB written between timed steps",
                   "sharding": ("every GPU draws its own batch of 64 utterances" if args.independent
                                else "one batch of 64 utterances per GPU, split over the GPUs by total "
                                     "frames, longest first; no collective on the data path")},
        "e2e": {"value": value_e, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": t_e,
                "call": "fltop_decode_host: pinned host emissions in, host hypotheses out; "
                        "the valid frames and the existing tokens are what crosses the bus"},
        "gpu_launches": launches,
        "clocks": clocks,
        "roofline": {"bound": "hbm",
                     "kernel": "decode_rows_kernel" if V <= 32 and BEAM <= 64 else "decode_kernel",
                     "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": (recorded_traffic() if args.workload == "wav2vec2" and not args.batch
                                 and world == 1 else None),
                     "peak_source": f"{peak_kind} copy bandwidth",
                     "bytes_per_launch": db, "ms_per_launch": dk_ms,
                     "note": "latency-bound serial frame chain: max_frames dependent steps"},
        "cpu_baseline": cpu,
        "detail": {
            "r0": {"value": value_0, "ms_per_step": t_0,
                   "decode_kernel_ms": statistics.mean(decode_0),
                   "prune_kernel_ms": statistics.mean(prune_0),
                   "mean_survivors": stats_0["survivors"] / max(1, stats_0["frames"]),
                   "mean_live_hypotheses": stats_0["live_hypotheses_sum"] / max(1, stats_0["frames"]),
                   "hbm_frac_step": (pb0 + db0) / (t_0 * 1e-3) / 1e9 / peak},
            "pruned_over_r0_speedup": t_0 / t_p,
            "utterances_per_s": n_global / (t_p * 1e-3),
            "prune_kernel_ms": statistics.mean(prune_p),
            "decode_kernel_ms": dk_ms,
            "ns_per_frame_step": 1e6 * dk_ms / int(wl.lengths.max()),
            "mean_survivors": stats_p["survivors"] / max(1, stats_p["frames"]),
            "mean_live_hypotheses": stats_p["live_hypotheses_sum"] / max(1, stats_p["frames"]),
            "trie_nodes_created": stats_p["trie_nodes_created"],
            "hbm_frac_step": (pb + db) / (t_p * 1e-3) / 1e9 / peak,
            "prune_kernel_gbs": (pb / (statistics.mean(prune_p) * 1e-3) / 1e9
                                 if statistics.mean(prune_p) > 0 else None),
            "pruning": "inside the decode kernel" if launches_per_step == 1 else "separate kernel",
            "beam_state_bytes": dec_p.beam_state_bytes,
            "beam_state_bytes_written": NODE_BYTES * stats_p["trie_nodes_created"],
            "step_ms_min": min(ms_p), "step_ms_median": statistics.median(ms_p),
        },
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def _time_decode(dec, x, ln, flush, reps=7, warm=2):
    """Best-of device times (ms) of the whole call and of its prune and decode kernels."""
    import torch
    best = None
    for i in range(warm + reps):
        flush.fill_(i & 0xff)
        t0, t1 = torch.cuda.Event(True), torch.cuda.Event(True)
        t0.record()
        dec.decode(x, ln)
        t1.record()
        t1.synchronize()
        if i >= warm:
            pk, dk = dec.last_kernel_ms()
            cur = (t0.elapsed_time(t1), pk, dk)
            best = cur if best is None or cur[0] < best[0] else best
    return best


def _oracle_top1(wl, K, r, threads):
    """Top-1 sequence of every utterance from the CPU oracle (utterances in parallel threads)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor

    def one(b):
        res = oracle.decode(wl.emissions[b:b + 1], wl.lengths[b:b + 1], wl.blank_id, K, r)
        return res.hyps(0)[0][0]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(one, range(len(wl.lengths))))


def run_report(args):
    """All five workloads on one GPU; a markdown table goes to args.report."""
    import torch
    from paper_2510_09085_b200 import binding, workloads
    peak, peak_kind = _peaks()
    cores = len(os.sched_getaffinity(0))
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    rows = []

    def measure(wl, K, r, label, top1_ref=None, top_n=0, theta=0.0, merge_max=False,
                dtype=torch.float32):
        B, T, V = wl.emissions.shape
        x = torch.from_numpy(wl.emissions).cuda().to(dtype)
        ln = torch.from_numpy(wl.lengths).cuda()
        # a trie arena of half the worst case first (peaked emissions use far less); a batch that
        # runs out of it says so in its status words and is measured again with the worst case
        for arena in (max(1024, K * T // 2), 0):
            dec = binding.Decoder(V, wl.blank_id, K, r, B, T, top_n=top_n, beam_threshold=theta,
                                  merge_max=merge_max, emission_dtype=dtype, max_trie_nodes=arena)
            dec.set_profiling(True)
            ms, pk, dk = _time_decode(dec, x, ln, flush)
            st = dec.last_call_stats()
            if int((dec.status != 0).sum()) == 0:
                break
            dec.close()
        assert int((dec.status != 0).sum()) == 0
        frames = int(wl.lengths.sum())
        pbytes, dbytes = _algorithmic_bytes(
            V, st, 4 * int(dec.lens.sum()) + 8 * int(dec.nhyp.sum()) + 8 * B, fused=(pk == 0.0),
            esize=x.element_size())
        agree = None
        if top1_ref is not None:
            agree = sum(dec.hyps(b)[0][0] == top1_ref[b] for b in range(B)) / B
        row = {"workload": label, "K": K, "r": r, "frames_per_s": frames / (ms * 1e-3),
               "utt_per_s": B / (ms * 1e-3), "ms": ms, "prune_ms": pk, "decode_ms": dk,
               "hbm_frac_step": (pbytes + dbytes) / (ms * 1e-3) / 1e9 / peak,
               "prune_gbs": pbytes / (pk * 1e-3) / 1e9 if pk > 0 else 0.0,
               "ns_per_frame_step": 1e6 * dk / max(1, int(wl.lengths.max())),
               "beam_state_bytes": dec.beam_state_bytes,
               "nodes_per_frame": st["max_node_ids_used"] / max(1, int(wl.lengths.max())),
               "exact_select_frames": st["exact_select_frames"],
               "mean_survivors": st["survivors"] / max(1, st["frames"]),
               "mean_live": st["live_hypotheses_sum"] / max(1, st["frames"]), "top1_agree": agree}
        rows.append(row)
        dec.close()
        print(json.dumps(row), file=sys.stderr, flush=True)
        return row

    pr1 = workloads.workload_pr1()
    for r in pr1.thresholds:
        measure(pr1, pr1.beam_width, r, "0 pr1")
    wav = workloads.workload_wav2vec2()
    for r in wav.thresholds:
        measure(wav, wav.beam_width, r, "1 wav2vec2")
    for K in workloads.SWEEP_BEAMS:
        t0 = time.perf_counter()
        ref = None if args.skip_oracle else _oracle_top1(wav, K, 0.0, cores)
        print(f"oracle r=0 K={K}: {time.perf_counter() - t0:.1f} s on {cores} threads",
              file=sys.stderr, flush=True)
        for r in workloads.SWEEP_THRESHOLDS:
            measure(wav, K, r, "2 sweep", ref)
    # the paper's own operating point (Sections 4.2-4.4): N = 4, R = 0.007, beam_threshold = 25,
    # against its baseline (all tokens, same beam_threshold) and Top-4 without R
    for K in (50, 1000):
        ref = None if args.skip_oracle or K > 50 else _oracle_top1(wav, K, 0.0, cores)
        measure(wav, K, 0.0, "P baseline (all tokens, bt 25)", ref, theta=25.0)
        measure(wav, K, 0.0, "P Top-4 (bt 25)", ref, top_n=4, theta=25.0)
        measure(wav, K, 0.007, "P FLToP N=4 R=0.007 (bt 25)", ref, top_n=4, theta=25.0)
    sub = workloads.workload_subword()
    for r in sub.thresholds:
        measure(sub, sub.beam_width, r, "3 subword")
    # variants: best-alignment scores (merge by max) and emissions stored in half precision
    measure(wav, wav.beam_width, R_PRUNED, "V wav2vec2, merge by max", merge_max=True)
    measure(wav, wav.beam_width, R_PRUNED, "V wav2vec2, fp16 emissions", dtype=torch.float16)
    measure(sub, sub.beam_width, R_PRUNED, "V subword, fp16 emissions", dtype=torch.float16)
    measure(sub, sub.beam_width, R_PRUNED, "V subword, bf16 emissions", dtype=torch.bfloat16)
    # streaming: 1024 streams, 16-frame chunks, beam state carried in the handle
    stw = workloads.workload_streaming()
    S, T, V = stw.emissions.shape
    C, K, r = stw.chunk_frames, stw.beam_width, stw.thresholds[0]
    x = torch.from_numpy(stw.emissions).cuda()
    dec = binding.Decoder(V, 0, K, r, S, T, max_chunk_frames=C)
    full = torch.full((S,), C, dtype=torch.int32, device="cuda")
    n = T // C
    chunks = [x[:, i * C:(i + 1) * C].contiguous() for i in range(n)]
    first = torch.full((S,), 1, dtype=torch.uint8, device="cuda")
    mid = torch.zeros((S,), dtype=torch.uint8, device="cuda")
    last = torch.full((S,), 2, dtype=torch.uint8, device="cuda")
    lat, total = [], None
    for rep in range(3):
        torch.cuda.synchronize()
        t_all = time.perf_counter()
        for i in range(n):
            flags = first if i == 0 else (last if i == n - 1 else mid)
            t0 = time.perf_counter()
            dec.stream_step(chunks[i], full, flags, readback=(i == n - 1))
            torch.cuda.synchronize()
            if rep > 0:
                lat.append(time.perf_counter() - t0)
        dt = time.perf_counter() - t_all
        total = dt if total is None or dt < total else total
    assert int((dec.status != 0).sum()) == 0
    lat = np.array(lat) * 1e3
    stream_row = {"workload": "4 streaming", "K": K, "r": r, "frames_per_s": S * T / total,
                  "p50_ms": float(np.percentile(lat, 50)), "p99_ms": float(np.percentile(lat, 99)),
                  "beam_state_bytes": dec.beam_state_bytes}
    print(json.dumps(stream_row), file=sys.stderr, flush=True)
    dec.close()

    # many more streams than SMs: chunks queued back to back, device time, with the decode kernel
    # the library picks by itself (one warp per stream) and with the block-per-stream kernel
    def many_streams(streams, mode):
        w = workloads.workload_streaming(streams=streams, chunks=8)
        S2, T2, _ = w.emissions.shape
        x2 = torch.from_numpy(w.emissions).cuda()
        d2 = binding.Decoder(V, 0, K, r, S2, T2, max_chunk_frames=C)
        d2.set_warp_decode(mode)
        full2 = torch.full((S2,), C, dtype=torch.int32, device="cuda")
        n2 = T2 // C
        ch = [x2[:, i * C:(i + 1) * C].contiguous() for i in range(n2)]
        fl = [torch.full((S2,), (1 if i == 0 else 0) | (2 if i == n2 - 1 else 0), dtype=torch.uint8,
                         device="cuda") for i in range(n2)]
        best = None
        for _ in range(3):
            e0, e1 = torch.cuda.Event(True), torch.cuda.Event(True)
            e0.record()
            for i in range(n2):
                d2.stream_step(ch[i], full2, fl[i], readback=(i == n2 - 1))
            e1.record()
            e1.synchronize()
            ms = e0.elapsed_time(e1)
            best = ms if best is None or ms < best else best
        assert int((d2.status != 0).sum()) == 0
        d2.close()
        return {"streams": S2, "frames_per_s": S2 * T2 / (best * 1e-3), "us_per_chunk": 1e3 * best / n2}
    many = [(many_streams(n_s, 1), many_streams(n_s, 0)) for n_s in (4096, 16384)]
    print(json.dumps(many), file=sys.stderr, flush=True)
    # CPU oracle, single thread, on a sample of the wav2vec2 workload (a reported baseline)
    order = np.argsort(wav.lengths)
    sample = [int(i) for i in order[::8]]
    cpu_p, _ = _oracle_frames_per_s(wav, R_PRUNED, sample)
    cpu_0, _ = _oracle_frames_per_s(wav, 0.0, sample)

    with open(args.report, "w") as f:
        f.write(f"Measured on one B200, HBM peak {peak:.0f} GB/s ({peak_kind}); host threads {cores}.\n\n")
        f.write("| cfg | K | r | frames/s | utt/s | step ms | HBM frac (step) | prune GB/s | "
                "ns / frame step | beam-state MB | trie nodes / frame (max utt) | mean survivors | mean live hyps | top-1 vs r=0 oracle |\n")
        f.write("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|\n")
        for w in rows:
            ag = "" if w["top1_agree"] is None else f"{100 * w['top1_agree']:.1f} %"
            f.write(f"| {w['workload']} | {w['K']} | {w['r']:g} | {w['frames_per_s']:.3g} | "
                    f"{w['utt_per_s']:.3g} | {w['ms']:.3f} | {100 * w['hbm_frac_step']:.3f} % | "
                    f"{(format(w['prune_gbs'], '.0f') if w['prune_gbs'] else 'in decode')} | "
                    f"{w['ns_per_frame_step']:.0f} | "
                    f"{w['beam_state_bytes'] / 1e6:.1f} | {w['nodes_per_frame']:.1f} | "
                    f"{w['mean_survivors']:.2f} | "
                    f"{w['mean_live']:.1f} | {ag} |\n")
        f.write(f"\nStreaming (cfg 4, K={K}, r={r:g}, 1024 streams x 100 chunks of 16 frames): "
                f"{stream_row['frames_per_s']:.3g} frames/s aggregate, chunk latency p50 "
                f"{stream_row['p50_ms']:.3f} ms, p99 {stream_row['p99_ms']:.3f} ms (host wall clock, "
                f"call to stream sync), beam state {stream_row['beam_state_bytes'] / 1e6:.1f} MB.\n")
        for auto, block in many:
            f.write(f"\nStreaming, {auto['streams']} streams (same K, r, chunks of {C} frames queued back to "
                    f"back, device time): {auto['frames_per_s']:.3g} frames/s, {auto['us_per_chunk']:.0f} us "
                    f"per chunk with the warp-per-stream kernel the library picks at this size; "
                    f"{block['frames_per_s']:.3g} frames/s, {block['us_per_chunk']:.0f} us with the "
                    f"block-per-stream kernel.\n")
        f.write(f"\nCPU oracle, one thread, 8 of the 64 wav2vec2 utterances, K=50: "
                f"{cpu_p:.0f} frames/s at r=1e-3, {cpu_0:.0f} frames/s at r=0.\n")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", choices=["wav2vec2", "subword"], default="wav2vec2",
                    help="default: the headline wav2vec2-shaped batch; subword: V=1024, K=32")
    ap.add_argument("--batch", type=int, default=0, help="utterances per GPU (0 = the workload's own)")
    ap.add_argument("--no-fusion", action="store_true",
                    help="prune with the separate kernel even where the decode kernel could do it")
    ap.add_argument("--independent", action="store_true",
                    help="N > 1: every rank draws a batch of its own instead of taking its share "
                         "of one batch of N x 64 utterances")
    ap.add_argument("--report", metavar="FILE", help="measure all five workloads, write a table")
    ap.add_argument("--skip-oracle", action="store_true", help="--report without top-1 agreement")
    args = ap.parse_args()
    if args.report:
        run_report(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
