#!/usr/bin/env python
"""Benchmark of the CPE decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c1..c5] [--impl ours|reference]

One decode is one pass of the whole path (decode+vote, peaks, candidate lists, assignment+labels) over one batch of
the chosen workload, replayed as one CUDA graph.  One "step" is `inner` decodes back to back (as many as make a step
last 2.5 ms, so that the timed region of the default run is long enough for clock samples and percentiles to mean
something); every decode has its own pair of CUDA events.  Prints ONE JSON line (rank 0).

The default workload is c5, the largest single-GPU configuration, decoded with sub-cell refined candidates
(`--candidates refined`, CPE_FLAG_REFINE); `--candidates bins` times the paper's own candidates (the palette rows of
the peaks' bins, Eq. 7 / Eq. 9), and the default run reports that figure beside the headline.

  value       whole-job megapixels/s, inputs resident in HBM, device time (CUDA events on the launching
              stream), max over ranks; weak scaling: every rank decodes its own frames, no collective.
  e2e         the same metric through the host-buffer entry point (pinned host memory in, host memory out),
              copies inside the timed region.
  roofline    the dominant stage: its algorithmic bytes (participating pixels' embeddings once, mask, labels) divided
              by its CUDA-event time, against the measured HBM copy bandwidth (MEASURED_PEAKS.json).
  cpu_baseline  the CPU oracle, as it stands, on this machine's host cores (rank 0, N = 1).

`--impl reference` times the CPU oracle itself (there is no other reference implementation of this path).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_16874_b200 import distributed as dist_util  # noqa: E402
from paper_2609_16874_b200 import workloads as wl  # noqa: E402

METRIC = "decode_megapixels_per_s"
UNIT = "MP/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0
MIN_STEP_MS = 2.5          # a step is made of as many decodes as it takes to last at least this long


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


class ClockSampler:
    """Polls NVML for SM clock and throttle reasons while the timed region runs (reading only)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._active = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def sample(self):
        """One reading, now (also called from the timing loop itself, while the GPU works through the queued steps:
        the polling thread gets few turns while the main thread is busy submitting)."""
        nv = self.nv
        if nv is None:
            return
        try:
            mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            try:
                r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            self.samples.append(mhz)
            for bit, name in self.REASONS.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _poll(self):
        while not self._stop.is_set():
            if self._active.is_set():
                self.sample()
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()

    def window(self, on: bool):
        (self._active.set if on else self._active.clear)()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=1.0)
        return {"sm_mhz": (float(np.median(self.samples)) if self.samples else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def algorithmic_bytes(cfg, fg_pixels: int, pruned: bool):
    """Bytes each stage must move per decode: participating pixels' embeddings once per pass, the mask once per
    pass, the label map once; with the pruned assignment each pixel's bin is written by the voting pass and read by
    the assignment (4 bytes each way); vote map / peak lists are small and counted where they are touched."""
    P, D, esz = cfg.pixels, cfg.D, cfg.esz
    cells = cfg.B * cfg.bins_w * cfg.bins_h
    cell_words = 4 * fg_pixels if pruned else 0
    return {
        "clear": 0,
        "decode_vote": fg_pixels * D * esz + P + cell_words,
        "peaks": 4 * cells + cells // 8,
        "lists": 0,
        "assign": fg_pixels * D * esz + P + 4 * P + cell_words,
    }


STAGE_KERNELS = {
    "decode_vote": "decode_vote_vec_kernel",
    "peaks": "peaks_kernel",
    "lists": "peak_rows_kernel + peak_graph_kernel",
    "assign": "assign_near_stream_kernel + assign_near_walk_kernel + assign_near_hard_kernel (pruned) / "
              "assign_kernel (few peaks) / assign_filter_kernel (handed on)",
}


def profiled_traffic(cfg_name: str, stage: str):
    """DRAM bytes per launch of the stage's kernel from the ncu summary under profiles/ (a line
    `traffic <workload> <stage>: <bytes>`), or None if no summary names it."""
    import re
    pdir = os.path.join(ROOT, "profiles")
    try:
        for fn in sorted(os.listdir(pdir)):
            with open(os.path.join(pdir, fn)) as f:
                m = re.search(r"^traffic %s %s: (\d+)" % (re.escape(cfg_name), re.escape(stage)), f.read(), re.M)
            if m:
                return int(m.group(1)), "profiles/" + fn
    except OSError:
        pass
    return None, None


def frames_needed(cfg):
    """Rotate over enough distinct frames that the inputs of consecutive decodes cannot all sit in L2."""
    return max(1, min(8, math.ceil(2.2 * L2_BYTES / cfg.emb_bytes)))


# ----------------------------------------------------------------------------------------- CPU oracle timing

def time_oracle(cfg, frame, budget_s: float, threads: int, refine: bool):
    """Seconds per full batch for the oracle as it stands: the vote and peak steps on the whole batch, the
    assignment on a sample of pixels (scaled up linearly: its cost is per pixel)."""
    import oracle
    oracle.set_threads(threads)
    emb, fg = frame["emb"], frame["fg"]
    t0 = time.perf_counter()
    ov = oracle.votes(emb, fg, cfg.bins_w, cfg.bins_h, want_est=refine, want_cell=refine)
    peaks = [oracle.peaks(ov["votes"][b], cfg.T_v, cfg.K_max)[0] for b in range(cfg.B)]
    rows = [None] * cfg.B
    if refine:
        sums = oracle.vote_sums(ov["est"], ov["cell"], cfg.bins_w, cfg.bins_h)
        rows = [oracle.refined_peaks(ov["votes"][b], sums[b], peaks[b], cfg.F, cfg.H, cfg.W)["peak_emb"]
                for b in range(cfg.B)]
    t_front = time.perf_counter() - t0
    HW = cfg.H * cfg.W
    # calibrate the per-pixel assignment cost on a small sample, then size the real sample to the budget
    rng = np.random.default_rng(0)
    n_cal = min(HW, 4096)
    idx = np.sort(rng.choice(HW, n_cal, replace=False)).astype(np.int64)
    t0 = time.perf_counter()
    oracle.assign_image(emb[0], fg[0], cfg.bins_w, cfg.bins_h, peaks[0], cfg.tau, idx=idx, peak_emb=rows[0])
    per_px = max((time.perf_counter() - t0) / n_cal, 1e-9)
    n = int(min(HW, max(n_cal, budget_s / per_px / cfg.B)))
    t_assign = 0.0
    for b in range(cfg.B):
        idx = None if n >= HW else np.sort(rng.choice(HW, n, replace=False)).astype(np.int64)
        t0 = time.perf_counter()
        oracle.assign_image(emb[b], fg[b], cfg.bins_w, cfg.bins_h, peaks[b], cfg.tau, idx=idx, peak_emb=rows[b])
        t_assign += (time.perf_counter() - t0) * (HW / min(n, HW))
    sample = (f"votes+peaks{'+refined candidates' if refine else ''} on the full batch; assignment on {min(n, HW)} of "
              f"{HW} pixels per image" + (" (all)" if n >= HW else ", scaled to the image"))
    return t_front + t_assign, sample


def workload_name(cfg, refine: bool) -> str:
    return cfg.describe() + (", candidates: refined centroids (CPE_FLAG_REFINE)" if refine
                             else ", candidates: palette rows of the peaks' bins (Eq. 7)")


def run_reference(args, cfg):
    """`--impl reference`: the CPU oracle, timed on the host cores, on the same workload and metric."""
    rank, _, world = dist_util.env_world()
    if rank != 0:
        return
    import oracle
    refine = args.candidates == "refined"
    threads = oracle.max_threads()
    frame = wl.make_frame(cfg, 0)
    total_steps = args.steps + args.warmup
    budget = max(0.05, min(2.0, 60.0 / max(1, total_steps)))
    times, sample = [], ""
    for i in range(total_steps):
        t, sample = time_oracle(cfg, frame, budget, threads, refine)
        if i >= args.warmup:
            times.append(t)
    sec = float(np.mean(times))
    value = cfg.pixels / sec / 1e6
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg, refine), "name": cfg.name,
                   "timing": "host wall clock; the oracle is CPU code"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------- the GPU arm

def timed_replays(dec, graphs, stream, flush, n_decodes, sampler=None):
    """`n_decodes` graph replays (frames in rotation), each between its own pair of CUDA events on the launching
    stream; returns the per-decode milliseconds."""
    import torch
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_decodes)]
    for i in range(n_decodes):
        if flush is not None:
            flush.fill_(i & 0xff)                     # evicts L2 between decodes; outside the event pair
        ev[i][0].record(stream)
        dec.replay(graphs[i % len(graphs)], stream=stream)
        ev[i][1].record(stream)
        if sampler is not None and i % 64 == 32:
            sampler.sample()                          # between two submissions; the decodes are timed by their own events
    stream.synchronize()
    return np.array([a.elapsed_time(b) for a, b in ev])


def run_ours(args, cfg):
    import torch
    from paper_2609_16874_b200 import binding as cb

    rank, local_rank, world = dist_util.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    dev = torch.device("cuda", local_rank if world > 1 else 0)
    torch.cuda.set_device(dev)
    if world > 1:
        dist_util.init("nccl", dev)
    K, Wm = args.steps, args.warmup
    refine = args.candidates == "refined"

    # inputs: this rank's own frames (weak scaling), resident in HBM before anything is timed
    n_frames = frames_needed(cfg)
    frame_ids = dist_util.frames_for_rank(rank, world, n_frames)
    frames = [wl.make_frame(cfg, f) for f in frame_ids]
    d_emb = [torch.from_numpy(f["emb"]).to(dev) for f in frames]
    d_fg = [torch.from_numpy(f["fg"]).to(dev) for f in frames]
    fg_pixels = [int(f["fg"].sum()) for f in frames]
    flush = None
    if cfg.emb_bytes < 2 * L2_BYTES and n_frames * cfg.emb_bytes < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)

    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max,
                     device=dev, refine=refine, flags=args.flags)
    pruned = cb.cpe_get_intermediate(dec.params, cb.CPE_INT_PRUNE_STATE, cfg.B, cfg.H, cfg.W, cfg.F)[0] == cb.CPE_OK
    stream = torch.cuda.Stream(device=dev)
    sampler = ClockSampler(dev.index)
    sampler.start()
    with torch.cuda.stream(stream):
        graphs = [dec.capture(d_emb[i], d_fg[i], stream=stream) for i in range(n_frames)]
        kernel_nodes = cb.cpe_graph_kernel_nodes(graphs[0])
        # bring the clocks up (idle parts sit at a few hundred MHz) and find out how long one decode takes
        t_end = time.perf_counter() + (0.0 if args.quick else 0.4)
        while True:
            probe = timed_replays(dec, graphs, stream, flush, 8)
            if time.perf_counter() >= t_end:
                break
        inner = args.inner if args.inner > 0 else max(1, int(math.ceil(MIN_STEP_MS / max(1e-3, float(np.median(probe))))))
        timed_replays(dec, graphs, stream, flush, Wm * inner)             # the W warm-up steps
        dist_util.barrier()
        torch.cuda.synchronize(dev)
        sampler.window(True)
        dec_ms = timed_replays(dec, graphs, stream, flush, K * inner, sampler)   # exactly K steps of `inner` decodes
        sampler.sample()
        torch.cuda.synchronize(dev)
        sampler.window(False)
        dist_util.barrier()
        step_ms = dec_ms.reshape(K, inner).sum(1)

        # per-stage device times of the same frames (events between the kernels; outside the graph)
        stage_ms = {k: 0.0 for k in cb.CPE_STAGE_NAMES}
        reps = max(3, min(20, K))
        for i in range(n_frames):
            if flush is not None:
                flush.fill_(1)
            ms = dec.profile(d_emb[i], d_fg[i], iters=reps if flush is None else 1, stream=stream)
            for k, v in ms.items():
                stage_ms[k] += v / n_frames
        counters = dec.intermediate(cb.CPE_INT_COUNTERS).cpu().numpy().astype(np.int64)
        handed_on = dec.intermediate(cb.CPE_INT_PRUNE_STATE).cpu().numpy()[:, 2].tolist() if pruned else None
        count_dev = dec.count.cpu().numpy().tolist()
    clocks = sampler.stop()

    # sum of the per-decode device times: excludes the L2 flush, includes every kernel and gap inside a decode
    total_ms = float(step_ms.sum())
    t_max, px_total = dist_util.reduce_measurement(total_ms, float(cfg.pixels) * K * inner, device=dev)
    value = px_total / (t_max * 1e-3) / 1e6
    p50, p95 = float(np.percentile(dec_ms, 50)), float(np.percentile(dec_ms, 95))
    voting = max(1, int(counters[:, cb.CPE_CNT_VOTING].sum()))
    assignment = {"pruned_assignment": pruned, "images_handed_to_filtered_kernel": handed_on,
                  "scored_pairs_per_voting_pixel": float(counters[:, cb.CPE_CNT_FILTER_PAIRS].sum()) / voting,
                  "pixels_with_several_candidates": int(counters[:, cb.CPE_CNT_RESCORED].sum()),
                  "pixels_scored_against_every_peak": int(counters[:, cb.CPE_CNT_FULL_SCORED].sum())}

    if args.quick:
        print(json.dumps({"quick": True, "name": cfg.name, "candidates": args.candidates, "flags": args.flags,
                          "p50_ms": p50, "value": value, "inner": inner, "stage_ms": stage_ms, "assignment": assignment,
                          "kernel_nodes": kernel_nodes}))
        dec.close()
        dist_util.shutdown()
        return

    # ---- end to end through the host-buffer entry point (rank-local wall clock, max over ranks)
    hd = cb.HostDecoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max,
                        refine=refine, flags=args.flags)
    h_emb = [torch.from_numpy(f["emb"]).pin_memory() for f in frames]
    h_fg = [torch.from_numpy(f["fg"]).pin_memory() for f in frames]
    # two sets of result buffers: two decodes are in flight (the copy of one's inputs overlaps the decode and
    # read-back of the one before); every decode still moves its own inputs and results
    h_out = [(torch.empty((cfg.B, cfg.H, cfg.W), dtype=torch.int32).pin_memory(),
              torch.empty((cfg.B, cfg.K_max, 2), dtype=torch.float32).pin_memory(),
              torch.empty((cfg.B,), dtype=torch.int32).pin_memory()) for _ in range(2)]
    e2e_n = max(3, min(K * inner, int(2.0 / max(1e-4, cfg.emb_bytes / 20e9))))
    for i in range(min(3, Wm)):
        hd.decode(h_emb[i % n_frames], h_fg[i % n_frames], *h_out[0])
    dist_util.barrier()
    t0 = time.perf_counter()
    for i in range(e2e_n):
        if i >= 2:
            hd.wait()
        hd.submit(h_emb[i % n_frames], h_fg[i % n_frames], *h_out[i & 1])
    for _ in range(min(2, e2e_n)):
        hd.wait()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    dist_util.barrier()
    e_max, e_px = dist_util.reduce_measurement(e2e_ms, float(cfg.pixels) * e2e_n, device=dev)
    e2e_value = e_px / (e_max * 1e-3) / 1e6
    count_last = h_out[(e2e_n - 1) & 1][2].numpy().copy()
    t0 = time.perf_counter()
    for i in range(e2e_n):                             # the synchronous call, one decode at a time, for comparison
        hd.decode(h_emb[i % n_frames], h_fg[i % n_frames], *h_out[0])
    e2e_sync_ms = (time.perf_counter() - t0) * 1e3 / e2e_n
    h2d, d2h = hd.h2d_bytes, hd.d2h_bytes
    hd.close()

    all_clocks = dist_util.gather_objects(clocks)
    if rank != 0:
        dist_util.shutdown()
        return

    # ---- roofline of the dominant stage: algorithmic bytes / its CUDA-event time / the measured copy bandwidth
    peak_gbs, peak_src = measured_peaks()
    alg = algorithmic_bytes(cfg, int(np.mean(fg_pixels)), pruned)
    dominant = max(stage_ms, key=lambda k: stage_ms[k])
    achieved = alg[dominant] / (stage_ms[dominant] * 1e-3) / 1e9
    one_read_us = cfg.emb_bytes / (peak_gbs * 1e9) * 1e6
    alg_total = sum(alg.values())
    traffic, traffic_src = profiled_traffic(cfg.name + ("-refined" if refine else "-bins"), dominant)
    roofline = {
        "bound": "hbm", "stage": dominant, "kernel": STAGE_KERNELS.get(dominant, dominant), "achieved": achieved,
        "peak": peak_gbs, "unit": "GB/s", "frac": achieved / peak_gbs, "traffic": traffic, "traffic_source": traffic_src,
        "peak_source": peak_src, "algorithmic_bytes_per_launch": alg[dominant], "kernel_ms": stage_ms[dominant],
        "derivation": "algorithmic_bytes_per_launch / kernel_ms / peak; bytes = participating pixels x 4F x element size "
                      "+ mask (1 B/pixel) (+ 4 B/pixel labels in the assignment, + 4 B per participating pixel for its bin)",
        "stage_ms": stage_ms,
        "stage_frac_of_peak": {k: (alg[k] / (v * 1e-3) / 1e9 / peak_gbs if v > 0 and alg[k] else None)
                               for k, v in stage_ms.items()},
        "end_to_end": {
            "p50_ms": p50,
            "one_read_embedding_roofline_us": one_read_us,
            "frac_of_one_read_roofline": one_read_us / (p50 * 1e3),
            "algorithmic_bytes": alg_total,
            "frac_of_algorithmic_bytes_roofline": alg_total / (peak_gbs * 1e9) / (p50 * 1e-3),
        },
    }

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        threads = oracle.max_threads()
        sec, sample = time_oracle(cfg, frames[0], 12.0, threads, refine)
        sec1, _ = time_oracle(cfg, frames[0], 4.0, 1, refine)
        cpu = {"value": cfg.pixels / sec / 1e6, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
               "single_thread_value": cfg.pixels / sec1 / 1e6}

    worst = [c for c in all_clocks if c.get("sm_mhz")]
    clk = dict(clocks)
    if worst:
        clk["sm_mhz"] = float(min(c["sm_mhz"] for c in worst))
        clk["reasons"] = sorted(set(r for c in all_clocks for r in c.get("reasons", [])))
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": t_max / K, "p50_decode_ms": p50, "p95_decode_ms": p95, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32" if cfg.dtype == "f32" else "f16", "data": "synthetic",
        "config": {
            "workload": workload_name(cfg, refine), "name": cfg.name, "candidates": args.candidates,
            "frames_per_rank": n_frames, "decodes_per_step": inner,
            "l2": ("every decode reads %.0f MB of embedding, more than L2 holds (%d frame%s in rotation)"
                   % (cfg.emb_bytes / 1e6, n_frames, "" if n_frames == 1 else "s")
                   if flush is None else "a 252 MB buffer is rewritten between decodes, outside the timed events"),
            "launch": "one CUDA graph replay per decode (%d kernel nodes)" % kernel_nodes,
            "timing": "sum of per-decode CUDA-event times on the launching stream (timed region %.1f ms)" % total_ms,
            "parallelism": "independent frames per rank, no collective",
            "instances_found": count_dev, "instances_found_last_e2e_step": count_last.tolist(),
            "assignment": assignment,
        },
        "clocks": clk,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_n, "ms_per_step": e_max / e2e_n,
                "timing": "host wall clock around cpe_host_submit / cpe_host_wait with two decodes in flight, pinned "
                          "buffers; every decode copies its inputs in and its results out (one decode per e2e step)",
                "synchronous_ms_per_step": e2e_sync_ms},
        "gpu_launches": kernel_nodes * K * inner,
        "roofline": roofline,
        "cpu_baseline": cpu,
    }
    dec.close()
    del d_emb, d_fg, graphs
    if world == 1 and not args.only_default:
        torch.cuda.empty_cache()
        try:   # the same workload with the other kind of candidates
            other_kind = "bins" if refine else "refined"
            line["%s_candidates" % other_kind] = measure_other(cfg, 30, 5, dev, refine=not refine)
        except Exception as exc:
            line["other_candidates"] = {"error": repr(exc)}
        others = {}
        for name in sorted(wl.CONFIGS):
            if name == cfg.name:
                continue
            for kind in (False, True):
                try:
                    others[name + ("-refined" if kind else "-bins")] = measure_other(wl.CONFIGS[name], 60, 5, dev, refine=kind)
                except Exception as exc:   # a parity-test workload must not take the headline line down with it
                    others[name + ("-refined" if kind else "-bins")] = {"error": repr(exc)}
        line["other_configs"] = others
        try:   # what the chain of launches costs by itself
            line["launch_floor"] = measure_launch_floor(wl.CONFIGS["c2"], 200, 10, dev)
        except Exception as exc:
            line["launch_floor"] = {"error": repr(exc)}
        try:   # the decode with the paper's own vote (Eq. 5-6, strict maxima, Eq. 7-8)
            sd = {}
            for n in ("c1", "c2"):
                thr = soft_threshold_for(wl.CONFIGS[n], dev)
                r = measure_other(wl.CONFIGS[n], 40, 5, dev, soft_threshold=thr)
                r["workload"] += ("; vote mode: soft (CPE_FLAG_SOFT_VOTE, soft_threshold %.4g = 0.3 x the histogram's "
                                  "maximum on frame 0; a global threshold cuts small instances and lets side lobes of large "
                                  "ones through: see instances_found)" % thr)
                sd[n] = r
            line["soft_vote_decode"] = sd
        except Exception as exc:
            line["soft_vote_decode"] = {"error": repr(exc)}
        try:
            line["soft_votes"] = {n: measure_soft_votes(wl.CONFIGS[n], 40, 5, dev) for n in ("c2", "c3")}
        except Exception as exc:
            line["soft_votes"] = {"error": repr(exc)}
        try:
            line["instance_masks"] = {n: measure_instance_masks(wl.CONFIGS[n], 20, 3, dev) for n in ("c2", "c5")}
        except Exception as exc:
            line["instance_masks"] = {"error": repr(exc)}
        try:
            line["channels_last_to_planar"] = {n: measure_layout(wl.CONFIGS[n], 20, 3, dev) for n in ("c2", "c5")}
        except Exception as exc:
            line["channels_last_to_planar"] = {"error": repr(exc)}
    print(json.dumps(line))
    dist_util.shutdown()


def soft_threshold_for(cfg, dev):
    """A peak threshold for the soft-vote decode of this workload: 0.3 of the histogram's maximum on frame 0 (the
    threshold is the caller's parameter; the paper's is "predefined")."""
    import torch
    from paper_2609_16874_b200 import binding as cb
    fr = wl.make_frame(cfg, 0)
    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, device=dev)
    h = dec.soft_votes(torch.from_numpy(fr["emb"]).to(dev), torch.from_numpy(fr["fg"]).to(dev))
    torch.cuda.synchronize(dev)
    thr = 0.3 * float(h.max().item())
    dec.close()
    return thr


def measure_other(cfg, steps, warmup, dev, refine=False, k_max=None, flags=0, soft_threshold=None):
    """Graph-replay timing of one more workload (no host leg, no CPU baseline): p50, MP/s, per-stage times.
    `refine`: with sub-cell refined centroids (CPE_FLAG_REFINE); `k_max`: max_instances other than the workload's."""
    import torch
    from paper_2609_16874_b200 import binding as cb
    n_frames = frames_needed(cfg)
    frames = [wl.make_frame(cfg, f) for f in range(n_frames)]
    d_emb = [torch.from_numpy(f["emb"]).to(dev) for f in frames]
    d_fg = [torch.from_numpy(f["fg"]).to(dev) for f in frames]
    flush = (torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
             if cfg.emb_bytes < 2 * L2_BYTES and n_frames * cfg.emb_bytes < 2 * L2_BYTES else None)
    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau,
                     k_max if k_max else cfg.K_max, device=dev, refine=refine, flags=flags, soft_threshold=soft_threshold)
    pruned = cb.cpe_get_intermediate(dec.params, cb.CPE_INT_PRUNE_STATE, cfg.B, cfg.H, cfg.W, cfg.F)[0] == cb.CPE_OK
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        graphs = [dec.capture(d_emb[i], d_fg[i], stream=stream) for i in range(n_frames)]
        nodes = cb.cpe_graph_kernel_nodes(graphs[0])
        timed_replays(dec, graphs, stream, flush, warmup)
        step_ms = timed_replays(dec, graphs, stream, flush, steps)
        stage = dec.profile(d_emb[0], d_fg[0], iters=3, stream=stream)
        counters = dec.intermediate(cb.CPE_INT_COUNTERS).cpu().numpy().astype(np.int64)
        handed_on = dec.intermediate(cb.CPE_INT_PRUNE_STATE).cpu().numpy()[:, 2].tolist() if pruned else None
    count = dec.count.cpu().numpy().tolist()
    dec.close()
    peak_gbs, _ = measured_peaks()
    p50 = float(np.percentile(step_ms, 50))
    one_read_us = cfg.emb_bytes / (peak_gbs * 1e9) * 1e6
    alg = sum(algorithmic_bytes(cfg, int(np.mean([f["fg"].sum() for f in frames])), pruned).values())
    voting = max(1, int(counters[:, cb.CPE_CNT_VOTING].sum()))
    return {"workload": workload_name(cfg, refine), "decodes": steps, "p50_ms": p50,
            "p95_ms": float(np.percentile(step_ms, 95)),
            "value": cfg.pixels / (float(step_ms.mean()) * 1e-3) / 1e6, "unit": UNIT, "kernel_nodes": nodes, "stage_ms": stage,
            "instances_found": count, "pruned_assignment": pruned, "images_handed_to_filtered_kernel": handed_on,
            "scored_pairs_per_voting_pixel": float(counters[:, cb.CPE_CNT_FILTER_PAIRS].sum()) / voting,
            "one_read_embedding_roofline_us": one_read_us,
            "frac_of_one_read_roofline": one_read_us / (p50 * 1e3),
            "frac_of_algorithmic_bytes_roofline": alg / (peak_gbs * 1e9) / (p50 * 1e-3)}


def measure_launch_floor(cfg, steps, warmup, dev):
    """The decode's graph on the workload's shape with an all-zero mask: no pixel votes, no peak is found, nothing is
    scored; the kernels still start, synchronise with their predecessors, read the mask and write the (all-zero) label
    map.  Its replay time is what the chain of dependent launches costs before any of the method's arithmetic."""
    import torch
    from paper_2609_16874_b200 import binding as cb
    dt = torch.float32 if cfg.dtype == "f32" else torch.float16
    emb = torch.zeros(cfg.B, cfg.D, cfg.H, cfg.W, dtype=dt, device=dev)
    fg = torch.zeros(cfg.B, cfg.H, cfg.W, dtype=torch.uint8, device=dev)
    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, device=dev)
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        graph = dec.capture(emb, fg, stream=stream)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(warmup + steps):
            j = i - warmup
            if j >= 0:
                ev[j][0].record(stream)
            dec.replay(graph, stream=stream)
            if j >= 0:
                ev[j][1].record(stream)
        stream.synchronize()
    step_ms = np.array([a.elapsed_time(b) for a, b in ev])
    dec.close()
    return {"workload": cfg.name + " shape, all-zero mask", "steps": steps, "p50_ms": float(np.percentile(step_ms, 50)),
            "mean_ms": float(step_ms.mean()),
            "note": "the same graph; no votes, no peaks, no scoring; mask read and label map written"}


# Ceiling of the special-function units: 148 SMs x 16 results per clock x 1.965 GHz.
SFU_PEAK_GOPS = 148 * 16 * 1.965


def measure_soft_votes(cfg, steps, warmup, dev):
    """The second vote mode (`cpe_soft_votes`, Eq. 6) on the same workload: device time per call over rotating
    frames.  Its floor is the special-function units: every (participating pixel, bin of either axis) pair costs
    one square root and one exponential."""
    import torch
    from paper_2609_16874_b200 import binding as cb
    n_frames = frames_needed(cfg)
    frames = [wl.make_frame(cfg, f) for f in range(n_frames)]
    d_emb = [torch.from_numpy(f["emb"]).to(dev) for f in frames]
    d_fg = [torch.from_numpy(f["fg"]).to(dev) for f in frames]
    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, device=dev)
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        out = dec.soft_votes(d_emb[0], d_fg[0], stream=stream)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(warmup + steps):
            j = i - warmup
            if j >= 0:
                ev[j][0].record(stream)
            dec.soft_votes(d_emb[i % n_frames], d_fg[i % n_frames], out=out, stream=stream)
            if j >= 0:
                ev[j][1].record(stream)
        stream.synchronize()
    ms = np.array([a.elapsed_time(b) for a, b in ev])
    dec.close()
    part = float(np.mean([f["fg"].sum() for f in frames]))
    n_ab, n_bb = -(-cfg.bins_w // 128), -(-cfg.bins_h // 128)
    pairs = part * (cfg.bins_w + cfg.bins_h)                       # the method's own count
    r32 = lambda n: min(128, -(-n // 32) * 32)
    issued = part * sum(r32(cfg.bins_w - 128 * i) + r32(cfg.bins_h - 128 * j) for i in range(n_ab) for j in range(n_bb))   # what the blocks evaluate
    p50 = float(np.percentile(ms, 50))
    return {"entry_point": "cpe_soft_votes", "p50_ms": p50, "value": cfg.pixels / (p50 * 1e-3) / 1e6, "unit": UNIT,
            "bound": "sfu", "pixel_bin_pairs": pairs, "sfu_ops_algorithmic": 2 * pairs, "sfu_ops_issued": 2 * issued,
            "achieved_gops": 2 * pairs / (p50 * 1e-3) / 1e9, "peak_gops": SFU_PEAK_GOPS,
            "frac": 2 * pairs / (p50 * 1e-3) / 1e9 / SFU_PEAK_GOPS,
            "note": "memset + one kernel per call; two tcgen05 contractions per 128-pixel tile, weights kept on the SM"}


def measure_instance_masks(cfg, steps, warmup, dev):
    """`cpe_instance_masks` (the paper's one-hot planes and pixel counters) after one decode of the workload: a
    store-bound pass, 4 bytes read and n_planes bytes written per pixel; planes = the number of instances found."""
    import torch
    from paper_2609_16874_b200 import binding as cb
    fr = wl.make_frame(cfg, 0)
    d_emb, d_fg = torch.from_numpy(fr["emb"]).to(dev), torch.from_numpy(fr["fg"]).to(dev)
    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, device=dev)
    dec.decode(d_emb, d_fg)
    torch.cuda.synchronize()
    n_planes = max(1, int(dec.count.max().item()))
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(warmup + steps):
            j = i - warmup
            if j >= 0:
                ev[j][0].record(stream)
            planes, pixels = dec.instance_masks(n_planes, stream=stream)
            if j >= 0:
                ev[j][1].record(stream)
            del planes, pixels
        stream.synchronize()
    ms = np.array([a.elapsed_time(b) for a, b in ev])
    dec.close()
    peak_gbs, _ = measured_peaks()
    p50 = float(np.percentile(ms, 50))
    nbytes = cfg.pixels * (4 + n_planes)
    return {"entry_point": "cpe_instance_masks", "n_planes": n_planes, "p50_ms": p50, "bound": "hbm",
            "algorithmic_bytes": nbytes, "achieved": nbytes / (p50 * 1e-3) / 1e9, "peak": peak_gbs, "unit": "GB/s",
            "frac": nbytes / (p50 * 1e-3) / 1e9 / peak_gbs,
            "note": "includes torch's allocation of the output planes on the stream and the counters' memset"}


def measure_layout(cfg, steps, warmup, dev):
    """`cpe_channels_last_to_planar` on an embedding of the workload's size: one read and one write of it."""
    import torch
    from paper_2609_16874_b200 import binding as cb
    dt = torch.float32 if cfg.dtype == "f32" else torch.float16
    src = torch.randn(cfg.B, cfg.H, cfg.W, cfg.D, device=dev).to(dt)
    dst = torch.empty(cfg.B, cfg.D, cfg.H, cfg.W, dtype=dt, device=dev)
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if 2 * cfg.emb_bytes < 2 * L2_BYTES else None
    stream = torch.cuda.Stream(device=dev)
    code = cb.CPE_F32 if cfg.dtype == "f32" else cb.CPE_F16
    with torch.cuda.stream(stream):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(warmup + steps):
            if flush is not None:
                flush.fill_(i & 0xff)
            j = i - warmup
            if j >= 0:
                ev[j][0].record(stream)
            rc = cb.cpe_channels_last_to_planar(stream.cuda_stream, src.data_ptr(), dst.data_ptr(), cfg.B, cfg.H, cfg.W, cfg.F, code)
            assert rc == 0, rc
            if j >= 0:
                ev[j][1].record(stream)
        stream.synchronize()
    ms = np.array([a.elapsed_time(b) for a, b in ev])
    peak_gbs, _ = measured_peaks()
    p50 = float(np.percentile(ms, 50))
    nbytes = 2 * cfg.emb_bytes
    return {"entry_point": "cpe_channels_last_to_planar", "p50_ms": p50, "bound": "hbm", "algorithmic_bytes": nbytes,
            "achieved": nbytes / (p50 * 1e-3) / 1e9, "peak": peak_gbs, "unit": "GB/s", "frac": nbytes / (p50 * 1e-3) / 1e9 / peak_gbs,
            "l2": "a 252 MB buffer is rewritten between calls" if flush is not None else "source + destination exceed L2"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="c5", choices=sorted(wl.CONFIGS),
                    help="workload; c5 (1x2048x2048, F=16, 300 instances) is the largest single-GPU one")
    ap.add_argument("--candidates", default="refined", choices=["refined", "bins"],
                    help="what the pixels are assigned to: gamma of the peaks' refined centroids (CPE_FLAG_REFINE), or the "
                         "palette rows of the peaks' bins (the paper's Eq. 7 as printed)")
    ap.add_argument("--inner", type=int, default=0, help="decodes per step (0: as many as make a step last 2.5 ms)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-default", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--quick", action="store_true",
                    help="profiling runs: no clock pre-heat, no host-buffer leg, no CPU baseline (few launches)")
    ap.add_argument("--flags", type=int, default=0, help="extra cpe_params.flags bits (A/B runs)")
    ap.add_argument("--soft-votes", action="store_true",
                    help="profiling runs: only the second vote mode (cpe_soft_votes) on the chosen workload")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)
    cfg = wl.CONFIGS[args.config]
    if args.soft_votes:
        import torch
        dev = torch.device("cuda", 0)
        torch.cuda.set_device(dev)
        print(json.dumps({"soft_votes": measure_soft_votes(cfg, args.steps, args.warmup, dev), "name": cfg.name}))
        return
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
