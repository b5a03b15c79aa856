#!/usr/bin/env python
"""Benchmark of the sparsity-aware IVFPQ query path on B200.

One "step" is one pass of the whole hot path - filtering, selective L2-LUT
construction, list scan, top-k - over one batch of synthetic queries through the C
ABI (`ivfpq_search_sparse` at the radius scale whose recall@100 is within 0.01 of
the dense search).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--nprobe 32]
    python bench.py --impl reference ...      # the CPU oracle on the host cores

Multi-GPU (torchrun, one rank per GPU): the index is replicated and every rank
searches its own query batch - no data-path collective ("scaling": "weak").
"""

from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import dataclasses  # noqa: E402

from ivfpq_inputs import (CONFIGS, DensityAccumulator, build_index_streamed, calibrate_radius,  # noqa: E402
                          calibrate_radius_ip, fit_threshold_model, recall_1_at_k, recall_at_k)
from ivfpq_inputs import generators as G  # noqa: E402
from ivfpq_inputs.groundtruth import ExactKnnAccumulator  # noqa: E402

METRIC = "queries/sec at recall@100 (1 B200) + scan HBM GB/s as % of peak"
UNIT = "queries/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per visited point of the dominant kernel
# at the default settings of a workload, from the ncu capture summarised in the named file under
# profiles/ (taken on a 1000-query batch: 7.309 GB for 475.8 M visited points; the traffic grows
# with the points visited).  An entry is dropped (traffic: null) when the kernel it describes changes.
SCAN_DRAM_BYTES_PER_VISIT = {"c5": (15.36, "profiles/scan16x8_1024_c5_nq1000.md")}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    REASONS = {
        0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
        0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
        0x100: "display_clock_setting",
    }

    def __init__(self, device_index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            uuid = torch.cuda.get_device_properties(device_index).uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # pragma: no cover
            log(f"[bench] NVML unavailable: {e}")
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for b, name in self.REASONS.items():
                    if bits & b:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self._period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------
# workload
# --------------------------------------------------------------------------------------------

def rank_config(name: str, nq: int | None, rank: int):
    """The workload of one rank: the index recipe is the same on every rank (replicated index), the
    query batch is drawn from a rank-specific seed (queries are sharded, no exchange)."""
    cfg = CONFIGS[name]
    if nq is not None:
        cfg = cfg.scaled(nq=nq)
    if rank:
        cfg = cfg.scaled(query_seed=cfg.query_seed + rank)
    return cfg


def max_over_ranks(total_ms: float, dist, device) -> float:
    """Device time of the slowest rank (all ranks search concurrently)."""
    if dist is None:
        return total_ms
    t = torch.tensor([total_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def build_workload(name: str, device: str, nq: int | None, query_seed_offset: int = 0, metric: int = 0,
                   dynamic: bool = False):
    """Index + queries + exact neighbours + calibrated radii for one of the synthetic configs.
    metric 1: the same index (clusters and codebooks trained under L2) searched by inner product,
    with exact maximum-inner-product neighbours as the ground truth."""
    cfg = rank_config(name, nq, query_seed_offset)
    t0 = time.time()
    spec = G.make_mixture(cfg, device)
    q = G.queries(cfg, spec)
    acc = ExactKnnAccumulator(q, cfg.k, metric=metric)
    on_chunk, dens, acc_cal, cal_q = acc.add, None, None, None
    if dynamic:
        # density maps of the base projections and exact neighbours of the training queries, gathered
        # in the same pass over the base vectors (unit-norm data: every projection lies in [-1, 1]^2)
        if cfg.dsub != 2 or not cfg.normalize:
            raise SystemExit("--dynamic-radius needs 2-d subspaces on unit-norm data (workload c3)")
        lo = torch.full((cfg.nsub, 2), -1.0, device=device)
        dens = DensityAccumulator(cfg.nsub, 100, (lo, -lo))
        cal_q = G.calibration_queries(cfg, spec, 1000)
        acc_cal = ExactKnnAccumulator(cal_q, cfg.k)

        def on_chunk(first_id, x):
            acc.add(first_id, x)
            acc_cal.add(first_id, x)
            dens.add(x)
    index = build_index_streamed(cfg, spec, on_chunk=on_chunk)
    true_ids, _ = acc.result()
    if dynamic:
        d_map, origin, inv_cell = dens.result()
        model = fit_threshold_model(index, d_map, origin, inv_cell, cal_q, acc_cal.result()[0], degree=2)
        log(f"[bench] built {name} with a threshold model (100 x 100 maps, degree 2) in {time.time() - t0:.1f}s")
        return cfg, index, q.cpu().numpy(), true_ids, model
    if metric == 1:
        index = dataclasses.replace(index, metric=1)
        radius = calibrate_radius_ip(index, G.calibration_queries(cfg, spec, 1000))
    else:
        radius = calibrate_radius(index, G.calibration_queries(cfg, spec, 1000))
    log(f"[bench] built {name}: N={index.ntotal} nlist={index.nlist} {index.nsub}x{index.dsub} "
        f"nq={q.shape[0]} in {time.time() - t0:.1f}s on {device}")
    return cfg, index, q.cpu().numpy(), true_ids, radius


def pick_scale(search_sparse, search_dense, true_ids, scales=(0.5, 0.75, 1.0, 1.25, 1.5, 2.0, 3.0, 4.0)):
    """Smallest radius scale whose recall@100 is within 0.01 of the dense search."""
    dense_ids = search_dense()
    r_dense = recall_at_k(dense_ids, true_ids)
    table = []
    chosen = None
    for s in scales:
        ids = search_sparse(s)
        r = recall_at_k(ids, true_ids)
        table.append((s, round(r, 4)))
        if chosen is None and r >= r_dense - 0.01:
            chosen = (s, r, recall_1_at_k(ids, true_ids))
            break
    if chosen is None:
        ids = search_sparse(float("inf"))
        chosen = (float("inf"), recall_at_k(ids, true_ids), recall_1_at_k(ids, true_ids))
    return r_dense, recall_1_at_k(dense_ids, true_ids), chosen, table


def pick_scale_for_counts(search_sparse, true_ids, scales=(0.5, 0.75, 1.0, 1.25, 1.5, 2.0, 3.0)):
    """Count scores never reproduce the dense ranking: take the radius scale with the best R1@100
    (the paper's quality measure for its hit-count configurations, Sec. 6.1)."""
    best, table = None, []
    for s in scales:
        ids = search_sparse(s)
        r, r1 = recall_at_k(ids, true_ids), recall_1_at_k(ids, true_ids)
        table.append((s, round(r, 4), round(r1, 4)))
        if best is None or r1 > best[2]:
            best = (s, r, r1)
    return best, table


SCORE_NAMES = {"distance": 0, "hit_count": 1, "reward_penalty": 2}


def scan_kernel_name(index) -> str:
    """Name of the kernel the library picks for this index (same rule as ivfpq_index_load)."""
    rot_shapes = {(16, 8), (48, 2), (50, 4), (8, 4), (12, 2)}
    if getattr(index, "metric", 0) == 1:
        return "scan_rot_kernel<inner product>" if (index.nsub, index.dsub) in rot_shapes else "scan_ip_kernel"
    if (index.nsub, index.dsub) == (16, 8):
        forced = os.environ.get("IVFPQ_SCAN_KERNEL")
        wide = forced == "warps32" or (forced != "warps16" and index.ntotal // index.nlist >= 2048)
        return "scan16x8_kernel<1024>" if wide else "scan16x8_kernel<512>"
    return "scan_rot_kernel"


def workload_string(cfg, index, nq, nprobe, k, scale) -> str:
    """One description of the workload for both arms."""
    return (f"{cfg.name}: N={index.ntotal} D={index.d} nlist={index.nlist} PQ {index.nsub}x{index.dsub} (uint8 codes), "
            f"nq={nq}/GPU, nprobe={nprobe}, k={k}, sparse search at radius scale {scale}")


def visits_per_batch(index, probe_ids: np.ndarray) -> int:
    lens = np.diff(index.list_offsets)
    return int(lens[probe_ids].sum())


def selection_stats(lib, h, index, qd, nprobe, k, rad_d, scale, score, sample=16):
    """What the selection does at this radius scale, from the stage dumps of a small query sample
    (outside any timed region): the mean fraction of codebook entries selected per (query, probed
    cluster, subspace), the fraction of visited points whose entry was selected in every subspace,
    and the mean fraction of subspaces selected per visited point."""
    n = min(sample, qd.shape[0])
    qs = qd[:n].contiguous()
    rad = rad_d if rad_d.dim() == 1 else rad_d[:n].contiguous()
    probe_ids = lib.ivfpq_debug_probes(h, qs, nprobe)[0].cpu().numpy()
    lens = np.diff(index.list_offsets)
    stride = int(lens[probe_ids].sum(axis=1).max())
    r = lib.ivfpq_debug_search(h, qs, nprobe, k, radius=rad, scale=scale, visit_stride=stride, score=score)
    masks = r["masks"].cpu().numpy().view(np.uint32)
    sel = float(np.unpackbits(masks.view(np.uint8)).sum()) / (masks.shape[0] * masks.shape[1] * index.nsub * index.ksub)
    vcount = r["visit_count"].cpu().numpy()
    hits = r["visit_hits"].cpu().numpy().view(np.uint64)
    full = np.uint64((1 << index.nsub) - 1)
    allhit = nvis = nbits = 0
    for i in range(n):
        hrow = hits[i, :vcount[i]]
        allhit += int((hrow == full).sum())
        nbits += int(np.unpackbits(hrow.view(np.uint8)).sum())
        nvis += int(vcount[i])
    return {"queries_sampled": n, "selected_entry_fraction": round(sel, 4),
            "all_hit_point_fraction": round(allhit / max(1, nvis), 5),
            "selected_subspaces_per_point": round(nbits / max(1, nvis) / index.nsub, 4)}


# --------------------------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------------------------

def run_cuda(args):
    import paper_2312_01712_b200 as lib

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus != world:
        if world == 1 and args.gpus > 1:
            raise SystemExit("launch with torch.distributed.run for --gpus > 1")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(dev))

    lib.load_library()
    metric = 1 if args.metric == "ip" else 0
    dynamic = bool(args.dynamic_radius)
    if dynamic and (metric != 0 or args.score != "distance"):
        raise SystemExit("--dynamic-radius goes with the L2 distance search")
    cfg, index, q_np, true_ids, radius = build_workload(args.workload, dev, args.nq, query_seed_offset=rank,
                                                        metric=metric, dynamic=dynamic)
    nprobe = args.nprobe or cfg.nprobes[len(cfg.nprobes) // 2]
    k = cfg.k
    nq = q_np.shape[0]
    h = lib.ivfpq_index_load(index, dev)
    has_map = (index.nsub, index.dsub) == (16, 8) and metric == 0
    if args.sparse_scan != "auto":
        if args.sparse_scan == "map" and not has_map:
            raise SystemExit("--sparse-scan map: this index shape has no entry->points map")
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN,
                                   lib.IVFPQ_SPARSE_SCAN_MAP if args.sparse_scan == "map" else lib.IVFPQ_SPARSE_SCAN_STREAM)
    map_scan = has_map and args.sparse_scan == "map"
    qd = torch.from_numpy(q_np).to(dev)
    model = mh = None
    if dynamic:
        # query-specific thresholds from the density maps and the regressor, computed on the device
        model, radius = radius, None
        mh = lib.ThresholdModelHandle(model, dev)
        rad_d = lib.ivfpq_query_thresholds(h, qd, mh)
    else:
        rad_d = torch.from_numpy(radius).to(dev)
    out = (torch.empty((nq, k), dtype=torch.float32, device=dev), torch.empty((nq, k), dtype=torch.int32, device=dev))

    def dense_ids():
        return lib.ivfpq_search_dense(h, qd, nprobe, k)[1].cpu().numpy()

    score = SCORE_NAMES[args.score]

    def sparse_ids(s):
        return lib.ivfpq_search_sparse(h, qd, nprobe, rad_d, k, scale=s, score=score)[1].cpu().numpy()

    if args.scale > 0:
        # a fixed radius scale (an operating point of lower quality than the recall-matched one)
        r_dense, r1_dense, (scale, r_sparse, r1_sparse), sweep = pick_scale(sparse_ids, dense_ids, true_ids, scales=(args.scale,))
        ids = sparse_ids(args.scale)
        scale, r_sparse, r1_sparse = args.scale, recall_at_k(ids, true_ids), recall_1_at_k(ids, true_ids)
    else:
        r_dense, r1_dense, (scale, r_sparse, r1_sparse), sweep = pick_scale(sparse_ids, dense_ids, true_ids)
    if score != 0 and args.scale <= 0:
        (scale, r_sparse, r1_sparse), sweep = pick_scale_for_counts(sparse_ids, true_ids)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    log(f"[bench] recall@100 dense {r_dense:.4f}, sparse {r_sparse:.4f} at scale {scale} (sweep {sweep})")

    sel_stats = selection_stats(lib, h, index, qd, nprobe, k, rad_d, scale, score)
    log(f"[bench] selection at scale {scale}: {sel_stats}")
    probe_ids = lib.ivfpq_debug_probes(h, qd, nprobe)[0].cpu().numpy()
    visits = visits_per_batch(index, probe_ids)
    scan_bytes = visits * index.nsub          # algorithmic: one code byte per subspace per visited point

    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)   # > L2 (126 MB)
    lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_TIMING, 1)

    def step_sparse():
        if dynamic:
            lib.ivfpq_query_thresholds(h, qd, mh, out=rad_d)
        lib.ivfpq_search_sparse(h, qd, nprobe, rad_d, k, scale=scale, out=out, score=score)

    def step_dense():
        lib.ivfpq_search_dense(h, qd, nprobe, k, out=out)

    def timed(step, steps, warmup, sampler=None, stage_acc=None):
        for _ in range(warmup):
            flush.zero_()
            step()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        ctx = sampler if sampler is not None else _Null()
        with ctx:
            for a, b in evs:
                flush.zero_()            # L2 flush between timed iterations (not timed)
                a.record()
                step()
                b.record()
                if stage_acc is not None:
                    stage_acc.append(lib.ivfpq_last_stage_ms(h))
            torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        return max_over_ranks(sum(a.elapsed_time(b) for a, b in evs), dist, dev)

    sampler = ClockSampler(local_rank)
    stages = []
    total_ms = timed(step_sparse, args.steps, args.warmup, sampler, stages)
    launches = (lib.ivfpq_last_launch_count(h) + (1 if dynamic else 0)) * args.steps
    dense_ms = timed(step_dense, max(3, args.steps // 4), 3)
    dense_steps = max(3, args.steps // 4)

    # end to end: host buffers, copies inside the timed region
    qh = torch.from_numpy(q_np).pin_memory()
    odh = torch.empty((nq, k), dtype=torch.float32).pin_memory()
    oih = torch.empty((nq, k), dtype=torch.int32).pin_memory()

    qd2 = torch.empty_like(qd)

    def step_host():
        if dynamic:   # the thresholds need the queries on the device before the search call
            qd2.copy_(qh, non_blocking=True)
            lib.ivfpq_query_thresholds(h, qd2, mh, out=rad_d)
            lib.ivfpq_search_sparse(h, qd2, nprobe, rad_d, k, scale=scale, out=out)
            odh.copy_(out[0], non_blocking=True)
            oih.copy_(out[1], non_blocking=True)
        else:
            lib.ivfpq_search_host(h, qh, nprobe, k, odh, oih, radius=rad_d, scale=scale, score=score)

    lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_TIMING, 0)
    e2e_steps = max(3, args.steps // 4)
    e2e_ms = timed(step_host, e2e_steps, 3)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK

    # the paper's comparison (Sec. 6.3 "Effectiveness of Dynamic Threshold Strategy"): one static
    # threshold per subspace set to the smallest / largest of the query-specific ones
    dyn_report = None
    if dynamic:
        lib.ivfpq_query_thresholds(h, qd, mh, out=rad_d)
        scaled = rad_d * scale
        dyn_report = {"threshold_min_mean_max": [float(scaled.min()), float(scaled.mean()), float(scaled.max())]}
        for name, stat in (("static_small", scaled.min(dim=0).values.contiguous()), ("static_large", scaled.max(dim=0).values.contiguous())):
            ids = lib.ivfpq_search_sparse(h, qd, nprobe, stat, k)[1].cpu().numpy()
            ms = timed(lambda: lib.ivfpq_search_sparse(h, qd, nprobe, stat, k, out=out), 5, 3)
            dyn_report[name] = {"recall@100": round(recall_at_k(ids, true_ids), 4), "queries_per_s": nq * world * 5 / (ms * 1e-3)}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = FALLBACK_HBM_GBS, "fallback"
    scan_ms = float(np.mean([s[1] for s in stages]))
    coarse_ms = float(np.mean([s[0] for s in stages]))
    props = torch.cuda.get_device_properties(local_rank)
    clk = sampler.summary()["sm_mhz"] or sampler.summary()["sm_max_mhz"] or 1965.0
    # Which ceiling binds the list scan depends on where the codes live.  Larger than the L2 cache:
    # the scan streams them from HBM, algorithmic bytes = one code byte per subspace per visited
    # point.  Inside the L2 cache: DRAM sees next to nothing and the ceiling is the shared-memory
    # table gather (one conflict-free 32-lane gather per SM per clock, one gather per code byte).
    code_bytes_total = int(index.ntotal) * index.nsub
    l2_bytes = int(getattr(props, "L2_cache_size", 126 << 20))
    hbm_gbs = scan_bytes / (scan_ms * 1e-3) / 1e9
    gather_peak = props.multi_processor_count * 32 * clk * 1e6 / 1e9            # G gathers/s
    kernel = ("scan16x8_map_kernel" if map_scan else scan_kernel_name(index)) + " (selective LUT + list scan + top-k)"
    default_run = args.nq is None and args.nprobe == 0 and score == 0 and metric == 0 and not dynamic
    per_visit = SCAN_DRAM_BYTES_PER_VISIT.get(args.workload) if (default_run and not map_scan) else None
    traffic = per_visit[0] * visits if per_visit else None
    common = {"kernel": kernel, "algorithmic_bytes_per_launch": int(scan_bytes), "visits_per_launch": int(visits),
              "kernel_ms": scan_ms, "traffic": traffic, "traffic_source": per_visit[1] if per_visit else None,
              "codes": f"{code_bytes_total / 1e6:.0f} MB of codes against {l2_bytes / 1e6:.0f} MB of L2"}
    if code_bytes_total > l2_bytes:
        roofline = {"bound": "hbm", "achieved": hbm_gbs, "peak": peak, "unit": "GB/s", "frac": hbm_gbs / peak,
                    "peak_source": f"of {peak_src}", **common,
                    "gather_frac": hbm_gbs / gather_peak}
    else:
        roofline = {"bound": "shared-memory gathers", "achieved": hbm_gbs, "peak": gather_peak, "unit": "Ggather/s",
                    "frac": hbm_gbs / gather_peak,
                    "peak_source": f"{props.multi_processor_count} SMs x 32 lanes x {clk:.0f} MHz", **common,
                    "hbm_equivalent_gbs": hbm_gbs,
                    "note": "the codes stay in L2, so HBM bandwidth does not bound this workload; the HBM-equivalent "
                            "rate (code bytes / kernel time) is context only"}

    cpu = cpu_baseline(index, q_np, nprobe, k, radius, scale, args.cpu_sample, score, model)

    line = {
        "metric": METRIC, "value": nq * world * args.steps / (total_ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_string(cfg, index, nq, nprobe, k, scale)
                               + ("" if score == 0 else f", ranked by {args.score}")
                               + ("" if metric == 0 else ", inner-product similarity")
                               + ("" if not dynamic else ", query-specific thresholds (density map + regressor) computed in the step"),
                   "l2": "512 MiB buffer written between timed iterations (L2 flush)",
                   "parallelism": "replicas only (index replicated, queries split)" if world > 1 else "1 GPU",
                   "radius_scale": scale, "nprobe": nprobe, "score": args.score, "similarity": args.metric},
        "recall@100": {"sparse": round(r_sparse, 4), "dense": round(r_dense, 4),
                       "R1@100_sparse": round(r1_sparse, 4), "R1@100_dense": round(r1_dense, 4)},
        "dense_queries_per_s": nq * world * dense_steps / (dense_ms * 1e-3),
        "sparse_over_dense": (dense_ms / dense_steps) / (total_ms / args.steps),
        "stages_ms": {"filtering": round(coarse_ms, 4), "lut_scan_topk": round(scan_ms, 4)},
        "e2e": {"value": nq * world * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": int(qh.numel() * 4), "d2h_bytes_per_step": int(odh.numel() * 4 + oih.numel() * 4)},
        "gpu_launches": int(launches),
        "clocks": sampler.summary(),
        "roofline": roofline,
        "selection": sel_stats,
        "cpu_baseline": cpu,
    }
    if dyn_report is not None:
        line["dynamic_threshold"] = dyn_report
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


# --------------------------------------------------------------------------------------------
# the CPU oracle: cpu_baseline leg and --impl reference
# --------------------------------------------------------------------------------------------

def oracle_sample_size(index, q_np, nprobe, k, radius, scale, score, want, target_s=15.0, model=None):
    """Number of queries for one timed oracle call: `want` if given, else as many as take about
    `target_s` seconds, estimated from a first call on 32 queries (which also pages the index in)."""
    import oracle
    nq = q_np.shape[0]
    if want and want > 0:
        return min(want, nq)
    n0 = min(32, nq)
    rad = radius if model is None else oracle.thresholds(index.d, index.nsub, index.dsub, q_np[:n0], model)
    oracle.search(index, q_np[:n0], nprobe, k, radius=rad, scale=scale, score=score)
    t0 = time.perf_counter()
    oracle.search(index, q_np[:n0], nprobe, k, radius=rad, scale=scale, score=score)
    rate = n0 / max(1e-6, time.perf_counter() - t0)
    return int(max(n0, min(nq, rate * target_s)))


def cpu_baseline(index, q_np, nprobe, k, radius, scale, sample, score=0, model=None):
    import oracle
    sample = oracle_sample_size(index, q_np, nprobe, k, radius, scale, score, sample, model=model)
    t0 = time.perf_counter()
    if model is not None:
        radius = oracle.thresholds(index.d, index.nsub, index.dsub, q_np[:sample], model)
    oracle.search(index, q_np[:sample], nprobe, k, radius=radius, scale=scale, score=score)
    dt = time.perf_counter() - t0
    return {"value": sample / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {sample} of the batch's {q_np.shape[0]} queries, one oracle.search call, {dt:.2f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"      # input generation only
    cfg, index, q_np, true_ids, radius = build_workload(args.workload, dev, args.nq,
                                                        metric=1 if args.metric == "ip" else 0)
    nprobe = args.nprobe or cfg.nprobes[len(cfg.nprobes) // 2]
    k = cfg.k
    scale = args.ref_scale
    if scale <= 0:
        # the same rule as the CUDA arm (smallest scale whose recall@100 is within 0.01 of dense),
        # decided by the oracle on a query sample that takes it a few seconds per scale
        ns = oracle_sample_size(index, q_np, nprobe, k, radius, 1.0, 0, 0, target_s=4.0)
        ns = min(ns, 1000)
        _, _, (scale, _, _), sweep = pick_scale(
            lambda sc: oracle.search(index, q_np[:ns], nprobe, k, radius=radius, scale=sc)["ids"],
            lambda: oracle.search(index, q_np[:ns], nprobe, k, dense=True)["ids"], true_ids[:ns])
        log(f"[bench] reference arm: radius scale {scale} from {ns} queries (sweep {sweep})")
    steps = min(args.steps, 5)
    # each step: a bounded sample of the batch, sized so that all steps take about 20 s together
    sample = oracle_sample_size(index, q_np, nprobe, k, radius, scale, 0, args.cpu_sample, target_s=20.0 / steps)
    for _ in range(min(args.warmup, 1)):
        oracle.search(index, q_np[:min(64, sample)], nprobe, k, radius=radius, scale=scale)
    t0 = time.perf_counter()
    for i in range(steps):
        lo = (i * sample) % max(1, q_np.shape[0] - sample + 1)
        oracle.search(index, q_np[lo:lo + sample], nprobe, k, radius=radius, scale=scale)
    dt = time.perf_counter() - t0
    value = sample * steps / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": dt / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_string(cfg, index, q_np.shape[0], nprobe, k, scale)
                               + ("" if args.metric == "l2" else ", inner-product similarity"),
                   "l2": "not applicable (host cores)", "parallelism": "1 process, OpenMP over queries",
                   "radius_scale": scale, "nprobe": nprobe, "score": "distance", "similarity": args.metric,
                   "reference_step": f"{sample} queries of the batch per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": f"{steps} steps x {sample} queries"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c5", choices=sorted(CONFIGS),
                    help="c5 (100 M points, 1.6 GB of codes: the one workload whose list scan streams from HBM) is "
                         "the headline; c1-c4 fit the L2 cache")
    ap.add_argument("--nprobe", type=int, default=0)
    ap.add_argument("--nq", type=int, default=None)
    ap.add_argument("--cpu-sample", type=int, default=0,
                    help="queries timed on the CPU oracle; 0 = as many as take about 15 s (at most the batch)")
    ap.add_argument("--ref-scale", type=float, default=0.0,
                    help="radius scale of the reference arm; 0 = chosen by the CUDA arm's recall rule")
    ap.add_argument("--scale", type=float, default=0.0,
                    help="radius scale of the sparse search; 0 = the smallest whose recall@100 is within 0.01 of dense")
    ap.add_argument("--dynamic-radius", action="store_true",
                    help="query-specific thresholds from density maps + polynomial regressor (workload c3)")
    ap.add_argument("--metric", default="l2", choices=["l2", "ip"],
                    help="similarity of the index (l2 = the headline path)")
    ap.add_argument("--sparse-scan", default="auto", choices=["auto", "stream", "map"],
                    help="list scan of the sparse search on the 16x8 shape: walk the entry->points map, stream the "
                         "codes, or let the library choose (it streams)")
    ap.add_argument("--score", default="distance", choices=sorted(SCORE_NAMES),
                    help="what the sparse search ranks by (distance = the headline path)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "cuda":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
