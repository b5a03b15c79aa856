"""Throughput against search quality on one of the synthetic workloads
(`python -m paper_2312_01712_b200.recall_curve --workload c5 --nprobes 32,64,128,256`): for every
probe count the dense search and the sparsity-aware search at the smallest radius scale whose
recall@100 stays within 0.01 of the dense one, each with queries/s (device time of the search call,
L2 flushed between iterations), recall@100 and R1@100 against exact brute-force neighbours (the
quality measure of the paper's evaluation, Sec. 6.1).  Prints one JSON line per probe count."""

from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from ivfpq_inputs import CONFIGS, build_index_streamed, calibrate_radius, recall_1_at_k, recall_at_k
from ivfpq_inputs import generators as G
from ivfpq_inputs.groundtruth import ExactKnnAccumulator

from . import binding as lib

SCALES = (0.5, 0.75, 1.0, 1.25, 1.5, 2.0, 3.0, 4.0)


def curve(workload: str, nprobes, nq: int | None, device: str = "cuda", iters: int = 5):
    cfg = CONFIGS[workload] if nq is None else CONFIGS[workload].scaled(nq=nq)
    spec = G.make_mixture(cfg, device)
    q = G.queries(cfg, spec)
    acc = ExactKnnAccumulator(q, cfg.k)
    index = build_index_streamed(cfg, spec, on_chunk=acc.add)
    true_ids, _ = acc.result()
    radius = torch.from_numpy(calibrate_radius(index, G.calibration_queries(cfg, spec, 1000))).to(device)
    h = lib.ivfpq_index_load(index, device)
    qd = q.to(device).contiguous()
    k = cfg.k
    out = (torch.empty((qd.shape[0], k), dtype=torch.float32, device=device),
           torch.empty((qd.shape[0], k), dtype=torch.int32, device=device))
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)   # larger than L2

    def timed(step):
        for _ in range(2):
            step()
        evs = []
        for _ in range(iters):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            step()
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        return float(np.median([a.elapsed_time(b) for a, b in evs]))

    rows = []
    for nprobe in nprobes:
        if nprobe > index.nlist:
            continue
        ids = lib.ivfpq_search_dense(h, qd, nprobe, k)[1].cpu().numpy()
        rd, r1d = recall_at_k(ids, true_ids), recall_1_at_k(ids, true_ids)
        ms_d = timed(lambda: lib.ivfpq_search_dense(h, qd, nprobe, k, out=out))
        scale, rs, r1s = float("inf"), rd, r1d
        for s in SCALES:
            ids = lib.ivfpq_search_sparse(h, qd, nprobe, radius, k, scale=s)[1].cpu().numpy()
            r = recall_at_k(ids, true_ids)
            if r >= rd - 0.01:
                scale, rs, r1s = s, r, recall_1_at_k(ids, true_ids)
                break
        ms_s = timed(lambda: lib.ivfpq_search_sparse(h, qd, nprobe, radius, k, scale=scale, out=out))
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        rows.append({"workload": workload, "nprobe": nprobe, "nq": int(qd.shape[0]),
                     "dense": {"queries_per_s": qd.shape[0] / (ms_d * 1e-3), "recall@100": round(rd, 4), "R1@100": round(r1d, 4)},
                     "sparse": {"queries_per_s": qd.shape[0] / (ms_s * 1e-3), "recall@100": round(rs, 4), "R1@100": round(r1s, 4),
                                "radius_scale": scale}})
        print(json.dumps(rows[-1]), flush=True)
    lib.ivfpq_index_free(h)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c5", choices=sorted(CONFIGS))
    ap.add_argument("--nprobes", default="32,64,128,256")
    ap.add_argument("--nq", type=int, default=None)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    curve(args.workload, [int(x) for x in args.nprobes.split(",")], args.nq)


if __name__ == "__main__":
    main()
