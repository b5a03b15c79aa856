"""Entry usage and locality of the exact neighbours on one of the synthetic workloads
(`python -m paper_2312_01712_b200.entry_stats_report --workload c3`): the two observations the
method rests on (paper Sec. 3.2: the top-100 neighbours of a query use a minority of the codebook
entries; Sec. 3.3: those entries are the ones closest to the query's projection), measured with
`ivfpq_entry_stats`.  Prints one JSON line."""

from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from ivfpq_inputs import CONFIGS, build_index_streamed
from ivfpq_inputs.groundtruth import ExactKnnAccumulator
from ivfpq_inputs import generators as G

from . import binding as lib


def report(workload: str, nq: int | None, device: str = "cuda") -> dict:
    cfg = CONFIGS[workload] if nq is None else CONFIGS[workload].scaled(nq=nq)
    spec = G.make_mixture(cfg, device)
    q = G.queries(cfg, spec)
    acc = ExactKnnAccumulator(q, cfg.k)
    index = build_index_streamed(cfg, spec, on_chunk=acc.add)
    true_ids, _ = acc.result()
    pos_of_id = np.empty(index.ntotal, np.int64)
    pos_of_id[index.ids] = np.arange(index.ntotal)
    pos = torch.from_numpy(pos_of_id[true_ids]).to(device)
    h = lib.ivfpq_index_load(index, device)
    codes = torch.from_numpy(np.ascontiguousarray(index.codes)).to(device)
    qd = q.to(device).contiguous()
    lib.ivfpq_entry_stats(h, codes, qd, pos)                       # warm-up
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    usage, hist, flags = lib.ivfpq_entry_stats(h, codes, qd, pos)
    t1.record()
    torch.cuda.synchronize()
    usage = usage.cpu().numpy() / index.ksub
    cdf = np.cumsum(hist.cpu().numpy().sum(axis=0)) / float(hist.sum().item())
    lib.ivfpq_index_free(h)
    at = lambda frac: float(cdf[max(int(round(frac * index.ksub)) - 1, 0)])
    return {"workload": f"{cfg.name}: N={index.ntotal} PQ {index.nsub}x{index.dsub}, nq={q.shape[0]}, "
                        f"exact top-{cfg.k} neighbours",
            "usage_ratio": {"mean": float(usage.mean()), "max_subspace_mean": float(usage.mean(axis=0).max()),
                            "max": float(usage.max())},
            "cdf_of_neighbours_over_closest_entries": {"1/16": at(1 / 16), "1/8": at(1 / 8), "1/4": at(0.25),
                                                       "1/2": at(0.5), "3/4": at(0.75)},
            "kernel_ms": t0.elapsed_time(t1), "flags": flags}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c3", choices=sorted(CONFIGS))
    ap.add_argument("--nq", type=int, default=None)
    a = ap.parse_args()
    print(json.dumps(report(a.workload, a.nq)), flush=True)


if __name__ == "__main__":
    main()
