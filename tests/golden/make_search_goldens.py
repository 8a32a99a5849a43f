"""Writes tests/golden/search_*.json: the oracle's exhaustive-search answers for the benchmark
configurations (optimum, top-k, feasible count), so that GPU parity at full size does not need a
multi-minute CPU enumeration inside the test run.

Calls only the CPU oracle and the input module.  Usage (from the repo root):
    python tests/golden/make_search_goldens.py [--threads N] [name-substring ...]
A full run over all 35 workloads enumerates about 9e10 mappings (about an hour on 8 cores).
"""
import argparse
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import mmee_inputs as mi   # noqa: E402
import oracle              # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def record_dict(r):
    return dict(idx=r.idx, t=r.t, row=r.row, bound=list(r.bound), phi=r.phi, pi=r.pi,
                beta=list(r.beta), sm=list(r.sm), recompute=r.recompute,
                bs=r.bs, bs_op1=r.bs_op1, bs_op2=r.bs_op2, br=r.br, cyc1=r.cyc1, cyc2=r.cyc2,
                n=list(r.n), e_key=r.e_key, l_key=r.l_key, edp_key_hex=float(r.edp_key).hex(),
                energy_pj_hex=float(r.energy_pj).hex(),
                latency_cycles_hex=float(r.latency_cycles).hex())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("names", nargs="*")
    args = ap.parse_args()
    for cfg in mi.golden_configs():
        if args.names and not any(s in cfg["name"] for s in args.names):
            continue
        path = os.path.join(HERE, "search_%s.json" % cfg["name"])
        out = dict(name=cfg["name"], workload=cfg["workload"], arch=cfg["arch"], searches=[])
        for obj in cfg["searches"]:
            p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
            t0 = time.time()
            res = oracle.search(p, args.threads)
            dt = time.time() - t0
            out["searches"].append(dict(objective=obj, n_total=res.n_total, n_feasible=res.n_feasible,
                                        topk=[record_dict(r) for r in res.topk]))
            print("%s obj=%d k=%d N=%d feasible=%d  %.1f s  %.1f M/s" %
                  (cfg["name"], obj["objective"], obj["topk"], res.n_total, res.n_feasible, dt,
                   res.n_total / dt / 1e6), flush=True)
        with open(path, "w") as f:
            json.dump(out, f, indent=1)
            f.write("\n")


if __name__ == "__main__":
    main()
