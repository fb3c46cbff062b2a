"""Small single-kernel cases for profiling under ncu (a few hundred MB on the device).

    python paper_2303_10837_b200/profile_case.py encrypt [--cts 296] [--reps 2]
    python paper_2303_10837_b200/profile_case.py ntt [--polys 256]
    python paper_2303_10837_b200/profile_case.py aggregate [--cts 64]

Each case touches more memory than the L2 holds so that DRAM counters mean something,
launches the kernel of interest a handful of times and exits.
"""
from __future__ import annotations

import argparse
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import paper_2303_10837_b200 as he
import synthetic_inputs as si


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["encrypt", "ntt", "aggregate", "decrypt"])
    ap.add_argument("--cts", type=int, default=296)
    ap.add_argument("--polys", type=int, default=256)
    ap.add_argument("--reps", type=int, default=2)
    ap.add_argument("--workload", choices=["resnet18", "tiny", "bert"], default="resnet18")
    a = ap.parse_args()
    base = {"resnet18": si.RESNET18, "tiny": si.TINY, "bert": si.bert(1.0)}[a.workload]
    w = si.scaled(base, a.cts * base.n, clients=base.clients)
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if a.case == "ntt":
        polys = torch.from_numpy(si.random_residues(7, (a.polys, w.L, w.N), w.primes).view(np.int64)).cuda()
        ev0.record()
        for _ in range(a.reps):
            he.he_ntt_forward(g, polys)
            he.he_ntt_inverse(g, polys)
        ev1.record()
    else:
        x = torch.from_numpy(si.client_update(w, 0)).cuda()
        sel, _ = he.he_pack(g, None, x)
        if a.case == "encrypt":
            ct = he.he_encrypt(g, keys, sel, 1, 0)
            ev0.record()
            for _ in range(a.reps):
                he.he_encrypt(g, keys, sel, 1, 0, out=ct)
            ev1.record()
        else:
            cts = [he.he_encrypt(g, keys, sel, 1, i) for i in range(w.clients)]
            alpha = si.client_weights(w)
            agg = he.he_weighted_aggregate(g, cts, alpha)
            ev0.record()
            for _ in range(a.reps):
                if a.case == "aggregate":
                    he.he_weighted_aggregate(g, cts, alpha, out=agg)
                else:
                    he.he_decrypt(g, keys, agg)
            ev1.record()
    torch.cuda.synchronize()
    print("%s: %.3f ms per repetition" % (a.case, ev0.elapsed_time(ev1) / a.reps))


if __name__ == "__main__":
    main()
