"""Small single-kernel cases for profiling under ncu (a few hundred MB on the device).

    python paper_2303_10837_b200/profile_case.py encrypt [--cts 296] [--reps 2]
    python paper_2303_10837_b200/profile_case.py ntt [--polys 256]
    python paper_2303_10837_b200/profile_case.py aggregate [--cts 64]
    python paper_2303_10837_b200/profile_case.py sweep [--prime-bits 45]   # kernel sweep table (no profiler)

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


def read_hbm_peak():
    import json
    try:
        return float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def timed(fn, reps):
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fn()
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(reps):
        fn()
    ev1.record()
    torch.cuda.synchronize()
    return ev0.elapsed_time(ev1) / reps


def sweep(bits=60):
    """Batched forward+inverse NTT and encode+encrypt over ring degrees, limb counts and batch
    sizes; GB/s counts 16 N bytes per limb transform (32 N for N > 2^14: two passes) and the
    ciphertext bytes written per encryption."""
    peak, src = read_hbm_peak()
    print("HBM peak %.1f GB/s (%s); %d-bit primes" % (peak, src, bits))
    print("%6s %3s %6s | %10s %9s %7s | %10s %9s %7s" % ("N", "L", "batch", "ntt us", "GB/s", "%HBM", "encrypt us", "GB/s", "%HBM"))
    for logn in (13, 14, 15, 16):
        N = 1 << logn
        for L in (2, 4, 8, 12):
            primes = (si.PRIMES_SWEEP if bits == 60 else si.PRIMES_SWEEP_45)[:L]
            g = he.he_ctx_create(N, list(primes), 40)
            keys = he.he_keygen(g, 5)
            for B in (1, 4, 16, 64, 256, 1024, 4096):
                words = B * L * N
                if words * 8 > 8 << 30 or 2 * words * 8 > 12 << 30:
                    continue
                polys = torch.randint(0, 1 << (bits - 1), (B, L, N), dtype=torch.int64, device="cuda")   # below every prime
                reps = 3 if words > (1 << 26) else 10

                def both():
                    he.he_ntt_forward(g, polys)
                    he.he_ntt_inverse(g, polys)
                t_ntt = timed(both, reps) / 2
                passes = 1 if logn <= 14 else 2
                gbs_ntt = 16.0 * N * L * B * passes / (t_ntt * 1e-3) / 1e9
                del polys
                sel = torch.randn(B * (N // 2), dtype=torch.float32, device="cuda") * 0.01
                ct = torch.empty((B, 2, L, N), dtype=torch.int64, device="cuda")
                t_enc = timed(lambda: he.he_encrypt(g, keys, sel, 3, 0, out=ct), reps)
                gbs_enc = (16.0 * N * L + 2.0 * N) * B / (t_enc * 1e-3) / 1e9
                del sel, ct
                print("%6d %3d %6d | %10.1f %9.1f %6.1f%% | %10.1f %9.1f %6.1f%%"
                      % (N, L, B, t_ntt * 1e3, gbs_ntt, 100 * gbs_ntt / peak, t_enc * 1e3, gbs_enc,
                         100 * gbs_enc / peak), flush=True)
            del keys, g


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["encrypt", "ntt", "aggregate", "decrypt", "sweep"])
    ap.add_argument("--cts", type=int, default=296)
    ap.add_argument("--polys", type=int, default=256)
    ap.add_argument("--reps", type=int, default=2)
    ap.add_argument("--workload", choices=["resnet18", "tiny", "bert"], default="resnet18")
    ap.add_argument("--prime-bits", type=int, choices=[60, 45], default=60,
                    help="sweep: 60-bit primes (integer transforms) or 45-bit primes (double-precision transforms)")
    a = ap.parse_args()
    if a.case == "sweep":
        sweep(a.prime_bits)
        return
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
