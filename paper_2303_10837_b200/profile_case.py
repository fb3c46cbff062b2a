"""Small single-kernel cases for profiling under ncu (a few hundred MB on the device).

    python paper_2303_10837_b200/profile_case.py encrypt [--cts 296] [--reps 2]
    python paper_2303_10837_b200/profile_case.py ntt [--polys 256]
    python paper_2303_10837_b200/profile_case.py aggregate [--cts 64]
    python paper_2303_10837_b200/profile_case.py sweep [--prime-bits 45]   # kernel sweep table (no profiler)
    python paper_2303_10837_b200/profile_case.py kernels [--workload W]    # every step alone, % of the HBM peak

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


def kernels(workload):
    """Every step of the round timed alone on one workload: algorithmic bytes (the minimum the
    step must move) / time as a share of the HBM peak, median of 11 runs."""
    peak, src = read_hbm_peak()
    base = {"resnet18": si.RESNET18, "tiny": si.TINY, "bert": si.bert(1.0)}[workload]
    w = si.scaled(base, min(base.P, 11_700_000), clients=base.clients)        # full encryption of at most 11.7 M parameters
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    C, L, N, n, T, P = w.clients, w.L, w.N, w.n, w.T, w.P
    xs = [torch.from_numpy(si.client_update(w, i)).cuda() for i in range(C)]
    alpha = si.client_weights(w)
    score = torch.rand(P, device="cuda")
    mask = he.he_select_mask(g, score, P // 10)
    sel, _ = he.he_pack(g, None, xs[0])
    cts = [he.he_encrypt(g, keys, he.he_pack(g, None, xs[i])[0], w.enc_seed, i) for i in range(C)]
    agg = he.he_weighted_aggregate(g, cts, alpha)
    z = he.he_decrypt(g, keys, agg)
    rests = [he.he_pack(g, mask, xs[i])[1] for i in range(C)]
    ravg = he.he_plain_aggregate(g, rests, alpha)

    # Short calls are timed as `burst` back-to-back calls between two events (one call alone would
    # time the launch latency, not the kernel), on rotating inputs and with the results kept alive so
    # that consecutive calls touch different memory (more than the L2 holds in total); long calls alone.
    keep = []

    def med(fn, burst):
        ts = []
        for _ in range(5):
            keep.clear()
            torch.cuda.synchronize()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            for i in range(burst):
                keep.append(fn(i))
            ev1.record()
            torch.cuda.synchronize()
            ts.append(ev0.elapsed_time(ev1) / burst)
        keep.clear()
        return sorted(ts)[2]

    outs = [torch.empty(P, dtype=torch.float64, device="cuda") for _ in range(3)]
    zs = [z, z.clone(), z.clone()]
    rows = [
        ("he_select_mask (k = P/10)", lambda i: he.he_select_mask(g, score, P // 10), 6 * 4.0 * P, 4),
        ("he_pack (full)", lambda i: he.he_pack(g, None, xs[i % C]), 8.0 * P, 8),
        ("he_pack (masked, 10 %)", lambda i: he.he_pack(g, mask, xs[i % C]), 8.0 * P + 4.0 * P / 10, 8),
        ("he_encode", lambda i: he.he_encode(g, sel), 4.0 * T * n + 8.0 * T * N, 4),
        ("he_encrypt (encode + encrypt)", lambda i: he.he_encrypt(g, keys, sel, w.enc_seed, 0, out=cts[i % C]),
         4.0 * T * n + 16.0 * L * N * T, 2),
        ("he_weighted_aggregate", lambda i: he.he_weighted_aggregate(g, cts, alpha, out=agg),
         16.0 * N * T * (L * C + (L - 1)), 1),
        ("he_plain_aggregate (90 %)", lambda i: he.he_plain_aggregate(g, rests, alpha), rests[0].numel() * (4.0 * C + 8), 4),
        ("he_decrypt (decrypt + decode)", lambda i: he.he_decrypt(g, keys, agg, out=zs[i % 3]), 16.0 * N * T + 8.0 * n * T, 2),
        ("he_unpack (full)", lambda i: he.he_unpack(g, None, zs[i % 3], None, P, out=outs[i % 3]), 16.0 * P, 6),
        ("he_unpack (masked, 10 %)", lambda i: he.he_unpack(g, mask, zs[i % 3], ravg, P, out=outs[i % 3]),
         4.0 * P / 10 + 8.0 * P + 8.0 * P, 6),
    ]
    print("workload %s: N %d, L %d, %d clients, %d ciphertexts per client; HBM peak %.1f GB/s (%s)"
          % (w.name, N, L, C, T, peak, src))
    print("%-34s %10s %12s %9s %7s" % ("call", "ms", "alg. MB", "GB/s", "%HBM"))
    for name, fn, nbytes, burst in rows:
        ms = med(fn, burst)
        gbs = nbytes / (ms * 1e-3) / 1e9
        print("%-34s %10.3f %12.1f %9.1f %6.1f%%" % (name, ms, nbytes / 1e6, gbs, 100 * gbs / peak))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["encrypt", "ntt", "aggregate", "decrypt", "sweep", "kernels"])
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
    if a.case == "kernels":
        kernels(a.workload)
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
