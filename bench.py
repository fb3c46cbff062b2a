#!/usr/bin/env python
"""Benchmark of the HE secure-aggregation round on B200.

One step = one whole round of the hot path over one batch of synthetic client
updates: for every client pack + CKKS-encode + encrypt, then the server's
weighted ciphertext sum with rescale (and the plaintext remainder average when
a mask is used), then decrypt + decode + unpack.  The headline value is model
parameters per second with the inputs already in HBM; ``e2e`` is the same round
through ``he_round_host`` with pinned host buffers, copies inside the timed
region.  ``--impl reference`` times the CPU oracle instead.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

For N > 1 launch under ``torch.distributed.run``; every rank processes its own
full batch (ciphertext indices are independent, so the path shards with no
collective) and the job time is the maximum over ranks.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import synthetic_inputs as si

METRIC = "HE-agg params/s (encrypt+weighted sum+decrypt); NTT % of HBM roofline"
UNIT = "params/s"

# Roofline of the transforms.  On B200 integer multiplies and double-precision
# operations draw on one budget of 64 slots per SM and clock (measured with the
# int_pipe_bench tool of the package: 63.7 32-bit multiply-adds, 63.6
# double-precision FMAs, and no gain from running half of each side by side);
# a 32x32->64 multiply-add costs 2.5 of those slots.  A 64-bit Shoup butterfly
# needs the high half of x*w' (4 wide products) and the low halves of x*w and
# hi*q (1 wide + 2 narrow each): 6 wide + 4 narrow = 19 slots.  Limbs whose
# prime is below 2^46 run in exact double-precision arithmetic instead: 6
# operations for the modular product, 2 for the sum and difference, and in the
# inverse transform 1 more per butterfly for keeping the sums small.
# Additions, shifts and logic go to another pipe.
# DRAM bytes (read + write) per ciphertext of encrypt_fused2_kernel at N = 16384,
# L = 4, from an ncu capture of the profile_case.py encrypt case (summary under profiles/)
# (363.1 MB for 296 ciphertexts; traffic grows in proportion to the count).
ENCRYPT_DRAM_BYTES_PER_CT_N16384_L4 = 363.052288e6 / 296
SLOTS_PER_SM_CLK = 64.0
WIDE_COST = 2.5
INT_SLOTS_PER_BUTTERFLY = 6 * WIDE_COST + 4
F64_SLOTS_FORWARD, F64_SLOTS_INVERSE = 8.0, 9.0
F64_PRIME_LIMIT = 1 << 46


def transform_slots(primes, N, forward, inverse):
    """Pipe slots of `forward` forward and `inverse` inverse transforms of every limb."""
    bf = (N // 2) * (N.bit_length() - 1)
    total = 0.0
    for q in primes:
        if q < F64_PRIME_LIMIT:
            total += bf * (forward * F64_SLOTS_FORWARD + inverse * F64_SLOTS_INVERSE)
        else:
            total += bf * (forward + inverse) * INT_SLOTS_PER_BUTTERFLY
    return total


def fallback_peaks():
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


def read_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {"hbm_gbs": float(d["hbm_gbs"]), "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)),
                    "source": "measured"}
        except Exception:
            pass
    return fallback_peaks()


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                   f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def reduce_job(units_local: float, seconds_local: float, world: int, backend_tensor_device="cpu"):
    """Whole-job units (sum over ranks) and time (max over ranks)."""
    if world == 1:
        return units_local, seconds_local
    import torch
    import torch.distributed as dist
    t = torch.tensor([seconds_local], dtype=torch.float64, device=backend_tensor_device)
    u = torch.tensor([units_local], dtype=torch.float64, device=backend_tensor_device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()), float(t.item())


# --------------------------------------------------------------------------- oracle arms

def oracle_sample(w: si.Workload, n_ct: int, rank_seed: int = 0):
    """Times the CPU oracle on the first n_ct ciphertext indices of the workload (all clients)."""
    import oracle
    n_ct = min(n_ct, w.T)
    P_s = min(w.P, n_ct * w.n)
    o = oracle.Context(w.N, w.primes, w.log2_delta)
    xs = [si.client_update(w, i, P_s) for i in range(w.clients)]
    alpha = si.client_weights(w)
    t0 = time.perf_counter()
    out = o.round(xs, alpha, None, P_s, w.key_seed, w.enc_seed + rank_seed, 0, n_ct)
    dt = time.perf_counter() - t0
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(out - want).max() < 1e-6
    return P_s, dt, oracle.num_threads()


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    n_ct = 256
    for _ in range(args.warmup):
        oracle_sample(w, 2)
    units, secs, cores = 0, 0.0, 1
    for _ in range(args.steps):
        p, dt, cores = oracle_sample(w, n_ct)
        units += p
        secs += dt
    value = units / secs
    sample = "first %d of %d ciphertext indices, all %d clients, per step" % (min(n_ct, w.T), w.T, w.clients)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
        "data": "synthetic", "config": config_dict(w, "oracle sample: " + sample),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def config_dict(w, note):
    return {"workload": w.name, "N": w.N, "slots": w.n, "limbs": w.L, "log2_delta": w.log2_delta,
            "clients": w.clients, "params": w.P, "encrypted_params": w.k, "ciphertexts_per_client": w.T,
            "l2": "inputs larger than L2 (%.1f GB of ciphertexts per step%s)"
                  % (w.clients * w.T * 2 * w.L * w.N * 8 / 1e9,
                     ", streamed in chunks of ciphertext indices" if w.clients * w.T * 2 * w.L * w.N * 8 > 40e9 else ""),
            "note": note}


# --------------------------------------------------------------------------- GPU arm

def run_ours(args, w):
    import torch
    import torch.distributed as dist
    import paper_2303_10837_b200 as he

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = read_peaks()

    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    alpha = si.client_weights(w)
    enc_seed = w.enc_seed + 1000 * rank
    # inputs: every rank has its own batch (weak scaling)
    xs_host = []
    for i in range(w.clients):
        rng = np.random.default_rng([w.seed, 1000 + i, rank])
        x = rng.standard_normal(w.P, dtype=np.float32)
        x *= np.float32(w.std)
        xs_host.append(torch.from_numpy(x).pin_memory())
    xs = [x.cuda() for x in xs_host]
    mask = None
    if w.k < w.P:
        mask = he.he_select_mask(g, torch.from_numpy(si.sensitivity_scores(w)).cuda(), w.k)
    T, n = w.T, w.n
    # ciphertext indices are streamed in chunks when all clients' ciphertexts exceed 40 GB
    ct_bytes = 8 * 2 * w.L * w.N
    Tc = T
    if w.clients * T * ct_bytes > 40e9:
        n_sm = torch.cuda.get_device_properties(local).multi_processor_count
        Tc = max(n_sm, int(16e9 // (w.clients * ct_bytes)) // n_sm * n_sm)
    cts = [torch.empty((Tc, 2, w.L, w.N), dtype=torch.int64, device="cuda") for _ in range(w.clients)]
    agg = torch.empty((Tc, 2, w.L - 1, w.N), dtype=torch.int64, device="cuda")
    z = torch.empty(T * n, dtype=torch.float64, device="cuda")
    out = torch.empty(w.P, dtype=torch.float64, device="cuda")
    he.he_ctx_reserve(g, w.k)
    enc_events = []

    def step_streamed(record):
        sels = [he.he_pack(g, mask, xs[i])[0] for i in range(w.clients)]
        for t0 in range(0, T, Tc):
            tc = min(Tc, T - t0)
            for i in range(w.clients):
                if record:
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                he.he_encrypt_range(g, keys, sels[i][t0 * n:(t0 + tc) * n], t0, tc, enc_seed, i, cts[i][:tc])
                if record:
                    e1.record()
                    enc_events.append((e0, e1, tc))
            he.he_weighted_aggregate(g, [c[:tc] for c in cts], alpha, out=agg[:tc])
            he.he_decrypt(g, keys, agg[:tc], out=z[t0 * n:(t0 + tc) * n])
        he.he_unpack(g, mask, z, None, w.P, out=out)

    transform = args.format == "transform"
    if transform and Tc < T:
        raise SystemExit("bench: --format transform is not wired to the streamed (chunked) round")
    enc = he.he_encrypt_ntt if transform else he.he_encrypt

    def step(record):
        if Tc < T:
            return step_streamed(record)
        rests = []
        for i in range(w.clients):
            sel, rest = he.he_pack(g, mask, xs[i])
            if record:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            enc(g, keys, sel, enc_seed, i, out=cts[i])
            if record:
                e1.record()
                enc_events.append((e0, e1, T))
            rests.append(rest)
        if transform:
            he.he_weighted_aggregate_ntt(g, cts, alpha, out=agg)
            he.he_decrypt_level_ntt(g, keys, agg, w.L - 1, out=z)
        else:
            he.he_weighted_aggregate(g, cts, alpha, out=agg)
            he.he_decrypt(g, keys, agg, out=z)
        avg = he.he_plain_aggregate(g, rests, alpha) if mask is not None else None
        he.he_unpack(g, mask, z, avg, w.P, out=out)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step(False)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = he.he_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step(True)
    ev1.record()
    barrier()
    launches = he.he_launch_count() - launches0
    secs = ev0.elapsed_time(ev1) * 1e-3
    # correctness of what was timed: plaintext FedAvg on every parameter
    want = sum(float(a) * x.double() for a, x in zip(alpha, xs))
    err = float((out - want).abs().max())
    if not err <= 1e-6 or he.he_ctx_status(g) != he.HE_OK:
        raise SystemExit("bench: aggregate differs from plaintext FedAvg by %g" % err)

    # dominant kernel: the fused encrypt.  Its duration = the event-bracketed
    # he_encrypt calls of the timed region minus the encode kernel that runs in
    # the same call, timed alone on the same inputs.
    # time of all he_encrypt calls of one client (T ciphertexts, one call unless streamed)
    enc_ms = sum(a.elapsed_time(b) for a, b, _ in enc_events) / (args.steps * w.clients)
    sel0, _ = he.he_pack(g, mask, xs[0])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 5
    he.he_encode(g, sel0)
    e0.record()
    for _ in range(reps):
        he.he_encode(g, sel0)
    e1.record()
    torch.cuda.synchronize()
    encode_ms = e0.elapsed_time(e1) / reps
    kern_ms = max(enc_ms - encode_ms, 1e-6)

    # standalone transform: forward + inverse over a batch larger than L2
    B = 256
    polys = torch.from_numpy(si.random_residues(7, (B, w.L, w.N), w.primes).view(np.int64)).cuda()
    he.he_ntt_forward(g, polys)
    he.he_ntt_inverse(g, polys)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        he.he_ntt_forward(g, polys)
        he.he_ntt_inverse(g, polys)
    e1.record()
    torch.cuda.synchronize()
    ntt_ms = e0.elapsed_time(e1) / (2 * reps)
    pass_bytes = 16.0 * w.N * w.L * B * (1 if w.N <= 16384 else 2)
    ntt_gbs = pass_bytes / (ntt_ms * 1e-3) / 1e9
    clocks = sampler.stop()

    # e2e through the host entry point
    host_out = torch.empty(w.P, dtype=torch.float64).pin_memory()
    he.he_round_host(g, keys, mask, xs_host, alpha, enc_seed, host_out)          # allocates its buffers
    barrier()
    e2e_steps = max(1, min(args.steps, 3))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        he.he_round_host(g, keys, mask, xs_host, alpha, enc_seed, host_out)
    torch.cuda.synchronize()
    e2e_secs = time.perf_counter() - t0
    if not float((host_out.cuda() - want).abs().max()) <= 1e-6:
        raise SystemExit("bench: host round differs from plaintext FedAvg")

    units, job_secs = reduce_job(float(w.P) * args.steps, secs, world, "cuda")
    e2e_units, e2e_job = reduce_job(float(w.P) * e2e_steps, e2e_secs, world, "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # roofline of the dominant kernel (bound by the multiply / double-precision pipe)
    logN = w.N.bit_length() - 1
    butterflies = 3 * w.L * (w.N // 2) * logN * T           # per launch: 3 limb transforms per limb
    # coefficient format: one forward and two inverse transforms per limb; transform format: three forward
    achieved = transform_slots(w.primes, w.N, 3 if transform else 1, 0 if transform else 2) * T / (kern_ms * 1e-3) / 1e12
    n_sm = torch.cuda.get_device_properties(local).multi_processor_count
    peak = n_sm * SLOTS_PER_SM_CLK * peaks["sm_max_mhz"] * 1e6 / 1e12
    alg_bytes = (16.0 + 32.0 * w.L) * n * T          # read m, write the ciphertext
    roofline = {
        "kernel": ("encrypt_fused2_kernel" if w.N == 16384 else "encrypt_fused_kernel") if w.N <= 16384
                  else "enc_block_forward_kernel + ntt_block_kernel (inside he_encrypt)",
        "bound": "alu", "achieved": achieved, "peak": peak,
        "unit": "T slots/s (integer-multiply / double-precision pipe)",
        "frac": achieved / peak,
        "traffic": ENCRYPT_DRAM_BYTES_PER_CT_N16384_L4 * T if (w.N == 16384 and w.L == 4) else None,
        "algorithmic_bytes": alg_bytes,
        "ms_per_launch": kern_ms, "launches_per_step": w.clients, "butterflies_per_launch": butterflies,
        "hbm_gbs_of_kernel": alg_bytes / (kern_ms * 1e-3) / 1e9,
        "hbm_frac_of_kernel": alg_bytes / (kern_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "ntt_standalone": {"gbs": ntt_gbs, "hbm_frac": ntt_gbs / peaks["hbm_gbs"], "ms": ntt_ms,
                           "batch_polys": B, "bytes_per_launch": pass_bytes,
                           "mul_pipe_frac": (B * transform_slots(w.primes, w.N, 0.5, 0.5)
                                             / (ntt_ms * 1e-3) / 1e12) / peak},
        "f64_limbs": sum(1 for q in w.primes if q < F64_PRIME_LIMIT),
        "peak_source": "multiply / double-precision pipe: SM count x 64 per clock (microbenchmark) x max SM clock; "
                       + peaks["source"] + " hbm_gbs for the HBM fractions",
    }

    cpu_ct = min(w.T, 768)
    cpu_p, cpu_dt, cores = oracle_sample(w, cpu_ct)
    cpu = {"value": cpu_p / cpu_dt, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": "first %d of %d ciphertext indices (%d params), all %d clients, %.1f s" % (cpu_ct, w.T, cpu_p, w.clients, cpu_dt)}

    line = {
        "metric": METRIC, "value": units / job_secs, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * job_secs / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u64 (limbs below 2^46: exact f64)", "data": "synthetic",
        "config": dict(config_dict(w, "every rank runs its own full batch; no collective on the path"),
                       format=args.format),
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"] or peaks["sm_max_mhz"],
                   "reasons": clocks["reasons"], "samples": clocks["samples"]},
        "e2e": {"value": e2e_units / e2e_job, "unit": UNIT, "h2d_bytes_per_step": 4 * w.P * w.clients,
                "d2h_bytes_per_step": 8 * w.P, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roofline, "cpu_baseline": cpu,
        "max_abs_err_vs_fedavg": err,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=["resnet18", "tiny", "resnet50-top10", "bert-1", "bert-10", "bert-100"],
                    default="resnet18")
    ap.add_argument("--format", choices=["coefficient", "transform"], default="coefficient",
                    help="ciphertext wire format of the timed round (the host-buffer leg always runs "
                         "he_round_host, which implements the coefficient format)")
    args = ap.parse_args()
    w = {"resnet18": si.RESNET18, "tiny": si.TINY, "resnet50-top10": si.RESNET50_TOP10,
         "bert-1": si.bert(0.01), "bert-10": si.bert(0.10), "bert-100": si.bert(1.0)}[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
