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

The default line carries the ResNet-18-sized workload (``value``) and, under
``workloads``, the ResNet-50-sized top-10 % round and the BERT-sized round at
100 % encryption (streamed in chunks of ciphertext indices), each with its own
time, roofline block, host-buffer leg and clocks.

For N > 1 launch under ``torch.distributed.run``.  ``--shard index`` (default):
ONE round is cut over the ranks, rank r taking the contiguous ciphertext
indices [T r / N, T (r+1) / N) and the same share of the plaintext remainder,
with context, keys and mask replicated and no collective on the path
(``--gather`` adds the one all-gather of the decoded pieces, for when one
place needs the whole model); fixed total work, "scaling": "strong".
``--shard batch``: every rank runs its own full round ("weak").  ``--shard
client``: the clients are spread over the ranks, whose weighted sums meet in
one reduce-scatter (the layout of a server that receives different clients on
different GPUs).  The job time is the maximum over ranks in every mode.
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
# DRAM bytes (read + write) per ciphertext of the encrypt kernel, by (N, L), from ncu captures of
# the profile_case.py encrypt case (summaries under profiles/; traffic grows in proportion to the
# number of ciphertexts).  An entry is dropped (None is reported) when the kernel has changed
# since its counters were taken.
ENCRYPT_DRAM_BYTES_PER_CT = {(16384, 4): 372.248832e6 / 296,       # encrypt_fused2_kernel, 296 ciphertexts
                             (32768, 6): 478.248704e6 / 148}       # encrypt_cluster_kernel, 148 ciphertexts
SLOTS_PER_SM_CLK = 64.0
WIDE_COST = 2.5
INT_SLOTS_PER_BUTTERFLY = 6 * WIDE_COST + 4
F64_SLOTS_FORWARD, F64_SLOTS_INVERSE = 8.0, 9.0
F64_PRIME_LIMIT = 1 << 46
ENCODE_SLOTS_PER_BUTTERFLY = 10.0     # complex product (4 multiplies, 2 add/sub) and complex sum and difference


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
            "l2": ("inputs larger than L2 (%.1f GB of ciphertexts per step%s)"
                   % (w.clients * w.T * 2 * w.L * w.N * 8 / 1e9,
                      ", streamed in chunks of ciphertext indices" if w.clients * w.T * 2 * w.L * w.N * 8 > 40e9 else "")
                   if w.clients * w.T * 2 * w.L * w.N * 8 > 126e6 else
                   "the small case: %.0f MB of ciphertexts per step fit the L2 and are not flushed between steps"
                   % (w.clients * w.T * 2 * w.L * w.N * 8 / 1e6)),
            "note": note}


# --------------------------------------------------------------------------- GPU arm

class Job:
    """Process-wide state of one bench run."""

    def __init__(self, args):
        import torch
        import torch.distributed as dist
        self.torch, self.dist = torch, dist
        self.rank, self.world, self.local = dist_env()
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
        torch.cuda.set_device(self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
        self.peaks = read_peaks()
        self.n_sm = torch.cuda.get_device_properties(self.local).multi_processor_count
        self.args = args

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()


def measure(job, w, steps, warmup, with_cpu_baseline):
    """One workload: W warm-up rounds, K timed rounds, the dominant kernel's roofline, the
    host-buffer leg.  Returns the fields of a bench line for this workload (rank 0) or None."""
    import paper_2303_10837_b200 as he
    from paper_2303_10837_b200.sharding import even_edges, gather_pieces, shard_range, slot_edges, slot_range
    torch, args = job.torch, job.args
    rank, world = job.rank, job.world
    by_index = world > 1 and args.shard == "index"
    transform = args.format == "transform"

    # one-off steps (not part of a round): timed on the host around a device synchronisation
    one_off = {}

    def timed(name, fn):
        torch.cuda.synchronize()
        t_start = time.perf_counter()
        r = fn()
        torch.cuda.synchronize()
        one_off[name] = 1e3 * (time.perf_counter() - t_start)
        return r

    g = timed("ctx_create", lambda: he.he_ctx_create(w.N, list(w.primes), w.log2_delta))
    keys = timed("keygen", lambda: he.he_keygen(g, w.key_seed))
    alpha = si.client_weights(w)
    T, n = w.T, w.n
    # what this rank works on: everything (one GPU, or one batch per rank), or its range of one round
    if by_index:
        tb, te, sb, se = slot_range(T, n, w.k, rank, world)
        rb, re = shard_range(w.P - w.k, rank, world)
        batch_seed, enc_seed = 0, w.enc_seed
    else:
        tb, te, sb, se = 0, T, 0, w.k
        rb, re = 0, w.P - w.k
        batch_seed, enc_seed = rank, w.enc_seed + 1000 * rank
    Tr = te - tb
    xs_host = []
    for i in range(w.clients):
        rng = np.random.default_rng([w.seed, 1000 + i, batch_seed])
        x = rng.standard_normal(w.P, dtype=np.float32)
        x *= np.float32(w.std)
        xs_host.append(torch.from_numpy(x).pin_memory())
    xs = [x.cuda() for x in xs_host]
    mask, idx = None, None
    if w.k < w.P:
        scores = torch.from_numpy(si.sensitivity_scores(w)).cuda()
        # the first call of a process also loads the kernels and makes the mask memory pool
        first = timed("select_mask_first_call", lambda: he.he_select_mask(g, scores, w.k))
        del first                                   # the handle is released with the object
        mask = timed("select_mask", lambda: he.he_select_mask(g, scores, w.k))
        del scores
        idx = he.he_mask_indices(mask).long()
    # ciphertext indices are streamed in chunks when all clients' ciphertexts of this rank exceed 40 GB
    ct_bytes = 8 * 2 * w.L * w.N
    Tc = max(Tr, 1)
    if w.clients * Tr * ct_bytes > 40e9:
        Tc = max(job.n_sm, int(16e9 // (w.clients * ct_bytes)) // job.n_sm * job.n_sm)
    if transform and (Tc < Tr or by_index):
        raise SystemExit("bench: --format transform is wired to the whole, unchunked round only")
    cts = [torch.empty((Tc, 2, w.L, w.N), dtype=torch.int64, device="cuda") for _ in range(w.clients)]
    agg = torch.empty((Tc, 2, w.L - 1, w.N), dtype=torch.int64, device="cuda")
    z = torch.empty(Tr * n, dtype=torch.float64, device="cuda")
    out = torch.empty(w.P, dtype=torch.float64, device="cuda")
    he.he_ctx_reserve(g, min(Tr, Tc) * n)
    enc_events = []
    result = {}

    def step(record):
        sels, rests = [], []
        for i in range(w.clients):
            if by_index and mask is None:           # full encryption: the rank's slots are a slice of x
                if se > sb:
                    sel, rest = he.he_pack(g, None, xs[i][sb:se])
                else:                               # more ranks than ciphertexts: nothing for this one
                    sel, rest = torch.empty(0, dtype=torch.float32, device="cuda"), None
            else:
                sel, rest = he.he_pack(g, mask, xs[i])
                sel = sel[tb * n:te * n]
            sels.append(sel)
            rests.append(rest[rb:re] if rest is not None else None)
        for t0 in range(0, Tr, Tc):
            tc = min(Tc, Tr - t0)
            for i in range(w.clients):
                if record:
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                if transform:
                    he.he_encrypt_ntt(g, keys, sels[i], enc_seed, i, out=cts[i])
                else:
                    he.he_encrypt_range(g, keys, sels[i][t0 * n:(t0 + tc) * n], tb + t0, tc, enc_seed, i, cts[i][:tc])
                if record:
                    e1.record()
                    enc_events.append((e0, e1, tc))
            if transform:
                he.he_weighted_aggregate_ntt(g, cts, alpha, out=agg)
                he.he_decrypt_level_ntt(g, keys, agg, w.L - 1, out=z)
            else:
                he.he_weighted_aggregate(g, [c[:tc] for c in cts], alpha, out=agg[:tc])
                he.he_decrypt(g, keys, agg[:tc], out=z[t0 * n:(t0 + tc) * n])
        avg = he.he_plain_aggregate(g, rests, alpha) if (mask is not None and re > rb) else None
        if by_index:
            # the rank's part of the model: z[: se - sb] and avg; gathered only on request
            if args.gather:
                zf = gather_pieces(z[: se - sb], slot_edges(T, n, w.k, world), rank)
                af = gather_pieces(avg, even_edges(w.P - w.k, world), rank) if mask is not None and w.k < w.P else None
                he.he_unpack(g, mask, zf, af, w.P, out=out)
            result["z"], result["avg"] = z, avg
        else:
            he.he_unpack(g, mask, z, avg, w.P, out=out)

    for _ in range(warmup):
        step(False)
    job.barrier()
    sampler = ClockSampler(job.local)
    sampler.start()
    launches0 = he.he_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        step(True)
    ev1.record()
    job.barrier()
    launches = he.he_launch_count() - launches0
    secs = ev0.elapsed_time(ev1) * 1e-3
    # correctness of what was timed: plaintext FedAvg on every parameter this rank produced
    want = sum(float(a) * x.double() for a, x in zip(alpha, xs))
    if by_index and not args.gather:
        pos = torch.arange(sb, se, device="cuda") if idx is None else idx[sb:se]
        err = float((result["z"][: se - sb] - want[pos]).abs().max()) if se > sb else 0.0
        if result["avg"] is not None:
            comp = torch.ones(w.P, dtype=torch.bool, device="cuda")
            comp[idx] = False
            err = max(err, float((result["avg"] - want[comp][rb:re]).abs().max()))
    else:
        err = float((out - want).abs().max())
    if not err <= 1e-6 or he.he_ctx_status(g) != he.HE_OK:
        raise SystemExit("bench: aggregate differs from plaintext FedAvg by %g" % err)

    # Dominant kernel: the encryption.  Duration of one client's he_encrypt calls in the timed
    # region (CUDA events on the launching stream); where the library still runs the encoder as a
    # launch of its own inside he_encrypt, that launch, timed alone on the same inputs, is taken off.
    enc_ms = sum(a.elapsed_time(b) for a, b, _ in enc_events) / (steps * w.clients)
    sel0 = he.he_pack(g, mask, xs[0])[0][tb * n:te * n]
    probe = min(Tr, Tc)
    c0 = he.he_launch_count()
    he.he_encrypt_range(g, keys, sel0[: probe * n], tb, probe, enc_seed, 0, cts[0][:probe])
    launches_per_encrypt = he.he_launch_count() - c0
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 5
    encode_ms = 0.0
    if launches_per_encrypt > 1 and Tr:
        he.he_encode(g, sel0)
        e0.record()
        for _ in range(reps):
            he.he_encode(g, sel0)
        e1.record()
        torch.cuda.synchronize()
        encode_ms = e0.elapsed_time(e1) / reps
    kern_ms = max(enc_ms - encode_ms, 1e-6)

    # standalone transform: forward + inverse over a batch larger than L2
    # (1024 polynomials: 256 seeded ones, repeated on the device; 0.5 to 1.6 GB)
    B = 1024
    polys = torch.from_numpy(si.random_residues(7, (B // 4, w.L, w.N), w.primes).view(np.int64)).cuda().repeat(4, 1, 1)
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
    del polys
    clocks = sampler.stop()

    # end to end through the host entry point (pinned host buffers, copies inside the timed region)
    e2e = None
    del cts, agg
    torch.cuda.empty_cache()
    if not by_index or mask is None:
        if by_index:
            xh = [x[sb:se] for x in xs_host]             # the rank's slots are a slice of every update
            Pe = se - sb
        else:
            xh, Pe = xs_host, w.P
        host_out = torch.empty(max(Pe, 1), dtype=torch.float64).pin_memory()[:Pe]
        if Pe:
            he.he_round_host(g, keys, mask, xh, alpha, enc_seed, host_out)          # allocates its buffers
        job.barrier()                                   # every rank, also one without work
        e2e_steps = max(1, min(steps, 3))
        t0 = time.perf_counter()
        for _ in range(e2e_steps if Pe else 0):
            he.he_round_host(g, keys, mask, xh, alpha, enc_seed, host_out)
        torch.cuda.synchronize()
        e2e_secs = time.perf_counter() - t0
        if Pe:
            ref = want[sb:se] if by_index else want
            if not float((host_out.cuda() - ref).abs().max()) <= 1e-6:
                raise SystemExit("bench: host round differs from plaintext FedAvg")
            e2e = (float(Pe) * e2e_steps, e2e_secs, e2e_steps, 4 * Pe * w.clients, 8 * Pe)

    # whole job: units = parameters every rank produced, time = the slowest rank
    mine = float(w.P) if not by_index else float((se - sb) + (re - rb))
    units, job_secs = reduce_job(mine * steps, secs, world, "cuda")
    e2e_line = None
    if not by_index or mask is None:                # the same on every rank: every rank joins the reduction
        mine_e2e = e2e if e2e is not None else (0.0, 0.0, 0, 0, 0)
        eu, es = reduce_job(mine_e2e[0], mine_e2e[1], world, "cuda")
    if e2e is not None:
        e2e_line = {"value": eu / es, "unit": UNIT, "h2d_bytes_per_step": e2e[3], "d2h_bytes_per_step": e2e[4],
                    "steps": e2e[2]}
        if by_index:
            e2e_line["note"] = "per rank: he_round_host on the rank's slice of every update (bytes are per rank)"
    del xs, xs_host, out, z, mask, keys, g
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    # roofline of the dominant kernel (bound by the multiply / double-precision pipe)
    logN = w.N.bit_length() - 1
    per_launch = Tr                                          # ciphertexts of one client's he_encrypt calls
    butterflies = 3 * w.L * (w.N // 2) * logN * per_launch
    # coefficient format: one forward and two inverse transforms per limb; transform format: three forward
    slots_per_ct = transform_slots(w.primes, w.N, 3 if transform else 1, 0 if transform else 2)
    if launches_per_encrypt == 1:
        # the encoder runs inside the kernel: (n/2) log2 n complex butterflies of 10 double-precision operations
        slots_per_ct += (n // 2) * (n.bit_length() - 1) * ENCODE_SLOTS_PER_BUTTERFLY
    achieved = slots_per_ct * per_launch / (kern_ms * 1e-3) / 1e12
    # Everything else the method makes the kernel compute on the same pipe, per ciphertext:
    # Philox4x32-10 (ten rounds of two 32x32->64 products for each of the N/4 + N/2 + N/2 blocks behind
    # u, e0, e1), the two products with the public key per coefficient and limb, and the factor 1/N
    # (one more product per butterfly of the last stage of both inverse transforms).
    ints = sum(1 for q in w.primes if q >= F64_PRIME_LIMIT)
    f64s = w.L - ints
    per_product = ints * INT_SLOTS_PER_BUTTERFLY + f64s * 6.0
    extra_per_ct = 1.25 * w.N * 20 * WIDE_COST + (2 * w.N + w.N) * per_product
    achieved_all = (slots_per_ct + (0 if transform else extra_per_ct)) * per_launch / (kern_ms * 1e-3) / 1e12
    peak = job.n_sm * SLOTS_PER_SM_CLK * job.peaks["sm_max_mhz"] * 1e6 / 1e12
    alg_bytes = (4.0 + 32.0 * w.L) * n * per_launch          # read the slots, write the ciphertext
    if w.N <= 16384:
        kname = "encrypt_fused2_kernel" if w.N == 16384 else "encrypt_fused_kernel"
    elif launches_per_encrypt == 1:
        kname = "encrypt_cluster_kernel"                     # one limb per pair of thread blocks (N = 32768)
    else:
        kname = "the %d kernels of he_encrypt on this ring, timed as one call" % launches_per_encrypt
    roofline = {
        "kernel": kname,
        "bound": "alu", "achieved": achieved, "peak": peak,
        "unit": "T slots/s (integer-multiply / double-precision pipe)",
        "frac": achieved / peak,
        "frac_all_required_work": achieved_all / peak,
        "traffic": (ENCRYPT_DRAM_BYTES_PER_CT[(w.N, w.L)] * per_launch
                    if (w.N, w.L) in ENCRYPT_DRAM_BYTES_PER_CT and not transform else None),
        "algorithmic_bytes": alg_bytes,
        "ms_per_launch": kern_ms, "launches_per_step": w.clients, "kernels_per_he_encrypt": int(launches_per_encrypt),
        "butterflies_per_launch": butterflies,
        "hbm_gbs_of_kernel": alg_bytes / (kern_ms * 1e-3) / 1e9,
        "hbm_frac_of_kernel": alg_bytes / (kern_ms * 1e-3) / 1e9 / job.peaks["hbm_gbs"],
        "ntt_standalone": {"gbs": ntt_gbs, "hbm_frac": ntt_gbs / job.peaks["hbm_gbs"], "ms": ntt_ms,
                           "batch_polys": B, "bytes_per_launch": pass_bytes,
                           "mul_pipe_frac": (B * transform_slots(w.primes, w.N, 0.5, 0.5)
                                             / (ntt_ms * 1e-3) / 1e12) / peak},
        "f64_limbs": sum(1 for q in w.primes if q < F64_PRIME_LIMIT),
        "peak_source": "multiply / double-precision pipe: SM count x 64 per clock (microbenchmark) x max SM clock; "
                       + job.peaks["source"] + " hbm_gbs for the HBM fractions",
    }
    if by_index:
        note = ("one round cut over %d ranks by ciphertext index (rank r: [T r / N, T (r+1) / N) and the same share of "
                "the plaintext remainder); no collective on the path%s" % (world, "; decoded pieces all-gathered" if args.gather else ""))
    elif world > 1:
        note = "every rank runs its own full batch; no collective on the path"
    else:
        note = "one GPU"
    fields = {
        "value": units / job_secs, "unit": UNIT, "ms_per_step": 1e3 * job_secs / steps, "steps": steps, "warmup": warmup,
        "config": dict(config_dict(w, note), format=args.format),
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"] or job.peaks["sm_max_mhz"],
                   "reasons": clocks["reasons"], "samples": clocks["samples"]},
        "e2e": e2e_line,
        "gpu_launches": int(launches),
        "roofline": roofline,
        "max_abs_err_vs_fedavg": err,
        # encrypted parameters / time of one client's he_encrypt calls (this rank's share when the round is cut)
        "param_encryptions_per_s": float(se - sb) / (enc_ms * 1e-3) if enc_ms > 0 else None,
        # not part of a round: once per task (context, keys) and once per mask (first round)
        "one_off_ms": {k_: round(v_, 3) for k_, v_ in one_off.items()},
    }
    if with_cpu_baseline:
        cpu_ct = min(w.T, 768)
        cpu_p, cpu_dt, cores = oracle_sample(w, cpu_ct)
        fields["cpu_baseline"] = {"value": cpu_p / cpu_dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                  "sample": "first %d of %d ciphertext indices (%d params), all %d clients, %.1f s"
                                            % (cpu_ct, w.T, cpu_p, w.clients, cpu_dt)}
    return fields


def measure_client_layout(job, w, steps, warmup):
    """The round with the clients spread over the ranks (`--shard client`): rank r encrypts the
    clients [C r / N, C (r+1) / N) on every ciphertext index and forms their weighted sum on all
    limbs; one reduce-scatter of 64-bit words sums over the clients and leaves rank r the
    ciphertext indices [T r / N, T (r+1) / N), which it rescales and decrypts.  The one layout with
    an exchange step on the path; wired to full encryption without chunked streaming."""
    import paper_2303_10837_b200 as he
    from paper_2303_10837_b200.sharding import scatter_sum, shard_range, slot_range
    torch = job.torch
    rank, world = job.rank, job.world
    if w.k < w.P:
        raise SystemExit("bench: --shard client is wired to full encryption")
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    alpha = si.client_weights(w)
    T, n = w.T, w.n
    cb, ce = shard_range(w.clients, rank, world)
    tb, te, sb, se = slot_range(T, n, w.k, rank, world)
    ct_bytes = 8 * 2 * w.L * w.N
    if (ce - cb + 2) * T * ct_bytes > 100e9:
        raise SystemExit("bench: --shard client keeps all ciphertexts of a rank's clients resident; this workload needs more ranks")
    xs = []
    for i in range(w.clients):
        rng = np.random.default_rng([w.seed, 1000 + i, 0])
        x = rng.standard_normal(w.P, dtype=np.float32)
        x *= np.float32(w.std)
        xs.append(torch.from_numpy(x).cuda())
    cts = [torch.empty((T, 2, w.L, w.N), dtype=torch.int64, device="cuda") for _ in range(cb, ce)]
    partial = torch.zeros((T, 2, w.L, w.N), dtype=torch.int64, device="cuda")
    agg = torch.empty((te - tb, 2, w.L - 1, w.N), dtype=torch.int64, device="cuda")
    z = torch.empty((te - tb) * n, dtype=torch.float64, device="cuda")
    he.he_ctx_reserve(g, T * n)

    def step():
        for j, i in enumerate(range(cb, ce)):
            sel, _ = he.he_pack(g, None, xs[i])
            he.he_encrypt(g, keys, sel, w.enc_seed, i, out=cts[j])
        if ce > cb:
            he.he_weighted_partial(g, cts, alpha[cb:ce], out=partial)
        mine = scatter_sum(partial, rank, world)
        if te > tb:
            he.he_rescale_partial_sum(g, mine, world, out=agg)
            he.he_decrypt(g, keys, agg, out=z)

    for _ in range(warmup):
        step()
    job.barrier()
    sampler = ClockSampler(job.local)
    sampler.start()
    launches0 = he.he_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    job.barrier()
    launches = he.he_launch_count() - launches0
    secs = ev0.elapsed_time(ev1) * 1e-3
    clocks = sampler.stop()
    want = sum(float(a) * x.double() for a, x in zip(alpha, xs))
    err = float((z[: se - sb] - want[sb:se]).abs().max()) if se > sb else 0.0
    if not err <= 1e-6 or he.he_ctx_status(g) != he.HE_OK:
        raise SystemExit("bench: aggregate differs from plaintext FedAvg by %g" % err)
    units, job_secs = reduce_job(float(se - sb) * steps, secs, world, "cuda")
    if rank != 0:
        return None
    note = ("clients spread over %d ranks (rank r: clients [C r / N, C (r+1) / N)); one reduce-scatter of the "
            "clients' weighted sums (%.1f MB of 64-bit words per rank and step), then every rank rescales and decrypts "
            "its ciphertext indices" % (world, T * ct_bytes / 1e6))
    return {"value": units / job_secs, "unit": UNIT, "ms_per_step": 1e3 * job_secs / steps, "steps": steps,
            "warmup": warmup, "config": dict(config_dict(w, note), format="coefficient"),
            "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"] or job.peaks["sm_max_mhz"],
                       "reasons": clocks["reasons"], "samples": clocks["samples"]},
            "e2e": None, "gpu_launches": int(launches), "roofline": None, "max_abs_err_vs_fedavg": err}


def run_ours(args, w, extras):
    job = Job(args)
    if args.shard == "client":
        main = measure_client_layout(job, w, args.steps, args.warmup)
        if job.rank == 0:
            line = {"metric": METRIC, "n_gpus": job.world, "higher_is_better": True, "scaling": "strong",
                    "vs_baseline": None, "dtype": "u64 (limbs below 2^46: exact f64)", "data": "synthetic"}
            line.update(main)
            print(json.dumps(line), flush=True)
        if job.world > 1:
            job.dist.destroy_process_group()
        return
    main = measure(job, w, args.steps, args.warmup, with_cpu_baseline=(job.world == 1))
    others = {}
    for name, ew in extras:
        # the further workloads take at most three timed rounds each (a BERT-sized round is 0.4 s)
        f = measure(job, ew, max(1, min(args.steps, 3)), max(3, min(args.warmup, 3)), with_cpu_baseline=False)
        if f is not None:
            others[name] = f
    if job.rank == 0:
        by_index = job.world > 1 and args.shard == "index"
        line = {"metric": METRIC, "n_gpus": job.world, "higher_is_better": True,
                "scaling": "strong" if by_index else "weak", "vs_baseline": None,
                "dtype": "u64 (limbs below 2^46: exact f64)", "data": "synthetic"}
        line.update(main)
        if others:
            line["workloads"] = others
        print(json.dumps(line), flush=True)
    if job.world > 1:
        job.dist.destroy_process_group()


WORKLOADS = {"resnet18": lambda: si.RESNET18, "tiny": lambda: si.TINY, "resnet50-top10": lambda: si.RESNET50_TOP10,
             "bert-1": lambda: si.bert(0.01), "bert-10": lambda: si.bert(0.10), "bert-100": lambda: si.bert(1.0)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default="resnet18")
    ap.add_argument("--also", default=None,
                    help="comma-separated further workloads reported under `workloads` (default: resnet50-top10,bert-100 "
                         "on one GPU when --workload is left at its default; 'none' for none)")
    ap.add_argument("--shard", choices=["index", "batch", "client"], default="index",
                    help="N > 1: cut one round over the ranks by ciphertext index (strong scaling), run one full "
                         "batch per rank (weak scaling), or spread the clients over the ranks with one "
                         "reduce-scatter of their weighted sums (client; also runs on one GPU)")
    ap.add_argument("--gather", action="store_true",
                    help="with --shard index: all-gather the decoded pieces so that every rank holds the whole model")
    ap.add_argument("--format", choices=["coefficient", "transform"], default="coefficient",
                    help="ciphertext wire format of the timed round (the host-buffer leg always runs "
                         "he_round_host, which implements the coefficient format)")
    args = ap.parse_args()
    w = WORKLOADS[args.workload]()
    if args.impl == "reference":
        run_reference(args, w)
        return
    _, world, _ = dist_env()
    if args.also is None:
        also = ["resnet50-top10", "bert-100"] if (world == 1 and args.workload == "resnet18" and args.format == "coefficient") else []
    else:
        also = [a for a in args.also.split(",") if a and a != "none"]
    run_ours(args, w, [(a, WORKLOADS[a]()) for a in also])


if __name__ == "__main__":
    main()
