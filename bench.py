#!/usr/bin/env python
"""Throughput of the SBC hot path on B200: encode + decode-aggregate of a flat 2^30-element update.

One step = for each sparsity p in {1e-2, 1e-3, 1e-4}: sbc_encode of the
update (residual carried from step to step, one residual per p) and
sbc_decode_accumulate of the resulting stream into a dense fp32 tensor.
Prints one JSON line (rank 0).  ``--impl reference`` times the CPU oracle on
a bounded sample of the same workload instead.
"""
import argparse
import concurrent.futures
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

P_SWEEP = (1e-2, 1e-3, 1e-4)
FULL_N = 1 << 30
METRIC = "sbc_encode_decode_throughput"
UNIT = "Gelem/s"
WORKLOAD = ("flat 2^30-element fp32 update, Student-t(nu=3) x 1e-3, p sweep {1e-2,1e-3,1e-4}: "
            "per p one sbc_encode (residual carried across steps) + one sbc_decode_accumulate")
ALGO_BYTES_PER_ELEM = 12  # read update, read residual, write residual
DECODE_BYTES_PER_POSITION = 64  # one 32-byte sector of the dense tensor read and written back per decoded position


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--numel", type=int, default=FULL_N, help="elements per update (default 2^30)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-sample", type=int, default=1 << 23, help="elements per p for the oracle timing")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows:
            f = [x.strip() for x in row.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm),
                "reasons": sorted(reasons)}


# ------------------------------------------------------------------ reference arm (CPU oracle)

def time_oracle(sample_n: int, seed: int):
    """Oracle encode + decode on `sample_n` elements per p, one core; returns (Gelem/s, seconds, description)."""
    import numpy as np
    import oracle
    from paper_1805_08768_b200 import workloads
    upd = workloads.student_t_flat(sample_n, seed)
    elems, t0 = 0, time.perf_counter()
    for p in P_SWEEP:
        res = np.zeros(sample_n, dtype=np.float32)
        stream, _ = oracle.encode(upd, res, p)
        dense = np.zeros(sample_n, dtype=np.float32)
        oracle.decode_accumulate([stream], dense)
        elems += sample_n
    dt = time.perf_counter() - t0
    desc = (f"{sample_n} elements of the same Student-t(3) x 1e-3 distribution per p, "
            f"p in {list(P_SWEEP)}, encode + decode each, zero residual")
    return elems / dt / 1e9, dt, desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_1805_08768_b200 import workloads
    for _ in range(max(args.warmup, 0) and 1):
        time_oracle(1 << 16, 1)
    total_t, total_elems = 0.0, 0
    sample_n = max(1 << 12, min(args.cpu_sample, (1 << 24) // max(args.steps, 1)))
    desc = ""
    for step in range(args.steps):
        g, dt, desc = time_oracle(sample_n, workloads.seed_for(5, step))
        total_t += dt
        total_elems += 3 * sample_n
    value = total_elems / total_t / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": WORKLOAD, "timed_on": "host CPU, bounded sample"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": desc + f" ({args.steps} steps)"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ our arm

# DRAM traffic of one k_add_collect launch, from an ncu capture at 2^26 elements, p = 1e-2 (its
# summary is kept with the other profile summaries).  Reads grow in proportion to the element count.
# Writes do not quite: when the kernel ends, a part of what it stored is still in L2 as dirty lines
# (written back during the next kernel), and that part does not grow with the tensor.  So a launch
# over `numel` elements is modelled as
#     reads(2^26) * numel / 2^26  +  stored(numel) - l2_residue,
#     stored(numel) = stored(2^26) * numel / 2^26,   l2_residue = stored(2^26) - writes(2^26),
# where stored(2^26) = 4 B per element plus the candidate lists the capture's launch wrote.
# Valid only for the kernel source it was taken from: a different hash of the file reports null.
NCU_READ_BYTES_AT_2P26 = 537.07e6      # dram__bytes_read.sum
NCU_WRITE_BYTES_AT_2P26 = 229.18e6     # dram__bytes_write.sum (during the kernel)
# 4 B x 2^26 of residual + 8 B x (717245 + 699450) ordered candidate entries + ~1.4 MB of band entries
# + 0.26 MB of span records
NCU_STORED_BYTES_AT_2P26 = 268.435456e6 + 11.33356e6 + 1.4e6 + 0.262144e6
NCU_TRAFFIC_SOURCE_SHA256 = "623b599fadbfc6197856f6d23ed7ffa42ed7a04d2353a8c38a418ec21f92cb26"


def measured_traffic(numel: int):
    import hashlib
    path = os.path.join(ROOT, "paper_1805_08768_b200", "csrc", "sbc_front.cuh")
    try:
        with open(path, "rb") as fh:
            if hashlib.sha256(fh.read()).hexdigest() != NCU_TRAFFIC_SOURCE_SHA256:
                return None
    except OSError:
        return None
    scale = numel / float(1 << 26)
    residue = NCU_STORED_BYTES_AT_2P26 - NCU_WRITE_BYTES_AT_2P26
    traffic = NCU_READ_BYTES_AT_2P26 * scale + NCU_STORED_BYTES_AT_2P26 * scale - (residue if scale >= 1.0 else residue * scale)
    # what the kernel must move can only be exceeded, never undercut
    return traffic if traffic >= ALGO_BYTES_PER_ELEM * numel else None


def reduce_max_over_ranks(value: float, dist, device) -> float:
    """Max of a per-rank scalar over all ranks (the slowest rank sets the job's time)."""
    if dist is None:
        return value
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def load_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except (OSError, KeyError, ValueError):
        return 6650.0, "fallback (6.65 TB/s: MEASURED_PEAKS.json not found)"


def run_ours(args):
    import torch
    from paper_1805_08768_b200 import binding as sbc
    from paper_1805_08768_b200 import workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    n = args.numel
    steps, warmup = args.steps, max(args.warmup, 3)
    sbc.lib()  # fail here, loudly, if the CUDA library is missing

    # ---- inputs, resident in HBM before anything is timed (each rank = one independent client)
    update = workloads.student_t_flat_torch(n, workloads.seed_for(5, 0, rank), dev)
    residual = [torch.zeros(n, dtype=torch.float32, device=dev) for _ in P_SWEEP]
    dense = torch.zeros(n, dtype=torch.float32, device=dev)
    ws = torch.empty(max(sbc.sbc_workspace_bytes(n, p) for p in P_SWEEP), dtype=torch.uint8, device=dev)
    streams = [torch.empty(sbc.sbc_stream_bytes(n, p), dtype=torch.uint8, device=dev) for p in P_SWEEP]
    mus = [torch.empty(1, dtype=torch.float32, device=dev) for _ in P_SWEEP]
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    cur = torch.cuda.current_stream()

    def new_events(count):
        return [torch.cuda.Event(enable_timing=True) for _ in range(count)]

    def one_step(record):
        """One pass of the hot path; `record` collects (p index, encode marks, decode events)."""
        for i, p in enumerate(P_SWEEP):
            marks = new_events(sbc.MARK_COUNT)
            for m in marks:
                m.record(cur)  # torch creates the CUDA event on first record; the library re-records it
            sbc.sbc_encode_ex(update, residual[i], p, streams[i], mus[i], ws, marks)
            dense.zero_()                      # the caller's zero fill: outside the timed intervals
            d0, d1 = new_events(2)
            d0.record(cur)
            sbc.sbc_decode_accumulate([streams[i]], dense, status=status)
            d1.record(cur)
            if record is not None:
                record.append((i, marks, d0, d1))

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(warmup):
        one_step(None)
    sync_all()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    sync_all()
    rec = []
    wall0 = time.perf_counter()
    for _ in range(steps):
        one_step(rec)
    sync_all()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop() if rank == 0 else None

    enc_ms = [0.0] * len(P_SWEEP)
    dec_ms = [0.0] * len(P_SWEEP)
    stage_ms = [[0.0] * (sbc.MARK_COUNT - 1) for _ in P_SWEEP]
    collect_ms_all = []
    for i, marks, d0, d1 in rec:
        enc_ms[i] += marks[0].elapsed_time(marks[-1])
        dec_ms[i] += d0.elapsed_time(d1)
        for s in range(sbc.MARK_COUNT - 1):
            stage_ms[i][s] += marks[s].elapsed_time(marks[s + 1])
        collect_ms_all.append(marks[sbc.MARK_BOUNDS].elapsed_time(marks[sbc.MARK_COLLECT]))
    timed_ms = sum(enc_ms) + sum(dec_ms)
    timed_ms = reduce_max_over_ranks(timed_ms, dist, dev)
    if int(status.item()) != 0:
        raise RuntimeError(f"decoder reported status {int(status.item())}")

    # The decode once more, per p, with the L2 cleaned between the caller's zero fill and the timed
    # call (a read of 512 MB that nothing wrote): the timed decodes above start with the L2 full of
    # the zero fill's dirty lines, which are written back while the decode's own lines come in.
    # Reported beside decode_ms, not part of `value`.
    dec_clean_ms = [0.0] * len(P_SWEEP)
    clean_reps = 5
    for i, p in enumerate(P_SWEEP):
        for _ in range(clean_reps):
            dense.zero_()
            update[: 1 << 27].sum()
            d0, d1 = new_events(2)
            d0.record(cur)
            sbc.sbc_decode_accumulate([streams[i]], dense, status=status)
            d1.record(cur)
            torch.cuda.synchronize()
            dec_clean_ms[i] += d0.elapsed_time(d1) / clean_reps

    infos = [sbc.sbc_stream_info_get(s) for s in streams]
    diags = []
    for i, p in enumerate(P_SWEEP):  # one more untimed encode per p to read back which route it takes
        sbc.sbc_encode(update, residual[i], p, streams[i], mus[i], ws)
        d = sbc.sbc_encode_diag_get(ws)
        diags.append({"exact_route": int(d.exact_route), "candidates": [int(d.candidates[0]), int(d.candidates[1])],
                      "capacity": int(d.capacity)})
    ms_per_step = timed_ms / steps
    elems_per_step = len(P_SWEEP) * n * world
    value = elems_per_step / (ms_per_step * 1e-3) / 1e9

    # ---- roofline of the dominant kernel (the streaming accumulate + collect pass)
    peak, peak_src = load_peak()
    collect_ms = sum(collect_ms_all) / len(collect_ms_all)
    achieved = ALGO_BYTES_PER_ELEM * n / (collect_ms * 1e-3) / 1e9
    traffic = measured_traffic(n)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic,
                "traffic_over_algorithmic": (traffic / (ALGO_BYTES_PER_ELEM * n)) if traffic else None,
                "kernel": "k_add_collect", "launches_timed": len(collect_ms_all),
                "avg_ms": collect_ms, "peak_source": peak_src,
                "algorithmic_bytes_per_launch": ALGO_BYTES_PER_ELEM * n}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    per_p = []
    for i, p in enumerate(P_SWEEP):
        e, d = enc_ms[i] / steps, dec_ms[i] / steps
        per_p.append({
            "p": p, "k": int(infos[i].k), "b": int(infos[i].b), "nbits": int(infos[i].nbits),
            "bits_per_position": infos[i].nbits / max(infos[i].k, 1),
            "container_bytes": int(infos[i].total_bytes),
            "encode_ms": e, "decode_ms": d,
            "encode_gelem_s": n / (e * 1e-3) / 1e9,
            "encode_algorithmic_gbs": ALGO_BYTES_PER_ELEM * n / (e * 1e-3) / 1e9,
            "encode_frac_of_peak": ALGO_BYTES_PER_ELEM * n / (e * 1e-3) / 1e9 / peak,
            "decode_positions_per_s": infos[i].k / (d * 1e-3),
            # decode as the blueprint counts it: dense-equivalent rate, and bytes = one 32-byte sector read
            # and written per position plus the container read once
            "decode_dense_gelem_s": n / (d * 1e-3) / 1e9,
            "decode_gbs": (DECODE_BYTES_PER_POSITION * infos[i].k + infos[i].total_bytes) / (d * 1e-3) / 1e9,
            "decode_frac_of_peak": (DECODE_BYTES_PER_POSITION * infos[i].k + infos[i].total_bytes) / (d * 1e-3) / 1e9 / peak,
            "decode_ms_clean_l2": dec_clean_ms[i],
            "stage_ms": {name: stage_ms[i][s] / steps for s, name in enumerate(sbc.MARK_NAMES)},
            "route": diags[i],
        })

    # the metric's second half: achieved (algorithmic) HBM rate of the encode over the whole p sweep
    sweep_ms = sum(enc_ms) / steps
    sweep_gbs = ALGO_BYTES_PER_ELEM * n * len(P_SWEEP) / (sweep_ms * 1e-3) / 1e9
    encode_sweep = {"ms": sweep_ms, "algorithmic_gbs": sweep_gbs, "frac_of_measured_peak": sweep_gbs / peak,
                    "frac_of_nominal_8tbs": sweep_gbs / 8000.0,
                    "decode_ms": sum(dec_ms) / steps}

    # ---- end to end through the host-buffer entry points (pinned host memory, copies timed)
    e2e = run_e2e(args, torch, sbc, dev, update, ws, n, world)

    # ---- the oracle on this machine's host cores, bounded sample
    cpu = None
    if not args.no_cpu_baseline:
        g, dt, desc = time_oracle(min(args.cpu_sample, n), workloads.seed_for(5))
        cpu = {"value": g, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc,
               "seconds": dt, "host_cores_available": len(os.sched_getaffinity(0))}

    try:
        network_shapes = run_network_shapes(torch, sbc, workloads, dev, with_oracle=not args.no_cpu_baseline)
    except Exception as exc:  # context numbers only: never fail the headline for them
        network_shapes = {"error": repr(exc)}

    launches = steps * sum(sbc.sbc_encode_launches() + sbc.sbc_decode_launches(1) for _ in P_SWEEP)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "numel": n, "p": list(P_SWEEP),
                   "l2": "inputs (8 bytes x numel per encode) are far larger than the 126 MB L2",
                   "timed": "CUDA events around every sbc_encode and sbc_decode_accumulate; the caller's "
                            "zero fill of the dense tensor is outside the intervals",
                   "parallelism": f"{world} independent client replica(s), no collective"},
        "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches,
        "clocks": clocks, "encode_sweep": encode_sweep, "per_p": per_p, "network_shapes": network_shapes, "wall_s": wall,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def _timed(torch, fn, reps=10):
    """Mean device time of fn() in ms: 3 warm-ups, then `reps` calls between two CUDA events."""
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def _oracle_round(tensors, p):
    """The oracle over one round of a model's tensors (zero residual), one core: (seconds, streams)."""
    import numpy as np
    import oracle
    t0 = time.perf_counter()
    streams = []
    for u in tensors:
        stream, _ = oracle.encode(u, np.zeros(u.size, dtype=np.float32), p)
        streams.append(stream)
    return time.perf_counter() - t0, streams


def run_network_shapes(torch, sbc, workloads, dev, with_oracle=True):
    """The four small configurations next to the headline: per configuration the device time of
    the calls (CUDA events, 10 repetitions after 3 warm-ups) and, beside it, the oracle on the same
    tensors (one core, wall clock, run whole unless it says otherwise)."""
    import numpy as np
    import oracle
    out = {}

    # ---- config 1: one tensor of 2^20 elements, N(0, 1e-3), p = 0.01, encode + decode round trip
    n1, p1 = 1 << 20, 0.01
    upd = workloads.normal_flat(n1, 1e-3, workloads.seed_for(1))
    u = torch.from_numpy(upd).to(dev)
    r = torch.zeros(n1, dtype=torch.float32, device=dev)
    ws1 = torch.empty(sbc.sbc_workspace_bytes(n1, p1), dtype=torch.uint8, device=dev)
    out1 = torch.empty(sbc.sbc_stream_bytes(n1, p1), dtype=torch.uint8, device=dev)
    mu1 = torch.empty(1, dtype=torch.float32, device=dev)
    dense1 = torch.zeros(n1, dtype=torch.float32, device=dev)
    enc_ms = _timed(torch, lambda: sbc.sbc_encode(u, r, p1, out_stream=out1, out_mu=mu1, workspace=ws1), 20)
    dec_ms = _timed(torch, lambda: sbc.sbc_decode_accumulate([out1], dense1), 20)
    out["config1_flat_2p20_p1e-2"] = {"elements": n1, "encode_us": 1e3 * enc_ms, "decode_us": 1e3 * dec_ms,
                                      "round_trip_gelem_s": n1 / (enc_ms + dec_ms) / 1e6}
    if with_oracle:
        t0 = time.perf_counter()
        stream, _ = oracle.encode(upd, np.zeros(n1, dtype=np.float32), p1)
        t1 = time.perf_counter()
        oracle.decode_accumulate([stream], np.zeros(n1, dtype=np.float32))
        t2 = time.perf_counter()
        out["config1_flat_2p20_p1e-2"]["oracle"] = {"encode_s": t1 - t0, "decode_s": t2 - t1, "cores": 1,
                                                     "round_trip_gelem_s": n1 / (t2 - t0) / 1e9}

    # ---- configs 2, 3, 4: the network-shaped rounds (batched calls)
    for name, sizes, p, gen in (
            ("resnet50_shapes_p1e-3", [int(np.prod(s)) for _, s, _ in workloads.resnet50_shapes()], 1e-3,
             workloads.resnet50_update),
            ("word_lstm_shapes_p1e-2", [int(np.prod(s)) for _, s in workloads.word_lstm_shapes()], 1e-2,
             workloads.word_lstm_update),
            ("word_lstm_shapes_p1e-3", [int(np.prod(s)) for _, s in workloads.word_lstm_shapes()], 1e-3,
             workloads.word_lstm_update)):
        n_clients = 8
        ps = [p] * len(sizes)
        ws = torch.empty(sbc.sbc_workspace_bytes_batch(sizes, ps), dtype=torch.uint8, device=dev)
        # one message per client and tensor, from eight different seeded updates; every client has
        # its own residuals, outputs and marshalled descriptors, as eight clients on one GPU would
        clients, first_host = [], None
        for c in range(n_clients):
            host = gen(1 + c)
            if c == 0:
                first_host = host
            ups = [torch.from_numpy(x).to(dev) for x in host]
            res = [torch.zeros(n, dtype=torch.float32, device=dev) for n in sizes]
            outs = [torch.empty(sbc.sbc_stream_bytes(n, p), dtype=torch.uint8, device=dev) for n in sizes]
            mus = [torch.empty(1, dtype=torch.float32, device=dev) for _ in sizes]
            clients.append((sbc.EncodeBatch(ups, res, ps, outs, mus, ws), outs))
        dense = [torch.zeros(n, dtype=torch.float32, device=dev) for n in sizes]
        dws = torch.empty(sbc.sbc_decode_workspace_bytes_batch(len(sizes)), dtype=torch.uint8, device=dev)
        dec = sbc.DecodeBatch([[clients[c][1][t] for c in range(n_clients)] for t in range(len(sizes))], dense, dws)

        def encode_all():
            for enc, _ in clients:
                enc.run()

        # the same eight rounds, every client on a stream and with a workspace of its own: the clients
        # are independent, so their (latency-bound) kernel chains can overlap on the one GPU
        streams8 = [torch.cuda.Stream(device=dev) for _ in range(n_clients)]
        ws8 = [ws] + [torch.empty_like(ws) for _ in range(n_clients - 1)]
        conc = [sbc.EncodeBatch(enc.keep[0], enc.keep[1], ps, enc.keep[2], enc.keep[3], ws8[c])
                for c, (enc, _) in enumerate(clients)]

        def encode_all_concurrently():
            here = torch.cuda.current_stream()
            fork = torch.cuda.Event()
            fork.record(here)
            for c in range(n_clients):
                streams8[c].wait_event(fork)
                conc[c].run(stream=streams8[c])
                here.wait_stream(streams8[c])

        one_ms = _timed(torch, clients[0][0].run)
        all_ms = _timed(torch, encode_all, 5)
        conc_ms = _timed(torch, encode_all_concurrently, 5)
        dec_ms = _timed(torch, dec.run)
        total = sum(sizes)
        out[name] = {"tensors": len(sizes), "elements": total, "encode_batch_us": 1e3 * one_ms,
                     "encode_gelem_s": total / one_ms / 1e6,
                     "encode_algorithmic_gbs": ALGO_BYTES_PER_ELEM * total / one_ms / 1e6,
                     "encode_algorithmic_frac_of_peak": ALGO_BYTES_PER_ELEM * total / one_ms / 1e6 / load_peak()[0],
                     "encode_8_clients_us": 1e3 * all_ms,
                     "encode_8_clients_on_8_streams_us": 1e3 * conc_ms,
                     "decode_batch_8_clients_us": 1e3 * dec_ms,
                     "encode_8_clients_plus_decode_us": 1e3 * (all_ms + dec_ms)}
        if with_oracle and name != "word_lstm_shapes_p1e-3":   # (the LSTM shapes are timed against the oracle at one p)
            secs, streams = _oracle_round(first_host, p)
            t0 = time.perf_counter()
            for t, n in enumerate(sizes):    # the same message eight times stands in for eight clients' messages
                oracle.decode_accumulate([streams[t]] * n_clients, np.zeros(n, dtype=np.float32))
            dsecs = time.perf_counter() - t0
            out[name]["oracle"] = {"encode_round_s": secs, "decode_8_clients_s": dsecs, "cores": 1,
                                   "encode_gelem_s": total / secs / 1e9,
                                   "sample": "one client's round (of eight), zero residual; decode of eight messages per tensor"}
    return out


def run_e2e(args, torch, sbc, dev, update, ws, n, world):
    """Same step through sbc_encode_host / sbc_decode_accumulate_host with pinned host buffers."""
    if args.e2e_steps <= 0:
        return None
    try:
        upd_host = torch.empty(n, dtype=torch.float32, pin_memory=True)
        dense_host = torch.empty(n, dtype=torch.float32, pin_memory=True)
    except RuntimeError as exc:  # not enough lockable host memory
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                "note": f"pinned host allocation failed: {exc}"}
    upd_host.copy_(update)
    cap = max(sbc.sbc_stream_bytes(n, p) for p in P_SWEEP)
    stream_host = [torch.empty(cap, dtype=torch.uint8, pin_memory=True) for _ in P_SWEEP]
    stream_dev = torch.empty(cap, dtype=torch.uint8, device=dev)
    staging = torch.empty(cap + 64, dtype=torch.uint8, device=dev)
    upd_dev = torch.empty(n, dtype=torch.float32, device=dev)
    dense_dev = torch.empty(n, dtype=torch.float32, device=dev)
    residual = [torch.zeros(n, dtype=torch.float32, device=dev) for _ in P_SWEEP]
    h2d = d2h = 0
    # Two CUDA streams and a second host thread: while the aggregate of one p travels back to the
    # host, the update for the next p already travels to the device (the link is full duplex).
    enc_stream, dec_stream = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    pool = concurrent.futures.ThreadPoolExecutor(max_workers=1)

    def decode(i, nbytes):
        return sbc.sbc_decode_accumulate_host([stream_host[i]], [nbytes], dense_host, dense_dev, staging,
                                              stream=dec_stream)

    def settle(pending):
        if pending is not None and pending.result():
            raise RuntimeError(f"decode status {pending.result()}")

    pending = None

    def step():
        nonlocal h2d, d2h, pending
        for i, p in enumerate(P_SWEEP):
            nbytes, _ = sbc.sbc_encode_host(upd_host, upd_dev, residual[i], p, stream_host[i], stream_dev, ws,
                                            stream=enc_stream)
            settle(pending)                       # one decode in flight at a time: it owns dense_host
            pending = pool.submit(decode, i, nbytes)
            h2d += 4 * n + nbytes
            d2h += nbytes + 4 + 64 + 4 * n + 4

    step()  # warm-up
    settle(pending)
    pending = None
    torch.cuda.synchronize()
    # the containers this first step brought back to the host are those of the device-buffer call
    # on the same input (zero residual), byte for byte, and the last aggregate is the decoded message
    chk_res = torch.zeros(n, dtype=torch.float32, device=dev)
    for i, p in enumerate(P_SWEEP):
        chk_res.zero_()
        out, _ = sbc.sbc_encode(update, chk_res, p, workspace=ws)
        info = sbc.sbc_stream_info_get(out)
        if not torch.equal(out[: info.total_bytes].cpu(), stream_host[i][: info.total_bytes]):
            raise RuntimeError(f"host-buffer encode at p={p} differs from sbc_encode")
        if i == len(P_SWEEP) - 1:
            chk_res.zero_()
            sbc.sbc_decode_accumulate([out], chk_res)
            if not torch.equal(chk_res.cpu().view(torch.int32), dense_host.view(torch.int32)):
                raise RuntimeError("host-buffer decode differs from sbc_decode_accumulate")
    del chk_res
    h2d = d2h = 0
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        step()                                    # the last decode of a step overlaps the next step's first encode
    settle(pending)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    return {"value": len(P_SWEEP) * n * world / (dt / args.e2e_steps) / 1e9, "unit": UNIT,
            "h2d_bytes_per_step": h2d // args.e2e_steps, "d2h_bytes_per_step": d2h // args.e2e_steps,
            "ms_per_step": 1e3 * dt / args.e2e_steps, "steps": args.e2e_steps,
            "note": "host wall clock around synchronising host-buffer calls; update H2D, stream D2H, "
                    "stream H2D, dense aggregate D2H every step; every encode overlaps the decode "
                    "of the previous encode's message (two streams, two host threads)"}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
