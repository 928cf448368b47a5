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

# DRAM traffic of one k_add_collect launch from an ncu capture at 2^26 elements (its summary
# is kept with the other profile summaries): (536.94 + 226.60) MB at 2^26 elements, p = 1e-2.
# Traffic is proportional to the element count, so it is scaled by numel / 2^26.  Valid only for
# the kernel source it was taken from: a different hash of the file reports null.
NCU_TRAFFIC_BYTES_AT_2P26 = 763.54e6
NCU_TRAFFIC_SOURCE_SHA256 = "7fde50810e202a03e25da00d8bce1e859be4aabb3c48e116afdef7a99eb21cda"


def measured_traffic(numel: int):
    import hashlib
    path = os.path.join(ROOT, "paper_1805_08768_b200", "csrc", "sbc_front.cuh")
    try:
        with open(path, "rb") as fh:
            if hashlib.sha256(fh.read()).hexdigest() != NCU_TRAFFIC_SOURCE_SHA256:
                return None
    except OSError:
        return None
    return NCU_TRAFFIC_BYTES_AT_2P26 * numel / float(1 << 26)


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
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


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
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": measured_traffic(n), "kernel": "k_add_collect", "launches_timed": len(collect_ms_all),
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
        network_shapes = run_network_shapes(torch, sbc, workloads, dev)
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


def run_network_shapes(torch, sbc, workloads, dev):
    """Batched encode (one round) and 8-client batched decode on the network-shaped workloads:
    context numbers next to the headline, timed with CUDA events over 10 repetitions."""
    import numpy as np
    out = {}
    for name, sizes, p, gen in (
            ("resnet50_shapes_p1e-3", [int(np.prod(s)) for _, s, _ in workloads.resnet50_shapes()], 1e-3,
             workloads.resnet50_update),
            ("word_lstm_shapes_p1e-2", [int(np.prod(s)) for _, s in workloads.word_lstm_shapes()], 1e-2,
             workloads.word_lstm_update)):
        n_clients = 8
        res = [torch.zeros(n, dtype=torch.float32, device=dev) for n in sizes]
        mus = [torch.empty(1, dtype=torch.float32, device=dev) for _ in sizes]
        ws = torch.empty(sbc.sbc_workspace_bytes_batch(sizes, [p] * len(sizes)), dtype=torch.uint8, device=dev)
        # one message per client and tensor, from eight different seeded updates (zero residual each)
        client_outs = []
        for c in range(n_clients):
            ups = [torch.from_numpy(u).to(dev) for u in gen(1 + c)]
            for r in res:
                r.zero_()
            outs = [torch.empty(sbc.sbc_stream_bytes(n, p), dtype=torch.uint8, device=dev) for n in sizes]
            sbc.EncodeBatch(ups, res, [p] * len(sizes), outs, mus, ws).run()
            torch.cuda.synchronize()
            client_outs.append(outs)
        enc = sbc.EncodeBatch(ups, res, [p] * len(sizes), client_outs[-1], mus, ws)  # timed: the last client's round
        dense = [torch.zeros(n, dtype=torch.float32, device=dev) for n in sizes]
        dws = torch.empty(sbc.sbc_decode_workspace_bytes_batch(len(sizes)), dtype=torch.uint8, device=dev)
        dec = sbc.DecodeBatch([[client_outs[c][t] for c in range(n_clients)] for t in range(len(sizes))], dense, dws)

        def timed(fn, reps=10):
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

        enc_ms, dec_ms = timed(enc.run), timed(dec.run)
        total = sum(sizes)
        out[name] = {"tensors": len(sizes), "elements": total, "encode_batch_us": 1e3 * enc_ms,
                     "encode_gelem_s": total / enc_ms / 1e6,
                     "encode_algorithmic_gbs": ALGO_BYTES_PER_ELEM * total / enc_ms / 1e6,
                     "decode_batch_8_clients_us": 1e3 * dec_ms}
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
