#!/usr/bin/env python
"""Benchmark of the exponent-reuse codec hot path on B200.

One *step* = one pass of the whole path over one iterate of the synthetic weight trajectory:
for every layer, sender-side encode, the device-to-device transport that stands where the
Allgather would be, and receiver-side decode -- layer-pipelined on two streams.

Workload at one GPU: the full OLMoE-1B-7B expert stack (16 layers x 64 experts x 3 matrices,
bf16, 6.44 G values = 12.9 GB), 16 simulated shards per matrix, block size 512, with the
clustered update model (a fraction f = 0.22 of 512-aligned segments receives an Adam-like
update each iteration; the rest is bit-identical), which reproduces the block change rate the
paper reports for OLMoE expert-FFN shards.  Two consecutive iterates are kept on the device and
the steps alternate between them (the set of changed exponents between A and B is the same in
both directions), so every step is a real encode against a cache left by the previous one and
the K timed steps run back to back.

Prints ONE JSON line (rank 0).  ``--impl reference`` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "encode/decode GB/s of weights"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# Measured DRAM traffic per value of the headline encode launch (dram__bytes_read.sum + dram__bytes_write.sum of
# one ncu capture, divided by the values of the launch; traffic grows in proportion to the values).  The figure
# lives in a small data file beside the ncu summaries, together with a digest of the kernel sources it was
# captured with; when the sources have changed since, the bench line says traffic: null and why.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")
CSRC_DIR = os.path.join(ROOT, "paper_2609_04609_b200", "csrc")


def csrc_digest() -> str:
    """sha256 over the kernel sources (names and contents, sorted by name)."""
    import hashlib

    h = hashlib.sha256()
    for name in sorted(os.listdir(CSRC_DIR)):
        h.update(name.encode())
        with open(os.path.join(CSRC_DIR, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_traffic(key: str, n_values: int):
    """(bytes per launch or None, note) for the capture stored under `key`."""
    try:
        entry = json.load(open(TRAFFIC_FILE))[key]
    except Exception:
        return None, "no ncu capture on record for this workload"
    if entry.get("csrc_sha256") != csrc_digest():
        return None, "kernel sources changed since the ncu capture on record; re-capture to fill this in"
    return float(entry["dram_bytes_per_value"]) * n_values, f"ncu capture on record ({entry.get('captured', '')})"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=16, help="layers of the expert stack (16 = full model)")
    ap.add_argument("--experts", type=int, default=64)
    ap.add_argument("--shards", type=int, default=16)
    ap.add_argument("--block", type=int, default=512)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp32", "fp16"])
    ap.add_argument("--update", default="clustered", choices=["clustered", "adam", "inject"])
    ap.add_argument("--inject", type=float, default=0.01, help="exponent change rate of the 'inject' update model")
    ap.add_argument("--inject-seg", type=int, default=0,
                    help="'inject' update model: 0 = every value changes independently; n = whole n-aligned segments change")
    ap.add_argument("--shapes", default="olmoe", choices=["olmoe", "mixed"],
                    help="olmoe: 64 experts x 3 matrices per layer; mixed: 256 fine-grained experts (2048x512, "
                         "2048x512, 512x2048) plus dense tensors of 4 KB ... 256 MB (the mixed-shape sweep)")
    ap.add_argument("--detect", default="compare", choices=["compare", "hash"],
                    help="sender-side change detection: exact comparison with an exponent cache, or a 128-bit "
                         "hash per block (ciera_encode_hashed)")
    ap.add_argument("--entropy", action="store_true",
                    help="rANS-code the changed exponents before the transport and restore them after it")
    ap.add_argument("--f", type=float, default=0.22, help="fraction of segments updated (clustered model)")
    ap.add_argument("--schedule", default="pipelined", choices=["pipelined", "serial"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-regimes", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the one-layer runs of the other configurations (config 2 worst case, fp32, mixed shapes, "
                         "small blocks, fp16, hashed sender, entropy stage)")
    ap.add_argument("--cpu-sample-units", type=int, default=3072, help="units per layer given to the CPU oracle")
    ap.add_argument("--cpu-sample-layers", type=int, default=4, help="layers given to the CPU oracle")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------------- ranks


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Slowest rank's time: every rank gets the maximum (needs an initialised process group when world > 1)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def host_memory_allows(need_bytes: int, world: int, device=None) -> bool:
    """True on every rank iff on every rank `need_bytes` is at most 60 % of the free host memory."""
    import psutil

    ok = 1.0 if need_bytes <= 0.6 * psutil.virtual_memory().available else 0.0
    if world > 1:
        import torch
        import torch.distributed as dist

        t = torch.tensor([ok], dtype=torch.float64, device=device if device is not None else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MIN)
        ok = float(t.item())
    return ok > 0.5


def whole_job_gbps(world: int, bytes_per_rank: int, ms_per_step: float) -> float:
    """Weak scaling: every rank processes its own stack; the job's throughput is the sum."""
    return world * bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def rank_seed(rank: int) -> int:
    """Seed base of a rank's synthetic stack (config id 3; ranks get different weights)."""
    return 1234 + 3 + 1000 * rank


# --------------------------------------------------------------------------------- clocks


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs
    (read-only queries)."""

    def __init__(self, index: int, uuid: str = "", period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if uuid else b"")
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                except Exception:
                    pass
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w": float(np.median(self.power)) if self.power else None}


# --------------------------------------------------------------------------------- workload


def build_stack(args, device, seed_base):
    """Layers of the expert stack with two consecutive iterates W_a, W_b per layer on the device."""
    import torch

    from paper_2609_04609_b200 import runtime
    from paper_2609_04609_b200 import workloads as wl

    shapes = layer_numels(args)
    layers, wa, wb = [], [], []
    for l in range(args.layers):
        codec = runtime.LayerCodec.from_tensors(shapes, args.shards, args.dtype, args.block, device)
        n = codec.weights_bytes // wl.VALUE_BYTES[args.dtype]
        gen = wl.make_generator(seed_base + l, device)
        w = wl.init_weights(n, args.dtype, gen)
        if args.update == "clustered":
            step = lambda x: wl.step_clustered(x, gen, f=args.f, seg=512)
        elif args.update == "adam":
            step = lambda x: wl.step_adam_like(x, gen)
        else:
            step = lambda x: wl.inject_exponent_changes(x, gen, args.inject, args.inject_seg)
        for _ in range(4):  # iterations 1..4 of the trajectory
            w = step(w)
        w5 = step(w)  # iteration 5
        layers.append(codec)
        wa.append(w.view(torch.uint8))
        wb.append(w5.view(torch.uint8))
        codec.init_caches(wa[-1])
        if args.detect == "hash":
            codec.init_hash_cache(wa[-1])
    torch.cuda.synchronize()
    return layers, wa, wb


def layer_numels(args):
    from paper_2609_04609_b200 import workloads as wl

    if args.shapes == "mixed":
        return [r * c for r, c in wl.fine_grained_layer_shapes(256)] + wl.dense_tensor_sizes()
    return [r * c for r, c in wl.olmoe_layer_shapes(args.experts)]


def selection_report(args, ciera, codec, enc_ms, dec_ms, alpha=20e-6, beta=8e9):
    """Every unit of one layer as a shard of the selection rule.  q_i comes from the last encode,
    T_cmp and T_decmp are the layer's measured kernel times shared out by size (the sender side is
    taken as overlapped), Comm(S) = alpha + (W - 1) S / beta with synthetic link parameters
    (W = the simulated shard count), and the budget is half of what caching every unit would take."""
    n = codec.units["n_values"].astype(np.int64)
    changed = codec.changed_blocks.cpu().numpy().astype(np.int64)
    blocks = np.maximum(-(-n // args.block), 1)
    total = max(int(n.sum()), 1)
    code = ciera.DTYPE_CODES[args.dtype]
    shards = [dict(n_values=int(ni), dtype=code, block=args.block, q=float(min(ci / bi, 1.0)), world_size=args.shards,
                   alpha=alpha, beta=beta, t_cmp=enc_ms * 1e-3 * ni / total, t_decmp=dec_ms * 1e-3 * ni / total,
                   overlapped=True) for ni, ci, bi in zip(n, changed, blocks)]
    everything = ciera.select_shards(shards, 1 << 62, True)
    budget = sum(everything["footprints"]) // 2
    got = ciera.select_shards(shards, budget, True)
    gains = np.array(got["gains"])
    sel = np.array(got["selected"], bool)
    return {
        "rule": "g_i > 0, ranked by g_i / M_i, greedy prefix under the budget (ciera_select_shards)",
        "comm_model": {"alpha_s": alpha, "beta_Bps": beta, "world_size": args.shards, "kind": "synthetic"},
        "units": int(n.size), "positive_gain": int((gains > 0).sum()), "selected": int(sel.sum()),
        "budget_bytes": int(budget), "used_bytes": int(got["used"]),
        "gain_ms_selected": float(gains[sel].sum() * 1e3), "gain_ms_all_positive": float(gains[gains > 0].sum() * 1e3),
    }


def algorithmic_bytes(n_values, q, dtype, block, detect="compare"):
    """HBM bytes per launch the method needs: (encode, transport, decode).  q = share of the
    exponent bytes that travel (changed blocks); the bitmap is one bit per block.  The hashed sender
    reads no exponent cache and writes none; it reads 16 bytes of HashCache per block and writes them back
    for the changed ones."""
    vb, smb = (2, 1) if dtype == "bf16" else (4, 3)
    bm = 1.0 / (8 * block)
    if dtype == "fp16":
        # packed on the wire (11 and 5 bits per value), one byte per value in the caches
        sm, ex = 11 / 8, 5 / 8
        enc = n_values * (2 + 1 + sm + bm + q * (ex + 1))
        tra = 2 * n_values * (sm + bm + q * ex)
        dec = n_values * (sm + bm + (1 - q) + q * ex + 2 + q)
        return enc, tra, dec
    if detect == "hash":
        enc = n_values * (vb + smb + bm + q + 16.0 * (1 + q) / block)
    else:
        enc = n_values * (vb + 1 + smb + bm + 2 * q)
    tra = 2 * n_values * (smb + bm + q)
    dec = n_values * (smb + bm + (1 - q) + q + vb + q)
    return enc, tra, dec


def oracle_roundtrip_units(units, w_prev, w_cur, dtype_code, block, vb, threads):
    """CPU oracle (as it stands) on a list of units: cache init from w_prev, encode + decode of
    w_cur.  Returns seconds of wall time with ``threads`` host threads."""
    from concurrent.futures import ThreadPoolExecutor

    from oracle import ciera_oracle as ora

    ora.build()
    wdt = np.uint32 if dtype_code == 1 else np.uint16
    prev = w_prev.view(wdt)
    cur = w_cur.view(wdt)
    jobs = []
    for u in units:
        lo, n = int(u["weights_off"]) // vb, int(u["n_values"])
        jobs.append((prev[lo : lo + n], cur[lo : lo + n]))
    caches = [ora.cache_init(p, p.size, dtype_code) for p, _ in jobs]
    caches_r = [c.copy() for c in caches]

    def work(i):
        m, wb, pb, cb = ora.encode(jobs[i][1], caches[i], dtype_code, block)
        out = ora.decode(m, caches_r[i], dtype_code, block)
        return np.array_equal(out, jobs[i][1])

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        ok = list(ex.map(work, range(len(jobs))))
    dt = time.perf_counter() - t0
    assert all(ok), "oracle round trip failed"
    return dt, sum(j[1].size for j in jobs)


# --------------------------------------------------------------------------------- reference arm


def run_reference(args):
    """Times the CPU oracle on the host cores, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch

    from paper_2609_04609_b200 import workloads as wl
    from oracle import ciera_oracle as ora

    ora.build()
    code = {"bf16": 0, "fp32": 1, "fp16": 2}[args.dtype]
    vb = wl.VALUE_BYTES[args.dtype]
    shapes = layer_numels(args)
    n_units = min(args.cpu_sample_units, len(shapes) * args.shards)
    units, wbytes, _, _ = wl.layout_units(shapes, args.shards, vb, lambda n: ora.message_capacity(n, code, args.block))
    units = units[:n_units]
    n = int(units[-1]["weights_off"]) // vb + int(units[-1]["n_values"])
    gen = wl.make_generator(1234 + 3)
    w = wl.init_weights(n, args.dtype, gen)
    if args.update == "clustered":
        w1 = wl.step_clustered(w, gen, f=args.f, seg=512)
    elif args.update == "adam":
        w1 = wl.step_adam_like(w, gen)
    else:
        w1 = wl.inject_exponent_changes(w, gen, args.inject, args.inject_seg)
    a = wl.as_bits(w).view(np.uint8)
    b = wl.as_bits(w1).view(np.uint8)
    threads = os.cpu_count() or 1
    times = []
    nvals = 0
    for i in range(args.warmup + args.steps):
        prev, cur = (a, b) if i % 2 == 0 else (b, a)
        dt, nvals = oracle_roundtrip_units(units, prev, cur, code, args.block, vb, threads)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    gbps = nvals * vb / (ms * 1e-3) / 1e9
    total_units = len(shapes) * args.shards * args.layers
    sample = f"{n_units} of {total_units} units ({nvals} values) per step"
    config = workload_config(args)
    config["workload"] += (f" -- each step of this arm is a sample of {n_units} of the {total_units} units; ms_per_step is "
                           f"the time of that sample, value (GB/s of weights) is what compares with the other arm")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbps, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": config,
        "cpu_baseline": {"value": gbps, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbps, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(args):
    full = args.layers == 16 and args.experts == 64 and args.shapes == "olmoe"
    upd = f"update model {args.update}" + (f" f={args.f}" if args.update == "clustered" else "") + (
        f" c={args.inject}" + (f" in segments of {args.inject_seg}" if args.inject_seg else "") if args.update == "inject" else "")
    if args.shapes == "mixed":
        what = (f"mixed-shape sweep (config 5), {args.layers} x [256 fine-grained experts x (2048x512, 2048x512, "
                f"512x2048) + dense tensors 4 KB..256 MB] {args.dtype}")
    else:
        name = "config3: full OLMoE-1B-7B expert stack" if full else "reduced OLMoE expert stack"
        what = (f"{name}, {args.layers} layers x {args.experts} experts x 3 matrices (2048x1024, 2048x1024, "
                f"1024x2048) {args.dtype}")
    return {
        "workload": f"{what}, {args.shards} simulated shards per matrix, block {args.block}, {upd}",
        "l2": "inputs larger than L2 (no flush needed)",
        "schedule": args.schedule,
        "round_trip": "encode + device-to-device transport + decode",
        "change_detection": "exact comparison with a sender-side exponent cache" if args.detect == "compare"
                            else "128-bit hash per block (HashCache), the persistent kernel in its HashCache form",
    }


def verify_stack(args, ciera, layers, last_w, prev_w, n_layer_picks, n_unit_picks, with_oracle=True):
    """After a finished step from `prev_w` to `last_w`: the reconstructed weights equal the input everywhere and
    the two caches agree (device-side comparison), and, for sampled units, message, length, changed-block count
    and cache equal the CPU oracle's.  Returns (all of it held, number of units the oracle checked)."""
    import torch

    vb = 4 if args.dtype == "fp32" else 2

    def same_weights(c, w):
        """Exact comparison over the units' own bytes (alignment gaps between units carry nothing)."""
        if int(c.units["n_values"].sum()) * vb == w.numel():
            return torch.equal(c.weights_out[: w.numel()], w)
        keep = np.zeros(w.numel(), dtype=bool)
        for u in c.units:
            keep[int(u["weights_off"]) : int(u["weights_off"]) + int(u["n_values"]) * vb] = True
        keep = torch.from_numpy(keep).to(w.device)
        return torch.equal(c.weights_out[: w.numel()][keep], w[keep])

    verified = all(same_weights(c, w) for c, w in zip(layers, last_w))
    if args.detect == "compare":
        verified = verified and all(torch.equal(c.sender_cache, c.receiver_cache) for c in layers)
    sampled = 0
    if with_oracle:
        from oracle import ciera_oracle as ora

        ora.build()
        code = ciera.DTYPE_CODES[args.dtype]
        wdt = np.uint32 if code == 1 else np.uint16
        rng = np.random.default_rng(0)
        for l in sorted(set(rng.integers(0, len(layers), n_layer_picks).tolist())):
            c = layers[l]
            for ui in sorted(set(rng.integers(0, len(c.units), n_unit_picks).tolist())):
                u = c.units[ui]
                lo, n, mo, co = int(u["weights_off"]), int(u["n_values"]), int(u["msg_off"]), int(u["cache_off"])
                w_prev = prev_w[l][lo : lo + n * vb].cpu().numpy().view(wdt)
                w_cur = last_w[l][lo : lo + n * vb].cpu().numpy().view(wdt)
                cache = ora.cache_init(w_prev, n, code)
                m, wbytes, _, cb = ora.encode(w_cur, cache, code, args.block)
                got = c.msg_recv[mo : mo + wbytes].cpu().numpy()
                verified = verified and int(c.wire_bytes[ui].item()) == wbytes and np.array_equal(got, m)
                verified = verified and int(c.changed_blocks[ui].item()) == cb
                verified = verified and np.array_equal(c.receiver_cache[co : co + n].cpu().numpy(), cache)
                sampled += 1
    return bool(verified), sampled


# --------------------------------------------------------------------------------- main arm


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    from paper_2609_04609_b200 import build as libbuild

    libbuild.ensure_library()  # a fresh checkout: built once, in-tree; an existing library is used as it is
    from paper_2609_04609_b200 import ciera, runtime
    from paper_2609_04609_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the codec has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peak, peak_kind = measured_peak()
    vb = wl.VALUE_BYTES[args.dtype]
    layers, wa, wb = build_stack(args, device, seed_base=rank_seed(rank))
    n_values = sum(c.plan.total_values for c in layers)
    weight_bytes = n_values * vb
    s_enc = torch.cuda.Stream()
    s_dec = s_enc if args.schedule == "serial" else torch.cuda.Stream()
    if args.entropy:  # the stage's scratch is only used between a layer's launches: one buffer serves all layers
        shared = layers[0]._entropy_scratch()
        for c in layers[1:]:
            c.entropy_scratch = shared
    pipe = runtime.LayerPipeline(layers, s_enc, s_dec, entropy=args.entropy)
    serial_pipe = runtime.LayerPipeline(layers, s_enc, s_enc, entropy=args.entropy)

    def weights_of(i):
        return wb if i % 2 == 0 else wa

    step_i = 0
    for _ in range(max(args.warmup, 3)):
        pipe.step(weights_of(step_i))
        step_i += 1
    barrier()

    # ---- timed region: exactly K steps, device-timed, launch accounting, clocks sampled
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(device).uuid)
    except Exception:
        uuid = ""
    sampler = ClockSampler(local_rank, uuid)
    timers = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ciera.kernel_launch_count()
    sampler.start()
    barrier()
    cur = torch.cuda.current_stream()
    ev0.record(cur)
    s_enc.wait_event(ev0)
    s_dec.wait_event(ev0)
    for _ in range(args.steps):
        pipe.step(weights_of(step_i), None, timers)
        step_i += 1
    cur.wait_stream(s_enc)
    cur.wait_stream(s_dec)
    ev1.record(cur)
    barrier()
    clocks = sampler.stop()
    launches = ciera.kernel_launch_count() - launches0
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), world, device)
    ms_per_step = ms_total / args.steps
    for c in layers:
        c.check_status()

    # ---- the same K steps once more on ONE stream: kernels do not overlap, so the CUDA events
    #      around each launch time that kernel alone (used for the roofline entries)
    serial_timers = []
    sev0, sev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sev0.record(s_enc)
    for _ in range(args.steps):
        serial_pipe.step(weights_of(step_i), None, serial_timers)
        step_i += 1
    sev1.record(s_enc)
    barrier()
    serial_ms_per_step = sev0.elapsed_time(sev1) / args.steps
    # spread over the steps (serial re-run: a step's first launch to its last; the paper reports p5 / p95 whiskers)
    nl = len(layers)
    per_step = [serial_timers[i * nl][0].elapsed_time(serial_timers[i * nl + nl - 1][5]) for i in range(args.steps)]
    step_spread = {"mean": float(np.mean(per_step)), "min": float(np.min(per_step)), "p5": float(np.percentile(per_step, 5)),
                   "p95": float(np.percentile(per_step, 95)), "max": float(np.max(per_step)), "steps": args.steps,
                   "per": "serial re-run on one stream, first launch to last of each step, ms"}
    for c in layers:
        c.check_status()

    # ---- what was moved: change rates and the paper's byte count of the last step
    # element change rate c of the workload (reporting only): exponent fields of the two iterates of layer 0
    shift, wdt_t, emask = {"bf16": (7, torch.int16, 0xFF), "fp32": (23, torch.int32, 0xFF),
                           "fp16": (10, torch.int16, 0x1F)}[args.dtype]
    ea = (wa[0].view(wdt_t) >> shift) & emask
    eb = (wb[0].view(wdt_t) >> shift) & emask
    element_change_rate = float((ea != eb).float().mean().item())
    del ea, eb
    changed = sum(int(c.changed_blocks.sum().item()) for c in layers)
    blocks = sum(c.n_blocks() for c in layers)
    q = changed / blocks
    paper_bytes = sum(c.paper_bytes() for c in layers)
    ovl_ms = [float(np.mean([t[2 * i].elapsed_time(t[2 * i + 1]) for t in timers])) for i in range(3)]
    enc_ms, tra_ms, dec_ms = [float(np.mean([t[2 * i].elapsed_time(t[2 * i + 1]) for t in serial_timers]))
                              for i in range(3)]
    ent_ms = [float(np.mean([t[i].elapsed_time(t[i + 1]) for t in serial_timers])) for i in (6, 8)] if args.entropy else None
    n_layer = layers[0].plan.total_values
    a_enc, a_tra, a_dec = algorithmic_bytes(n_layer, q, args.dtype, args.block, args.detect)
    enc_gbs = a_enc / (enc_ms * 1e-3) / 1e9
    dec_gbs = a_dec / (dec_ms * 1e-3) / 1e9
    tra_gbs = a_tra / (tra_ms * 1e-3) / 1e9
    path_gbs = len(layers) * (a_enc + a_tra + a_dec) / (ms_per_step * 1e-3) / 1e9

    # ---- correctness at full size: exact round trip everywhere, oracle on sampled units
    last_w = weights_of(step_i - 1)
    prev_w = weights_of(step_i)  # the iterate before the last one (the steps alternate)
    verified, sampled = verify_stack(args, ciera, layers, last_w, prev_w, n_layer_picks=4, n_unit_picks=16,
                                     with_oracle=rank == 0)

    coded = None
    if args.entropy:
        # one more (untimed) step, stopped after the entropy stage of every layer to read the coded sizes
        nxt = weights_of(step_i)
        coded_bytes = 0
        for c, w in zip(layers, nxt):
            c.encode(w)
            raw_bytes_layer = c.paper_bytes()
            c.entropy_encode()
            coded_bytes += c.paper_bytes()
            c.transport()
            c.entropy_decode()
            c.decode()
        torch.cuda.synchronize()
        for c in layers:
            c.check_status()
        step_i += 1
        coded = {"bytes_ratio_coded": coded_bytes / weight_bytes,
                 "entropy_encode_ms": ent_ms[0], "entropy_decode_ms": ent_ms[1],
                 "per": "layer launch, serial re-run",
                 "note": "rANS of the changed exponents, static 12-bit model per unit; one block per unit"}

    traffic, traffic_note = None, "no ncu capture on record for this workload"
    if args.dtype == "bf16" and args.block == 512 and args.update == "clustered" and args.f == 0.22 and args.shapes == "olmoe":
        traffic, traffic_note = measured_traffic("encode_exact_bf16_B512_clustered_f0.22" if args.detect == "compare"
                                                 else "encode_hashed_bf16_B512_clustered_f0.22", n_layer)

    out = {
        "metric": METRIC,
        "value": whole_job_gbps(world, weight_bytes, ms_per_step),
        "unit": "GB/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "u32",
        "data": "synthetic",
        "config": workload_config(args),
        "gpu_launches": int(launches),
        "clocks": clocks,
        "verified_bit_exact": verified,
        "element_change_rate_c": element_change_rate,
        "entropy_stage": coded,
        "oracle_sampled_units": sampled,
        "block_change_rate_q": q,
        "bytes_ratio": paper_bytes / weight_bytes,
        "encode_GBps_of_weights": n_layer * vb / (enc_ms * 1e-3) / 1e9,
        "decode_GBps_of_weights": n_layer * vb / (dec_ms * 1e-3) / 1e9,
        "kernel_ms": {"encode": enc_ms, "transport": tra_ms, "decode": dec_ms,
                      "per": "layer launch; serial re-run of the timed steps on one stream"},
        "kernel_ms_overlapped": {"encode": ovl_ms[0], "transport": ovl_ms[1], "decode": ovl_ms[2],
                                 "per": "layer launch inside the two-stream timed region (kernels overlap)"},
        "serial_ms_per_step": serial_ms_per_step,
        "serial_step_ms_spread": step_spread,
        "kernel_ms_x_sm_mhz": ({"encode": enc_ms * clocks["sm_mhz"], "transport": tra_ms * clocks["sm_mhz"],
                                "decode": dec_ms * clocks["sm_mhz"],
                                "note": "launch time x median SM MHz sampled in the timed region: constant across runs "
                                        "for a kernel bound by the SM clock, proportional to the clock for one bound by HBM"}
                               if clocks.get("sm_mhz") else None),
        "roofline": {
            "bound": "hbm", "kernel": ("encode_kernel" if args.detect == "compare" else "encode_kernel (HashCache form)"), "achieved": enc_gbs, "peak": peak, "unit": "GB/s",
            "frac": enc_gbs / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBps": enc_gbs / NOMINAL_HBM_GBS,
            "traffic": traffic, "traffic_note": traffic_note,
            "algorithmic_bytes_per_launch": a_enc,
            "timed": "CUDA events around every encode launch, same K steps re-run on one stream so that "
                     "no other kernel overlaps it",
        },
        "roofline_other": {
            "decode_kernel": {"achieved": dec_gbs, "frac": dec_gbs / peak, "algorithmic_bytes_per_launch": a_dec},
            "transport_kernel": {"achieved": tra_gbs, "frac": tra_gbs / peak, "algorithmic_bytes_per_launch": a_tra},
            "whole_step_pipelined": {"achieved": path_gbs, "frac": path_gbs / peak,
                                     "note": "algorithmic bytes of all three kernels over the two-stream step time"},
        },
    }

    # ---- which shards would be compressed: the gain rule and the selection under a cache budget,
    #      fed with this run's measured change rates and kernel times (host arithmetic only)
    if rank == 0:
        out["selection"] = selection_report(args, ciera, layers[-1], enc_ms, dec_ms)

    # ---- per-kernel numbers with each kernel alone on the GPU, three change regimes (one layer)
    if not args.no_regimes and rank == 0 and args.detect == "compare":
        out["kernels_alone"] = kernels_alone(args, layers[0], wa[0], wb[0], peak)

    # ---- the other configurations, one layer each (rank 0, one GPU only)
    if not args.no_other_configs and rank == 0 and world == 1:
        out["other_configs"] = other_configs(args, device, peak, clocks.get("sm_mhz"))
        out["block_size_sweep"] = block_size_sweep(args, device, peak)
        out["graph_replay"] = graph_replay_latency(device)

    # ---- end to end through the host-buffer entry point (weights start and end in host memory)
    if not args.no_e2e:
        # three pinned host copies of the stack per rank; all ranks of the node share its memory
        need = 3 * sum(w.numel() for w in wa) * int(os.environ.get("LOCAL_WORLD_SIZE", str(world)))
        if host_memory_allows(need, world, device):
            out["e2e"] = e2e(args, layers, wa, wb, world, rank, barrier)
        else:
            out["e2e"] = {"value": None, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                          "skipped": f"{need} bytes of pinned host memory would be more than 60 % of what is free"}

    # ---- the oracle on this machine's host cores (rank 0, one GPU only)
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        threads = os.cpu_count() or 1
        code = ciera.DTYPE_CODES[args.dtype]
        dt = nv = nu = 0
        for l in range(min(len(layers), args.cpu_sample_layers)):  # a bounded sample: some seconds of CPU work
            units = layers[l].units[: args.cpu_sample_units]
            hi = int(units[-1]["weights_off"]) + int(units[-1]["n_values"]) * vb
            a = wa[l][:hi].cpu().numpy()
            b = wb[l][:hi].cpu().numpy()
            d, n = oracle_roundtrip_units(units, a, b, code, args.block, vb, threads)
            dt, nv, nu = dt + d, nv + n, nu + len(units)
        units1 = layers[0].units[: max(1, min(args.cpu_sample_units, 256))]
        hi = int(units1[-1]["weights_off"]) + int(units1[-1]["n_values"]) * vb
        d1, n1 = oracle_roundtrip_units(units1, wa[0][:hi].cpu().numpy(), wb[0][:hi].cpu().numpy(), code, args.block, vb, 1)
        out["cpu_baseline"] = {"value": nv * vb / dt / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
                               "sample": f"{nu} of {sum(len(c.units) for c in layers)} units ({nv} values), "
                                         f"encode+decode round trip, {dt:.2f} s wall on {threads} threads",
                               "single_thread_value": n1 * vb / d1 / 1e9}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# The other workloads of the build's configuration list, one layer each, kernels timed one after the other on one
# stream (CUDA events around every launch).  They ride along in the bench line as `other_configs`; `value` is
# never taken from them.
OTHER_CONFIGS = [
    # name, overrides of the command-line defaults
    ("config2_one_layer_adam_like_update", dict(update="adam")),
    ("config4_fp32_clustered", dict(dtype="fp32")),
    ("config4_fp32_adam_like_update", dict(dtype="fp32", update="adam")),
    ("config5_mixed_8_shards_1pct_iid", dict(shapes="mixed", shards=8, update="inject", inject=0.01, inject_seg=0)),
    ("config5_mixed_64_shards_10pct_segments", dict(shapes="mixed", shards=64, update="inject", inject=0.1, inject_seg=512)),
    ("block1_adam_like_update", dict(block=1, update="adam")),
    ("block2_adam_like_update", dict(block=2, update="adam")),
    ("block4_adam_like_update", dict(block=4, update="adam")),
    ("block8_adam_like_update", dict(block=8, update="adam")),
    ("block1_half_of_the_exponents_change", dict(block=1, update="inject", inject=0.5, inject_seg=0)),
    ("block64_adam_like_update", dict(block=64, update="adam")),
    ("fp16_clustered", dict(dtype="fp16")),
    ("fp16_block1_adam_like_update", dict(dtype="fp16", block=1, update="adam")),
    ("hashed_sender_bf16_block512", dict(detect="hash")),
    ("hashed_sender_bf16_block32_adam_like_update", dict(detect="hash", block=32, update="adam")),
    ("hashed_sender_fp32_block512", dict(detect="hash", dtype="fp32")),
    ("entropy_stage_bf16_block512", dict(entropy=True)),
    ("entropy_stage_fp16_block512", dict(entropy=True, dtype="fp16")),
]


def raw_payload_symbols(codec, a):
    """Changed exponents (one symbol each) that the entropy stage codes: the raw payload bytes of the last encode
    (fp16: five bits per exponent on the wire, so 8 symbols to 5 payload bytes; a short last block rounds up)."""
    from paper_2609_04609_b200 import ciera

    wire = codec.wire_bytes.cpu().numpy()
    payload = int(sum(int(w) - ciera.payload_offset(int(u["n_values"]), codec.dtype, a.block)
                      for u, w in zip(codec.units, wire) if int(u["n_values"])))
    return payload * 8 // 5 if a.dtype == "fp16" else payload


def entropy_roofline(symbols, enc_ms, dec_ms, sm_mhz, sms=148):
    """The entropy stage moves little and computes a lot per byte: its bound is instruction issue.  Peak = SMs x 4
    warp schedulers x one warp instruction per clock at the SM clock sampled during the run; the work is the ncu
    count of warp instructions per coded symbol on record (profiles/) x the symbols of this launch."""
    try:
        rec = json.load(open(TRAFFIC_FILE))["entropy_stage_bf16_B512_clustered_f0.22"]
    except Exception:
        return None
    peak = sms * 4 * (sm_mhz or 1965.0) * 1e6  # warp instructions per second
    out = {"bound": "issue", "unit": "G warp-instructions/s", "peak": peak / 1e9, "symbols_per_launch": symbols,
           "derivation": "148 SMs x 4 schedulers x 1 warp instruction per clock x sampled SM MHz"}
    for name, ms, key in (("encode", enc_ms, "warp_instructions_per_symbol_encode"),
                          ("decode", dec_ms, "warp_instructions_per_symbol_decode")):
        ach = rec[key] * symbols / (ms * 1e-3)
        out[name] = {"warp_instructions_per_symbol": rec[key], "achieved": ach / 1e9, "frac": ach / peak,
                     "payload_GBps": symbols / (ms * 1e-3) / 1e9}
    if rec.get("csrc_sha256") != csrc_digest():
        out["note"] = "instruction counts per symbol are from an ncu capture of earlier kernel sources"
    return out


def one_layer_case(args, device, peak, over, steps=5, clocks_mhz=None):
    """One layer of the workload `args` + `over`: three warm-up steps, then `steps` timed ones, all on one stream."""
    import torch

    from paper_2609_04609_b200 import ciera, runtime
    from paper_2609_04609_b200 import workloads as wl

    a = argparse.Namespace(**{**vars(args), "layers": 1, "experts": 64, "shards": 16, "block": 512, "dtype": "bf16",
                              "update": "clustered", "f": 0.22, "shapes": "olmoe", "detect": "compare",
                              "entropy": False, **over})
    layers, wa, wb = build_stack(a, device, seed_base=4321)
    codec = layers[0]
    vb = wl.VALUE_BYTES[a.dtype]
    stream = torch.cuda.Stream()
    pipe = runtime.LayerPipeline(layers, stream, stream, entropy=a.entropy)
    i = 0
    for _ in range(3):
        pipe.step(wb if i % 2 == 0 else wa)
        i += 1
    timers = []
    for _ in range(steps):
        pipe.step(wb if i % 2 == 0 else wa, None, timers)
        i += 1
    torch.cuda.synchronize()
    codec.check_status()
    last_w, prev_w = (wb, wa) if (i - 1) % 2 == 0 else (wa, wb)
    verified, sampled = verify_stack(a, ciera, layers, last_w, prev_w, n_layer_picks=1, n_unit_picks=6)
    n = codec.plan.total_values
    q = int(codec.changed_blocks.sum().item()) / max(codec.n_blocks(), 1)
    enc_ms, tra_ms, dec_ms = [float(np.mean([t[2 * k].elapsed_time(t[2 * k + 1]) for t in timers])) for k in range(3)]
    a_enc, a_tra, a_dec = algorithmic_bytes(n, q, a.dtype, a.block, a.detect)
    res = {
        "workload": workload_config(a)["workload"], "values": n, "units": len(codec.units),
        "block_change_rate_q": q, "bytes_ratio": codec.paper_bytes() / (n * vb),
        "encode_ms": enc_ms, "transport_ms": tra_ms, "decode_ms": dec_ms,
        "encode_frac": a_enc / (enc_ms * 1e-3) / 1e9 / peak, "transport_frac": a_tra / (tra_ms * 1e-3) / 1e9 / peak,
        "decode_frac": a_dec / (dec_ms * 1e-3) / 1e9 / peak,
        "encode_GBps_of_weights": n * vb / (enc_ms * 1e-3) / 1e9, "decode_GBps_of_weights": n * vb / (dec_ms * 1e-3) / 1e9,
        "verified_bit_exact": verified, "oracle_sampled_units": sampled,
    }
    if a.block < 32 and a.detect == "compare":
        # Blocks smaller than a 32-byte DRAM sector: the caches (one byte per value) can only be refreshed by whole
        # sectors, so the bytes that have to move are the sectors holding a changed exponent, not q bytes per value.
        # s = share of the 32-value groups of the layer in which some exponent differs between the two iterates.
        shift, wdt_t, emask = {"bf16": (7, torch.int16, 0xFF), "fp32": (23, torch.int32, 0xFF),
                               "fp16": (10, torch.int16, 0x1F)}[a.dtype]
        ea = (wa[0].view(wdt_t) >> shift) & emask
        eb = (wb[0].view(wdt_t) >> shift) & emask
        diff = ea != eb
        m = diff.numel() // 32 * 32
        s_rate = float(diff[:m].view(-1, 32).any(dim=1).float().mean().item())
        del ea, eb, diff
        extra = n * max(s_rate - q, 0.0)  # cache bytes beyond the q per value already counted
        res["cache_sector_rate"] = s_rate
        res["encode_frac_sector_granular"] = (a_enc + extra) / (enc_ms * 1e-3) / 1e9 / peak
        res["decode_frac_sector_granular"] = (a_dec + extra) / (dec_ms * 1e-3) / 1e9 / peak
        res["sector_note"] = ("the *_frac_sector_granular figures count the cache refresh as whole 32-byte sectors "
                              "(cache_sector_rate bytes per value) instead of q bytes per value")
    if a.entropy:
        res["entropy_encode_ms"], res["entropy_decode_ms"] = [
            float(np.mean([t[k].elapsed_time(t[k + 1]) for t in timers])) for k in (6, 8)]
        # the coded size: one more sender step, read between the entropy stage and the transport
        w = wb if i % 2 == 0 else wa
        codec.encode(w[0])
        raw = codec.paper_bytes()
        symbols = raw_payload_symbols(codec, a)
        codec.entropy_encode()
        if a.dtype == "fp16":  # no instruction count on record for the unpacking and packing around the coder
            res["entropy_symbols_per_launch"] = symbols
            res["entropy_symbols_G_per_s"] = [symbols / (res[k] * 1e-3) / 1e9 for k in ("entropy_encode_ms", "entropy_decode_ms")]
        else:
            res["entropy_roofline"] = entropy_roofline(symbols, res["entropy_encode_ms"],
                                                       res["entropy_decode_ms"], clocks_mhz)
        coded = codec.paper_bytes()
        fixed = sum(ciera.message_bytes(int(u["n_values"]), codec.dtype, a.block, 0) for u in codec.units if int(u["n_values"]))
        res["bytes_ratio_coded"] = coded / (n * vb)
        res["payload_coded_over_raw"] = (coded - fixed) / (raw - fixed) if raw > fixed else None
        codec.transport()
        codec.entropy_decode()
        codec.decode()
        torch.cuda.synchronize()
        codec.check_status()
    del layers, wa, wb, pipe
    torch.cuda.empty_cache()
    return res


def graph_replay_latency(device, reps=200):
    """Small tables are bound by launch latency, not by HBM: config 1 (1024 x 512 bf16, 4 shards) and one expert's
    three matrices on 16 shards, stepped eagerly through the binding and replayed from a CUDA graph that holds two
    steps (A -> B -> A).  Microseconds per step (encode + transport + decode), CUDA events around `reps` pairs."""
    import torch

    from paper_2609_04609_b200 import runtime
    from paper_2609_04609_b200 import workloads as wl

    out = {"per": "step = encode + transport + decode of the whole table, one stream; us"}
    cases = {"config1_1024x512_bf16_4_shards": ([1024 * 512], 4),
             "one_expert_3_matrices_bf16_16_shards": ([r * c for r, c in wl.olmoe_layer_shapes(1)], 16)}
    for name, (sizes, shards) in cases.items():
        try:
            codec = runtime.LayerCodec.from_tensors(sizes, shards, "bf16", 512, device)
            gen = wl.make_generator(11, device)
            n = codec.weights_bytes // 2
            wa = wl.init_weights(n, "bf16", gen)
            wb = wl.step_clustered(wa, gen, f=0.22)
            a, b = wa.view(torch.uint8), wb.view(torch.uint8)
            codec.init_caches(a)
            stream = torch.cuda.Stream(device)
            with torch.cuda.stream(stream):
                for _ in range(3):
                    codec.step(b)
                    codec.step(a)
                stream.synchronize()

                def timed(fn):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    for _ in range(reps):
                        fn()
                    e1.record()
                    e1.synchronize()
                    return e0.elapsed_time(e1) * 1e3 / (2 * reps)

                def eager():
                    codec.step(b)
                    codec.step(a)

                eager_us = timed(eager)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                codec.step(b)
                codec.step(a)
            with torch.cuda.stream(stream):
                graph.replay()
                graph_us = timed(graph.replay)
            torch.cuda.synchronize()
            codec.check_status()
            ok = all(torch.equal(codec.weights_out[int(u["weights_off"]): int(u["weights_off"]) + 2 * int(u["n_values"])],
                                 a[int(u["weights_off"]): int(u["weights_off"]) + 2 * int(u["n_values"])])
                     for u in codec.units)
            out[name] = {"values": int(codec.plan.total_values), "units": len(codec.units), "eager_us": eager_us,
                         "graph_us": graph_us, "verified_bit_exact": bool(ok)}
        except Exception as e:
            out[name] = {"error": f"{type(e).__name__}: {e}"}
    return out


def block_size_sweep(args, device, peak):
    """The paper's block-size sensitivity (64 ... 4096 values per block, default 512) on one synthetic layer: how the
    share of changed blocks, the message size and the kernels' pace move with B, under the clustered update (changes
    concentrated in 512-aligned segments) and under the literal Adam-like update (independent changes)."""
    out = {"per": "one layer, bf16; kernels one after the other on one stream; fractions of the measured copy bandwidth"}
    for update in ("clustered", "adam"):
        for block in (16, 32, 64, 128, 256, 512, 1024, 2048, 4096):
            try:
                r = one_layer_case(args, device, peak, dict(block=block, update=update), steps=3)
                out[f"{update}_B{block}"] = {k: r[k] for k in ("block_change_rate_q", "bytes_ratio", "encode_ms", "decode_ms",
                                                                 "encode_frac", "transport_frac", "decode_frac",
                                                                 "verified_bit_exact")}
            except Exception as e:
                out[f"{update}_B{block}"] = {"error": f"{type(e).__name__}: {e}"}
    return out


def other_configs(args, device, peak, clocks_mhz=None):
    out = {"per": "one layer; kernels one after the other on one stream, CUDA events around every launch; fractions "
                  "are algorithmic bytes per launch over the measured copy bandwidth"}
    for name, over in OTHER_CONFIGS:
        try:
            out[name] = one_layer_case(args, device, peak, over, clocks_mhz=clocks_mhz)
        except Exception as e:  # one failing side case must not take the headline line with it
            out[name] = {"error": f"{type(e).__name__}: {e}"}
    return out


def kernels_alone(args, codec, w_a, w_b, peak):
    """Each kernel timed alone (events on its stream, nothing else running) on one layer, at block
    change rates ~0 (nothing changed), the workload's own, and 1 (every block changed)."""
    import torch

    res = {}
    vb = 4 if args.dtype == "fp32" else 2
    n = codec.plan.total_values
    # lowest exponent bit flipped everywhere: every block changes
    if args.dtype == "bf16":
        w_c = (w_a.view(torch.int16) ^ 0x0080).view(torch.uint8)
    elif args.dtype == "fp16":
        w_c = (w_a.view(torch.int16) ^ 0x0400).view(torch.uint8)
    else:
        w_c = (w_a.view(torch.int32) ^ 0x00800000).view(torch.uint8)

    def timed(fn, reps=5):
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            torch.cuda._sleep(300_000)  # keeps the stream busy while the host enqueues: no launch latency between the events
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    for name, first, second in (("q0", w_a, w_a), ("workload", w_a, w_b), ("q1", w_a, w_c)):
        enc, tra, dec = [], [], []
        for _ in range(5):
            codec.init_caches(first)
            enc.append(timed(lambda: codec.encode(second), 1))
            tra.append(timed(lambda: codec.transport(), 1))
            dec.append(timed(lambda: codec.decode(), 1))
        q = int(codec.changed_blocks.sum().item()) / codec.n_blocks()
        a_enc, a_tra, a_dec = algorithmic_bytes(n, q, args.dtype, args.block)
        e, t, d = float(np.median(enc)), float(np.median(tra)), float(np.median(dec))
        res[name] = {
            "q": q,
            "encode_ms": e, "encode_hbm_GBps": a_enc / e / 1e6, "encode_frac": a_enc / e / 1e6 / peak,
            "encode_GBps_of_weights": n * vb / e / 1e6,
            "transport_ms": t, "transport_hbm_GBps": a_tra / t / 1e6, "transport_frac": a_tra / t / 1e6 / peak,
            "decode_ms": d, "decode_hbm_GBps": a_dec / d / 1e6, "decode_frac": a_dec / d / 1e6 / peak,
            "decode_GBps_of_weights": n * vb / d / 1e6,
        }
    codec.init_caches(w_a)
    return res


def e2e(args, layers, wa, wb, world, rank, barrier):
    """Same step, but the weights start in pinned host memory and the reconstructed weights end
    there: every layer goes through ciera_roundtrip_host (H2D copy, encode, transport, decode,
    D2H copy), two streams so that the copies of neighbouring layers overlap."""
    import torch
    import torch.distributed as dist

    host_a = [torch.empty(w.numel(), dtype=torch.uint8, pin_memory=True) for w in wa]
    host_b = [torch.empty(w.numel(), dtype=torch.uint8, pin_memory=True) for w in wb]
    host_out = [torch.empty(w.numel(), dtype=torch.uint8, pin_memory=True) for w in wa]
    wire_host = [torch.empty(len(c.units), dtype=torch.int64, pin_memory=True) for c in layers]
    for h, w in zip(host_a, wa):
        h.copy_(w)
    for h, w in zip(host_b, wb):
        h.copy_(w)
    for c, w in zip(layers, wa):
        c.init_caches(w)
    staging = [torch.empty_like(wa[0]) for _ in range(2)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()

    def step(src):
        for l, c in enumerate(layers):
            c.step_host(src[l], host_out[l], staging[l % 2], wire_host[l], streams[l % 2])

    steps = max(1, min(args.steps, 3))
    step(host_b)
    step(host_a)
    barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    t0.record(cur)
    for s in streams:
        s.wait_event(t0)
    for i in range(steps):
        step(host_b if i % 2 == 0 else host_a)
    for s in streams:
        cur.wait_stream(s)
    t1.record(cur)
    barrier()
    ms = max_over_ranks(t0.elapsed_time(t1) / steps, world, wa[0].device)
    ok = all(torch.equal(o, (host_b if (steps - 1) % 2 == 0 else host_a)[l]) for l, o in enumerate(host_out))
    nbytes = sum(h.numel() for h in host_a)
    # what the link alone does on this machine: one layer's bytes in each direction at the same time, nothing else running
    # (the end-to-end step cannot be faster than this; reported so that its figure can be read against the link)
    link = None
    try:
        up, down = torch.empty_like(wa[0]), wa[0]
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        c0.record(cur)
        for s in streams:
            s.wait_event(c0)
        for _ in range(4):
            with torch.cuda.stream(streams[0]):
                up.copy_(host_a[0], non_blocking=True)
            with torch.cuda.stream(streams[1]):
                host_out[0].copy_(down, non_blocking=True)
        for s in streams:
            cur.wait_stream(s)
        c1.record(cur)
        torch.cuda.synchronize()
        link = 4 * host_a[0].numel() / (c0.elapsed_time(c1) * 1e-3) / 1e9
    except Exception:
        pass
    return {"value": whole_job_gbps(world, nbytes, ms), "unit": "GB/s", "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": nbytes + 8 * sum(len(c.units) for c in layers),
            "bit_exact": bool(ok), "api": "ciera_roundtrip_host (pinned host weights in, host weights out)",
            "link_GBps_each_way_both_at_once": link,
            "frac_of_link": (whole_job_gbps(1, nbytes, ms) / link) if link else None}


if __name__ == "__main__":
    main()
