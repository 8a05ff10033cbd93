#!/usr/bin/env python
"""Throughput of one LQ-SGD compression round on synthetic gradient sets.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one full round (Algorithm 1 body: error feedback, both power steps,
orthonormalisation, quantise / pack / average / dequantise of P and Q, reconstruction, error
update) over one gradient set.  The metric is GB/s of fp32 gradient processed:
4 bytes x W workers x all gradient elements / step time.  Prints ONE JSON line on rank 0.

--impl ours       the CUDA library through its C ABI (device-resident inputs for `value`,
                  host buffers through lqsgd_step_host for `e2e`).
--impl reference  the CPU oracle as it stands, on the host cores, on a bounded sample.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "LQ-SGD compress+decompress GB/s of fp32 gradient"
UNIT = "GB/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def csrc_digest(files=None) -> str:
    """SHA-256 over kernel sources (all of csrc, or the named files): ties a stored ncu figure to the
    code it was taken from."""
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2506_17974_b200", "csrc")
    names = sorted(files) if files else sorted(n for n in os.listdir(d) if n.endswith((".cu", ".cuh", ".h")))
    for name in names:
        h.update(name.encode())
        with open(os.path.join(d, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def recorded_traffic(workload: str, phase: str):
    """DRAM bytes (read + write) per launch of that phase's kernel from the ncu capture summarised under
    profiles/, or None when there is no capture of this workload or the kernel's sources changed since."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f)
    for e in rec.get("entries", []):
        if e.get("workload") == workload and e.get("phase") == phase:
            return e["dram_bytes"] if e.get("sha256") == csrc_digest(e.get("sources")) else None
    return None


def kernel_name(phase: str, rank: int) -> str:
    """The kernel that carries a pass for layers with 16-byte aligned rows at this rank (unaligned layers,
    a few KB in the ResNet set, run on the register kernels of the same phase)."""
    if phase == "round":
        return "resident_round_kernel"
    n = phase[-1]
    if rank > 8:
        return f"tc_pass{n}_kernel"
    return "pass2_kernel" if n == "2" else f"stream_pass{n}_kernel"


def get_workload(name: str):
    from paper_2506_17974_b200 import workloads as wl
    if name == "resnet18":
        return wl.config3(), "resnet18_cifar W=8 r=2 b=4 (ResNet-18 gradient set, Student-t nu=3)"
    if name == "mnist":
        return wl.config2(), "mnist_cnn W=4 r=4 b=4"
    if name == "single":
        return wl.config1(), "single 256x576 W=1 r=2 b=4"
    if name.startswith("large_"):
        a, b = name[len("large_"):].split("x")
        return wl.config4(int(a), int(b)), f"large layer {a}x{b} W=1 r=8 b=4, N(0, 0.01^2)"
    if name.startswith("config5_r"):
        r, b = name[len("config5_r"):].split("_b")
        return wl.config5(int(r), int(b)), f"resnet18_cifar100 W=16 r={r} b={b} (ResNet-18 gradient set, Student-t nu=3)"
    raise SystemExit(f"unknown workload {name}")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        # gpu_id: what nvidia-smi --id takes - the device's UUID ("GPU-..."), so that the samples are this
        # process's GPU whatever CUDA_VISIBLE_DEVICES maps ordinal 0 to (an index only as a last resort)
        self.index, self.rows, self.proc = gpu_id, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()          # the exact child started above
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "gpu": self.index}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm),
                "gpu": self.index}


def gpu_smi_id(torch, local: int) -> str:
    """The UUID nvidia-smi knows this CUDA device by (read-only query)."""
    try:
        u = str(torch.cuda.get_device_properties(local).uuid)
        return u if u.startswith("GPU-") else "GPU-" + u
    except Exception:
        return str(local)


def phase_bytes(wl_obj):
    """Algorithmic HBM bytes one launch of each streaming pass moves (three-pass streaming with M
    kept in place of E): pass 1 reads G and E and writes M, pass 2 reads M, pass 3 reads M,
    writes E per worker and G_hat once per layer."""
    from paper_2506_17974_b200 import workloads as wl
    W = wl_obj.workers
    nm = wl.matrix_elements(wl_obj.layers)
    return {"pass1": 12 * W * nm, "pass2": 4 * W * nm, "pass3": 8 * W * nm + 4 * nm}


def time_oracle(wl_obj, budget_s: float, max_steps: int):
    """Runs the CPU oracle on whole rounds of the workload until about budget_s has passed."""
    import numpy as np
    import torch
    from oracle import lqsgd_oracle as orc
    from paper_2506_17974_b200 import workloads as wl
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    rng = np.random.default_rng(0)
    Q0 = {li: rng.standard_normal((m, min(wl_obj.rank, n, m)))
          for li, (n, m) in enumerate(wl_obj.layers) if wl.is_matrix((n, m))}
    o = orc.Oracle(wl_obj.layers, wl_obj.rank, wl_obj.bits, wl_obj.bits, wl_obj.alpha, wl_obj.workers, Q0)
    grads = [[t.numpy() for t in per] for per in wl.draw_gradients(wl_obj, 0, device="cpu")]
    times = []
    t_all = time.perf_counter()
    while len(times) < max_steps and (not times or time.perf_counter() - t_all < budget_s):
        t0 = time.perf_counter()
        o.step(grads)
        times.append(time.perf_counter() - t0)
    return times, cores


def gradient_bytes(wl_obj):
    return 4 * wl_obj.workers * sum(n * m for n, m in wl_obj.layers)


def config_dict(wl_obj, desc):
    """What both arms print as `config`: the workload, and nothing that depends on the arm."""
    return {"workload": desc, "rank": wl_obj.rank, "bits": wl_obj.bits, "workers": wl_obj.workers,
            "alpha": wl_obj.alpha,
            "l2": f"inputs larger than L2: each step streams a gradient set of {gradient_bytes(wl_obj) / 1e6:.0f} MB "
                  "plus the error buffers; the CUDA arm rotates gradient sets between steps"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl_obj, desc = get_workload(args.workload)
    # whole rounds until warm-up + steps are done or 150 s have passed, whichever comes first (the line
    # says how many rounds were timed): the run ends within a few minutes on any host
    times, cores = time_oracle(wl_obj, budget_s=150.0, max_steps=args.warmup + args.steps)
    timed = times[args.warmup:] or times
    t = sum(timed) / len(timed)
    value = gradient_bytes(wl_obj) / t / 1e9
    sample = f"{len(timed)} whole rounds of the workload (all layers, all W workers), numpy fp64"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(timed), "warmup": args.warmup, "ms_per_step": 1e3 * t, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(wl_obj, desc),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(args):
    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry
    from paper_2506_17974_b200 import binding as B
    from paper_2506_17974_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py --impl ours needs a CUDA device: there is no CPU fallback")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"rank {rank} has no GPU: {torch.cuda.device_count()} visible, {world} ranks asked for")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    peak, peak_kind = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def allmax(x):
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def allmax_list(xs):
        if world == 1:
            return list(xs)
        t = torch.tensor(list(xs), dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return [float(v) for v in t.tolist()]

    def bench_workload(wl_obj, steps, warmup, nsets, want_e2e, sample_clocks, want_graph=False, min_ms=0.0,
                       one_launch=False):
        comp = B.LQSGD(wl_obj.layers, wl_obj.rank, wl_obj.bits, alpha=wl_obj.alpha, workers=wl_obj.workers,
                       seed=wl_obj.seed + rank, device=dev, one_launch=one_launch)
        seeded = dataclasses.replace(wl_obj, seed=wl_obj.seed + 1000 * rank)
        sets = [wl.draw_gradients(seeded, t, device=dev) for t in range(nsets)]
        ghat = [torch.empty_like(g) for g in sets[0][0]]
        ptrs = [comp.make_pointer_arrays(s, ghat) for s in sets]
        stream = torch.cuda.current_stream()
        for t in range(warmup):
            comp.step_ptrs(*ptrs[t % nsets], stream)
        psteps = min(steps, 20)            # steps of the per-kernel profile loop that follows the timed region
        events = [[torch.cuda.Event(enable_timing=True) for _ in range(B.N_PHASES + 1)] for _ in range(psteps)]
        for evs in events:                 # torch creates event handles lazily: do it before the timed region
            for e in evs:
                e.record(stream)
        barrier()
        sampler = ClockSampler(gpu_smi_id(torch, local)) if sample_clocks else None
        if sampler:
            sampler.__enter__()
            time.sleep(0.15)
        barrier()
        # The timed region: blocks of exactly `steps` steps, each bracketed by a barrier + synchronize and timed with
        # CUDA events on the launching stream; the block is repeated until min_ms of device time has passed
        # (every rank runs the same number of blocks: the count comes from the slowest rank's first block), so that
        # the region is long enough for the clock samples whatever `steps` the caller passed.
        blocks = []
        repeats, pos = 1, warmup
        while len(blocks) < repeats:
            start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record(stream)
            for t in range(steps):         # nothing but the steps
                comp.step_ptrs(*ptrs[(pos + t) % nsets], stream)
            stop.record(stream)
            barrier()
            pos += steps
            blocks.append(start.elapsed_time(stop) / steps)
            if len(blocks) == 1 and min_ms > 0:
                repeats = int(min(1000, max(1, -(-min_ms // max(allmax(blocks[0]) * steps, 1e-6)))))
        # per-kernel times: the same steps again, with CUDA events recorded at the phase boundaries
        # on the launching stream (the records cost a little, so they stay out of the timed region)
        for t in range(psteps):
            comp.set_phase_events(events[t])
            comp.step_ptrs(*ptrs[(pos + t) % nsets], stream)
        barrier()
        if sampler:
            sampler.__exit__(None, None, None)
        # the same step replayed from a CUDA graph (kernels only): what launch overhead is left in `ms`
        graph_ms = None
        if want_graph:
            comp.set_phase_events(None)
            comp.step_ptrs(*ptrs[0], stream)               # the captured call must repeat these pointers
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(stream)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
                comp.step_ptrs(*ptrs[0], torch.cuda.current_stream())
            stream.wait_stream(side)
            for _ in range(3):
                graph.replay()
            barrier()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(stream)
            for _ in range(steps):
                graph.replay()
            g1.record(stream)
            barrier()
            graph_ms = g0.elapsed_time(g1) / steps
            del graph
        blocks = sorted(allmax_list(blocks))      # per block: the slowest rank; then the median block
        ms = blocks[len(blocks) // 2]
        phases = [sum(events[t][i].elapsed_time(events[t][i + 1]) for t in range(psteps)) / psteps
                  for i in range(B.N_PHASES)]
        per_step = sorted(events[t][0].elapsed_time(events[t][B.N_PHASES]) for t in range(psteps))
        status = comp.status()
        # a dependent column or a zero scale is a property of the data (it happens with 2-bit codes);
        # a non-finite value or an expired wait would make the timing meaningless
        assert all(s & (B.STATUS_NONFINITE | B.STATUS_TIMEOUT) == 0 for s in status), f"device status flags: {status}"
        # the library's own figures of the last round (outside the timed region): codes that sit within one fp32 step
        # of a decision threshold, the only ones a correct implementation may code differently
        lst = [comp.step_stats(l) for l in range(len(comp.layers)) if comp.is_matrix(l)]
        n_codes = sum(x["codes_p"] + x["codes_q"] for x in lst)
        n_near = sum(x["near_p"] + x["near_q"] for x in lst)
        quantiser = {"codes": n_codes, "within_one_ulp_of_a_threshold": n_near,
                     "fraction": n_near / n_codes if n_codes else 0.0,
                     "min_pivot_ratio": min((x["pivot_ratio"] for x in lst), default=0.0),
                     "what": "last timed round, all workers, from lqsgd_step_stats"}
        out = {"ms": ms, "repeats": len(blocks), "block_ms_min_max": [blocks[0], blocks[-1]], "quantiser": quantiser,
               "phases_ms": dict(zip(B.PHASE_NAMES, phases)), "launches": comp.launches_per_step,
               "payload": comp.payload_nbytes, "clocks": sampler.summary() if sampler else None, "graph_ms": graph_ms,
               "flagged_layers": sum(1 for x in status if x),
               "profiled_step_ms": {"min": per_step[0], "median": per_step[len(per_step) // 2], "max": per_step[-1],
                                    "steps": psteps}}
        del comp
        if want_e2e:
            comp = B.LQSGD(wl_obj.layers, wl_obj.rank, wl_obj.bits, alpha=wl_obj.alpha, workers=wl_obj.workers,
                           seed=wl_obj.seed + rank, host_staging=True, device=dev)
            # host side as a trainer keeps it: one pinned flat buffer per worker (and one for G_hat), every tensor on
            # a 16-byte boundary; lqsgd_step_host then moves each buffer in a few large copies
            offs, total = [], 0
            for t in ghat:
                offs.append(total)
                total += (t.numel() + 3) // 4 * 4

            def flat_views(src):
                buf = torch.empty(total, dtype=torch.float32).pin_memory()
                views = [buf[o:o + t.numel()].view(t.shape) for o, t in zip(offs, ghat)]
                if src is not None:
                    for v, x in zip(views, src):
                        v.copy_(x)
                return views
            hg = [flat_views(per) for per in sets[0]]
            hh = flat_views(None)
            hp = torch.empty(wl_obj.workers * comp.payload_nbytes, dtype=torch.uint8).pin_memory()
            e2e_steps = max(1, min(steps, 5))
            comp.step_host(hg, hh, hp)
            barrier()
            t0 = time.perf_counter()
            for _ in range(e2e_steps):
                comp.step_host(hg, hh, hp)            # synchronises its stream before returning
            torch.cuda.synchronize()
            out["e2e_ms"] = 1e3 * (time.perf_counter() - t0) / e2e_steps
            out["h2d"] = gradient_bytes(wl_obj)
            out["d2h"] = 4 * sum(n * m for n, m in wl_obj.layers) + wl_obj.workers * comp.payload_nbytes
            del comp
        del sets, ghat
        torch.cuda.empty_cache()
        return out

    def residual_rel(wl_obj, steps):
        """||M - G_hat||_F / ||M||_F (Eq. 7: the new error buffer against what was compressed), over all 2-D
        layers and workers, at step `steps` of a fresh context."""
        comp = B.LQSGD(wl_obj.layers, wl_obj.rank, wl_obj.bits, alpha=wl_obj.alpha, workers=wl_obj.workers,
                       seed=wl_obj.seed, device=dev)
        mats = [l for l in range(len(wl_obj.layers)) if comp.is_matrix(l)]
        num = den = 0.0
        for t in range(steps):
            g = wl.draw_gradients(wl_obj, t, device=dev)
            last = t == steps - 1
            if last:
                for l in mats:
                    for w in range(wl_obj.workers):
                        den += float((g[w][l].double() + comp.get_state(B.STATE_E, l, w).double()).pow(2).sum())
            ghat = [torch.empty_like(x) for x in g[0]]
            comp.step(g, ghat)
            if last:
                for l in mats:
                    for w in range(wl_obj.workers):
                        num += float(comp.get_state(B.STATE_E, l, w).double().pow(2).sum())
        torch.cuda.synchronize()
        return (num / den) ** 0.5

    def oracle_reconstruction_error(wl_obj):
        """Part of the CPU-baseline leg (the one place this arm runs the oracle): one round of the workload on the
        device and, on the same inputs and the same Q_0, one round of the oracle running free on the host;
        returns ||G_hat - G_hat_oracle||_F / ||G_hat_oracle||_F over all matrices, the share of codes that
        differ (a code next to a decision threshold moves its entry by a whole level) and the oracle's time."""
        import numpy as np
        from oracle import lqsgd_oracle as orc
        comp = B.LQSGD(wl_obj.layers, wl_obj.rank, wl_obj.bits, alpha=wl_obj.alpha, workers=wl_obj.workers,
                       seed=wl_obj.seed, device=dev)
        mats = [l for l in range(len(wl_obj.layers)) if comp.is_matrix(l)]
        Q0 = {l: comp.get_state(B.STATE_Q, l).cpu().numpy() for l in mats}
        g = wl.draw_gradients(wl_obj, 0, device=dev)
        ghat = [torch.empty_like(x) for x in g[0]]
        comp.step(g, ghat)
        torch.cuda.synchronize()
        o = orc.Oracle(wl_obj.layers, wl_obj.rank, wl_obj.bits, wl_obj.bits, wl_obj.alpha, wl_obj.workers, Q0)
        t0 = time.perf_counter()
        out = o.step([[x.cpu().numpy() for x in per] for per in g])
        secs = time.perf_counter() - t0
        num = den = 0.0
        differ = total = 0
        for l in mats:
            d = ghat[l].cpu().numpy().astype(np.float64) - out[l]["G_hat"]
            num += float((d * d).sum())
            den += float((out[l]["G_hat"] ** 2).sum())
            for w in range(wl_obj.workers):
                for which, key in ((B.STATE_CODES_P, "xp"), (B.STATE_CODES_Q, "xq")):
                    c = comp.get_state(which, l, w).cpu().numpy()
                    differ += int((c != out[l][key]["codes"][w]).sum())
                    total += c.size
        # The same round stage by stage: every stage of the device against the oracle's stage ON THE DEVICE'S OWN INPUT
        # to that stage (how the tolerances are stated: <= 1e-4 relative Frobenius error per stage, codes equal), so
        # that one code next to a threshold does not carry over into everything computed after it.
        def rel(a, b):
            nb = float(np.linalg.norm(b))
            return float(np.linalg.norm(np.asarray(a, dtype=np.float64) - b)) / nb if nb > 0 else 0.0
        hostf = lambda which, l, w=0: comp.get_state(which, l, w).cpu().numpy()
        stage = {"P_raw": 0.0, "P": 0.0, "Q_w": 0.0, "G_hat": 0.0, "E": 0.0}
        sdiffer = 0
        for l in mats:
            n, m = wl_obj.layers[l]
            sc = hostf(B.STATE_SCALES, l)
            P_bar, Q_bar = hostf(B.STATE_P_BAR, l), hostf(B.STATE_Q, l)
            G_hat = orc.reconstruct(P_bar, Q_bar)
            stage["G_hat"] = max(stage["G_hat"], rel(ghat[l].cpu().numpy(), G_hat))
            for w in range(wl_obj.workers):
                M = orc.error_feedback(g[w][l].cpu().numpy().reshape(n, m), np.zeros((n, m)))     # E_0 = 0
                P_raw, P, Qw = hostf(B.STATE_P_RAW, l, w), hostf(B.STATE_P, l, w), hostf(B.STATE_Q_W, l, w)
                stage["P_raw"] = max(stage["P_raw"], rel(P_raw, orc.power_step_p(M, Q0[l])))
                stage["P"] = max(stage["P"], rel(P, orc.orthonormalize(P_raw)[0]))
                stage["Q_w"] = max(stage["Q_w"], rel(Qw, orc.power_step_q(M, P_bar)))
                stage["E"] = max(stage["E"], rel(hostf(B.STATE_E, l, w), orc.error_update(M, G_hat)))
                sdiffer += int((hostf(B.STATE_CODES_P, l, w) != orc.log_quantize(P, np.float32(sc[0]), wl_obj.bits, wl_obj.alpha)).sum())
                sdiffer += int((hostf(B.STATE_CODES_Q, l, w) != orc.log_quantize(Qw, np.float32(sc[1]), wl_obj.bits, wl_obj.alpha)).sum())
        near = sum(comp.step_stats(l)["near_p"] + comp.step_stats(l)["near_q"] for l in mats)
        del comp
        return {"ghat_vs_oracle_rel": (num / den) ** 0.5 if den > 0 else 0.0, "codes_differing": differ,
                "codes": total, "oracle_s": secs,
                "stage_by_stage": dict(stage, codes_differing=sdiffer, codes_within_one_ulp_of_a_threshold=near,
                                       what="max over layers and workers of the relative Frobenius error of each stage "
                                            "against the oracle's stage on the device's own input; codes from the "
                                            "device's own factors")}

    wl_obj, desc = get_workload(args.workload)
    if args.workers:
        wl_obj = dataclasses.replace(wl_obj, workers=args.workers)
        desc += f" [workers overridden: W={args.workers}]"
    gbytes = gradient_bytes(wl_obj)
    nsets_main = max(3, min(16, -(-int(2.5e8) // gbytes)))          # a rotation streams more than twice the L2
    res = bench_workload(wl_obj, args.steps, args.warmup, nsets=nsets_main, want_e2e=not args.no_e2e, sample_clocks=True,
                         want_graph=not args.no_graph, min_ms=args.min_ms, one_launch=args.one_launch)

    ms = res["ms"]
    e2e_ms = allmax(res.get("e2e_ms", float("nan")))
    value = world * gbytes / (ms * 1e-3) / 1e9
    pb = phase_bytes(wl_obj)
    dom = max(("pass1", "pass2", "pass3"), key=lambda k: res["phases_ms"][k])
    achieved = pb[dom] / (res["phases_ms"][dom] * 1e-3) / 1e9
    round_bytes = sum(v for k, v in pb.items() if k != "round")
    traffic = recorded_traffic(args.workload, dom)
    one_launch = res["launches"] == 1 and args.one_launch
    if one_launch:
        # the whole round is one kernel that reads G and E and writes E and G_hat: 12 + 4/W bytes per worker-element
        from paper_2506_17974_b200 import workloads as _wl
        nm = _wl.matrix_elements(wl_obj.layers)
        dom = "round"
        pb = dict(pb, round=12 * wl_obj.workers * nm + 4 * nm)
        res["phases_ms"] = dict(res["phases_ms"], round=ms)
        achieved = pb["round"] / (ms * 1e-3) / 1e9
        traffic = recorded_traffic(args.workload, "round")
    cfg = config_dict(wl_obj, desc)
    if args.one_launch:
        cfg["one_launch"] = bool(one_launch)
    cfg["parallelism"] = f"{world} independent replica(s), one per GPU, no collective"
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": cfg,
        "repeats": res["repeats"],
        "timed_region": {"what": f"{res['repeats']} block(s) of {args.steps} steps, each bracketed by barrier + synchronize; "
                                 "ms_per_step is the median over blocks of the per-block mean (max over ranks)",
                         "block_ms_min": res["block_ms_min_max"][0], "block_ms_max": res["block_ms_min_max"][1]},
        "gpu_launches": res["repeats"] * args.steps * res["launches"],
        "clocks": res["clocks"],
        "e2e": {"value": world * gbytes / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                "h2d_bytes_per_step": res.get("h2d"), "d2h_bytes_per_step": res.get("d2h"), "ms_per_step": e2e_ms}
        if "e2e_ms" in res else None,
        # frac: algorithmic bytes of the pass / its CUDA-event time / peak.  traffic: DRAM bytes per launch of that
        # kernel from the ncu capture summarised under profiles/ (a stored figure, not measured by this run; null when
        # the kernel's sources changed since).  frac_min_bytes counts min(stored traffic, algorithmic bytes): bytes that
        # an earlier pass left in L2 are not credited.
        "roofline": {"bound": "hbm", "kernel": kernel_name(dom, wl_obj.rank), "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                     "traffic_source": "stored: profiles/dram_traffic.json (ncu capture of this workload)" if traffic else None,
                     "frac_min_bytes": (min(traffic, pb[dom]) / (res["phases_ms"][dom] * 1e-3) / 1e9 / peak) if traffic else None,
                     "bytes_per_launch": pb[dom], "kernel_ms": res["phases_ms"][dom]},
        "round": {"algorithmic_bytes": round_bytes, "achieved_gbs": round_bytes / (ms * 1e-3) / 1e9,
                  "frac_of_peak": round_bytes / (ms * 1e-3) / 1e9 / peak, "frac_of_nominal_8tbs": round_bytes / (ms * 1e-3) / 8e12,
                  "phases_ms": res["phases_ms"], "profiled_step_ms": res["profiled_step_ms"]},
        "cuda_graph": {"ms_per_step": res["graph_ms"], "what": "one captured step replayed on one gradient set "
                       "(larger than L2); the timed `value` above uses plain launches"} if res.get("graph_ms") else None,
        "compression_ratio": 4 * sum(n * m for n, m in wl_obj.layers) / res["payload"],
        "payload_bytes_per_worker": res["payload"],
        "quantiser": res["quantiser"],
    }

    def compact(w, r):
        rb = sum(phase_bytes(w).values())
        return {"gbs_gradient": gradient_bytes(w) / (r["ms"] * 1e-3) / 1e9, "ms_per_step": r["ms"],
                "round_frac_of_peak": rb / (r["ms"] * 1e-3) / 1e9 / peak, "round_frac_of_nominal_8tbs": rb / (r["ms"] * 1e-3) / 8e12,
                "launches_per_step": r["launches"], "phases_ms": r["phases_ms"]}

    if rank == 0 and world == 1 and not args.no_sweep:
        sweep = {}
        for a, b in wl.CONFIG4_SIZES:
            w4 = wl.config4(a, b)
            # enough gradient sets that a rotation streams more than twice the L2 (126 MB) before a set returns
            nsets4 = max(2, min(16, -(-int(2.5e8) // gradient_bytes(w4))))
            r4 = bench_workload(w4, steps=max(20, 2 * nsets4), warmup=3, nsets=nsets4, want_e2e=False, sample_clocks=False,
                                min_ms=50.0)
            sweep[f"{a}x{b}"] = dict(compact(w4, r4), gradient_sets_rotated=nsets4)
        line["large_layer_sweep"] = sweep
        # the other configurations, briefly (each a few tens of ms of device time)
        others = {}
        for name in ("single", "mnist", "config5_r1_b4", "config5_r8_b4", "config5_r16_b4"):
            wo, _ = get_workload(name)
            nso = max(2, min(16, -(-int(2.5e8) // gradient_bytes(wo))))
            ro = bench_workload(wo, steps=20, warmup=3, nsets=nso, want_e2e=False, sample_clocks=False, min_ms=30.0)
            others[name] = dict(compact(wo, ro), gradient_sets_rotated=nso,
                                compression_ratio=4 * sum(n * m for n, m in wo.layers) / ro["payload"])
            if name in ("single", "mnist"):
                # the same set as ONE cooperative launch with M resident in shared memory (LQSGD_FLAG_ONE_LAUNCH)
                r1 = bench_workload(wo, steps=20, warmup=3, nsets=nso, want_e2e=False, sample_clocks=False, min_ms=30.0,
                                    one_launch=True)
                others[name]["one_launch"] = {"ms_per_step": r1["ms"], "launches_per_step": r1["launches"]}
        w4 = wl.config4(1024, 4096)
        r1 = bench_workload(w4, steps=30, warmup=3, nsets=15, want_e2e=False, sample_clocks=False, min_ms=50.0, one_launch=True)
        line["large_layer_sweep"]["1024x4096"]["one_launch"] = {"ms_per_step": r1["ms"], "launches_per_step": r1["launches"]}
        line["other_configs"] = others
    if rank == 0 and world == 1 and args.config5_sweep:
        # rank x bits grid on the 16-worker ResNet-18 (100 classes) set: throughput, compression ratio and
        # what the round loses, ||M - G_hat||_F / ||M||_F over all layers and workers at the last step
        grid = {}
        for r5 in (1, 2, 4, 8, 16):
            for b5 in (2, 3, 4, 8):
                w5 = wl.config5(r5, b5)
                r = bench_workload(w5, steps=min(args.steps, 100), warmup=3, nsets=2, want_e2e=False, sample_clocks=False)
                grid[f"r{r5}_b{b5}"] = dict(
                    compact(w5, r), compression_ratio=4 * sum(n * m for n, m in w5.layers) / r["payload"],
                    payload_bytes_per_worker=r["payload"], residual_rel=residual_rel(w5, 10),
                    layers_with_dependent_column_or_zero_scale=r["flagged_layers"])
        line["config5_sweep"] = grid
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # The CPU-baseline leg: the oracle as it stands, on the host cores, on a bounded sample.
        times, cores = time_oracle(wl_obj, budget_s=12.0, max_steps=8)
        t = sum(times) / len(times)
        line["cpu_baseline"] = {"value": gbytes / t / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{len(times)} whole rounds of the same workload, numpy fp64, "
                                          f"{t:.2f} s each"}
        # and, with the oracle's output at hand, the reconstruction error against it on points of the rank / bit grid
        # (one round each: what the rank / bit sweep asks to be reported next to the throughput)
        if not args.no_sweep:
            err = {}
            for r5, b5 in ((1, 4), (8, 4), (16, 4)):
                err[f"config5_r{r5}_b{b5}"] = oracle_reconstruction_error(wl.config5(r5, b5))
            line["cpu_baseline"]["reconstruction_error_vs_oracle"] = err
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_exchange(args):
    """Opt-in (--exchange): the workers of all ranks take part in ONE average, with the real
    exchange of Algorithm 1 between the GPUs (two MAX all-reduces of the scales and two
    all-gathers of the packed codes per step, NCCL).  Every rank simulates the workload's W
    workers, so the average is over W x n_gpus workers (weak scaling)."""
    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry
    from paper_2506_17974_b200 import binding as B
    from paper_2506_17974_b200 import distributed as D
    from paper_2506_17974_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device(dev))
    if rank == 0:
        entry.build()
    dist.barrier()
    peak, peak_kind = load_peaks()
    wl_obj, desc = get_workload(args.workload)
    def make(layers):
        return B.LQSGD(layers, wl_obj.rank, wl_obj.bits, alpha=wl_obj.alpha, workers=wl_obj.workers,
                       seed=wl_obj.seed, device=dev, world_workers=wl_obj.workers * world)
    comp = make(wl_obj.layers)
    seeded = dataclasses.replace(wl_obj, seed=wl_obj.seed + 1000 * rank)
    sets = [wl.draw_gradients(seeded, t, device=dev) for t in range(3)]
    ghat = [torch.empty_like(g) for g in sets[0][0]]
    one_round = lambda t: D.distributed_round(comp, sets[t % 3], ghat)
    if args.overlap:
        # the layer table cut in two, one context per half on its own stream: one half's collectives run under the
        # other half's streaming passes
        idx = D.split_layers(wl_obj.layers)
        halves = [make([wl_obj.layers[i] for i in part]) for part in idx]
        streams = [torch.cuda.Stream(device=dev) for _ in range(2)]
        main = torch.cuda.current_stream()

        def one_round(t):
            for s in streams:
                s.wait_stream(main)
            D.distributed_round_overlapped([(halves[h], [[per[i] for i in idx[h]] for per in sets[t % 3]], [ghat[i] for i in idx[h]])
                                            for h in range(2)], streams=streams)
            for s in streams:
                main.wait_stream(s)
    for t in range(args.warmup):
        one_round(t)
    dist.barrier()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for t in range(args.steps):
        one_round(args.warmup + t)
    stop.record()
    dist.barrier()
    torch.cuda.synchronize()
    tms = torch.tensor([start.elapsed_time(stop) / args.steps], dtype=torch.float64, device=dev)
    dist.all_reduce(tms, op=dist.ReduceOp.MAX)
    ms = float(tms.item())
    gbytes = gradient_bytes(wl_obj)
    rb = sum(phase_bytes(wl_obj).values())
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": world * gbytes / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": desc, "l2": "inputs larger than L2; 3 gradient sets rotate",
                       "parallelism": f"{wl_obj.workers} workers per GPU x {world} GPUs in one average: 2 MAX "
                                      "all-reduces of scales + 2 all-gathers of packed codes + 1 SUM all-reduce of the 1-D "
                                      "tensors per step (NCCL)" + (", layer table in two halves on two streams" if args.overlap else "")},
            "gpu_launches": args.steps * (comp.launches_per_step + 5),
            "roofline": {"bound": "hbm", "kernel": "whole round per GPU", "achieved": rb / (ms * 1e-3) / 1e9, "peak": peak,
                         "unit": "GB/s", "frac": rb / (ms * 1e-3) / 1e9 / peak, "peak_kind": f"of {peak_kind}", "traffic": None},
            "exchange_bytes_per_rank_per_step": int(comp.exchange_view(B.XCHG_STREAMS_P).numel()
                                                    + comp.exchange_view(B.XCHG_STREAMS_Q).numel()),
        }))
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18")
    ap.add_argument("--no-sweep", action="store_true", help="skip the large-layer sweep")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer (end-to-end) measurement")
    ap.add_argument("--source-digest", action="store_true",
                    help="print the digest of the kernel sources that profiles/dram_traffic.json is keyed on, and exit")
    ap.add_argument("--config5-sweep", action="store_true",
                    help="also time the rank x bits grid on the 16-worker ResNet-18 set (a few minutes)")
    ap.add_argument("--workers", type=int, default=0,
                    help="override the workload's worker count (smaller cases for profiler captures)")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay measurement")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip timing the CPU oracle")
    ap.add_argument("--min-ms", type=float, default=500.0,
                    help="repeat the block of --steps steps until this much device time has been timed (0: one block)")
    ap.add_argument("--one-launch", action="store_true",
                    help="run the round as one cooperative kernel with M resident in shared memory, if the set qualifies")
    ap.add_argument("--overlap", action="store_true",
                    help="with --exchange: the layer table cut in two halves on two streams, collectives under compute")
    ap.add_argument("--exchange", action="store_true",
                    help="workers of all GPUs in one average, with the real NCCL exchange (default: independent replicas)")
    args = ap.parse_args()
    if args.source_digest:
        for group in (["lqsgd_stream.cu", "lqsgd_stream_common.cuh", "lqsgd_dev.h"],
                      ["lqsgd_kernels.cu", "lqsgd_dev.h"],
                      ["lqsgd_tc.cu", "lqsgd_stream_common.cuh", "lqsgd_dev.h"],
                      ["lqsgd_resident.cu", "lqsgd_factor.cuh", "lqsgd_stream_common.cuh", "lqsgd_dev.h"]):
            print(" ".join(group), csrc_digest(group))
        return
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # plain `python bench.py --gpus N`: become N ranks, one per GPU, under torchrun on this node
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        os.execv(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                  f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1", "--master-port", str(port),
                                  os.path.abspath(__file__)] + sys.argv[1:])
    if args.impl == "reference":
        run_reference(args)
    elif args.exchange:
        run_exchange(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
