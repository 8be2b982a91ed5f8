"""Benchmark of the LOOK-M prefill-time KV-cache compression path on B200.

A step is one pass of the whole path (score -> select -> match -> merge/compact) over one layer
of the 8192-token, 32-head LLaVA-1.5-7B-shaped synthetic prompt (budget 20 %, window 32, merge
mode cycling averaged / pivotal / weighted).  The metric is prompt tokens x KV heads compressed
per second.  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

--impl reference times the fp64 CPU oracle, as it stands, on the host cores.
With N > 1 (launched by torch.distributed.run) every rank compresses its own replica of the
workload (layers with different seeds); there is no data-path collective.
"""
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

from paper_2406_18139_b200 import synth  # noqa: E402

METRIC = "prompt tokens*heads compressed/s per layer at 8K prompt"
UNIT = "token*heads/s"
N_INPUT_SETS = 3          # distinct layers rotated through, 192 MiB each (> the 126 MB L2)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "tflops": p["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops": 1400.0, "source": "fallback"}


def workload(args=None):
    """The 8K-prompt 7B-shape workload; --seq-len / --heads shrink it (profiling captures only)."""
    w = synth.config2(seed=0)
    if args is not None and (args.seq_len or args.heads):
        L = args.seq_len or 8192
        H = args.heads or 32
        n_img = max(1, int(0.84 * L) // synth.IMAGE_TOKENS)
        text = L - n_img * synth.IMAGE_TOKENS
        seg = [text // (n_img + 1)] * (n_img + 1)
        seg[-1] += text - sum(seg)
        r = synth.Request(L, n_img, seg, int(0.2 * L), 32, 0, synth.interleave(n_img, seg))
        w = synth.Workload("c2_shape_reduced_%dx%d" % (L, H), 2, 0, 32, H, H, 128, True, [r])
    return w


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._halt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def sample(self):
        if not self.nv:
            return
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(
                nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                     "sw_thermal_slowdown": 0x20, "hw_power_brake_slowdown": 0x80}
            for n, bit in names.items():
                if r & bit:
                    self.reasons.add(n)
        except Exception:
            pass

    def run(self):
        while not self._halt.is_set():
            self.sample()
            time.sleep(0.004)

    def stop(self):
        self._halt.set()
        self.join()
        self.sample()
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def rank_layers(rank):
    """Layers (seeds) whose inputs rank `rank` compresses: every rank gets its own replica."""
    return [rank * N_INPUT_SETS + s for s in range(N_INPUT_SETS)]


def max_over_ranks(values, world, device):
    """Element-wise maximum of a list of floats over all ranks (the job is as slow as its slowest rank)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(world, steps, units_per_step, ms):
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return world * steps * units_per_step / (ms * 1e-3)


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------

def oracle_sample(w, heads, threads, bits):
    """Times the oracle's whole path on `heads` KV heads of one layer; returns (seconds, units)."""
    from oracle import lookm_oracle as orc
    qf, kf, vf = (synth.bf16_to_f32(t) for t in bits)
    req = w.requests[0]
    t0 = time.perf_counter()
    orc.compress_layer(qf, kf, vf, req.mask, req.budget, req.window, req.merge_mode, kv_heads=heads,
                       threads=threads)
    return time.perf_counter() - t0, req.seq_len * len(heads)


def cpu_baseline(w, bits):
    from oracle import lookm_oracle as orc
    cores = orc.default_threads()
    heads = list(range(min(cores, w.n_kv_heads)))
    sec, units = oracle_sample(w, heads, cores, bits)
    return {"value": units / sec, "unit": UNIT, "cores": min(cores, len(heads)), "kind": "oracle",
            "sample": "whole path on %d of %d KV heads of one 8192-token layer, one head per thread, %.1f s"
                      % (len(heads), w.n_kv_heads, sec)}


def run_reference(args):
    """--impl reference: the fp64 oracle on the host cores; a step = one head per core."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import lookm_oracle as orc
    w = workload(args)
    cores = orc.default_threads()
    heads = list(range(min(cores, w.n_kv_heads)))
    qb, kb, vb = synth.layer_tensors(w, 0)
    qf, kf, vf = (synth.bf16_to_f32(t) for t in (qb, kb, vb))
    req = w.requests[0]

    def step(i):
        orc.compress_layer(qf, kf, vf, req.mask, req.budget, req.window, i % 3, kv_heads=heads, threads=cores)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(i)
    sec = time.perf_counter() - t0
    value = args.steps * req.seq_len * len(heads) / sec
    sample = "whole path on %d of %d KV heads of one 8192-token layer per step, one head per thread" % (
        len(heads), w.n_kv_heads)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "gpu_launches": 0,
        "config": {"workload": w.name, "seq_len": req.seq_len, "n_kv_heads": w.n_kv_heads,
                   "budget": req.budget, "window": req.window, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, len(heads)), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2406_18139_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B.lib()

    w = workload(args)
    req = w.requests[0]
    L, Hq, Hkv, budget, window = req.seq_len, w.n_q_heads, w.n_kv_heads, req.budget, req.window
    dev = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    host_sets, dev_sets, first_bits = [], [], None
    for layer in rank_layers(rank):
        qb, kb, vb = synth.layer_tensors(w, layer=layer)
        first_bits = first_bits or (qb, kb, vb)
        host_sets.append(tuple(torch.from_numpy(t.view(np.int16)).view(torch.bfloat16).pin_memory()
                               for t in (qb, kb, vb)))
        dev_sets.append(tuple(dev(t) for t in (qb, kb, vb)))
    mask_host = torch.from_numpy(req.mask).pin_memory()
    mask = mask_host.cuda()
    lay = B.make_layout(dev_sets[0][0], dev_sets[0][1])
    ws = B.alloc_workspace(lay, [L])
    out_k = torch.zeros(Hkv, budget, 128, dtype=torch.bfloat16, device="cuda")
    out_v = torch.zeros_like(out_k)

    def step(i, tensors=None):
        q, k, v = tensors if tensors is not None else dev_sets[i % N_INPUT_SETS]
        st, _ = B.lookm_compress_layer(q, k, v, mask, L, budget, window, i % 3, lay, out_k, out_v, ws)
        if st != B.OK:
            raise RuntimeError("lookm_compress_layer: " + B.lookm_strerror(st))
        return B.lookm_last_launch_count()

    def fence():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing ------------------------------------------------------------------
    # Inside the timed region only the events around the two score sweeps (the dominant kernels)
    # are recorded; every further event between two kernels costs about 2 us.  The full per-stage
    # breakdown comes from a second, untimed pass below.
    n_ev = B.N_STAGE_EVENTS
    stage_events = [[torch.cuda.Event(enable_timing=True) if s < 3 else None for s in range(n_ev)]
                    for _ in range(args.steps)]
    for evs in stage_events:
        for e in evs:
            if e is not None:
                e.record()
    for i in range(args.warmup):
        step(i)
    B.check(B.lookm_device_status(ws))
    sampler = ClockSampler(physical_gpu_index(local_rank))
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches = 0
    fence()
    sampler.start()
    t_begin.record()
    for i in range(args.steps):
        B.lookm_set_stage_events(stage_events[i])
        launches += step(i)
    t_end.record()
    fence()
    clocks = sampler.stop()
    B.lookm_set_stage_events(None)
    B.check(B.lookm_device_status(ws))
    ms_total = t_begin.elapsed_time(t_end)

    # ---- per-stage breakdown: same steps again with every stage event recorded (not timed) -----
    n_detail = max(3, min(args.steps, 20))
    detail_events = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(n_detail)]
    for evs in detail_events:
        for e in evs:
            e.record()
    fence()
    for i in range(n_detail):
        B.lookm_set_stage_events(detail_events[i])
        step(i)
    fence()
    B.lookm_set_stage_events(None)

    # ---- end to end through the public call with host buffers -----------------------------------
    # Every step copies its inputs from pinned host memory, compresses, and copies the compacted
    # cache back.  The three phases run on three streams with two sets of staging buffers, so
    # the upload of step i + 1 and the download of step i - 1 overlap the kernels of step i (the
    # PCIe link carries 201 MB up and 27 MB down per step and is the limit).
    n_sets = 2
    stage = [tuple(torch.empty_like(t) for t in dev_sets[0]) + (torch.empty_like(mask),) for _ in range(n_sets)]
    outs = [(torch.zeros_like(out_k), torch.zeros_like(out_v)) for _ in range(n_sets)]
    host_out = [(torch.empty(out_k.shape, dtype=out_k.dtype).pin_memory(),
                 torch.empty(out_v.shape, dtype=out_v.dtype).pin_memory()) for _ in range(n_sets)]
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    in_ready = [torch.cuda.Event() for _ in range(n_sets)]
    run_done = [torch.cuda.Event() for _ in range(n_sets)]
    out_done = [torch.cuda.Event() for _ in range(n_sets)]

    def e2e_step(i):
        b = i % n_sets
        hq, hk, hv = host_sets[i % N_INPUT_SETS]
        sq, sk, sv, sm = stage[b]
        with torch.cuda.stream(s_in):
            s_in.wait_event(run_done[b])                 # the kernels that read this set are done
            sq.copy_(hq, non_blocking=True); sk.copy_(hk, non_blocking=True)
            sv.copy_(hv, non_blocking=True); sm.copy_(mask_host, non_blocking=True)
            in_ready[b].record(s_in)
        with torch.cuda.stream(s_run):
            s_run.wait_event(in_ready[b])
            s_run.wait_event(out_done[b])                # its previous result has left the device
            st, _ = B.lookm_compress_layer(sq, sk, sv, sm, L, budget, window, i % 3, lay, outs[b][0], outs[b][1], ws)
            if st != B.OK:
                raise RuntimeError("lookm_compress_layer: " + B.lookm_strerror(st))
            run_done[b].record(s_run)
        with torch.cuda.stream(s_out):
            s_out.wait_event(run_done[b])
            host_out[b][0].copy_(outs[b][0], non_blocking=True); host_out[b][1].copy_(outs[b][1], non_blocking=True)
            out_done[b].record(s_out)

    e2e_steps = max(3, min(args.steps, 20))
    for i in range(2):
        e2e_step(i)
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fence()
    e_begin.record()
    for st_ in (s_in, s_run, s_out):
        st_.wait_event(e_begin)
    for i in range(e2e_steps):
        e2e_step(i)
    cur = torch.cuda.current_stream()
    for ev in out_done + run_done + in_ready:
        cur.wait_event(ev)
    e_end.record()
    fence()
    e2e_ms = e_begin.elapsed_time(e_end)
    B.check(B.lookm_device_status(ws))
    # the last step's download must equal what the device holds
    last = (e2e_steps - 1) % n_sets
    if not torch.equal(host_out[last][0], outs[last][0].cpu()):
        raise RuntimeError("end-to-end result differs from the device result")

    ms_total, e2e_ms = max_over_ranks([ms_total, e2e_ms], world, "cuda")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    units_per_step = L * Hkv
    value = job_throughput(world, args.steps, units_per_step, ms_total)
    stage_ms = np.zeros(n_ev - 1)
    for evs in detail_events:
        for s in range(n_ev - 1):
            stage_ms[s] += evs[s].elapsed_time(evs[s + 1])
    stage_ms /= n_detail
    # the two sweeps as timed inside the timed region (these feed the roofline)
    for s in range(2):
        stage_ms[s] = sum(evs[s].elapsed_time(evs[s + 1]) for evs in stage_events) / args.steps
    peaks = measured_peaks()
    d = w.head_dim
    sweep_flops = float(d) * L * (L + 1) * Hq                 # one causal QK^T over all query heads
    match_flops = 2.0 * (L - budget) * budget * d * Hkv
    merge_bytes = float(L + budget) * d * 2 * 2 * Hkv
    names = B.STAGE_NAMES
    stages = {}
    for s, n in enumerate(names):
        stages[n] = {"ms": round(float(stage_ms[s]), 4)}
    for n in ("score_sweep1", "score_sweep2"):
        tf = sweep_flops / (stages[n]["ms"] * 1e-3) / 1e12
        stages[n].update({"tflops": round(tf, 1), "frac_of_%s_bf16" % peaks["source"]: round(tf / peaks["tflops"], 4)})
    tf = match_flops / (stages["match"]["ms"] * 1e-3) / 1e12
    stages["match"].update({"tflops": round(tf, 1), "frac_of_%s_bf16" % peaks["source"]: round(tf / peaks["tflops"], 4)})
    gbs = merge_bytes / (stages["merge"]["ms"] * 1e-3) / 1e9
    stages["merge"].update({"gbs": round(gbs, 1), "frac_of_%s_hbm" % peaks["source"]: round(gbs / peaks["hbm_gbs"], 4)})
    dom = max(("score_sweep1", "score_sweep2"), key=lambda n: stages[n]["ms"])
    achieved = sweep_flops / (stages[dom]["ms"] * 1e-3) / 1e12
    # DRAM traffic per launch of the dominant kernel: dram__bytes_read + write of one ncu capture
    # on the 4096-token x 16-head case (profiles/tile_kernels_4096x16.txt), scaled by tokens x heads
    # (the kernels read Q and K once from DRAM and re-read tiles from L2, so traffic grows with
    # the input size).  Must be set to None when the tile kernels change after the capture.
    captured = {"score_sweep1": 33.594624e6, "score_sweep2": 35.689984e6}
    traffic = captured[dom] * (L * Hq) / (4096.0 * 16.0)
    roofline = {"kernel": "tile_kernel<%s>" % dom, "bound": "tensor", "achieved": round(achieved, 2),
                "peak": peaks["tflops"], "peak_source": peaks["source"] + " (cuBLAS bf16, sustained)",
                "unit": "TFLOP/s", "frac": round(achieved / peaks["tflops"], 4), "traffic": traffic,
                "traffic_unit": "bytes per launch (ncu capture of a 4096x16 case, scaled)"}
    e2e_value = job_throughput(world, e2e_steps, units_per_step, e2e_ms)
    h2d = sum(t.numel() * t.element_size() for t in host_sets[0]) + mask_host.numel()
    d2h = (out_k.numel() + out_v.numel()) * 2
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "seq_len": L, "n_q_heads": Hq, "n_kv_heads": Hkv, "head_dim": d,
                   "budget": budget, "window": window, "merge_mode": "average/pivotal/weighted by step",
                   "l2": "inputs rotate over %d layers of 192 MiB each, larger than L2" % N_INPUT_SETS,
                   "parallelism": "replicas x%d" % world},
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
        "roofline": roofline, "stages": stages,
        "stages_note": "sweeps timed inside the timed region; other stages from a second pass with all stage events",
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w, first_bits)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--seq-len", type=int, default=0, help="reduced prompt length (profiling only)")
    ap.add_argument("--heads", type=int, default=0, help="reduced head count (profiling only)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 60 if args.impl == "ours" else 5
    if args.warmup is None:
        args.warmup = 5 if args.impl == "ours" else 1
    if args.impl == "ours":
        args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
