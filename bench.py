#!/usr/bin/env python
"""Benchmark of the LoRDS dequantize-and-multiply hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--case NAME]

A *step* is one pass of the whole hot path (unpack, level lookup, scale reconstruction,
Hadamard product, contraction, epilogue) over one batch of synthetic layers: `rounds` rounds over
`copies` distinct weight sets of the case's shape, one forward call each, so that a round touches
more than twice the L2 capacity and every launch reads its weights from HBM.  `rounds` is chosen
from a short calibration so that the K timed steps together last about a second whatever K is: the
clock sampler then has samples and the tensor-bound case runs at sustained clocks.

The headline case is the Llama-3-8B q_proj decode (m = n = 4096, NF4, r = 32, M = 1) and
the headline metric is algorithmic HBM bytes per second (packed Q + B + A + x + y).  The
other cases (M = 8, the 3-bit MLP shapes, the M = 2048 prefill) are reported under "cases".

With N > 1 (torchrun) every rank runs the same workload on its own GPU: the path has no
exchange step, so the ranks are independent replicas ("weak" scaling, no collective on the
data path); the time is the max over ranks and the value the sum of all ranks' bytes.

`--impl reference` times the fp64 CPU oracle (the only reference implementation there is)
on the host cores, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1024 * 1024

# name -> (m, n, bits, r, M, outlier_frac, bound)
CASES = {
    "decode_q_m1":    dict(m=4096, n=4096, bits=4, r=32, M=1, outliers=0.0, bound="hbm"),
    "decode_q_m8":    dict(m=4096, n=4096, bits=4, r=32, M=8, outliers=0.0, bound="hbm"),
    "mlp3_gate_m1":   dict(m=14336, n=4096, bits=3, r=48, M=1, outliers=0.0, bound="hbm"),
    "mlp3_down_m1":   dict(m=4096, n=14336, bits=3, r=48, M=1, outliers=0.0, bound="hbm"),
    "mlp3_down_m16":  dict(m=4096, n=14336, bits=3, r=48, M=16, outliers=0.0, bound="hbm"),
    "prefill_m2048":  dict(m=4096, n=14336, bits=4, r=32, M=2048, outliers=0.01, bound="tensor"),
}
# the step before the path (Alg. 1, step 2.1) on the same shapes: name -> (m, n, r, bits)
QUANTIZE_CASES = {"quantize_q_nf4": (4096, 4096, 32, 4), "quantize_gate_nf3": (14336, 4096, 48, 3)}
# the backward with the codes fixed (Sec. 3.4): name -> (m, n, r, bits, M)
BACKWARD_CASES = {"backward_q_m512": (4096, 4096, 32, 4, 512)}
HEADLINE = "decode_q_m1"
METRIC = "LoRDS dequant-GEMM: HBM GB/s at M=1, TFLOP/s at M=2048, % of roofline"


def algorithmic_bytes(c):
    """Packed Q + B + A + x + y, each moved once."""
    return c["m"] * c["n"] * c["bits"] // 8 + 2 * c["r"] * (c["m"] + c["n"]) + 2 * c["M"] * (c["n"] + c["m"])


def useful_flops(c):
    return 2 * c["M"] * c["m"] * c["n"]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised
# under profiles/ (None until a capture of that case exists).
NCU_TRAFFIC_BYTES = {
    "decode_q_m1": 8976640,         # profiles/decode_kernel_decode_q_m1.md
    "decode_q_m8": 9029632,         # profiles/decode16_kernel_decode_q_m8_down_m16.md
    "mlp3_gate_m1": 23850496,       # profiles/decode_kernel_mlp3_gate_m1_down_m1.md
    "mlp3_down_m1": 23938560,       # same
    "mlp3_down_m16": 24299520,      # profiles/decode16_kernel_decode_q_m8_down_m16.md
    "prefill_m2048": 145443072,     # profiles/umma_kernel_prefill_m2048.md (the scale-MMA kernel; the pre-pass moves 73.7 MB more)
    "quantize_q_nf4": 34120448,     # profiles/quantize_kernel_q_nf4_gate_nf3.md (8.4 MB of codes were still in L2 at the end)
    "quantize_gate_nf3": 130577408,
    "backward_q_m512": 19691008,    # profiles/backward_tc_kernel_backward_q_m512.md (the factor-gradient kernel)
}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.splitlines():
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(ms, device, world):
    """A job's step time is that of its slowest rank: MAX-reduce the per-rank device time."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(per_rank_value, world):
    """Replicas only: every rank processes the same amount of work, so the job's throughput is the
    per-rank throughput (at the slowest rank's time) times the number of ranks."""
    return per_rank_value * world


def make_case_layers(case, copies, device):
    """One host-seeded layer per case; the other weight copies are row-rotations of it
    (distinct HBM addresses, same statistics), built on the device."""
    import numpy as np
    import torch
    from paper_2601_22716_b200 import binding as lords
    from paper_2601_22716_b200 import inputs as gen

    c = CASES[case]
    lay = gen.make_layer(c["m"], c["n"], c["r"], c["M"], bits=c["bits"], seed=0, outlier_frac=c["outliers"])
    packed = lords.lords_pack_codes(lay.codes, c["bits"])
    q0 = torch.from_numpy(packed).to(device)
    B0 = torch.from_numpy(lay.B.view(np.int16)).to(device)
    A0 = torch.from_numpy(lay.A.view(np.int16)).to(device)
    x0 = torch.from_numpy(lay.x.view(np.int16)).to(device)
    sets = []
    for l in range(copies):
        if l == 0:
            sets.append((q0, B0, A0, x0))
        else:
            sets.append((torch.roll(q0, l, 0).contiguous(), torch.roll(B0, l, 0).contiguous(),
                         A0.clone(), x0.clone()))
    return lay, packed, sets


def copies_for(case):
    c = CASES[case]
    per = algorithmic_bytes(c)
    return max(2, -(-2 * L2_BYTES // per) + 1)


MIN_TIMED_SECONDS = 1.0   # the K timed steps together last at least about this long


def time_case(case, steps, warmup, device, rank, world, sampler=None, do_e2e=True, min_seconds=MIN_TIMED_SECONDS):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2601_22716_b200 import binding as lords

    c = CASES[case]
    copies = copies_for(case)
    lay, packed, sets = make_case_layers(case, copies, device)
    M, m, n, r, bits = c["M"], c["m"], c["n"], c["r"], c["bits"]
    ys = [torch.zeros((M, m), dtype=torch.int16, device=device) for _ in range(copies)]

    def one_step():
        for (q, B, A, x), y in zip(sets, ys):
            lords.lords_linear_forward_bits(x, q, B, A, lay.codebook, bits, M, m, n, r, y)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    one_step()
    torch.cuda.synchronize()
    launches_per_call = lords.lords_last_launch_count()
    path = lords.lords_last_path()

    # capture one step in a CUDA graph (launch-bound inner loop); warm up on a side stream first
    graph = None
    try:
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            one_step()
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            one_step()
        graph = g
    except Exception as e:  # capture is an optimisation, not a requirement
        print(f"[bench] CUDA graph capture unavailable ({type(e).__name__}: {e}); launching directly",
              file=sys.stderr)
        torch.cuda.synchronize()

    one_round = (graph.replay if graph is not None else one_step)
    # calibration: rounds per step so that `steps` steps take about min_seconds (all ranks agree on the
    # slowest rank's figure)
    for _ in range(3):
        one_round()
    torch.cuda.synchronize()
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record()
    for _ in range(3):
        one_round()
    c1.record()
    torch.cuda.synchronize()
    round_ms = max_over_ranks(c0.elapsed_time(c1) / 3.0, device, world)
    rounds = int(max(1, min(100000, -(-min_seconds * 1e3 // max(steps * round_ms, 1e-6)))))

    def run():
        for _ in range(rounds):
            one_round()

    for _ in range(max(warmup, 3)):
        run()
    # A device-side status (a bounded wait that gave up) invalidates the measurement: it is reported
    # and the measurement taken once more; a second one is an error.
    status_retries = 0
    while True:
        barrier()
        if sampler is not None:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(steps):
            run()
        e1.record()
        barrier()
        clocks = sampler.stop() if sampler is not None else None
        ms = max_over_ranks(e0.elapsed_time(e1), device, world)
        ms_per_step = ms / steps
        status = lords.lords_poll_status()
        if status == 0:
            break
        d0, d1 = lords.lords_read_status_detail()
        print(f"[bench] device status {status} during {case} (first expired wait: tag {d0 & 0xFF}, parity {(d0 >> 8) & 1}, "
              f"warp {(d0 >> 16) & 0xFF}, CTA {(d0 >> 32) & 0x7FFFFFFF}, barrier 0x{d1 & 0xFFFFFFFF:x}, "
              f"{d1 >> 32} rounds of 64 tries); measuring once more", file=sys.stderr)
        status_retries += 1
        if status_retries > 1:
            raise RuntimeError(f"device status {status} during {case}, twice")

    # end to end through the host-buffer entry point: H2D of x and D2H of y inside the timed region
    e2e = None
    if do_e2e:
        xh = [torch.from_numpy(lay.x.view(np.int16)).clone().pin_memory() for _ in range(copies)]
        yh = [torch.zeros((M, m), dtype=torch.int16).pin_memory() for _ in range(copies)]

        def e2e_round():
            for (q, B, A, _x), xx, yy in zip(sets, xh, yh):
                lords.lords_linear_forward_host(xx, q, B, A, lay.codebook, bits, M, m, n, r, yy)

        for _ in range(3):
            e2e_round()
        torch.cuda.synchronize()
        # the host-buffer calls are stream-ordered, so a round of them (copy in, kernel, copy out, per call)
        # is captured once and replayed like the device-resident round above: every replay copies
        # every x from pinned host memory and every y back
        e2e_graph = None
        if graph is not None:
            try:
                s2 = torch.cuda.Stream()
                s2.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(s2):
                    e2e_round()
                torch.cuda.current_stream().wait_stream(s2)
                torch.cuda.synchronize()
                g2 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g2):
                    e2e_round()
                e2e_graph = g2
            except Exception as e:
                print(f"[bench] CUDA graph capture of the host-buffer round unavailable ({type(e).__name__}: {e})",
                      file=sys.stderr)
                torch.cuda.synchronize()
        one_e2e_round = e2e_graph.replay if e2e_graph is not None else e2e_round

        def e2e_step():
            for _ in range(rounds):
                one_e2e_round()

        for _ in range(3):
            one_e2e_round()
        barrier()
        e0.record()
        e2e_steps = max(1, min(steps, int(2.0 / (rounds * copies * 30e-6)) or 1))
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        ems = max_over_ranks(e0.elapsed_time(e1), device, world)
        e2e = {"ms_per_step": ems / e2e_steps, "h2d_bytes_per_step": rounds * copies * M * n * 2,
               "d2h_bytes_per_step": rounds * copies * M * m * 2, "steps": e2e_steps, "cuda_graph": e2e_graph is not None}
        if e2e_graph is not None:
            # the replayed copies really ran: the last y of the round equals the device-resident result
            torch.cuda.synchronize()
            assert torch.equal(yh[-1], ys[-1].cpu()), "host-buffer round did not reproduce the device result"


    peaks = measured_peaks()
    calls = copies * rounds
    us_per_launch = ms_per_step * 1e3 / calls
    byt, flo = algorithmic_bytes(c), useful_flops(c)
    gbs = byt / (us_per_launch * 1e-6) / 1e9
    tfs = flo / (us_per_launch * 1e-6) / 1e12
    if c["bound"] == "hbm":
        roof = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBs": gbs / 8000.0}
    else:
        # the kernel is timed inside a loop of about a second: the matching denominator is the library GEMM
        # measured the same way (sustained under the power cap); a loop far shorter takes the burst figure
        long_loop = ms_per_step * steps >= 300.0
        peak = peaks["bf16_tflops_sustained"] if long_loop else peaks["bf16_tflops"]
        roof = {"bound": "tensor", "achieved": tfs, "peak": peak, "unit": "TFLOP/s",
                "peak_kind": "sustained" if long_loop else "burst", "frac": tfs / peak,
                "frac_of_burst": tfs / peaks["bf16_tflops"], "frac_of_sustained": tfs / peaks["bf16_tflops_sustained"],
                "frac_of_nominal_2.25PF": tfs / 2250.0}
    roof["peak_source"] = peaks["source"]
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(case)
    roof["algorithmic_bytes_per_launch"] = byt
    roof["us_per_launch"] = us_per_launch
    res = {
        "case": case, "path": path, "copies": copies, "rounds": rounds, "ms_per_step": ms_per_step, "us_per_call": us_per_launch,
        "gbs": whole_job_value(gbs, world), "tflops": whole_job_value(tfs, world), "roofline": roof, "clocks": clocks,
        "launches_per_call": launches_per_call, "gpu_launches": steps * calls * launches_per_call,
        "graph": graph is not None, "status_retries": status_retries,
    }
    if e2e is not None:
        eus = e2e["ms_per_step"] * 1e3 / calls
        e2e["gbs"] = byt / (eus * 1e-6) / 1e9 * world
        e2e["tflops"] = flo / (eus * 1e-6) / 1e12 * world
        res["e2e"] = e2e
    res["_lay"] = (lay, packed)
    return res


STACK_LAYERS = ["q", "k", "v", "o", "gate", "up", "down"]


def time_stack(M, mlp_bits, steps, device, qkv_one_call=False, gate_up_one_call=False):
    """Full Llama-3-8B linear stack: 32 layers x {q, k, v, o, gate, up, down}, one forward call per
    module (224 calls) from one CUDA graph.  Attention modules are NF4 (r = 32; r = 16 for k/v); the
    MLP modules are NF4 r = 32, NF3 r = 48 or NF2 r = 32 (the NF4/NF2 layer mix of the paper's low-bit setting).  Each of the 224 modules has its own weights (3.5 GB
    at 4 bits: far beyond L2) and its own activations.

    qkv_one_call / gate_up_one_call: the projections of a block that read the same activations go through
    one call as one layer (rows and ranks concatenated, B block-diagonal: packing.concat_layers) -- 160 or
    128 calls; bytes and flops are still counted per original module."""
    import dataclasses

    import numpy as np
    import torch
    from paper_2601_22716_b200 import binding as lords
    from paper_2601_22716_b200 import inputs as gen
    from paper_2601_22716_b200 import packing

    lays = {}
    for idx, name in enumerate(STACK_LAYERS):
        m, n = gen.LLAMA3_8B_SHAPES[name]
        mlp = name in ("gate", "up", "down")
        bits = mlp_bits if mlp else 4
        r = (48 if bits == 3 else 32) if mlp else (16 if name in ("k", "v") else 32)
        lays[name] = gen.make_layer(m, n, r, M, bits=bits, seed=idx)
    byt = flo = 0
    for lay in lays.values():
        c = dict(m=lay.m, n=lay.n, bits=lay.bits, r=lay.r, M=M)
        byt += 32 * algorithmic_bytes(c)
        flo += 32 * useful_flops(c)
    modules = list(STACK_LAYERS)
    groups = []
    if qkv_one_call:
        groups.append(("qkv", ("q", "k", "v")))
    if gate_up_one_call:
        groups.append(("gate_up", ("gate", "up")))
    for joined, names in groups:
        parts = [lays.pop(k) for k in names]
        codes, Bc, Ac = packing.concat_layers([p.codes for p in parts], [p.B for p in parts], [p.A for p in parts])
        lays[joined] = dataclasses.replace(parts[0], m=codes.shape[0], r=Ac.shape[0], codes=codes, B=Bc, A=Ac)
        at = modules.index(names[0])
        modules = modules[:at] + [joined] + modules[at + len(names):]
    protos = {}
    for name in modules:
        lay = lays[name]
        packed = lords.lords_pack_codes(lay.codes, lay.bits)
        protos[name] = (lay, torch.from_numpy(packed).to(device), torch.from_numpy(lay.B.view(np.int16)).to(device),
                        torch.from_numpy(lay.A.view(np.int16)).to(device), torch.from_numpy(lay.x.view(np.int16)).to(device))
    calls = []
    for layer in range(32):
        for name in modules:
            lay, q0, B0, A0, x0 = protos[name]
            q = q0 if layer == 0 else torch.roll(q0, layer, 0).contiguous()
            B = B0 if layer == 0 else torch.roll(B0, layer, 0).contiguous()
            y = torch.zeros((M, lay.m), dtype=torch.int16, device=device)
            calls.append((lay, q, B, A0.clone(), x0.clone(), y))

    def one_pass():
        for lay, q, B, A, x, y in calls:
            lords.lords_linear_forward_bits(x, q, B, A, lay.codebook, lay.bits, M, lay.m, lay.n, lay.r, y)

    one_pass()
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        one_pass()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        one_pass()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    status_retries = 0
    while True:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        status = lords.lords_poll_status()
        if status == 0:
            break
        print(f"[bench] device status {status} during the M = {M} stack; measuring once more", file=sys.stderr)
        status_retries += 1
        if status_retries > 1:
            raise RuntimeError(f"device status {status} during the M = {M} stack, twice")
    peaks = measured_peaks()
    gbs, tfs = byt / (ms * 1e-3) / 1e9, flo / (ms * 1e-3) / 1e12
    return {"case": f"stack_m{M}_mlp{mlp_bits}bit" + ("_qkv_one_call" if qkv_one_call else "") + ("_gate_up_one_call" if gate_up_one_call else ""),
            "ms_per_pass": ms, "ms_per_token": ms / M, "calls": len(calls),
            "algorithmic_bytes": byt, "gbs": gbs, "tflops": tfs, "frac_hbm": gbs / peaks["hbm_gbs"],
            "frac_tensor": tfs / peaks["bf16_tflops"], "steps": steps, "status_retries": status_retries}


def time_quantize(name, m, n, r, bits, device, min_seconds=0.3):
    """The step before the path (Alg. 1, step 2.1): weights -> packed codes on the device.  HBM-bound:
    algorithmic bytes = W (bf16) + packed codes + B + A, each moved once."""
    import numpy as np
    import torch
    from paper_2601_22716_b200 import binding as lords
    from paper_2601_22716_b200 import inputs as gen

    lay = gen.make_layer(m, n, r, 1, bits=bits, seed=0)
    byt = 2 * m * n + m * n * bits // 8 + 2 * r * (m + n)
    copies = max(2, -(-2 * L2_BYTES // byt) + 1)
    W0 = torch.from_numpy(gen.make_weight(m, n, seed=1).view(np.int16)).to(device)
    B0 = torch.from_numpy(lay.B.view(np.int16)).to(device)
    A0 = torch.from_numpy(lay.A.view(np.int16)).to(device)
    sets = [(torch.roll(W0, l, 0).contiguous(), torch.roll(B0, l, 0).contiguous(), A0.clone(),
             torch.empty(m * n * bits // 8, dtype=torch.uint8, device=device)) for l in range(copies)]

    def one_round():
        for W, B, A, Q in sets:
            lords.lords_quantize_codes(W, B, A, lay.codebook, bits, m, n, r, Q)

    one_round()
    torch.cuda.synchronize()
    path = lords.lords_last_path()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        one_round()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        one_round()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    reps = int(max(3, min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)))
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps / copies
    status = lords.lords_poll_status()
    peaks = measured_peaks()
    gbs = byt / (us * 1e-6) / 1e9
    return {"case": name, "path": path, "us_per_call": us, "gbs": gbs, "tflops": None, "copies": copies, "rounds": reps,
            "steps": 1, "status_retries": 0 if status == 0 else 1,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": NCU_TRAFFIC_BYTES.get(name),
                         "algorithmic_bytes_per_launch": byt, "us_per_launch": us}}


# fp32 FMA throughput of the CUDA cores: 148 SMs x 128 lanes x 2 flops at the 1965 MHz boost clock
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def time_backward(name, m, n, r, bits, M, device, min_seconds=0.3):
    """The backward with the codes fixed (Sec. 3.4) on one layer shape: dx = g W^ on the forward
    kernels (transposed codes, made once outside the timed region; the per-call transposition of the
    factors inside it), then dB and dA on the CUDA cores.  Reported separately."""
    import numpy as np
    import torch
    from paper_2601_22716_b200 import binding as lords
    from paper_2601_22716_b200 import inputs as gen

    lay = gen.make_layer(m, n, r, M, bits=bits, seed=0)
    q = torch.from_numpy(lords.lords_pack_codes(lay.codes, bits)).to(device)
    qt = torch.empty(lords.lords_packed_bytes(n, m, bits), dtype=torch.uint8, device=device)
    lords.lords_transpose_codes(q, bits, m, n, qt)
    B = torch.from_numpy(lay.B.view(np.int16)).to(device)
    A = torch.from_numpy(lay.A.view(np.int16)).to(device)
    x = torch.from_numpy(lay.x.view(np.int16)).to(device)
    g = torch.from_numpy(gen.make_layer(m, m, 1, M, bits=4, seed=1).x[:, :m].copy().view(np.int16)).to(device)
    dx = torch.zeros((M, n), dtype=torch.int16, device=device)
    dB = torch.zeros((m, r), dtype=torch.float32, device=device)
    dA = torch.zeros((r, n), dtype=torch.float32, device=device)
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        path = lords.lords_last_path()
        total, reps = 0.0, 0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        while reps < 1 or (total < min_seconds * 1e3 / 2 and reps < 200):
            flush.zero_()                      # L2 flush between timed calls (a write larger than L2)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1)
            reps += 1
        return total / reps * 1e3, path, reps

    us_dx, path_dx, reps_dx = timed(lambda: lords.lords_linear_backward_input(g, qt, B, A, lay.codebook, bits, M, m, n, r, dx))
    us_f, path_f, reps_f = timed(lambda: lords.lords_linear_backward_factors(g, x, q, B, A, lay.codebook, bits, M, m, n, r, dB, dA))
    # the straight-through gradients of quantisation-aware training (Eq. 4-5) on the same layer: dW, dB, dA
    Wd = torch.from_numpy(gen.make_weight(m, n, seed=2).view(np.int16)).to(device)
    dW = torch.zeros((m, n), dtype=torch.float32, device=device)
    us_q, path_q, _ = timed(lambda: lords.lords_linear_backward_qat(g, x, Wd, q, B, A, lay.codebook, bits, M, m, n, r, dW, dB, dA))
    status = lords.lords_poll_status()
    peaks = measured_peaks()
    flops = 2.0 * M * m * n
    tf_dx = flops / (us_dx * 1e-6) / 1e12
    # CUDA-core work of the factor gradients: the two folds and the level multiply; with the schedules that
    # form g^T x on the CUDA cores as well, that product too (once: one CTA per tile of W)
    alu_flops = 4.0 * m * n * r + m * n + (0.0 if path_f == "backward_tensor" else flops)
    tf_f = alu_flops / (us_f * 1e-6) / 1e12
    return {"case": name, "path": f"{path_dx}+{path_f}", "us_per_call": us_dx + us_f, "gbs": None, "tflops": None,
            "copies": 1, "rounds": reps_dx, "steps": 1, "status_retries": 0 if status == 0 else 1,
            "input_gradient": {"us": us_dx, "path": path_dx, "tflops": tf_dx,
                               "roofline": {"bound": "tensor", "achieved": tf_dx, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                            "frac": tf_dx / peaks["bf16_tflops"], "peak_kind": "burst", "traffic": None}},
            "factor_gradients": {"us": us_f, "path": path_f, "alu_tflops": tf_f,
                                 "tile_product_tflops": flops / (us_f * 1e-6) / 1e12,
                                 "tile_product_on": "tensor cores" if path_f == "backward_tensor" else "CUDA cores"},
            "qat_gradients": {"us": us_q, "path": path_q},
            "roofline": {"bound": "alu", "achieved": tf_f, "peak": FP32_ALU_TFLOPS, "unit": "TFLOP/s",
                         "frac": tf_f / FP32_ALU_TFLOPS, "peak_source": "148 SMs x 128 fp32 lanes x 2 flops x 1.965 GHz",
                         "traffic": NCU_TRAFFIC_BYTES.get(name), "us_per_launch": us_f}}


def time_comparators(device, min_seconds=0.25):
    """Sec. 4.4 / Table 6 restated on this GPU, q_proj shape at one token: the LoRDS layer (r = 32) against a
    block-scaled NF4 layer (block 64: the same number of scale parameters) and against that layer with an
    additive rank-32 adapter, each replayed from a CUDA graph over distinct weight copies."""
    import numpy as np
    import torch
    from paper_2601_22716_b200 import binding as lords
    from paper_2601_22716_b200 import inputs as gen

    m = n = 4096
    M, r, blk, bits = 1, 32, 64, 4
    copies = copies_for("decode_q_m1")
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=0)
    blay, s = gen.make_blockwise_layer(m, n, blk, M, bits=bits, seed=0)
    g = torch.Generator().manual_seed(3)
    Al = torch.from_numpy(gen.bf16_bits(torch.randn(r, n, generator=g) * 0.05).view(np.int16)).to(device)
    Bl = torch.from_numpy(gen.bf16_bits(torch.randn(m, r, generator=g) * 0.05).view(np.int16)).to(device)
    q0 = torch.from_numpy(lords.lords_pack_codes(lay.codes, bits)).to(device)
    B = torch.from_numpy(lay.B.view(np.int16)).to(device)
    A = torch.from_numpy(lay.A.view(np.int16)).to(device)
    sd = torch.from_numpy(s.view(np.int16)).to(device)
    x = torch.from_numpy(lay.x.view(np.int16)).to(device)
    qs = [q0 if l == 0 else torch.roll(q0, l, 0).contiguous() for l in range(copies)]
    ys = [torch.zeros((M, m), dtype=torch.int16, device=device) for _ in range(copies)]
    variants = {
        "lords_r32": lambda q, y: lords.lords_linear_forward_bits(x, q, B, A, lay.codebook, bits, M, m, n, r, y),
        "blockscale_nf4_b64": lambda q, y: lords.lords_blockscale_forward(x, q, sd, lay.codebook, bits, blk, M, m, n, y),
        "blockscale_nf4_b64_plus_adapter_r32":
            lambda q, y: lords.lords_adapter_forward(x, q, sd, Al, Bl, lay.codebook, bits, blk, M, m, n, r, y),
    }
    out = {}
    for name, fn in variants.items():
        def one_round():
            for q, y in zip(qs, ys):
                fn(q, y)
        one_round()
        torch.cuda.synchronize()
        path = lords.lords_last_path()
        st = torch.cuda.Stream()
        st.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(st):
            one_round()
        torch.cuda.current_stream().wait_stream(st)
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            one_round()
        for _ in range(3):
            gr.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        gr.replay()
        e1.record()
        torch.cuda.synchronize()
        reps = int(max(3, min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)))
        e0.record()
        for _ in range(reps):
            gr.replay()
        e1.record()
        torch.cuda.synchronize()
        out[name] = {"us_per_call": e0.elapsed_time(e1) * 1e3 / reps / copies, "path": path}
    base = out["lords_r32"]["us_per_call"]
    return {"case": "compare_q_m1", "shape": "q_proj 4096x4096 NF4, one token", "variants": out,
            "adapter_over_lords": out["blockscale_nf4_b64_plus_adapter_r32"]["us_per_call"] / base,
            "blockscale_over_lords": out["blockscale_nf4_b64"]["us_per_call"] / base,
            "status_retries": 0 if lords.lords_poll_status() == 0 else 1}


def run_sweep(device):
    """The measurement behind the per-M choice of kernel: every tensor-core path that accepts the
    shape, at M in {1, 2, 3, 4, 8, 16}, on the q_proj (NF4, r = 32), gate and down (NF3, r = 48) shapes.
    Microseconds per forward call, graph replay over distinct weight sets as in the main measurement."""
    from paper_2601_22716_b200 import binding as lords
    shapes = [("q_proj 4096x4096 NF4 r=32", dict(m=4096, n=4096, bits=4, r=32)),
              ("gate 14336x4096 NF3 r=48", dict(m=14336, n=4096, bits=3, r=48)),
              ("down 4096x14336 NF3 r=48", dict(m=4096, n=14336, bits=3, r=48))]
    paths = ["decode", "decode16", "umma"]
    rows = []
    for label, shp in shapes:
        for M in (1, 2, 3, 4, 8, 16):
            CASES["_sweep"] = dict(shp, M=M, outliers=0.0, bound="hbm")
            entry = {"shape": label, "M": M}
            for path in paths:
                lords.lords_set_option("path", path)
                try:
                    r = time_case("_sweep", 5, 3, device, 0, 1, None, do_e2e=False, min_seconds=0.12)
                    r.pop("_lay")
                    entry[path] = round(r["us_per_call"], 2)
                except lords.LordsError:
                    entry[path] = None           # the path declines this shape
                finally:
                    lords.lords_set_option("path", "auto")
            lords.lords_set_option("path", "auto")
            r = time_case("_sweep", 5, 3, device, 0, 1, None, do_e2e=False, min_seconds=0.12)
            r.pop("_lay")
            entry["auto"] = round(r["us_per_call"], 2)
            entry["auto_path"] = r["path"]
            rows.append(entry)
            print(f"[sweep] {label} M={M}: " + ", ".join(f"{k}={entry[k]}" for k in paths) +
                  f", auto={entry['auto']} ({entry['auto_path']})", file=sys.stderr)
    CASES.pop("_sweep", None)
    return rows


def cpu_baseline(case, lay, packed, budget_s=12.0):
    """The oracle as it stands, on the host cores, on a bounded sample of the case."""
    import numpy as np
    import oracle

    c = CASES[case]
    # sample = a subset of output rows sized from a quick probe so the run takes about budget_s
    probe_rows = np.arange(min(c["m"], 64), dtype=np.int64)
    t0 = time.perf_counter()
    _, threads = oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, lay.bits, rows=probe_rows,
                                return_threads=True)
    dt = max(time.perf_counter() - t0, 1e-4)
    nrows = int(min(c["m"], max(64, probe_rows.size * budget_s / dt)))
    rows = np.arange(nrows, dtype=np.int64)
    # a whole layer may take far less than the budget: repeat it (the oracle has no state to warm)
    reps = 1
    if nrows == c["m"]:
        reps = int(max(1, min(2000, budget_s / max(dt * c["m"] / probe_rows.size, 1e-4))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, lay.bits, rows=rows)
    dt = (time.perf_counter() - t0) / reps
    frac = nrows / c["m"]
    sec_full = dt / frac
    byt, flo = algorithmic_bytes(c), useful_flops(c)
    if c["bound"] == "hbm":
        value, unit = byt / sec_full / 1e9, "GB/s"
    else:
        value, unit = flo / sec_full / 1e12, "TFLOP/s"
    return {"value": value, "unit": unit, "cores": int(threads), "kind": "oracle",
            "sample": f"{nrows} of {c['m']} output rows of one {case} layer, all {c['M']} tokens, "
                      f"{reps} repetition(s) of {dt:.3f} s, scaled to the full layer"}


def run_reference(args):
    """--impl reference: the fp64 oracle on the host cores (there is no other reference)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import numpy as np
    import oracle
    from paper_2601_22716_b200 import inputs as gen

    case = args.case or HEADLINE
    c = CASES[case]
    lay = gen.make_layer(c["m"], c["n"], c["r"], c["M"], bits=c["bits"], seed=0, outlier_frac=c["outliers"])
    packed = oracle.pack_codes(lay.codes, c["bits"])
    # each step = the oracle over a fixed sample of output rows of one layer
    probe = np.arange(min(64, c["m"]), dtype=np.int64)
    t0 = time.perf_counter()
    _, threads = oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, lay.bits, rows=probe, return_threads=True)
    dt = max(time.perf_counter() - t0, 1e-4)
    total = max(1, args.steps + args.warmup)
    nrows = int(min(c["m"], max(64, 64 * (60.0 / total) / dt)))
    rows = np.arange(nrows, dtype=np.int64)
    for _ in range(args.warmup):
        oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, lay.bits, rows=rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, lay.bits, rows=rows)
    dt = (time.perf_counter() - t0) / args.steps
    sec_full = dt * c["m"] / nrows
    byt, flo = algorithmic_bytes(c), useful_flops(c)
    value, unit = (byt / sec_full / 1e9, "GB/s") if c["bound"] == "hbm" else (flo / sec_full / 1e12, "TFLOP/s")
    sample = f"{nrows} of {c['m']} output rows of one {case} layer per step, scaled to the full layer"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": case, **{k: c[k] for k in ("m", "n", "bits", "r", "M")}},
        "cpu_baseline": {"value": value, "unit": unit, "cores": int(threads), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--case", default=None, help="time only this case (default: headline plus the others)")
    ap.add_argument("--no-extras", action="store_true", help="headline case only")
    ap.add_argument("--path", default="auto", help="force a kernel path (auto|simt|decode|umma)")
    ap.add_argument("--stack", action="store_true", help="(default) time the full Llama-3-8B linear stack as well")
    ap.add_argument("--no-stack", action="store_true", help="skip the 224-module Llama-3-8B linear stack")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="floor on the headline case's timed region (0: exactly --steps rounds, for profiler captures)")
    ap.add_argument("--sweep", action="store_true",
                    help="time every kernel path at M in {1, 2, 3, 4, 8, 16} on the q_proj, gate and down shapes and print the table")
    args = ap.parse_args()

    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2601_22716_b200 import binding as lords   # raises if liblords.so is missing: no fallback

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the hot path has no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device(f"cuda:{local}")
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    lords.lords_init(local, 0)
    lords.lords_set_option("path", args.path)

    if args.sweep:
        rows = run_sweep(device) if rank == 0 else []
        if rank == 0:
            print(json.dumps({"sweep": rows, "unit": "us per forward call"}))
        lords.lords_shutdown()
        if world > 1:
            dist.destroy_process_group()
        return 0

    if args.case == "compare_q_m1":
        if rank == 0:
            print(json.dumps(time_comparators(device)))
        lords.lords_shutdown()
        if world > 1:
            dist.destroy_process_group()
        return 0
    if args.case in BACKWARD_CASES:
        if rank == 0:
            print(json.dumps(time_backward(args.case, *BACKWARD_CASES[args.case], device, min_seconds=min(args.min_seconds, 0.3))))
        lords.lords_shutdown()
        if world > 1:
            dist.destroy_process_group()
        return 0
    if args.case in QUANTIZE_CASES:
        if rank == 0:
            print(json.dumps(time_quantize(args.case, *QUANTIZE_CASES[args.case], device, min_seconds=min(args.min_seconds, 0.3))))
        lords.lords_shutdown()
        if world > 1:
            dist.destroy_process_group()
        return 0

    head = args.case or HEADLINE
    sampler = ClockSampler(local) if rank == 0 else None
    res = time_case(head, args.steps, args.warmup, device, rank, world, sampler, min_seconds=args.min_seconds)
    lay, packed = res.pop("_lay")
    c = CASES[head]
    cases = []
    if not args.case and not args.no_extras:
        for name in CASES:
            if name == head:
                continue
            # the other cases get a fixed, short budget (about a quarter of a second each)
            k = {"decode_q_m8": 400, "mlp3_gate_m1": 800, "mlp3_down_m1": 800, "mlp3_down_m16": 300,
                 "prefill_m2048": 60}.get(name, 20)
            k = max(3, min(args.steps, k))
            # every case has its clocks sampled while it is timed (the prefill case runs under the power cap)
            r2 = time_case(name, k, 3, device, rank, world, ClockSampler(local) if rank == 0 else None, do_e2e=False,
                           min_seconds=0.4)
            r2.pop("_lay")
            cases.append({"case": name, "path": r2["path"], "us_per_call": r2["us_per_call"],
                          "gbs": r2["gbs"], "tflops": r2["tflops"], "roofline": r2["roofline"], "clocks": r2["clocks"],
                          "copies": r2["copies"], "rounds": r2["rounds"], "steps": k, "status_retries": r2["status_retries"]})

    if not args.case and not args.no_extras and world == 1:
        for name, shape in QUANTIZE_CASES.items():
            cases.append(time_quantize(name, *shape, device))
        for name, shape in BACKWARD_CASES.items():
            cases.append(time_backward(name, *shape, device))
        comparators = time_comparators(device)

    stack = []
    if not (not args.case and not args.no_extras and world == 1):
        comparators = None
    if not args.no_stack and not args.no_extras and not args.case and world == 1:
        # the last two lines: projections that share their input as one call (q, k, v; at one token also gate, up)
        for (M, mlp_bits, k, qkv, gate_up) in [(1, 4, 30, False, False), (8, 4, 30, False, False), (512, 4, 5, False, False),
                                               (1, 3, 30, False, False), (1, 2, 30, False, False),
                                               (1, 4, 30, True, True), (8, 4, 30, True, False)]:
            stack.append(time_stack(M, mlp_bits, k, device, qkv_one_call=qkv, gate_up_one_call=gate_up))
            torch.cuda.empty_cache()

    if rank == 0:
        hbm = c["bound"] == "hbm"
        value = res["gbs"] if hbm else res["tflops"]
        unit = "GB/s" if hbm else "TFLOP/s"
        base = cpu_baseline(head, lay, packed) if world == 1 else None
        e2e = res.get("e2e")
        line = {
            "metric": METRIC, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": res["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16",
            "data": "synthetic",
            "config": {"workload": head, **{k: c[k] for k in ("m", "n", "bits", "r", "M")},
                       "copies_per_step": res["copies"], "rounds_per_step": res["rounds"],
                       "calls_per_step": res["copies"] * res["rounds"], "path": res["path"], "cuda_graph": res["graph"],
                       "l2": f"every round of a step rotates over {res['copies']} distinct weight sets "
                             f"({res['copies'] * algorithmic_bytes(c) / 1e6:.0f} MB > 2 x L2), no explicit flush",
                       "parallelism": "replicas" if world > 1 else "single"},
            "us_per_call": res["us_per_call"],
            "roofline": res["roofline"], "clocks": res["clocks"], "gpu_launches": res["gpu_launches"],
            "status_retries": res["status_retries"],
            "e2e": None if e2e is None else {
                "value": e2e["gbs"] if hbm else e2e["tflops"], "unit": unit,
                "h2d_bytes_per_step": e2e["h2d_bytes_per_step"], "d2h_bytes_per_step": e2e["d2h_bytes_per_step"],
                "ms_per_step": e2e["ms_per_step"], "cuda_graph": e2e["cuda_graph"]},
            "cpu_baseline": base, "cases": cases,
        }
        if stack:
            line["stack"] = stack
        if comparators is not None:
            line["comparators"] = comparators
        print(json.dumps(line))
    lords.lords_shutdown()
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
