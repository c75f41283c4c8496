#!/usr/bin/env python
"""Benchmark of causal Polysketch attention (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl psk|reference]

One "step" is one pass of the whole hot path over one batch: psk_causal_attn_fwd
followed by psk_causal_attn_bwd (forward only for forward-only workloads).  Prints ONE
JSON line (rank 0).  Inputs are synthetic (seeded Gaussians with row-normalised Q, K).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "causal polysketch attn fwd+bwd tokens/s at n=32k GPT-2-small shape; % bf16 TC peak"
UNIT = "model-tokens/s"


# ---------------------------------------------------------------------------
# flop model (GEMM flops only, per head-token); "nominal" follows the paper's statement
# of the algorithm (r^2 features, h+1 columns, full b x b diagonal tiles)
# ---------------------------------------------------------------------------
def nominal_flops_per_head_token(w, local=False):
    """local: exact same-block weights (Section 3.2): the b x b tiles contract over h, not r."""
    h, r, b = w.h, w.r, w.b
    kd = h if local else r
    fwd = 8 * h * r + 4 * r * r * (h + 1) + 2 * b * (kd + h + 1)
    bwd = 10 * r * r * (h + 1) + 6 * b * kd + 4 * b * (h + 1) + 16 * h * r
    return fwd, (bwd if w.backward else 0)


def kernel_flops_per_head_token(name, w, local=False):
    """Executed flops of one launch of a library kernel, per head-token it covers."""
    h, r, b = w.h, w.r, w.b
    k = h + 1
    half = (b + 1) / 2.0                       # causal pairs per row inside a block
    table = {
        # CUDA-core path
        "sketch_kernel": 4 * h * r,
        "rows_prep_kernel": 2 * h,
        "state_kernel": 2 * r * r * k + r * r,
        "scan_kernel": r * r * k / b,
        "fwd_out_kernel": 2 * r * r * k + r * r + half * 2 * (r + k),
        "bwd_q_kernel": 2 * r * r * k + 2 * r * r + half * 2 * (2 * r + k),
        "bwd_k_kernel": 4 * r * r * k + 3 * r * r + half * 2 * (2 * r + 2 * k),
        "sketch_bwd_kernel": 8 * h * r,
    }
    # tensor-core path: MMA flops actually issued (symmetric features: F = r(r+1)/2, padded)
    F = r * (r + 1) // 2
    FK = (F + 15) // 16 * 16            # contraction extent over features
    FP = (F + 127) // 128 * 128         # stored / accumulated feature rows
    nt = b // 128
    other = (nt + 1) / 2.0              # other-side 128-row tiles met per own tile, averaged
    sk = 2 * h * 2 * r                  # one half-sketch GEMM
    tile_fwd = sk + 2 * 128 * 3 * r + 2 * 128 * h
    tile_bwd = sk + 2 * 128 * 3 * r + 2 * 128 * h + 2 * 128 * 64
    if local:                           # scores over h, no sketch of the other tile; dX product 64 wide
        tile_fwd = 2 * 128 * h + 2 * 128 * h
        tile_bwd = 2 * 128 * h + 2 * 128 * h + 2 * 128 * 64
    table.update({
        # (r = 64: a state set is built by five launches that split the feature tiles between them and
        # each redo the half sketch; the figure is the average launch)
        "tc_state_kernel": sk + 2 * FP * 80 / (1 if r <= 32 else 5),
        "tc_fwd_out_kernel": sk + 2 * FK * 80 + other * tile_fwd,
        "tc_bwd_recompute_kernel": sk + 2 * FK * 80 + other * tile_fwd,
        "tc_bwd_q_kernel": 2 * sk + 2 * FK * 80 + other * tile_bwd + 2 * 2 * r * 64,
        "tc_bwd_k_kernel": 2 * sk + 2 * FK * 80 + 2 * FK * 64 + other * (tile_bwd + 2 * 128 * 64) + 2 * 2 * r * 64,
        "tc_vmean_kernel": None, "tc_bwd_prep_kernel": None,
    })
    return table.get(name)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"],
                "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# fp32 FMA peak of the CUDA cores: 148 SMs x 128 lanes x 2 flop x 1.965 GHz (max SM clock)
ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons during the timed region."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for nm, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_step(w, inp_host, head, local=False):
    """One bounded sample of the workload for the CPU oracle: forward (+ backward) of one
    (batch, head) slice at full n.  Returns seconds."""
    from oracle import polysketch as orc
    Q, K, V, dO, G1, G2 = inp_host[head]
    diag = "exact" if local else "LR"
    t0 = time.perf_counter()
    orc.causal_polysketch_attention_blocked(Q, K, V, G1, G2, w.b, diagonal=diag)
    if w.backward:
        orc.causal_polysketch_attention_backward_blocked(Q, K, V, G1, G2, dO, w.b, diagonal=diag)
    return time.perf_counter() - t0


def host_head_inputs(w, heads):
    """Oracle inputs for a few heads, drawn on the host with the workload's recipe."""
    import numpy as np
    import torch
    from paper_2310_01655_b200 import inputs as wl
    small = wl.Workload(w.name, 1, len(heads), w.n, w.h, w.r, w.p, w.b, w.dtype, w.backward,
                        w.data_seed, w.g_seed, w.correlated)
    inp = wl.make_inputs(small, "cpu", with_dO=True)
    out = []
    for i, _ in enumerate(heads):
        f = lambda k: inp[k][0, i].to(torch.float64).numpy()
        out.append((f("Q"), f("K"), f("V"), f("dO"), inp["G1"][i].double().numpy(), inp["G2"][i].double().numpy()))
    return out


def cpu_threads():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args, w):
    """--impl reference: the CPU oracle, as it stands, on bounded samples of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    heads = list(range(max(1, min(2, args.steps + args.warmup))))
    data = host_head_inputs(w, heads)
    for i in range(args.warmup):
        oracle_step(w, data, i % len(data), args.local_exact)
    times = [oracle_step(w, data, i % len(data), args.local_exact) for i in range(args.steps)]
    total = sum(times)
    value = (w.n * args.steps / total) / w.H          # head-tokens/s -> model-tokens/s
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "n": w.n, "h": w.h, "r": w.r, "p": w.p, "b": w.b,
                   "passes": "fwd+bwd" if w.backward else "fwd",
                   "variant": "local_exact" if args.local_exact else "polysketch",
                   "step": "oracle on one (batch, head) slice at full n; value extrapolated over heads"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                         "sample": "%d steps x 1 head slice of %s at n=%d" % (args.steps, w.name, w.n)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def executed_flops_per_step(w, kernels, local):
    """Sum over the library's kernels of the MMA flops they issued in one step (None-flop kernels are
    memory-bound helpers and add nothing)."""
    total = 0.0
    for name, (cnt, _ms, steps) in kernels.items():
        key = {"tc_state_total_kernel": "tc_state_kernel"}.get(name, name)
        fl = kernel_flops_per_head_token(key, w, local)
        if fl:
            total += fl * w.head_tokens * cnt / steps
    return total


def time_other_config(psk, wl, name, steps, warmup, local, pk, device_index):
    """A short timed run of another benchmark configuration (same step definition as the headline):
    ms per step, nominal and executed TFLOP/s with their fractions of the measured peaks, clocks."""
    import torch
    w = wl.WORKLOADS[name]
    inp = wl.make_inputs(w, "cuda", with_dO=True)
    Q, K, V, dO, G1, G2 = (inp[k] for k in ("Q", "K", "V", "dO", "G1", "G2"))
    flags = (psk.FLAG_KEEP_STATES if w.backward else 0) | (psk.FLAG_LOCAL_EXACT if local else 0)
    shp = psk.binding.make_shape(Q, G1, w.r, w.b, w.p, psk.PATH_AUTO, flags)
    ws = torch.empty(max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, True) if w.backward else 0),
                     dtype=torch.uint8, device="cuda")
    O = torch.empty_like(Q)
    den = torch.empty((w.B, w.H, w.n), dtype=torch.float32, device="cuda")
    grads = tuple(torch.empty_like(Q) for _ in range(3)) if w.backward else None

    def step():
        psk.causal_attn_fwd(Q, K, V, G1, G2, w.b, w.p, psk.PATH_AUTO, ws, O, den, flags)
        if w.backward:
            psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, w.b, w.p, psk.PATH_AUTO, ws, grads, flags)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(device_index)
    sampler.start()
    psk.profile_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    clocks = sampler.stop()
    agg = {}
    for kname, t in psk.profile_records():
        a = agg.setdefault(kname, [0, 0.0, steps])
        a[0] += 1; a[1] += t
    psk.profile_enable(False)
    if psk.check(ws) != 0:
        raise RuntimeError("device-side error while timing %s" % name)
    f_fwd, f_bwd = nominal_flops_per_head_token(w, local)
    nominal = (f_fwd + f_bwd) * w.head_tokens / (ms / 1e3) / 1e12
    executed = executed_flops_per_step(w, agg, local) / (ms / 1e3) / 1e12
    return {"B": w.B, "H": w.H, "n": w.n, "r": w.r, "b": w.b, "passes": "fwd+bwd" if w.backward else "fwd",
            "steps": steps, "warmup": warmup, "ms_per_step": ms, "model_tokens_per_s": w.model_tokens / (ms / 1e3),
            "nominal_tflops": nominal, "executed_tflops": executed,
            "frac_nominal": {"burst": nominal / pk["bf16_burst"], "sustained": nominal / pk["bf16_sustained"]},
            "frac_executed": {"burst": executed / pk["bf16_burst"], "sustained": executed / pk["bf16_sustained"]},
            "kernels_ms_per_launch": {k: round(v[1] / v[0], 3) for k, v in sorted(agg.items(), key=lambda kv: -kv[1][1])},
            "clocks": clocks}


def time_lt_multiply(psk, base, steps, warmup, device_index):
    """psk_lt_multiply_bf16 (Section 3.1's block algorithm on GIVEN feature matrices, tensor cores) on a
    quarter of the headline's (batch, head) slices with m = r^2 = 1024 features of unit-variance rows:
    memory-bound by construction (the features are read, not generated), so the figure of merit is
    bytes: compulsory = A, B, C once + Out."""
    import torch
    batch, n, m, b = max(1, base.B * base.H // 4), base.n, 1024, 256
    gen = torch.Generator(device="cuda").manual_seed(base.data_seed)
    A, B = ((torch.randn(batch, n, m, generator=gen, device="cuda") / 32).bfloat16() for _ in range(2))
    C = torch.randn(batch, n, 64, generator=gen, device="cuda").bfloat16()
    ws = None
    for _ in range(warmup):
        out, ws = psk.lt_multiply_bf16(A, B, C, b, ws)
    torch.cuda.synchronize()
    psk.profile_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        out, ws = psk.lt_multiply_bf16(A, B, C, b, ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    agg = {}
    for kname, t in psk.profile_records():
        agg[kname] = agg.get(kname, 0.0) + t
    psk.profile_enable(False)
    if psk.check(ws) != 0:
        raise RuntimeError("device-side error while timing lt_multiply_bf16")
    compulsory = 2 * A.numel() * 2 + C.numel() * 2 + out.numel() * 4
    hbm = peaks()["hbm_gbs"]
    gbs = compulsory / (ms / 1e3) / 1e9
    return {"batch": batch, "n": n, "m": m, "k": 64, "b": b, "passes": "fwd", "steps": steps, "warmup": warmup, "ms_per_step": ms,
            "compulsory_bytes": compulsory, "compulsory_gbs": gbs, "frac_hbm_peak": gbs / hbm,
            "kernels_ms_per_step": {k: round(v / steps, 3) for k, v in sorted(agg.items(), key=lambda kv: -kv[1])}}


def time_variant(psk, wl, name, base, steps, warmup, device_index):
    """A short timed run of another member of the family at the headline configuration's B, H, n
    (forward + backward, bf16): "learned" = the learnable sketch of the appendix (r = 32, b = 256, parameter
    gradients included), "learned_local" = the same with exact same-block weights (the paper's
    "learned + local"), "p2" = exact degree-2 attention (r = h = 64, b = 512), "p8" = degree 8 (r = 32)."""
    import torch
    binding = psk.binding
    if name == "lt":
        return time_lt_multiply(psk, base, steps, warmup, device_index)
    r, b, p = {"learned": (32, 256, 4), "learned_local": (32, 256, 4), "p2": (64, 512, 2), "p8": (32, 256, 8)}[name]
    w = wl.Workload(name, base.B, base.H, base.n, base.h, r, 4, b, "bf16", True, base.data_seed, base.g_seed)
    inp = wl.make_inputs(w, "cuda", with_dO=True)
    Q, K, V, dO = (inp[k] for k in ("Q", "K", "V", "dO"))
    flags = psk.FLAG_KEEP_STATES
    O = torch.empty_like(Q)
    den = torch.empty((w.B, w.H, w.n), dtype=torch.float32, device="cuda")
    grads = tuple(torch.empty_like(Q) for _ in range(3))
    if name in ("learned", "learned_local"):
        lflags = flags | (psk.FLAG_LOCAL_EXACT if name == "learned_local" else 0)      # kept states, like the headline
        if name == "learned_local":
            Q.mul_(0.35); K.mul_(0.35)      # (q.k)^4 next to sketch weights bounded by r^2: the same scale
        flat = binding.pack_learned_params(*wl.learned_network_params(w.h, r, base.g_seed))
        ws = torch.empty(binding.learned_workspace_bytes(Q, r, b, lflags), dtype=torch.uint8, device="cuda")

        def step():
            o, d = binding.learned_attn_fwd(Q, K, V, flat, r, b, lflags, ws)
            binding.learned_attn_bwd(Q, K, V, flat, o, d, dO, r, b, lflags, ws)
    else:
        if p == 2:
            Q.mul_(0.5); K.mul_(0.5)        # (q.k)^2 with |q|^2 = 64: keep the weights on the headline's scale
            G1 = G2 = None
        else:
            Q.mul_(0.5); K.mul_(0.5)
            gen = torch.Generator(device="cpu").manual_seed(base.g_seed)
            G1 = torch.randn(w.H, 2 * w.h + r, r, generator=gen).to(Q.dtype).cuda()
            G2 = torch.randn(w.H, 2 * w.h + r, r, generator=gen).to(Q.dtype).cuda()
        shp = binding.make_shape(Q, G1, r, b, p, psk.PATH_AUTO, flags)
        ws = torch.empty(max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, True)), dtype=torch.uint8, device="cuda")

        def step():
            psk.causal_attn_fwd(Q, K, V, G1, G2, b, p, psk.PATH_AUTO, ws, O, den, flags)
            psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, p, psk.PATH_AUTO, ws, grads, flags)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(device_index)
    sampler.start()
    psk.profile_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    clocks = sampler.stop()
    agg = {}
    for kname, t in psk.profile_records():
        agg[kname] = agg.get(kname, 0.0) + t
    psk.profile_enable(False)
    if psk.check(ws) != 0:
        raise RuntimeError("device-side error while timing %s" % name)
    return {"B": w.B, "H": w.H, "n": w.n, "r": r, "b": b, "p": p, "passes": "fwd+bwd", "steps": steps, "warmup": warmup,
            "ms_per_step": ms, "model_tokens_per_s": w.model_tokens / (ms / 1e3),
            "kernels_ms_per_step": {k: round(v / steps, 3) for k, v in sorted(agg.items(), key=lambda kv: -kv[1])},
            "clocks": clocks}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--impl", default="psk", choices=["psk", "reference"])
    ap.add_argument("--path", default="auto", choices=["auto", "cuda_cores", "tensor_cores"])
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--cpu-heads", type=int, default=12, help="head slices the CPU baseline leg times")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--local-exact", action="store_true",
                    help="exact polynomial weights inside each block (Section 3.2) instead of the headline variant")
    ap.add_argument("--others", default="c1,c3,c4",
                    help="other configurations timed briefly after the headline one (N = 1 only); '' for none")
    ap.add_argument("--other-steps", type=int, default=5)
    ap.add_argument("--variants", default="learned,learned_local,p2,p8,lt",
                    help="other members of the family timed briefly at the headline's B, H, n (N=1 only; '' = none)")
    ap.add_argument("--variant-steps", type=int, default=2)
    ap.add_argument("--seq-segments", type=int, default=0,
                    help="runs a head's blocks are cut into for the state scan (0: the library chooses)")
    ap.add_argument("--no-keep-states", action="store_true",
                    help="let the backward rebuild the prefix states instead of reading the forward's")
    args = ap.parse_args()

    from paper_2310_01655_b200 import inputs as wl
    w = wl.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import paper_2310_01655_b200 as psk
    from paper_2310_01655_b200 import dist_util as du

    rank, world, local = du.env_rank()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the library")
    torch.cuda.set_device(local)
    du.init("nccl", torch.device("cuda", local))
    psk.lib()
    path = {"auto": psk.PATH_AUTO, "cuda_cores": psk.PATH_CUDA_CORES, "tensor_cores": psk.PATH_TENSOR_CORES}[args.path]

    # every rank holds its own batch of the workload (independent (batch, head) problems:
    # no data-path collective), seeded differently per rank
    wr = wl.Workload(**dict(w.asdict(), data_seed=du.rank_seed(w.data_seed, rank)))
    inp = wl.make_inputs(wr, "cuda", with_dO=True)
    Q, K, V, dO, G1, G2 = (inp[k] for k in ("Q", "K", "V", "dO", "G1", "G2"))
    # forward and backward of one step share the workspace: the backward reads the forward's states
    flags = psk.FLAG_KEEP_STATES if (w.backward and not args.no_keep_states) else 0
    keep = bool(flags)
    if args.local_exact:
        flags |= psk.FLAG_LOCAL_EXACT
    segs = args.seq_segments
    shp = psk.binding.make_shape(Q, G1, w.r, w.b, w.p, path, flags, segs)
    ws_bytes = max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, True) if w.backward else 0)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    O = torch.empty_like(Q)
    den = torch.empty((w.B, w.H, w.n), dtype=torch.float32, device="cuda")
    grads = tuple(torch.empty_like(Q) for _ in range(3)) if w.backward else None
    launches = [0]

    def step():
        psk.causal_attn_fwd(Q, K, V, G1, G2, w.b, w.p, path, ws, O, den, flags, segs)
        n = psk.last_launch_count()
        if w.backward:
            psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, w.b, w.p, path, ws, grads, flags, segs)
            n += psk.last_launch_count()
        launches[0] += n

    def barrier():
        du.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if psk.check(ws) != 0:
        raise RuntimeError("device-side error during warm-up")

    # ---- timed region: K steps, CUDA events on the launch stream, per-kernel events on ----
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    psk.profile_enable(True)
    launches[0] = 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    records = psk.profile_records()
    psk.profile_enable(False)
    if psk.check(ws) != 0:
        raise RuntimeError("device-side error during the timed region")
    ms = du.max_over_ranks(ms, "cuda")
    value = du.aggregate_throughput(w.model_tokens, args.steps, ms, world)

    # ---- end to end through the same C-ABI call with HOST buffers ----
    # Every step copies its inputs from pinned host memory and copies every result back.  Steps are
    # software-pipelined over two device buffer sets and three streams (H2D of step i+1 and D2H of
    # step i-1 overlap the kernels of step i); the timed region runs from the first copy-in to
    # the last copy-out.
    e2e = None
    if not args.no_e2e:
        names = ["Q", "K", "V"] + (["dO"] if w.backward else [])
        host_in = {k: torch.empty(inp[k].shape, dtype=inp[k].dtype, pin_memory=True).copy_(inp[k]) for k in names}
        nouts = 4 if w.backward else 1
        dev_in = [inp, {k: torch.empty_like(inp[k]) for k in names}]
        dev_out = [[torch.empty_like(Q) for _ in range(nouts)] for _ in range(2)]
        dev_den = [torch.empty_like(den) for _ in range(2)]
        host_out = [[torch.empty(Q.shape, dtype=Q.dtype, pin_memory=True) for _ in range(nouts)] for _ in range(2)]
        host_den = [torch.empty(den.shape, dtype=den.dtype, pin_memory=True) for _ in range(2)]
        bi = sum(t.numel() * t.element_size() for t in host_in.values())
        bo = sum(t.numel() * t.element_size() for t in host_out[0]) + host_den[0].numel() * 4
        s_in, s_out, s_comp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()

        def e2e_run(nsteps):
            ev_in = [None, None]; ev_comp = [None, None]; ev_out = [None, None]
            for i in range(nsteps):
                k = i & 1
                with torch.cuda.stream(s_in):
                    if ev_comp[k] is not None:
                        s_in.wait_event(ev_comp[k])          # step i-2 has read this input set
                    for nm in names:
                        dev_in[k][nm].copy_(host_in[nm], non_blocking=True)
                    ev_in[k] = torch.cuda.Event(); ev_in[k].record(s_in)
                s_comp.wait_event(ev_in[k])
                if ev_out[k] is not None:
                    s_comp.wait_event(ev_out[k])             # step i-2's results have left this output set
                d = dev_in[k]
                psk.causal_attn_fwd(d["Q"], d["K"], d["V"], G1, G2, w.b, w.p, path, ws, dev_out[k][0], dev_den[k], flags, segs)
                if w.backward:
                    psk.causal_attn_bwd(d["Q"], d["K"], d["V"], G1, G2, dev_out[k][0], dev_den[k], d["dO"], w.b, w.p,
                                        path, ws, tuple(dev_out[k][1:]), flags, segs)
                ev_comp[k] = torch.cuda.Event(); ev_comp[k].record(s_comp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_comp[k])
                    for o, ho in zip(dev_out[k], host_out[k]):
                        ho.copy_(o, non_blocking=True)
                    host_den[k].copy_(dev_den[k], non_blocking=True)
                    ev_out[k] = torch.cuda.Event(); ev_out[k].record(s_out)
            s_comp.wait_stream(s_out)
            s_comp.wait_stream(s_in)

        e2e_run(2)
        barrier()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        e2e_run(args.e2e_steps)
        b_.record()
        barrier()
        t2 = du.max_over_ranks(a.elapsed_time(b_), "cuda")
        e2e = {"value": du.aggregate_throughput(w.model_tokens, args.e2e_steps, t2, world), "unit": UNIT,
               "h2d_bytes_per_step": bi, "d2h_bytes_per_step": bo, "steps": args.e2e_steps,
               "ms_per_step": t2 / args.e2e_steps, "pipelined": True}
        del host_in, host_out, dev_in, dev_out

    if rank != 0:
        du.shutdown()
        return

    # ---- roofline of the dominant kernel ----
    pk = peaks()
    agg = {}
    for name, t in records:
        a = agg.setdefault(name, [0, 0.0])
        a[0] += 1; a[1] += t
    total_kernel_ms = sum(v[1] for v in agg.values()) or 1.0
    top = max(agg.items(), key=lambda kv: kv[1][1]) if agg else (None, [0, 0.0])
    roof = None
    if top[0] is not None:
        name, (cnt, tot) = top
        fl = kernel_flops_per_head_token(name, w, args.local_exact)
        tensor = name.startswith("tc_")
        peak = pk["bf16_sustained"] if tensor else ALU_PEAK_TFLOPS
        achieved = (fl * w.head_tokens / ((tot / cnt) / 1e3) / 1e12) if fl else None
        # DRAM bytes per launch: ncu capture on the profiling-sized slice, scaled by head-tokens
        traffic = None
        tname = "dram_traffic_c2s_local_exact.json" if args.local_exact else "dram_traffic_c2s.json"
        tpath = os.path.join(ROOT, "profiles", tname)
        if os.path.exists(tpath) and w.r == 32 and w.b == 256:
            per = json.load(open(tpath))["kernels"].get(name)
            if per:
                traffic = per["dram_bytes_per_head_token"] * w.head_tokens
        roof = {"kernel": name, "bound": "tensor" if tensor else "alu", "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": (achieved / peak) if achieved else None,
                "frac_sustained": (achieved / pk["bf16_sustained"]) if (achieved and tensor) else None,
                "frac_burst": (achieved / pk["bf16_burst"]) if (achieved and tensor) else None, "traffic": traffic,
                "traffic_source": ("profiles/%s (ncu on the c2s slice, scaled by head-tokens)" % tname) if traffic else None,
                "flops_per_launch": fl * w.head_tokens if fl else None,
                "peak_source": (pk["source"] + " (sustained bf16)") if tensor else "derived: 148 SM x 128 FMA x 1.965 GHz",
                "launches": cnt, "avg_ms": tot / cnt, "share_of_kernel_time": tot / total_kernel_ms}
    kernels = {k: {"launches": v[0], "ms_total": round(v[1], 3), "share": round(v[1] / total_kernel_ms, 4)}
               for k, v in sorted(agg.items(), key=lambda kv: -kv[1][1])}

    # ---- CPU baseline: the oracle on a bounded sample ----
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        heads = list(range(args.cpu_heads))
        data = host_head_inputs(w, heads)
        secs = sum(oracle_step(w, data, i, args.local_exact) for i in range(len(heads)))
        cpu = {"value": (w.n * len(heads) / secs) / w.H, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
               "sample": "%d (batch, head) slices of %s at full n=%d, %s; extrapolated linearly over heads"
                         % (len(heads), w.name, w.n, "fwd+bwd" if w.backward else "fwd"),
               "seconds": secs}

    f_fwd, f_bwd = nominal_flops_per_head_token(w, args.local_exact)
    nominal_tflops = (f_fwd + f_bwd) * w.head_tokens * world * args.steps / (ms / 1e3) / 1e12
    # flops the kernels actually issued (symmetric features, masked tiles skipped): the figure the
    # fraction of peak is claimed on; the nominal one counts the paper's statement of the algorithm
    executed_tflops = executed_flops_per_step(w, {k: (v[0], v[1], args.steps) for k, v in agg.items()},
                                              args.local_exact) * world / (ms / args.steps / 1e3) / 1e12
    # the headline tensors go before the other configurations are built
    others = None
    if world == 1 and args.others:
        del Q, K, V, dO, O, den, grads, ws, inp
        torch.cuda.empty_cache()
        others = {}
        for name in [x for x in args.others.split(",") if x and x != w.name]:
            others[name] = time_other_config(psk, wl, name, args.other_steps, args.warmup, args.local_exact, pk, local)
            torch.cuda.empty_cache()
    variants = None
    if world == 1 and args.variants:
        variants = {}
        for name in [x for x in args.variants.split(",") if x]:
            variants[name] = time_variant(psk, wl, name, w, args.variant_steps, 1, local)
            torch.cuda.empty_cache()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "n": w.n, "h": w.h, "r": w.r, "p": w.p, "b": w.b,
                   "passes": "fwd+bwd" if w.backward else "fwd", "path": args.path,
                   "variant": "local_exact" if args.local_exact else "polysketch",
                   "keep_states": keep, "seq_segments": segs,
                   "l2": "inputs larger than L2 (no flush)", "per_gpu_batch": w.B},
        "nominal_tflops": nominal_tflops, "executed_tflops": executed_tflops,
        "frac_bf16_peak": {"burst": nominal_tflops / world / pk["bf16_burst"],
                           "sustained": nominal_tflops / world / pk["bf16_sustained"],
                           "nominal_2250": nominal_tflops / world / 2250.0, "source": pk["source"],
                           "flops": "nominal (paper's statement: r^2 features, full b x b tiles)"},
        "frac_bf16_peak_executed": {"burst": executed_tflops / world / pk["bf16_burst"],
                                    "sustained": executed_tflops / world / pk["bf16_sustained"],
                                    "nominal_2250": executed_tflops / world / 2250.0, "source": pk["source"],
                                    "flops": "executed MMA flops (symmetric features, masked tiles skipped)"},
        "ms_x_sm_mhz": (ms / args.steps) * clocks["sm_mhz"] if (clocks and clocks.get("sm_mhz")) else None,
        "other_configs": others, "variants": variants,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches[0], "roofline": roof, "kernels": kernels,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    du.shutdown()


if __name__ == "__main__":
    main()
