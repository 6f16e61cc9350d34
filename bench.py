#!/usr/bin/env python
"""Benchmark of the UniQL hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--detail]

Workload (N = 1 and every rank at N > 1): the Llama-3-8B-shaped SwiGLU MLP in decode, the
configuration the headline metric is quoted on -- hidden 4096, intermediate 14336, uint4 g=128
weights, batch M = 1, intermediate channels truncated at keep rates 1.0 / 0.85 / 0.75 / 0.65.
One step = for every keep rate one gate|up launch (two matrices, one launch) and one down launch,
i.e. the whole decode path (truncation, unpack, de-quantise, contraction) over one batch.
metric = effective weight GB/s: 0.53125 bytes per RETAINED weight (codes + fp16 scale and zero per
128) divided by device time.  Each launch reads a different one of four weight copies (375 MB in
rotation, L2 is 126 MB), so every byte comes from HBM.  Synthetic seeded inputs stand in for the
paper's checkpoints.  The step is captured in a CUDA graph and replayed, timed with CUDA events.
"""
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

import numpy as np  # noqa: E402

HIDDEN, INTER = 4096, 14336
KEEP_RATES = (1.0, 0.85, 0.75, 0.65)
BYTES_PER_WEIGHT = 0.5 + 4.0 / 128.0
N_COPIES = 4
METRIC = "qlinear effective weight GB/s, Llama-3-8B MLP decode M=1, keep rates 1.0/0.85/0.75/0.65"


def keep_count(rate, D):
    return int(4 * round(rate * D / 4.0))


def step_bytes(rates=KEEP_RATES):
    return sum(BYTES_PER_WEIGHT * 3 * HIDDEN * keep_count(r, INTER) for r in rates)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    except Exception:
        return 6650.0, 1590.0, "fallback"


class ClockSampler:
    """nvidia-smi clocks / throttle reasons while the GPU is under load."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.rows.append((time.time(), ln.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for (t, ln) in self.rows:
            if t < t0 - 0.05 or t > t1 + 0.15:
                continue
            f = [c.strip() for c in ln.split(",")]
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except Exception:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------- CPU oracle leg
class OracleStep:
    """The oracle as it stands, on the host cores: one whole MLP step at M=1 (all four keep rates)."""

    def __init__(self):
        import oracle
        from paper_2512_03383_b200 import synth
        self.oracle = oracle
        rng = np.random.default_rng(0)
        self.mats = [synth.random_qweight_fast(rng, INTER, HIDDEN), synth.random_qweight_fast(rng, INTER, HIDDEN),
                     synth.random_qweight_fast(rng, HIDDEN, INTER)]
        self.pk = [oracle.pack_u4(w.codes) for w in self.mats]
        self.x = synth.draw_x(rng, 1, HIDDEN, "f16")
        self.h = synth.draw_x(rng, 1, INTER, "f16")
        oracle.qlinear(self.x, self.pk[0][:64], self.mats[0].scales[:64], self.mats[0].zeros[:64],
                       oracle.leading(64), oracle.leading(HIDDEN))

    def step(self):
        o, (gate, up, down), pk = self.oracle, self.mats, self.pk
        t0 = time.time()
        for r in KEEP_RATES:
            k = keep_count(r, INTER)
            o.qlinear(self.x, pk[0], gate.scales, gate.zeros, o.leading(k), o.leading(HIDDEN))
            o.qlinear(self.x, pk[1], up.scales, up.zeros, o.leading(k), o.leading(HIDDEN))
            o.qlinear(self.h[:, :k], pk[2], down.scales, down.zeros, o.leading(HIDDEN), o.leading(k))
        return time.time() - t0

    def describe(self, sec, steps):
        return {"value": step_bytes() / sec / 1e9, "unit": "GB/s", "cores": self.oracle.threads(), "kind": "oracle",
                "sample": "%d whole steps (gate, up, down at 4 keep rates, M=1; the full workload), "
                          "%.3f s per step" % (steps, sec)}


def oracle_leg(budget_s):
    """Bounded CPU-baseline sample: whole steps until `budget_s` seconds have passed; best step counts."""
    o = OracleStep()
    t0, per = time.time(), []
    while True:
        per.append(o.step())
        if time.time() - t0 > budget_s:
            break
    return o.describe(min(per), len(per))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    o = OracleStep()
    for _ in range(args.warmup):
        o.step()
    per = [o.step() for _ in range(args.steps)]
    sec = sum(per) / len(per)
    val = step_bytes() / sec / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "llama3-8b-mlp-decode-M1 (BASELINE configs[1])", "keep_rates": list(KEEP_RATES),
                       "M": 1},
            "cpu_baseline": o.describe(sec, args.steps),
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


# --------------------------------------------------------------------------------------- GPU leg
class MlpDecode:
    """Device-resident weights (N_COPIES rotating copies) and the launches of one step."""

    def __init__(self, B, torch, M, seed=0):
        from paper_2512_03383_b200 import synth
        self.B, self.torch, self.M = B, torch, M
        rng = np.random.default_rng(seed)
        mats = [synth.random_qweight_fast(rng, INTER, HIDDEN), synth.random_qweight_fast(rng, INTER, HIDDEN),
                synth.random_qweight_fast(rng, HIDDEN, INTER)]
        codes_d = [torch.from_numpy(m.codes).cuda() for m in mats]
        self.copies = []
        for c in range(N_COPIES):
            cp = []
            for m, cd in zip(mats, codes_d):
                packed = torch.empty((m.N, m.K // 2), dtype=torch.uint8, device="cuda")
                B.pack_u4(cd, packed)                   # the library's own packer
                cp.append((packed, torch.from_numpy(m.scales).cuda().clone(), torch.from_numpy(m.zeros).cuda().clone()))
            self.copies.append(cp)
        del codes_d
        # one pinned host buffer and one device buffer for the step's inputs (x | h), one of each for its results
        # (gate, up, down outputs of every keep rate): the end-to-end step copies each of them once
        xs = torch.from_numpy(synth.draw_x(rng, M, HIDDEN, "f16")).half()
        hs = torch.from_numpy(synth.draw_x(rng, M, INTER, "f16", outlier_frac=0.0)).half()
        self.in_host = torch.cat([xs.reshape(-1), hs.reshape(-1)]).pin_memory()
        self.in_dev = self.in_host.cuda()
        self.x = self.in_dev[:M * HIDDEN].view(M, HIDDEN)
        self.h = self.in_dev[M * HIDDEN:].view(M, INTER)
        per_rate = M * (2 * INTER + HIDDEN)
        self.out_dev = torch.zeros(len(KEEP_RATES) * per_rate, dtype=torch.float16, device="cuda")
        self.out_host = torch.zeros(len(KEEP_RATES) * per_rate, dtype=torch.float16).pin_memory()
        self.ygs, self.yus, self.yds = [], [], []
        for i in range(len(KEEP_RATES)):
            o = self.out_dev[i * per_rate:(i + 1) * per_rate]
            self.ygs.append(o[:M * INTER].view(M, INTER))
            self.yus.append(o[M * INTER:2 * M * INTER].view(M, INTER))
            self.yds.append(o[2 * M * INTER:].view(M, HIDDEN))
        self.yg, self.yu, self.yd = self.ygs[0], self.yus[0], self.yds
        self.launches_per_step = 2 * len(KEEP_RATES)
        self.turn = 0

    def step(self, e2e=False):
        B, M = self.B, self.M
        h2d = d2h = 0
        if e2e:
            self.in_dev.copy_(self.in_host, non_blocking=True)
            h2d = self.in_host.numel() * 2
        for i, r in enumerate(KEEP_RATES):
            k = keep_count(r, INTER)
            g, u, d = self.copies[self.turn % N_COPIES]
            self.turn += 1
            jobs = [dict(packed_w=g[0], scales=g[1], zeros=g[2], N=INTER, k_out=k, y=self.ygs[i], ldy=INTER),
                    dict(packed_w=u[0], scales=u[1], zeros=u[2], N=INTER, k_out=k, y=self.yus[i], ldy=INTER)]
            B.qlinear_multi(self.x, HIDDEN, M, HIDDEN, None, HIDDEN, jobs)
            B.qlinear_ex(self.h, INTER, d[0], d[1], d[2], None, M, INTER, HIDDEN, None, k, None, HIDDEN,
                         self.yds[i], HIDDEN)
        if e2e:
            self.out_host.copy_(self.out_dev, non_blocking=True)
            d2h = self.out_dev.numel() * 2
        return h2d, d2h


class Eager:
    """Stand-in for a captured graph that launches the step directly (profiler launch lists:
    ncu could not launch this kernel as a node of a replayed graph on this pool)."""

    def __init__(self, fn):
        self.fn = fn

    def replay(self):
        self.fn()


def capture(torch, fn, eager=False):
    if eager:
        return Eager(fn), fn()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        fn()                                     # warm: library workspace, function attributes
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    with torch.cuda.graph(g, stream=s):
        out = fn()
    return g, out


def time_graph(torch, g, steps, barrier=None):
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    if barrier:
        barrier()
    a.record()
    for _ in range(steps):
        g.replay()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e-3


def detail_tables(B, torch, steps):
    """Extra, reported next to the headline: decode at M = 4 and 16 and (when available) prefill."""
    out = {}
    hbm, tf, which = measured_peaks()
    for M in (1, 4, 16):
        w = MlpDecode(B, torch, M)
        rows = {}
        for r in KEEP_RATES:
            k = keep_count(r, INTER)

            def one(r=r, k=k, w=w):
                for _ in range(N_COPIES):
                    g, u, d = w.copies[w.turn % N_COPIES]
                    w.turn += 1
                    jobs = [dict(packed_w=g[0], scales=g[1], zeros=g[2], N=INTER, k_out=k, y=w.yg, ldy=INTER),
                            dict(packed_w=u[0], scales=u[1], zeros=u[2], N=INTER, k_out=k, y=w.yu, ldy=INTER)]
                    B.qlinear_multi(w.x, HIDDEN, M, HIDDEN, None, HIDDEN, jobs)
                    B.qlinear_ex(w.h, INTER, d[0], d[1], d[2], None, M, INTER, HIDDEN, None, k, None, HIDDEN,
                                 w.yd[0], HIDDEN)
            g, _ = capture(torch, one)
            for _ in range(5):
                g.replay()
            sec = time_graph(torch, g, steps) / (steps * N_COPIES)
            gbs = BYTES_PER_WEIGHT * 3 * HIDDEN * k / sec / 1e9
            rows["%.2f" % r] = {"us_per_mlp": round(sec * 1e6, 2), "GBps": round(gbs, 1),
                                "frac_hbm_%s" % which: round(gbs / hbm, 3), "tokens_per_s_mlp": round(M / sec, 1)}
        out["decode_M%d" % M] = rows
        # the MLP block through its own entry point: gate|up with the gated product as epilogue, then down
        # (two launches), and both products in one launch where the shapes allow it
        hbuf = torch.zeros((M, INTER), dtype=torch.float16, device="cuda")
        for fuse, name in ((0, "mlp_swiglu_two_launches_M%d" % M), (1, "mlp_swiglu_one_launch_M%d" % M)):
            rows = {}
            for r in KEEP_RATES:
                k = keep_count(r, INTER) // 8 * 8

                def one(k=k, w=w, fuse=fuse):
                    for _ in range(N_COPIES):
                        g, u, d = w.copies[w.turn % N_COPIES]
                        w.turn += 1
                        B.mlp_swiglu_decode(w.x, HIDDEN, g[0], g[1], g[2], u[0], u[1], u[2], d[0], d[1], d[2], M,
                                            HIDDEN, INTER, k, hbuf, INTER, w.yd[0], HIDDEN, fuse=fuse)
                try:
                    g, _ = capture(torch, one)
                except RuntimeError as e:                      # one launch: M > 8, or the activations do not fit
                    rows["%.2f" % r] = {"unsupported": str(e)[:80]}
                    torch.cuda.synchronize()
                    continue
                for _ in range(5):
                    g.replay()
                sec = time_graph(torch, g, steps) / (steps * N_COPIES)
                gbs = BYTES_PER_WEIGHT * 3 * HIDDEN * k / sec / 1e9
                rows["%.2f" % r] = {"us_per_mlp": round(sec * 1e6, 2), "GBps": round(gbs, 1),
                                    "frac_hbm_%s" % which: round(gbs / hbm, 3)}
            out[name] = rows
        del w, hbuf
        torch.cuda.empty_cache()
    return out


def max_over_ranks(dist, torch, values, device):
    """Replicas share nothing on the data path; the job's time is the slowest rank's (weak scaling)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(bytes_per_rank_step, steps, world, sec):
    """Aggregate metric over all replicas: bytes every rank processed, divided by the slowest rank's time."""
    return bytes_per_rank_step * steps * world / sec / 1e9


def run_ours(args):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    from paper_2512_03383_b200 import binding as B

    work = MlpDecode(B, torch, 1)
    graph, _ = capture(torch, work.step, args.no_graph)
    graph_e2e, (h2d, d2h) = capture(torch, lambda: work.step(e2e=True), args.no_graph)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t_load = time.time()
    for _ in range(max(args.warmup, 3)):
        graph.replay()
    # keep the device under load for a moment so that the sampled clocks are the clocks of the timed region
    torch.cuda.synchronize()
    while time.time() - t_load < 0.6:
        for _ in range(50):
            graph.replay()
        torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    sec = time_graph(torch, graph, args.steps, barrier)
    barrier()
    for _ in range(3):
        graph_e2e.replay()
    sec_e2e = time_graph(torch, graph_e2e, args.steps, barrier)
    t_end = time.time()
    clocks = sampler.stop(t_load, t_end) if rank == 0 else None

    sec, sec_e2e = max_over_ranks(dist, torch, [sec, sec_e2e], "cuda")

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    hbm, tf, which = measured_peaks()
    value = whole_job_value(step_bytes(), args.steps, world, sec)
    launches = work.launches_per_step * args.steps
    per_launch_bytes = step_bytes() / work.launches_per_step
    per_launch_sec = sec / launches
    achieved = per_launch_bytes / per_launch_sec / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": sec / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": "llama3-8b-mlp-decode-M1 (BASELINE configs[1])", "hidden": HIDDEN,
                   "intermediate": INTER, "keep_rates": list(KEEP_RATES), "M": 1,
                   "l2": "4 rotating weight copies (375 MB) > 126 MB L2", "parallelism": "replicas x%d" % world,
                   "timing": ("eager launches (profiling mode, host-bound: not a bench value), CUDA events" if args.no_graph
                              else "CUDA graph of one step replayed, CUDA events")},
        "tokens_per_s_mlp": args.steps * len(KEEP_RATES) * world / sec,
        "gpu_launches": launches,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm,
                     "traffic": None if DRAM_TRAFFIC_RATIO is None else DRAM_TRAFFIC_RATIO * per_launch_bytes, "peak_source": which,
                     "kernel": "decode_kernel (integer path, M=1)", "algorithmic_bytes_per_launch": per_launch_bytes,
                     "frac_of_nominal_8TBs": achieved / 8000.0},
        "e2e": {"value": whole_job_value(step_bytes(), args.steps, world, sec_e2e), "unit": "GB/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "the step's activations copied from pinned host memory before its first launch, all its results to pinned host memory after its last, every step; weights resident"},
    }
    if world == 1:
        line["cpu_baseline"] = oracle_leg(3.0)
        if args.detail:
            line["detail"] = detail_tables(B, torch, max(20, min(args.steps, 200)))
            line["detail"].update(prefill_tables(B, torch))
            line["detail"].update(attention_tables(B, torch, 20))
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


QWEN_HIDDEN, QWEN_INTER = 3584, 18944


class QwenPrefill:
    """Qwen2.5-7B-shaped gate (output rows pruned) and down (input columns pruned) projections, bf16."""

    def __init__(self, B, torch, M, seed=0):
        from paper_2512_03383_b200 import synth
        self.B, self.torch, self.M = B, torch, M
        rng = np.random.default_rng(seed)
        self.w = {}
        for name, N, K in (("gate", QWEN_INTER, QWEN_HIDDEN), ("down", QWEN_HIDDEN, QWEN_INTER)):
            m = synth.random_qweight_fast(rng, N, K)
            cd = torch.from_numpy(m.codes).cuda()
            packed = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
            B.pack_u4(cd, packed)
            self.w[name] = (packed, torch.from_numpy(m.scales).cuda(), torch.from_numpy(m.zeros).cuda(), N, K)
            del cd
        self.x = torch.randn((M, QWEN_HIDDEN), device="cuda").to(torch.bfloat16)
        self.h = torch.randn((M, QWEN_INTER), device="cuda").to(torch.bfloat16)
        self.yg = torch.zeros((M, QWEN_INTER), dtype=torch.bfloat16, device="cuda")
        self.yd = torch.zeros((M, QWEN_HIDDEN), dtype=torch.bfloat16, device="cuda")

    def gate(self, rate):
        k = keep_count(rate, QWEN_INTER)
        pw, s, z, N, K = self.w["gate"]
        self.B.qlinear_ex(self.x, QWEN_HIDDEN, pw, s, z, None, self.M, K, N, None, K, None, k, self.yg, QWEN_INTER)
        return 2.0 * self.M * K * k

    def down(self, rate):
        k = keep_count(rate, QWEN_INTER)
        pw, s, z, N, K = self.w["down"]
        self.B.qlinear_ex(self.h, QWEN_INTER, pw, s, z, None, self.M, K, N, None, k, None, N, self.yd, QWEN_HIDDEN)
        return 2.0 * self.M * k * N


def prefill_tables(B, torch):
    """Tensor-core path: TFLOP/s of Qwen2.5-7B gate / down at M = 512, 2048 per keep rate (bf16)."""
    hbm, tf, which = measured_peaks()
    out = {}
    for M in (512, 2048):
        q = QwenPrefill(B, torch, M)
        for name, fn in (("gate", q.gate), ("down", q.down)):
            rows = {}
            for r in (1.0, 0.85, 0.65):
                for _ in range(3):
                    flops = fn(r)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                a.record()
                for _ in range(10):
                    fn(r)
                b.record()
                torch.cuda.synchronize()
                sec = a.elapsed_time(b) * 1e-3 / 10
                rows["%.2f" % r] = {"us": round(sec * 1e6, 1), "TFLOPs": round(flops / sec / 1e12, 1),
                                    "frac_bf16_%s" % which: round(flops / sec / 1e12 / tf, 3),
                                    "tokens_per_s": round(M / sec, 1)}
            out["prefill_qwen_%s_M%d" % (name, M)] = rows
        del q
        torch.cuda.empty_cache()
    # the whole Llama-3-8B SwiGLU block through its entry point (gate and up as a pair job with the gated product
    # in the epilogue, then down), bf16 and fp16
    from paper_2512_03383_b200 import synth
    rng = np.random.default_rng(11)
    ws = []
    for N, K in ((INTER, HIDDEN), (INTER, HIDDEN), (HIDDEN, INTER)):
        m = synth.random_qweight_fast(rng, N, K)
        cd = torch.from_numpy(m.codes).cuda()
        pw = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
        B.pack_u4(cd, pw)
        del cd
        ws.append((pw, torch.from_numpy(m.scales).cuda(), torch.from_numpy(m.zeros).cuda()))
    (wg, sg, zg), (wu, su, zu), (wd, sd, zd) = ws
    for M in (512, 2048):
        for dt, dname in ((torch.bfloat16, "bf16"), (torch.float16, "f16")):
            rows = {}
            x = torch.randn((M, HIDDEN), device="cuda").to(dt)
            for r in (1.0, 0.85, 0.65):
                k = keep_count(r, INTER) // 8 * 8
                h = torch.zeros((M, k), dtype=dt, device="cuda")
                y = torch.zeros((M, HIDDEN), dtype=dt, device="cuda")

                def one():
                    B.mlp_swiglu(x, HIDDEN, wg, sg, zg, wu, su, zu, wd, sd, zd, M, HIDDEN, INTER, k, h, k, y, HIDDEN)
                for _ in range(3):
                    one()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                a.record()
                for _ in range(10):
                    one()
                b.record()
                torch.cuda.synchronize()
                sec = a.elapsed_time(b) * 1e-3 / 10
                flops = 2.0 * M * HIDDEN * k * 3
                rows["%.2f" % r] = {"us": round(sec * 1e6, 1), "TFLOPs": round(flops / sec / 1e12, 1),
                                    "frac_bf16_%s" % which: round(flops / sec / 1e12 / tf, 3),
                                    "tokens_per_s": round(M / sec, 1)}
            out["prefill_llama_mlp_swiglu_%s_M%d" % (dname, M)] = rows
    return out


def attention_tables(B, torch, steps):
    """Llama-3-8B Q and K projection with the fused pruned RoPE (one launch): decode at M = 1, 16 and the
    tensor-core path at M = 512, per retained head dim.  Weights rotate over enough copies to exceed L2."""
    from paper_2512_03383_b200 import synth
    hbm, tf, which = measured_peaks()
    rng = np.random.default_rng(3)
    Hq, Hkv, D, K, theta = 32, 8, 128, HIDDEN, 500000.0
    n_copies = 12                                   # 12 x 13.4 MB (q, k, v) > 126 MB
    wq, wk = synth.random_qweight_fast(rng, Hq * D, K), synth.random_qweight_fast(rng, Hkv * D, K)
    wv = synth.random_qweight_fast(rng, Hkv * D, K)
    copies = []
    for _ in range(n_copies):
        c = []
        for m in (wq, wk, wv):
            cd = torch.from_numpy(m.codes).cuda()
            packed = torch.empty((m.N, m.K // 2), dtype=torch.uint8, device="cuda")
            B.pack_u4(cd, packed)
            c.append((packed, torch.from_numpy(m.scales).cuda().clone(), torch.from_numpy(m.zeros).cuda().clone()))
        copies.append(c)
    out = {}
    for M in (1, 16, 512):
        x = torch.from_numpy(synth.draw_x(rng, M, K, "f16")).cuda().half()
        pos = torch.from_numpy(synth.draw_pos(rng, M)).cuda()
        rows = {}
        for keep in (128, 108, 96, 84):
            idx = torch.from_numpy(synth.draw_idx(rng, Hkv, D, keep)).cuda()
            qo = torch.zeros((M, Hq * keep), dtype=torch.float16, device="cuda")
            ko = torch.zeros((M, Hkv * keep), dtype=torch.float16, device="cuda")
            turn = [0]

            def one():
                for _ in range(n_copies):
                    (q, k, _v) = copies[turn[0] % n_copies]
                    turn[0] += 1
                    B.qk_rope_proj(x, K, q[0], q[1], q[2], k[0], k[1], k[2], None, None, M, K, Hq, Hkv, D, keep, idx, pos,
                                   theta, None, qo, Hq * keep, ko, Hkv * keep)
            g, _ = capture(torch, one)
            for _ in range(3):
                g.replay()
            sec = time_graph(torch, g, steps) / (steps * n_copies)
            weights = (Hq + Hkv) * keep * K
            row = {"us": round(sec * 1e6, 2), "tokens_per_s": round(M / sec, 1)}
            if M <= 16:
                gbs = BYTES_PER_WEIGHT * weights / sec / 1e9
                row.update({"GBps": round(gbs, 1), "frac_hbm_%s" % which: round(gbs / hbm, 3)})
            else:
                tfl = 2.0 * M * weights / sec / 1e12
                row.update({"TFLOPs": round(tfl, 1), "frac_bf16_%s" % which: round(tfl / tf, 3)})
            rows["d%d" % keep] = row
            # Q, K and V in one launch, against the Q|K launch followed by a V launch
            vo = torch.zeros((M, Hkv * keep), dtype=torch.float16, device="cuda")
            vmap = synth.map_per_head(Hkv, D, keep)

            def one_qkv():
                for _ in range(n_copies):
                    (q, k, v) = copies[turn[0] % n_copies]
                    turn[0] += 1
                    B.qkv_rope_proj(x, K, q[0], q[1], q[2], k[0], k[1], k[2], v[0], v[1], v[2], None, None, None, M, K,
                                    Hq, Hkv, D, keep, keep, idx, pos, theta, None, qo, Hq * keep, ko, Hkv * keep, vo,
                                    Hkv * keep)

            def two_launches():
                for _ in range(n_copies):
                    (q, k, v) = copies[turn[0] % n_copies]
                    turn[0] += 1
                    B.qk_rope_proj(x, K, q[0], q[1], q[2], k[0], k[1], k[2], None, None, M, K, Hq, Hkv, D, keep, idx, pos,
                                   theta, None, qo, Hq * keep, ko, Hkv * keep)
                    B.qlinear_ex(x, K, v[0], v[1], v[2], None, M, K, Hkv * D, None, K, vmap, 0, vo, Hkv * keep)
            for name, fn in (("qkv_one_launch", one_qkv), ("qk_then_v", two_launches)):
                g, _ = capture(torch, fn)
                for _ in range(3):
                    g.replay()
                sec = time_graph(torch, g, steps) / (steps * n_copies)
                rows["d%d" % keep][name + "_us"] = round(sec * 1e6, 2)
        out["llama_qk_rope_M%d" % M] = rows
    return out


def run_case(args):
    """A few plain (un-graphed) launches of one kernel on a small set-up, for ncu captures:
    --case decode-gateup | decode-down | prefill-gate | prefill-down, with --M and --keep."""
    import torch
    from paper_2512_03383_b200 import binding as B
    torch.cuda.set_device(0)
    if args.case.startswith("prefill"):
        q = QwenPrefill(B, torch, args.M)
        for _ in range(args.launches):
            (q.gate if args.case == "prefill-gate" else q.down)(args.keep)
        torch.cuda.synchronize()
        print("case %s M=%d keep=%.2f: %d launches done" % (args.case, args.M, args.keep, args.launches))
        return 0
    w = MlpDecode(B, torch, args.M)
    k = keep_count(args.keep, INTER)
    for _ in range(args.launches):
        g, u, d = w.copies[w.turn % N_COPIES]
        w.turn += 1
        if args.case == "decode-gateup":
            jobs = [dict(packed_w=g[0], scales=g[1], zeros=g[2], N=INTER, k_out=k, y=w.yg, ldy=INTER),
                    dict(packed_w=u[0], scales=u[1], zeros=u[2], N=INTER, k_out=k, y=w.yu, ldy=INTER)]
            B.qlinear_multi(w.x, HIDDEN, args.M, HIDDEN, None, HIDDEN, jobs)
        elif args.case == "decode-down":
            B.qlinear_ex(w.h, INTER, d[0], d[1], d[2], None, args.M, INTER, HIDDEN, None, k, None, HIDDEN,
                         w.yd[0], HIDDEN)
        else:
            raise SystemExit("unknown case " + args.case)
    torch.cuda.synchronize()
    print("case %s M=%d keep=%.2f: %d launches done" % (args.case, args.M, args.keep, args.launches))
    return 0


# DRAM bytes (read + write) per algorithmic byte of a decode launch, from the ncu captures summarised in
# profiles/decode_kernel_llama3_gateup_m1.md (62.49 MB read + 0.14 MB written, mean of two launches, for 62.39 MB of retained weights)
# and profiles/decode_kernel_llama3_down_m1.md (31.31 MB for 31.20 MB); traffic grows in proportion to the
# retained weights, so the per-launch average of the step is scaled from the two.
# None once the kernel has changed since the captures.
DRAM_TRAFFIC_RATIO = (62.63 + 31.32) / (62.39 + 31.20)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true",
                    help="launch eagerly instead of replaying a CUDA graph (for profiler launch lists only)")
    ap.add_argument("--detail", action="store_true", help="also report M=4/16 and per-keep-rate tables")
    ap.add_argument("--case", default=None, help="run a few plain launches of one kernel (for ncu)")
    ap.add_argument("--M", type=int, default=1)
    ap.add_argument("--keep", type=float, default=1.0)
    ap.add_argument("--launches", type=int, default=4)
    args = ap.parse_args()
    if args.case:
        return run_case(args)
    if args.impl == "reference":
        if args.steps > 50:
            args.steps, args.warmup = 5, 1       # the oracle runs ~1 s per step
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
