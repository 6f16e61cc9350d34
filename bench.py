#!/usr/bin/env python
"""Benchmark of the UniQL hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--no-tables]

Workload (N = 1 and every rank at N > 1): the Llama-3-8B-shaped SwiGLU MLP in decode, the
configuration the headline metric is quoted on -- hidden 4096, intermediate 14336, uint4 g=128
weights, batch M = 1, intermediate channels truncated at keep rates 1.0 / 0.85 / 0.75 / 0.65.
One step = for every keep rate one gate|up launch (two matrices, one launch) and one down launch,
i.e. the whole decode path (truncation, unpack, de-quantise, contraction) over one batch.
metric = effective weight GB/s: 0.53125 bytes per RETAINED weight (codes + fp16 scale and zero per
128) divided by device time.  Each launch reads a different one of four weight copies (375 MB in
rotation, L2 is 126 MB), so every byte comes from HBM.  Synthetic seeded inputs stand in for the
paper's checkpoints.  The step is captured in a CUDA graph and replayed, timed with CUDA events: the headline is the median of
REPEATS timed regions of --steps replays each (min and max are printed beside it).

The same line carries compact sub-records ("tables") for the rest of the metric, each with microseconds per
launch, achieved GB/s or TFLOP/s and the fraction of the measured peak: the decode MLP at M = 1, 4, 16 per keep
rate, the Llama-3-8B attention projections (q|k|v with the fused pruned RoPE in one launch, o_proj with per-head
input pruning) at M = 1, 16, 512 per retained head dim, the Qwen2.5-7B prefill linears (gate, down, q|k with RoPE)
at M = 512, 2048, the Mamba2-2.7B in/out projections at M = 1, 1024, and the two M = 1 MLP launches in isolation.
--no-tables skips them.
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
REPEATS = 11
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


def sustained_tflops():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"])
    except Exception:
        return 1400.0


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
            "config": {"workload": "llama3-8b-mlp-decode-M1", "keep_rates": list(KEEP_RATES),
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


QWEN_HIDDEN, QWEN_INTER = 3584, 18944


# --------------------------------------------------------------------------------------- sub-records
def dev_qweight(torch, N, K, seed):
    """Device-side seeded synthetic weights for the timing tables (values do not affect timing): uniform codes,
    scales of the magnitude the quantiser yields for N(0, 0.02) weights, zero-points around 8."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    packed = torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device="cuda", generator=g)
    s = (0.0075 * (1.0 + 0.1 * torch.randn((N, K // 128), device="cuda", generator=g))).half()
    z = torch.randint(6, 10, (N, K // 128), device="cuda", generator=g).half()
    return packed, s, z


def dev_x(torch, M, K, dtype, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return torch.randn((M, K), device="cuda", generator=g).to(dtype)


def time_rotating(torch, launch, n_copies, reps):
    """`launch(i)` enqueues one launch on copy i; a graph of n_copies launches is replayed reps times."""
    def seq():
        for i in range(n_copies):
            launch(i)
    g, _ = capture(torch, seq)
    for _ in range(3):
        g.replay()
    return time_graph(torch, g, reps) / (reps * n_copies)


def time_plain(torch, launch, reps):
    for _ in range(3):
        launch(0)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(reps):
        launch(0)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e-3 / reps


def rec_hbm(sec, weights, hbm, M):
    gbs = BYTES_PER_WEIGHT * weights / sec / 1e9
    return {"us": round(sec * 1e6, 2), "GBps": round(gbs, 1), "frac": round(gbs / hbm, 3), "tok_s": round(M / sec)}


def rec_tc(sec, flops, tf, tf_sus, M):
    t = flops / sec / 1e12
    return {"us": round(sec * 1e6, 1), "TFLOPs": round(t, 1), "frac": round(t / tf, 3),
            "frac_sustained": round(t / tf_sus, 3), "tok_s": round(M / sec)}


def tables(B, torch, work, reps=20):
    """The rest of the metric, per keep rate.  Decode-size launches (M <= 16) run as CUDA graphs over enough weight
    copies to exceed L2 and report effective weight GB/s against the measured HBM copy peak; launches of M >= 512
    report effective TFLOP/s against the measured bf16 GEMM peaks (burst, and sustained as frac_sustained)."""
    from paper_2512_03383_b200 import synth
    hbm, tf, which = measured_peaks()
    tf_sus = sustained_tflops()
    f16, bf16 = torch.float16, torch.bfloat16
    out = {"peaks": {"hbm_GBps": hbm, "bf16_TFLOPs_burst": tf, "bf16_TFLOPs_sustained": tf_sus, "source": which},
           "note": "frac = achieved / measured peak; decode rows: retained weight bytes only, rotating weight copies "
                   "larger than L2, CUDA graph; M >= 512 rows: 2*M*k_in*k_out flops, plain launches, CUDA events"}

    # ---- Llama-3-8B MLP at decode sizes: gate|up (one launch) + down, per keep rate; the M = 1 launches alone
    mlp = {}
    for M in (1, 4, 16):
        w = work if M == 1 else MlpDecode(B, torch, M)
        rows = {}
        for r in KEEP_RATES:
            k = keep_count(r, INTER)

            def one(i, k=k, w=w, M=M):
                g, u, d = w.copies[i]
                jobs = [dict(packed_w=g[0], scales=g[1], zeros=g[2], N=INTER, k_out=k, y=w.yg, ldy=INTER),
                        dict(packed_w=u[0], scales=u[1], zeros=u[2], N=INTER, k_out=k, y=w.yu, ldy=INTER)]
                B.qlinear_multi(w.x, HIDDEN, M, HIDDEN, None, HIDDEN, jobs)
                B.qlinear_ex(w.h, INTER, d[0], d[1], d[2], None, M, INTER, HIDDEN, None, k, None, HIDDEN, w.yd[0], HIDDEN)
            rows["%.2f" % r] = rec_hbm(time_rotating(torch, one, N_COPIES, reps), 3 * HIDDEN * k, hbm, M)
        mlp["M%d" % M] = rows
        if M == 1:
            iso = {}
            for r in (1.0, 0.65):
                k = keep_count(r, INTER)

                def gu(i, k=k, w=w):
                    g, u, d = w.copies[i]
                    jobs = [dict(packed_w=g[0], scales=g[1], zeros=g[2], N=INTER, k_out=k, y=w.yg, ldy=INTER),
                            dict(packed_w=u[0], scales=u[1], zeros=u[2], N=INTER, k_out=k, y=w.yu, ldy=INTER)]
                    B.qlinear_multi(w.x, HIDDEN, 1, HIDDEN, None, HIDDEN, jobs)

                def dn(i, k=k, w=w):
                    d = w.copies[i][2]
                    B.qlinear_ex(w.h, INTER, d[0], d[1], d[2], None, 1, INTER, HIDDEN, None, k, None, HIDDEN, w.yd[0], HIDDEN)
                for nm, fn, wts in (("gate_up", gu, 2 * HIDDEN * k), ("down", dn, HIDDEN * k)):
                    # the same launch repeated in a graph (back to back, overlapping launch set-up), and one launch at a
                    # time with the device idle before it (a synchronize between launches: the stand-alone latency)
                    row = rec_hbm(time_rotating(torch, fn, N_COPIES, reps), wts, hbm, 1)
                    ts = []
                    for j in range(12):
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        torch.cuda.synchronize()
                        a.record()
                        fn(j % N_COPIES)
                        b.record()
                        torch.cuda.synchronize()
                        ts.append(a.elapsed_time(b) * 1e-3)
                    row["isolated_us"] = round(statistics.median(ts[2:]) * 1e6, 2)
                    iso["%s_%.2f" % (nm, r)] = row
            mlp["M1_single_launches"] = iso
        if M != 1:
            del w
            torch.cuda.empty_cache()
    out["llama3_mlp_decode"] = mlp

    # ---- Llama-3-8B attention projections: q|k|v + pruned RoPE in one launch, o_proj with per-head input pruning
    Hq, Hkv, D, K, theta = 32, 8, 128, HIDDEN, 500000.0
    n_cp = 8                                               # 8 x 22 MB of q, k, v, o weights > L2
    att_w = [[dev_qweight(torch, n, K, 100 + 4 * c + j) for j, n in enumerate((Hq * D, Hkv * D, Hkv * D, HIDDEN))]
             for c in range(n_cp)]
    rng = np.random.default_rng(3)
    att = {}
    for M in (1, 16, 512):
        x = dev_x(torch, M, K, f16, 7)
        pos = torch.from_numpy(synth.draw_pos(rng, M)).cuda()
        rows = {}
        for keep in (128, 108, 96, 84):
            idx = torch.from_numpy(synth.draw_idx(rng, Hkv, D, keep)).cuda()
            qo = torch.zeros((M, Hq * keep), dtype=f16, device="cuda")
            ko = torch.zeros((M, Hkv * keep), dtype=f16, device="cuda")
            vo = torch.zeros((M, Hkv * keep), dtype=f16, device="cuda")
            ao = dev_x(torch, M, Hq * keep, f16, 8)        # attention output: the o_proj input, compact per head
            yo = torch.zeros((M, HIDDEN), dtype=f16, device="cuda")
            omap = synth.map_per_head(Hq, D, keep)

            def qkv(i):
                q, k, v, _ = att_w[i]
                B.qkv_rope_proj(x, K, q[0], q[1], q[2], k[0], k[1], k[2], v[0], v[1], v[2], None, None, None, M, K, Hq,
                                Hkv, D, keep, keep, idx, pos, theta, None, qo, Hq * keep, ko, Hkv * keep, vo, Hkv * keep)

            def oproj(i):
                o = att_w[i][3]
                B.qlinear_ex(ao, Hq * keep, o[0], o[1], o[2], None, M, Hq * D, HIDDEN, omap, 0, None, HIDDEN, yo, HIDDEN)
            w_qkv, w_o = (Hq + 2 * Hkv) * keep * K, Hq * keep * HIDDEN
            if M <= 16:
                rows["d%d" % keep] = {"qkv_rope": rec_hbm(time_rotating(torch, qkv, n_cp, reps), w_qkv, hbm, M),
                                      "o_proj": rec_hbm(time_rotating(torch, oproj, n_cp, reps), w_o, hbm, M)}
            else:
                rows["d%d" % keep] = {"qkv_rope": rec_tc(time_plain(torch, qkv, 10), 2.0 * M * w_qkv, tf, tf_sus, M),
                                      "o_proj": rec_tc(time_plain(torch, oproj, 10), 2.0 * M * w_o, tf, tf_sus, M)}
        att["M%d" % M] = rows
    del att_w
    torch.cuda.empty_cache()
    out["llama3_attention"] = att

    # ---- Qwen2.5-7B prefill linears (bf16): gate (rows pruned), down (columns pruned), q|k with the fused RoPE
    QH, QI, QHq, QHkv, qtheta = QWEN_HIDDEN, QWEN_INTER, 28, 4, 1e6
    wgate, wdown = dev_qweight(torch, QI, QH, 201), dev_qweight(torch, QH, QI, 202)
    wq, wk = dev_qweight(torch, QHq * 128, QH, 203), dev_qweight(torch, QHkv * 128, QH, 204)
    qwen = {}
    for M in (512, 2048):
        x = dev_x(torch, M, QH, bf16, 9)
        hh = dev_x(torch, M, QI, bf16, 10)
        yg = torch.zeros((M, QI), dtype=bf16, device="cuda")
        yd = torch.zeros((M, QH), dtype=bf16, device="cuda")
        pos = torch.from_numpy(synth.draw_pos(rng, M)).cuda()
        rows = {}
        for r in (1.0, 0.85, 0.65):
            k = keep_count(r, QI)
            keep = keep_count(r, 128)
            idx = torch.from_numpy(synth.draw_idx(rng, QHkv, 128, keep)).cuda()
            qo = torch.zeros((M, QHq * keep), dtype=bf16, device="cuda")
            ko = torch.zeros((M, QHkv * keep), dtype=bf16, device="cuda")

            def gate(i):
                B.qlinear_ex(x, QH, wgate[0], wgate[1], wgate[2], None, M, QH, QI, None, QH, None, k, yg, QI)

            def down(i):
                B.qlinear_ex(hh, QI, wdown[0], wdown[1], wdown[2], None, M, QI, QH, None, k, None, QH, yd, QH)

            def qk(i):
                B.qk_rope_proj(x, QH, wq[0], wq[1], wq[2], wk[0], wk[1], wk[2], None, None, M, QH, QHq, QHkv, 128, keep,
                               idx, pos, qtheta, None, qo, QHq * keep, ko, QHkv * keep)
            rows["%.2f" % r] = {"gate": rec_tc(time_plain(torch, gate, 10), 2.0 * M * QH * k, tf, tf_sus, M),
                                "down": rec_tc(time_plain(torch, down, 10), 2.0 * M * QH * k, tf, tf_sus, M),
                                "qk_rope": rec_tc(time_plain(torch, qk, 10), 2.0 * M * QH * (QHq + QHkv) * keep, tf, tf_sus, M)}
        qwen["M%d" % M] = rows
        del x, hh, yg, yd
    del wgate, wdown, wq, wk
    torch.cuda.empty_cache()
    out["qwen25_prefill_bf16"] = qwen

    # ---- Mamba2-2.7B in_proj (rows z|x|B|C|dt, z and x pruned per SSM head) and out_proj (columns per head), fp16
    d_model, d_inner, d_state, headdim, nheads = 2560, 5120, 128, 64, 80
    rows_in = 2 * d_inner + 2 * d_state + nheads
    n_cp = 8                                               # 8 x 21 MB > L2
    mw = [(dev_qweight(torch, rows_in, d_model, 300 + c), dev_qweight(torch, d_model, d_inner, 320 + c)) for c in range(n_cp)]
    mamba = {}
    for M in (1, 1024):
        x = dev_x(torch, M, d_model, f16, 11)
        rows = {}
        for keep in (64, 56, 48):
            om = synth.map_mamba_in_proj(d_inner, headdim, keep, d_state, 1, nheads)
            im = synth.map_per_head(nheads, headdim, keep)
            n_out = synth.map_size(om)
            yin = torch.zeros((M, n_out), dtype=f16, device="cuda")
            xo = dev_x(torch, M, nheads * keep, f16, 12)
            yo = torch.zeros((M, d_model), dtype=f16, device="cuda")

            def inp(i):
                w = mw[i][0]
                B.qlinear_ex(x, d_model, w[0], w[1], w[2], None, M, d_model, rows_in, None, d_model, om, 0, yin, n_out)

            def outp(i):
                w = mw[i][1]
                B.qlinear_ex(xo, nheads * keep, w[0], w[1], w[2], None, M, d_inner, d_model, im, 0, None, d_model, yo, d_model)
            w_in, w_out = n_out * d_model, d_model * nheads * keep
            if M == 1:
                rows["hd%d" % keep] = {"in_proj": rec_hbm(time_rotating(torch, inp, n_cp, reps), w_in, hbm, M),
                                       "out_proj": rec_hbm(time_rotating(torch, outp, n_cp, reps), w_out, hbm, M)}
            else:
                rows["hd%d" % keep] = {"in_proj": rec_tc(time_plain(torch, inp, 10), 2.0 * M * w_in, tf, tf_sus, M),
                                       "out_proj": rec_tc(time_plain(torch, outp, 10), 2.0 * M * w_out, tf, tf_sus, M)}
        mamba["M%d" % M] = rows
    del mw
    torch.cuda.empty_cache()
    out["mamba2_27b_fp16"] = mamba

    # ---- Hybrid model (the Mamba2 mixer of a Bamba-v2-9B-shaped layer: d_model 4096, d_inner 8192, 128 SSM heads of
    #      64 channels, one group of 128 states; shapes from the public model card, synthetic weights), fp16:
    #      in_proj with z / x pruned per SSM head AND the state dimension D_s pruned (the leading rows of B and of C:
    #      Section 3.2, SSM paragraph), out_proj with its input columns pruned per head.  Its attention and MLP
    #      blocks have the Llama-3-8B shapes of the tables above.
    d_model, d_inner, d_state, headdim, nheads = 4096, 8192, 128, 64, 128
    rows_in = 2 * d_inner + 2 * d_state + nheads
    n_cp = 3                                               # 3 x 53 MB > L2
    hw = [(dev_qweight(torch, rows_in, d_model, 400 + c), dev_qweight(torch, d_model, d_inner, 420 + c)) for c in range(n_cp)]
    hybrid = {}
    for M in (1, 1024):
        x = dev_x(torch, M, d_model, f16, 13)
        rows = {}
        for (keep, skeep) in ((64, 128), (56, 112), (48, 96), (40, 80)):
            om = synth.map_mamba_in_proj(d_inner, headdim, keep, d_state, 1, nheads, state_keep=skeep)
            im = synth.map_per_head(nheads, headdim, keep)
            n_out = synth.map_size(om)
            yin = torch.zeros((M, n_out), dtype=f16, device="cuda")
            xo = dev_x(torch, M, nheads * keep, f16, 14)
            yo = torch.zeros((M, d_model), dtype=f16, device="cuda")

            def inp(i):
                w = hw[i][0]
                B.qlinear_ex(x, d_model, w[0], w[1], w[2], None, M, d_model, rows_in, None, d_model, om, 0, yin, n_out)

            def outp(i):
                w = hw[i][1]
                B.qlinear_ex(xo, nheads * keep, w[0], w[1], w[2], None, M, d_inner, d_model, im, 0, None, d_model, yo, d_model)
            w_in, w_out = n_out * d_model, d_model * nheads * keep
            key = "hd%d_ds%d" % (keep, skeep)
            if M == 1:
                rows[key] = {"in_proj": rec_hbm(time_rotating(torch, inp, n_cp, reps), w_in, hbm, M),
                             "out_proj": rec_hbm(time_rotating(torch, outp, n_cp, reps), w_out, hbm, M)}
            else:
                rows[key] = {"in_proj": rec_tc(time_plain(torch, inp, 10), 2.0 * M * w_in, tf, tf_sus, M),
                             "out_proj": rec_tc(time_plain(torch, outp, 10), 2.0 * M * w_out, tf, tf_sus, M)}
        hybrid["M%d" % M] = rows
    del hw
    torch.cuda.empty_cache()
    out["hybrid_bamba_v2_9b_mixer_fp16"] = hybrid

    # derived per-model decode figure (layer counts are the public model-card values, not the paper's): the MLP
    # and attention-projection launches of one Llama-3-8B layer at M = 1, keep 1.0 and 0.65, times 32 layers
    try:
        d = {}
        for r, dk in (("1.00", "d128"), ("0.65", "d84")):
            us = mlp["M1"][r]["us"] + att["M1"][dk]["qkv_rope"]["us"] + att["M1"][dk]["o_proj"]["us"]
            d["keep_" + r] = {"us_per_layer_linears": round(us, 2), "tok_s_32_layers_linears_only": round(1e6 / (32 * us), 1)}
        out["derived_llama3_8b_decode"] = d
    except Exception:
        pass
    return out


def prefill_oracle_slab(budget_rows=64):
    """The oracle as it stands on a bounded slab of the largest prefill launch (Qwen2.5-7B gate, M = 2048, keep 1.0):
    64 token rows (tile-boundary rows included) x all 18944 outputs, reported as GFLOP/s."""
    import oracle
    from paper_2512_03383_b200 import synth
    rng = np.random.default_rng(1)
    qw = synth.random_qweight_fast(rng, QWEN_INTER, QWEN_HIDDEN)
    pk = oracle.pack_u4(qw.codes)
    M = 2048
    rows = sorted(set([0, 63, 64, 127, 128, M - 1] + list(range(256, 256 + budget_rows - 6))))
    x = synth.draw_x(rng, len(rows), QWEN_HIDDEN, "bf16")
    t0 = time.time()
    oracle.qlinear(x, pk, qw.scales, qw.zeros, oracle.leading(QWEN_INTER), oracle.leading(QWEN_HIDDEN))
    sec = time.time() - t0
    flops = 2.0 * len(rows) * QWEN_INTER * QWEN_HIDDEN
    return {"value": round(flops / sec / 1e9, 2), "unit": "GFLOP/s", "cores": oracle.threads(), "kind": "oracle",
            "sample": "qwen2.5-7b gate, keep 1.0: %d of 2048 token rows x 18944 outputs, %.2f s" % (len(rows), sec)}


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

    # REPEATS timed regions of --steps replays each (every region bracketed by a barrier + synchronize, CUDA events on
    # the stream the graph runs on); the headline is the median region, max over ranks
    secs = [time_graph(torch, graph, args.steps, barrier) for _ in range(REPEATS)]
    barrier()
    for _ in range(3):
        graph_e2e.replay()
    secs_e2e = [time_graph(torch, graph_e2e, args.steps, barrier) for _ in range(REPEATS)]
    t_end = time.time()
    clocks = sampler.stop(t_load, t_end) if rank == 0 else None

    secs = max_over_ranks(dist, torch, secs, "cuda")
    secs_e2e = max_over_ranks(dist, torch, secs_e2e, "cuda")
    sec, sec_e2e = statistics.median(secs), statistics.median(secs_e2e)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    hbm, tf, which = measured_peaks()
    value = whole_job_value(step_bytes(), args.steps, world, sec)
    launches = work.launches_per_step * args.steps
    traffic_ratio, traffic_note = dram_traffic_ratio()
    per_launch_bytes = step_bytes() / work.launches_per_step
    per_launch_sec = sec / launches
    achieved = per_launch_bytes / per_launch_sec / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": sec / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": "llama3-8b-mlp-decode-M1", "hidden": HIDDEN,
                   "intermediate": INTER, "keep_rates": list(KEEP_RATES), "M": 1,
                   "l2": "4 rotating weight copies (375 MB) > 126 MB L2", "parallelism": "replicas x%d" % world,
                   "timing": ("eager launches (profiling mode, host-bound: not a bench value), CUDA events" if args.no_graph
                              else "CUDA graph of one step replayed, CUDA events")},
        "tokens_per_s_mlp": args.steps * len(KEEP_RATES) * world / sec,
        "repeats": {"n": REPEATS, "statistic": "median", "GBps_min": whole_job_value(step_bytes(), args.steps, world, max(secs)),
                    "GBps_max": whole_job_value(step_bytes(), args.steps, world, min(secs)),
                    "ms_per_step_min": min(secs) / args.steps * 1e3, "ms_per_step_max": max(secs) / args.steps * 1e3},
        "gpu_launches": launches * REPEATS,
        "gpu_launches_note": "%d launches per step x %d steps x %d timed regions (the e2e regions launch as many again)" % (
            work.launches_per_step, args.steps, REPEATS),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm,
                     "traffic": None if traffic_ratio is None else traffic_ratio * per_launch_bytes,
                     "traffic_source": traffic_note, "peak_source": which,
                     "kernel": "decode_kernel (integer path, M=1)", "algorithmic_bytes_per_launch": per_launch_bytes,
                     "frac_of_nominal_8TBs": achieved / 8000.0},
        "e2e": {"value": whole_job_value(step_bytes(), args.steps, world, sec_e2e), "unit": "GB/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "the step's activations copied from pinned host memory before its first launch, all its results to pinned host memory after its last, every step; weights resident"},
    }
    if world == 1:
        line["cpu_baseline"] = oracle_leg(3.0)
        if not args.no_tables:
            line["tables"] = tables(B, torch, work)
            line["tables"]["qwen25_prefill_bf16"]["cpu_baseline"] = prefill_oracle_slab()
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


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


def run_case(args):
    """A few plain (un-graphed) launches of one kernel on a small set-up, for ncu captures:
    --case decode-gateup | decode-down | decode-big | prefill-gate | prefill-down, with --M and --keep (and --gemv)."""
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
    if args.gemv:
        B.set_option("gemv_first", 1)           # the streaming kernel wherever it applies (M <= 4)
    if args.case == "decode-big":
        # one tall matrix (65536 x 4096, 140 MB: larger than L2), plain launches
        N = 65536
        ws = [dev_qweight(torch, N, HIDDEN, 50 + i) for i in range(2)]
        x = dev_x(torch, args.M, HIDDEN, torch.float16, 5)
        y = torch.zeros((args.M, N), dtype=torch.float16, device="cuda")
        for i in range(args.launches):
            w = ws[i % 2]
            B.qlinear_ex(x, HIDDEN, w[0], w[1], w[2], None, args.M, HIDDEN, N, None, HIDDEN, None, N, y, N)
        torch.cuda.synchronize()
        print("case %s M=%d gemv=%d: %d launches done" % (args.case, args.M, int(args.gemv), args.launches))
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


TRAFFIC_FILE = os.path.join(ROOT, "profiles", "decode_kernel_dram_traffic.txt")
KERNEL_SOURCES = ("decode.cu", "common.cuh", "quant.cuh")


def kernel_source_hash():
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2512_03383_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def dram_traffic_ratio():
    """DRAM bytes (read + write) per algorithmic byte of a decode launch, from the ncu captures recorded in
    profiles/decode_kernel_dram_traffic.txt together with a hash of the kernel's sources at capture time.  Traffic
    grows in proportion to the retained weights, so the step's per-launch average is scaled from the two captured
    launches (gate|up and down at keep 1.0).  None once the sources have changed since the capture."""
    try:
        kv = {}
        with open(TRAFFIC_FILE) as f:
            for ln in f:
                if "=" in ln and not ln.startswith("#"):
                    k, v = ln.split("=", 1)
                    kv[k.strip()] = v.strip()
        if kv["kernel_source_sha256_16"] != kernel_source_hash():
            return None, "stale: kernel sources changed since the capture in profiles/decode_kernel_dram_traffic.txt"
        dram = float(kv["gateup_dram_bytes"]) + float(kv["down_dram_bytes"])
        algo = float(kv["gateup_algorithmic_bytes"]) + float(kv["down_algorithmic_bytes"])
        return dram / algo, "profiles/decode_kernel_dram_traffic.txt"
    except Exception as e:                                   # no capture on record
        return None, "no capture on record (%s)" % type(e).__name__


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true",
                    help="launch eagerly instead of replaying a CUDA graph (for profiler launch lists only)")
    ap.add_argument("--no-tables", action="store_true", help="headline only: skip the per-configuration sub-records")
    ap.add_argument("--traffic-hash", action="store_true", help="print the hash of the decode kernel's sources")
    ap.add_argument("--case", default=None, help="run a few plain launches of one kernel (for ncu)")
    ap.add_argument("--M", type=int, default=1)
    ap.add_argument("--keep", type=float, default=1.0)
    ap.add_argument("--launches", type=int, default=4)
    ap.add_argument("--gemv", action="store_true", help="with --case: run the streaming kernel wherever it applies")
    args = ap.parse_args()
    if args.traffic_hash:
        print(kernel_source_hash())
        return 0
    if args.case:
        return run_case(args)
    if args.impl == "reference":
        if args.steps > 50:
            args.steps, args.warmup = 5, 1       # the oracle runs ~1 s per step
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
