"""GPU parity of the tensor-core (tcgen05) prefill kernel against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_output, dev_weight, dev_x
from paper_2512_03383_b200 import synth
from test_gpu_parity import run_ex, run_rope

pytestmark = pytest.mark.gpu

# The weights are de-quantised exactly in fp32 and rounded once to the activation type before they
# enter the tensor cores: up to 2^-11 relative per weight for fp16, 2^-8 for bf16; the errors are
# independent, so the output carries a few 1e-4 (fp16) or about 1e-3 (bf16) of its r.m.s., less relative
# to the largest output (measured: 2.1e-4 fp16).  fp32 accumulation adds ~1e-6.  fp16 is held to a quarter
# of the stated bar; so is bf16, whose tensor-core operands are fp16 as well (activations converted in shared memory).
TOL = {"f16": 5e-4, "bf16": 5e-4}


@pytest.fixture(scope="module")
def B():
    from paper_2512_03383_b200 import binding
    return binding


@pytest.fixture(autouse=True)
def _reset_path(B):
    yield
    B.set_path(B.PATH_AUTO)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M", [17, 64, 100, 128, 257, 600])
def test_prefill_m_sweep(B, M, dtype):
    B.set_path(B.PATH_PREFILL)
    rng = np.random.default_rng(500 + M)
    qw = synth.draw_qweight(rng, 300, 768)
    dw = dev_weight(qw)
    for (k_in, k_out) in [(768, 300), (652, 256), (72, 4), (200, 132)]:
        x = synth.draw_x(rng, M, k_in, dtype)
        y, ref = run_ex(B, qw, dw, x, dtype, None, k_in, None, k_out, ldx_pad=8 - k_in % 8 if k_in % 8 else 0, ldy_pad=3)
        check_output(y, ref, dtype, TOL[dtype], "prefill M=%d %s k=(%d,%d)" % (M, dtype, k_in, k_out))
    assert B.workspace_status() == 0


def test_prefill_auto_dispatch_and_bias(B):
    rng = np.random.default_rng(600)
    qw = synth.draw_qweight(rng, 384, 512)
    dw = dev_weight(qw)
    bias = synth.to_dtype_values(rng.standard_normal(384).astype(np.float32), "f16")
    x = synth.draw_x(rng, 192, 512, "f16")
    y, ref = run_ex(B, qw, dw, x, "f16", None, 512, None, 384, bias=bias)
    check_output(y, ref, "f16", TOL["f16"], "auto M=192 with bias")
    y2, _ = run_ex(B, qw, dw, x, "f16", None, 512, None, 384, bias=bias)
    assert torch.equal(y, y2)


@pytest.mark.parametrize("M", [64, 160])
def test_prefill_output_maps(B, M):
    """V-projection rows per head and Mamba in_proj rows (z|x per SSM head, then B, C, dt)."""
    B.set_path(B.PATH_PREFILL)
    rng = np.random.default_rng(610 + M)
    qw = synth.draw_qweight(rng, 512, 384)
    dw = dev_weight(qw)
    for keep in (128, 84):
        om = synth.map_per_head(4, 128, keep)
        x = synth.draw_x(rng, M, 384, "bf16")
        y, ref = run_ex(B, qw, dw, x, "bf16", None, 384, om, 0)
        check_output(y, ref, "bf16", TOL["bf16"], "per-head rows keep %d" % keep)
    nheads, headdim, d_state = 4, 64, 32
    d_inner = nheads * headdim
    rows = 2 * d_inner + 2 * d_state + nheads
    qin = synth.draw_qweight(rng, rows, 256)
    din = dev_weight(qin)
    om = synth.map_mamba_in_proj(d_inner, headdim, 48, d_state, 1, nheads)
    x = synth.draw_x(rng, M, 256, "f16")
    y, ref = run_ex(B, qin, din, x, "f16", None, 256, om, 0)
    check_output(y, ref, "f16", TOL["f16"], "mamba in_proj")


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M", [64, 200])
@pytest.mark.parametrize("keep", [128, 84])
def test_prefill_qk_rope(B, M, keep, dtype):
    B.set_path(B.PATH_PREFILL)
    rng = np.random.default_rng(700 + keep + M)
    for (g, ref) in run_rope(B, rng, M, 256, 6, 2, 128, keep, 1e6, dtype, bias=(keep == 84)):
        check_output(g, ref, dtype, TOL[dtype], "prefill rope keep %d M=%d %s" % (keep, M, dtype))


def test_prefill_bf16_converted_in_kernel(B, monkeypatch):
    """The fallback for workspaces too small for an fp16 copy of the activations: tiles are converted in
    shared memory.  Same result as the copy-first path, bit for bit."""
    B.set_path(B.PATH_PREFILL)
    rng = np.random.default_rng(650)
    qw = synth.draw_qweight(rng, 300, 768)
    dw = dev_weight(qw)
    x = synth.draw_x(rng, 300, 652, "bf16")
    y1, ref = run_ex(B, qw, dw, x, "bf16", None, 652, None, 256, ldx_pad=4)
    monkeypatch.setenv("UNIQL_PREFILL_CONVERT", "kernel")
    y2, _ = run_ex(B, qw, dw, x, "bf16", None, 652, None, 256, ldx_pad=4)
    check_output(y2, ref, "bf16", TOL["bf16"], "bf16 converted in kernel")
    assert torch.equal(y1, y2)


def test_prefill_multi_job(B):
    rng = np.random.default_rng(800)
    gate, up = synth.draw_qweight(rng, 352, 512), synth.draw_qweight(rng, 352, 512)
    dg, du = dev_weight(gate), dev_weight(up)
    M, k = 130, 300
    x = synth.draw_x(rng, M, 512, "bf16")
    xd = dev_x(x, "bf16")
    yg = torch.zeros((M, k), dtype=torch.bfloat16, device="cuda")
    yu = torch.zeros((M, k), dtype=torch.bfloat16, device="cuda")
    jobs = [dict(packed_w=dg[1], scales=dg[2], zeros=dg[3], N=352, k_out=k, y=yg, ldy=k),
            dict(packed_w=du[1], scales=du[2], zeros=du[3], N=352, k_out=k, y=yu, ldy=k)]
    B.qlinear_multi(xd, 512, M, 512, None, 512, jobs)
    torch.cuda.synchronize()
    for (q, d, y) in ((gate, dg, yg), (up, du, yu)):
        ref = oracle.qlinear(x, d[0], q.scales, q.zeros, oracle.leading(k), oracle.leading(512))
        check_output(y, ref, "bf16", TOL["bf16"], "multi")
