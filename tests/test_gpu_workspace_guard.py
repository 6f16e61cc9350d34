"""A caller workspace of exactly the advertised size is enough and nothing is written behind it: the workspace
sits in front of a band of canary bytes that must survive every kind of launch (split input channels, streamed
activations of 5..16 rows, re-laid activations, tiles split along K on the tensor cores, the fp16 copy of bf16
activations, the SwiGLU block)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_output, dev_weight, dev_x
from paper_2512_03383_b200 import synth
from test_gpu_parity import run_ex
from test_gpu_mlp import draw_mlp, run_mlp, TOL_H, TOL_Y

pytestmark = pytest.mark.gpu
BAND = 1 << 20
CANARY = 0xA5


@pytest.fixture(scope="module")
def B():
    from paper_2512_03383_b200 import binding
    return binding


@pytest.fixture(autouse=True)
def _reset(B):
    yield
    B.set_path(B.PATH_AUTO)
    B.reset_options()


def guarded(B, nbytes):
    buf = torch.full((nbytes + BAND,), CANARY, dtype=torch.uint8, device="cuda")
    ws = buf[:nbytes]
    B.workspace_init(ws)
    return buf, ws


def band_intact(buf, nbytes):
    torch.cuda.synchronize()
    return bool((buf[nbytes:] == CANARY).all())


@pytest.mark.parametrize("M", [1, 4, 7, 8, 9, 16, 40, 300, 700])
def test_linear_layers_stay_inside_the_advertised_workspace(B, M):
    rng = np.random.default_rng(1200 + M)
    dtype = "f16"
    for (N, K, k_in, k_out) in [(200, 2304, 2304, 200), (70, 8192, 8192, 70), (330, 1024, 1020, 330), (1100, 512, 512, 1100)]:
        qw = synth.draw_qweight(rng, N, K)
        dw = dev_weight(qw)
        nbytes = B.workspace_bytes(M, K, N)
        buf, ws = guarded(B, nbytes)
        x = synth.draw_x(rng, M, k_in, dtype)
        for opts in ({}, {"decode_kp": 3, "decode_rp": 5}, {"decode_xstream": 1}, {"prefill_streamk": 1, "prefill_grid": 5},
                     {"prefill_streamk": 1, "prefill_grid": 5, "prefill_dual": 1}):
            B.reset_options()
            for k, v in opts.items():
                B.set_option(k, v)
            y, ref = run_ex(B, qw, dw, x, dtype, None, k_in, None, k_out, ldy_pad=3, workspace=ws)
            check_output(y, ref, dtype, 5e-4, "M=%d %s %s" % (M, (N, K, k_in, k_out), opts))
            assert band_intact(buf, nbytes), "wrote behind the workspace: M=%d %s %s" % (M, (N, K), opts)
            assert B.workspace_status(ws) == 0
    # per-head input maps with keep counts off the 8-channel grid: the activations are re-laid inside the workspace
    qw = synth.draw_qweight(rng, 256, 1024)
    dw = dev_weight(qw)
    im = synth.map_per_head(8, 128, 108)
    nbytes = B.workspace_bytes(M, 1024, 256)
    buf, ws = guarded(B, nbytes)
    x = synth.draw_x(rng, M, synth.map_size(im), dtype)
    y, ref = run_ex(B, qw, dw, x, dtype, im, 0, None, 256, workspace=ws)
    check_output(y, ref, dtype, 5e-4, "re-laid M=%d" % M)
    assert band_intact(buf, nbytes)


@pytest.mark.parametrize("M", [40, 300, 600])
def test_bf16_copy_and_split_tiles_stay_inside(B, M):
    rng = np.random.default_rng(1300 + M)
    qw = synth.draw_qweight(rng, 300, 1024)
    dw = dev_weight(qw)
    nbytes = B.workspace_bytes(M, 1024, 300)
    buf, ws = guarded(B, nbytes)
    x = synth.draw_x(rng, M, 1024, "bf16")
    for opts in ({}, {"prefill_streamk": 1, "prefill_grid": 7}, {"prefill_streamk": 1, "prefill_grid": 7, "prefill_dual": 1}):
        B.reset_options()
        for k, v in opts.items():
            B.set_option(k, v)
        y, ref = run_ex(B, qw, dw, x, "bf16", None, 1024, None, 300, workspace=ws)
        check_output(y, ref, "bf16", 5e-4, "bf16 M=%d %s" % (M, opts))
        assert band_intact(buf, nbytes), "wrote behind the workspace: bf16 M=%d %s" % (M, opts)
        assert B.workspace_status(ws) == 0


@pytest.mark.parametrize("M", [1, 5, 8, 11, 16, 64])
def test_mlp_block_stays_inside(B, M):
    _, qs, ds = draw_mlp(77, 512, 1024)
    x = synth.draw_x(np.random.default_rng(1400 + M), M, 512, "f16")
    nbytes = B.mlp_workspace_bytes(M, 512, 1024)
    buf, ws = guarded(B, nbytes)
    for k_int in (1024, 872):
        h, h_ref, y, y_ref = run_mlp(B, qs, ds, x, k_int, -1, workspace=ws)
        # (above 16 rows the block runs on the tensor cores, whose weights are rounded to fp16 first: 5e-4 there)
        check_output(h, h_ref, "f16", TOL_H if M <= 16 else 6e-4, "h M=%d" % M)
        check_output(y, y_ref, "f16", TOL_Y, "y M=%d" % M)
        assert band_intact(buf, nbytes), "wrote behind the workspace: MLP M=%d" % M
