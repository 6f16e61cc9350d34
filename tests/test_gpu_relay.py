"""Input maps on 4- but not 8-channel boundaries above four rows (head dims 108 and 84 on the input side of o_proj /
out_proj, 1740 leading channels with a row pitch of 1740): the activations are re-laid with every kept block padded
to a multiple of 8 channels by a small kernel in front, and the launch then runs on the integer path of the decode
kernel (5..16 rows) or on the tensor cores (more rows, bf16).  Forcing those paths must succeed for such maps, and
the results must match the oracle; a caller workspace without room for the copy still gives correct results."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_output, dev_weight, dev_x
from paper_2512_03383_b200 import synth

pytestmark = pytest.mark.gpu

TOL = {"decode": 4e-4, "prefill": 5e-4}


@pytest.fixture(scope="module")
def B():
    from paper_2512_03383_b200 import binding
    return binding


@pytest.fixture(autouse=True)
def _reset(B):
    yield
    B.set_path(B.PATH_AUTO)
    B.reset_options()


def run(B, qw, dw, x32, dtype, in_map, k_in, ldx_pad=0, workspace=None):
    packed, wp, ws, wz = dw
    M = x32.shape[0]
    n_in = synth.map_size(in_map) if in_map else k_in
    td = torch.float16 if dtype == "f16" else torch.bfloat16
    xd = torch.full((M, n_in + ldx_pad), 7.0, device="cuda", dtype=td)
    xd[:, :n_in] = dev_x(x32, dtype)
    y = torch.full((M, qw.N + 3), -77.0, device="cuda", dtype=td)
    B.qlinear_ex(xd, xd.stride(0), wp, ws, wz, None, M, qw.K, qw.N, in_map, k_in, None, qw.N, y, y.stride(0),
                 workspace=workspace)
    torch.cuda.synchronize()
    assert B.workspace_status(workspace) == 0
    assert (y[:, qw.N:] == -77.0).all()
    I = oracle.expand_map(in_map) if in_map else oracle.leading(k_in)
    return y[:, :qw.N], oracle.qlinear(x32, packed, qw.scales, qw.zeros, oracle.leading(qw.N), I)


@pytest.mark.parametrize("M", [5, 8, 9, 16])
@pytest.mark.parametrize("forced", [False, True])
def test_decode_sizes_per_head_108_84(B, M, forced):
    B.set_path(B.PATH_DECODE if forced else B.PATH_AUTO)
    rng = np.random.default_rng(820 + M)
    qw = synth.draw_qweight(rng, 256, 1024)
    dw = dev_weight(qw)
    for keep in (108, 84, 4):
        in_map = synth.map_per_head(8, 128, keep)
        x = synth.draw_x(rng, M, synth.map_size(in_map), "f16")
        y, ref = run(B, qw, dw, x, "f16", in_map, 0, ldx_pad=2)
        check_output(y, ref, "f16", TOL["decode"], "decode per-head keep %d M=%d" % (keep, M))
    x = synth.draw_x(rng, M, 876, "f16")                       # a leading block of 876 channels, pitch 876 + 2
    y, ref = run(B, qw, dw, x, "f16", None, 876, ldx_pad=2)
    check_output(y, ref, "f16", TOL["decode"], "decode leading 876 M=%d" % M)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M", [5, 17, 64, 300])
@pytest.mark.parametrize("forced", [False, True])
def test_tensor_core_sizes_per_head_108_84(B, M, dtype, forced):
    if M <= 16 and dtype == "f16" and forced:
        pytest.skip("fp16 decode sizes are covered above")
    B.set_path(B.PATH_PREFILL if forced else B.PATH_AUTO)       # forcing the tensor-core path must not be refused
    rng = np.random.default_rng(840 + M)
    qw = synth.draw_qweight(rng, 200, 1024)
    dw = dev_weight(qw)
    for (hd, keep) in ((128, 108), (128, 84), (64, 52)):
        in_map = synth.map_per_head(1024 // hd, hd, keep)
        x = synth.draw_x(rng, M, synth.map_size(in_map), dtype)
        y, ref = run(B, qw, dw, x, dtype, in_map, 0, ldx_pad=4)
        check_output(y, ref, dtype, TOL["prefill"], "tensor cores per-head keep %d of %d M=%d %s" % (keep, hd, M, dtype))
    x = synth.draw_x(rng, M, 1740 // 2, dtype)                  # 870 leading channels, pitch 870: rows 4-byte aligned only
    y, ref = run(B, qw, dw, x, dtype, None, 870)
    check_output(y, ref, dtype, TOL["prefill"], "tensor cores leading 870 M=%d %s" % (M, dtype))


def test_workspace_without_room_still_correct(B):
    """A caller workspace that holds the kernel's own needs but not the copy: the launch falls back to the kernels
    that read the activations where they are."""
    rng = np.random.default_rng(860)
    qw = synth.draw_qweight(rng, 128, 1024)
    dw = dev_weight(qw)
    in_map = synth.map_per_head(8, 128, 108)
    for M in (8, 40):
        need = B.workspace_bytes(M, 1024, 128)
        small = need - (M * (1024 + 8) * 2 + 255) // 256 * 256 - 512          # what the size query adds for the copy
        ws = torch.zeros(small, dtype=torch.uint8, device="cuda")
        B.workspace_init(ws)
        x = synth.draw_x(rng, M, synth.map_size(in_map), "f16")
        y, ref = run(B, qw, dw, x, "f16", in_map, 0, workspace=ws)
        check_output(y, ref, "f16", 5e-4, "small workspace M=%d" % M)
        ws2 = torch.zeros(need, dtype=torch.uint8, device="cuda")
        B.workspace_init(ws2)
        y2, _ = run(B, qw, dw, x, "f16", in_map, 0, workspace=ws2)
        check_output(y2, ref, "f16", 5e-4, "full workspace M=%d" % M)


@pytest.mark.parametrize("M", [1, 7, 16])
def test_fp16_mma_path_of_the_decode_kernel(B, M):
    """The second arithmetic path of the persistent decode kernel (fp16 MMAs on exact fp16 operands), switched on for
    shapes the integer path would take."""
    B.set_path(B.PATH_DECODE)
    B.set_option("decode_i8", 0)
    rng = np.random.default_rng(880 + M)
    qw = synth.draw_qweight(rng, 200, 1024)
    dw = dev_weight(qw)
    for k_in in (1024, 872):
        x = synth.draw_x(rng, M, k_in, "f16")
        y, ref = run(B, qw, dw, x, "f16", None, k_in)
        check_output(y, ref, "f16", 4e-4, "fp16 MMA path k_in=%d M=%d" % (k_in, M))
