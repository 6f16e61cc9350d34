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
    B.reset_options()


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
    B.set_option("prefill_convert", 1)
    y2, _ = run_ex(B, qw, dw, x, "bf16", None, 652, None, 256, ldx_pad=4)
    check_output(y2, ref, "bf16", TOL["bf16"], "bf16 converted in kernel")
    assert torch.equal(y1, y2)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M", [64, 200])
@pytest.mark.parametrize("grid", [0, 3])
def test_prefill_per_head_input_maps(B, monkeypatch, M, dtype, grid):
    """The input side of o_proj / out_proj: every head keeps its leading channels.  Heads of 128 and of 64
    channels; keep counts that end a head on a k-block boundary (128, 64), inside its second block (104, 96),
    inside its first (40, 8): a partly kept block reads the next head's activations against zero weights."""
    B.set_path(B.PATH_PREFILL)
    if grid:
        B.set_option("prefill_streamk", 1)
        B.set_option("prefill_grid", grid)
    rng = np.random.default_rng(950 + M)
    qw = synth.draw_qweight(rng, 200, 1024)
    dw = dev_weight(qw)
    for (hd, keep) in ((128, 128), (128, 104), (128, 96), (128, 64), (128, 40), (64, 64), (64, 48), (64, 8)):
        im = synth.map_per_head(1024 // hd, hd, keep)
        x = synth.draw_x(rng, M, synth.map_size(im), dtype)
        y, ref = run_ex(B, qw, dw, x, dtype, im, 0, None, 200, ldx_pad=8)
        check_output(y, ref, dtype, TOL[dtype], "per-head input map %d/%d M=%d" % (keep, hd, M))
    # a map whose first head does not start at channel 0, with per-head output rows as well
    im = [(256, 128, 96, 5)]
    om = synth.map_per_head(3, 64, 56)
    x = synth.draw_x(rng, M, synth.map_size(im), dtype)
    y, ref = run_ex(B, qw, dw, x, dtype, im, 0, om, 0, ldx_pad=8)
    check_output(y, ref, dtype, TOL[dtype], "offset per-head input map")
    assert B.workspace_status() == 0
    # not on the tensor-core path: keep counts that are not multiples of 8 (the call falls back to the generic kernel)
    B.set_path(B.PATH_AUTO)
    im = synth.map_per_head(8, 128, 108)
    x = synth.draw_x(rng, M, synth.map_size(im), dtype)
    y, ref = run_ex(B, qw, dw, x, dtype, im, 0, None, 200)
    check_output(y, ref, dtype, TOL[dtype], "keep 108 via auto")


@pytest.mark.parametrize("form", [1, 2])
@pytest.mark.parametrize("grid", [1, 3, 5, 7, 11])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_prefill_stream_k(B, monkeypatch, grid, dtype, form):
    """Stream-K: blocks take contiguous ranges of (tile, k-block) units; the fp32 parts of a tile cut by a range
    boundary go to slots of their own in the workspace and the last block to arrive adds them in block order and
    finishes the tile: results repeat bit for bit however many blocks share a tile."""
    B.set_path(B.PATH_PREFILL)
    B.set_option("prefill_streamk", form)                        # 1: a slot per part; 2: one sum per tile, added in L2
    B.set_option("prefill_grid", grid)
    B.set_option("prefill_dual", 0)                              # tiles of 256 tokens (the counts below assume them)
    rng = np.random.default_rng(900 + grid)
    qw = synth.draw_qweight(rng, 300, 1024)
    dw = dev_weight(qw)
    x = synth.draw_x(rng, 300, 1024, dtype)                      # 3 weight tiles x 2 token tiles, 16 k-blocks
    y, ref = run_ex(B, qw, dw, x, dtype, None, 1024, None, 300)
    check_output(y, ref, dtype, TOL[dtype], "stream-K grid %d" % grid)
    y2, _ = run_ex(B, qw, dw, x, dtype, None, 1024, None, 300)
    if form == 1 or grid in (1, 3, 7):
        # the parts of a split tile are added in block order, whatever the order of arrival; with one sum per tile
        # only where no tile, or no tile with more than two parts, is split (6 whole tiles; 7 ranges of 13 to 14 units)
        assert torch.equal(y, y2)
    else:
        check_output(y2, ref, dtype, TOL[dtype], "stream-K grid %d, second run" % grid)
    for (g, r) in run_rope(B, rng, 200, 512, 6, 2, 128, 84, 5e5, dtype):
        check_output(g, r, dtype, TOL[dtype], "stream-K rope grid %d" % grid)
    assert B.workspace_status() == 0


@pytest.mark.parametrize("grid", [0, 1, 2, 5])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M", [257, 300, 513, 700, 1100])
def test_prefill_tiles_on_both_accumulators(B, M, dtype, grid):
    """Above 256 tokens a tile may take both accumulators (512 tokens: two activation boxes per de-quantised weight
    stage).  Forced on, against the oracle and against tiles of 256 tokens: token counts that end inside the first
    box of a tile, inside the second and on a tile boundary; one block running many tiles in a row (accumulators
    re-used tile after tile), whole tiles and tiles split along K; bias, ragged rows, the rotary epilogue,
    per-head input maps, and bf16 activations converted inside the kernel."""
    B.set_path(B.PATH_PREFILL)
    if grid:
        B.set_option("prefill_grid", grid)
    B.set_option("prefill_streamk", (1 + M % 2) if grid == 5 else 0)      # both forms of the hand-over
    rng = np.random.default_rng(990 + M)
    qw = synth.draw_qweight(rng, 300, 1024)
    dw = dev_weight(qw)
    bias = synth.to_dtype_values(rng.standard_normal(300).astype(np.float32), dtype)
    outs = {}
    for dual in (1, 0):
        B.set_option("prefill_dual", dual)
        for (k_in, k_out) in [(1024, 300), (652, 132)]:
            x = synth.draw_x(np.random.default_rng(M + k_in), M, k_in, dtype)
            y, ref = run_ex(B, qw, dw, x, dtype, None, k_in, None, k_out, bias=bias, ldx_pad=8 - k_in % 8 if k_in % 8 else 0,
                            ldy_pad=3)
            check_output(y, ref, dtype, TOL[dtype], "dual=%d M=%d %s k=(%d,%d) grid %d" % (dual, M, dtype, k_in, k_out, grid))
            outs[(dual, k_in)] = y.clone()
    if grid != 5:        # whole tiles: one block sums a tile's k-blocks in the same order, whatever the tile's width
        for k_in in (1024, 652):
            assert torch.equal(outs[(1, k_in)], outs[(0, k_in)]), "tile width changed the result"
    B.set_option("prefill_dual", 1)
    im = synth.map_per_head(8, 128, 104)
    x = synth.draw_x(rng, M, synth.map_size(im), dtype)
    y, ref = run_ex(B, qw, dw, x, dtype, im, 0, None, 200, ldx_pad=8)
    check_output(y, ref, dtype, TOL[dtype], "dual per-head input map M=%d" % M)
    for (g, r) in run_rope(B, rng, M, 512, 6, 2, 128, 84, 5e5, dtype, bias=True):
        check_output(g, r, dtype, TOL[dtype], "dual rope M=%d grid %d" % (M, grid))
    if dtype == "bf16":
        B.set_option("prefill_convert", 1)
        x = synth.draw_x(rng, M, 652, dtype)
        y, ref = run_ex(B, qw, dw, x, dtype, None, 652, None, 256, ldx_pad=4)
        check_output(y, ref, dtype, TOL[dtype], "dual, converted in kernel, M=%d" % M)
    assert B.workspace_status() == 0


@pytest.mark.parametrize("dual", [0, 1])
@pytest.mark.parametrize("streamk", [0, 1])
@pytest.mark.parametrize("grid", [1, 2, 3])
def test_many_short_tiles_in_one_block(B, grid, streamk, dual):
    """Few k-blocks per tile and many tiles per block: the de-quantiser warps finish their part of the last tile
    while the MMAs are still several tiles back, and then help with that tile's epilogue; they must not mistake an
    earlier tile's "accumulator full" for the last one's."""
    B.set_path(B.PATH_PREFILL)
    B.set_option("prefill_grid", grid)
    B.set_option("prefill_streamk", streamk)
    B.set_option("prefill_dual", dual)
    rng = np.random.default_rng(1700 + grid)
    qw = synth.draw_qweight(rng, 900, 256)
    dw = dev_weight(qw)
    for (M, k_in) in ((300, 256), (600, 128), (1100, 64), (40, 192)):
        x = synth.draw_x(rng, M, k_in, "f16")
        y, ref = run_ex(B, qw, dw, x, "f16", None, k_in, None, 900, ldy_pad=3)
        check_output(y, ref, "f16", TOL["f16"], "short tiles M=%d k_in=%d grid %d streamk %d dual %d" % (M, k_in, grid, streamk, dual))
        y2, _ = run_ex(B, qw, dw, x, "f16", None, k_in, None, 900, ldy_pad=3)
        assert torch.equal(y, y2), "run-to-run results differ"
    assert B.workspace_status() == 0


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


# ---------------------------------------------------------------- full benchmark sizes, sampled token rows
def _sampled_rows(M):
    rows = sorted(set([0, 1, 31, 32, 63, 64, 127, 128, 255, 256, M // 2, M - 2, M - 1]))
    return [r for r in rows if 0 <= r < M]


@pytest.mark.parametrize("M", [512, 2048])
def test_qwen_gate_down_full_size_sampled(B, M):
    """Configuration 4 (Qwen2.5-7B-shaped MLP in prefill, bf16) in the launch configuration of the bench:
    sampled token rows of the full output against the oracle."""
    rng = np.random.default_rng(4)
    gate = synth.random_qweight_fast(rng, 18944, 3584)
    dg = dev_weight(gate)
    for rate in (1.0, 0.85, 0.65):
        k = synth.keep_count(rate, 18944)
        x = synth.draw_x(rng, M, 3584, "bf16")
        xd = dev_x(x, "bf16")
        y = torch.zeros((M, k), dtype=torch.bfloat16, device="cuda")
        B.qlinear_ex(xd, 3584, dg[1], dg[2], dg[3], None, M, 3584, 18944, None, 3584, None, k, y, k)
        torch.cuda.synchronize()
        rows = _sampled_rows(M)
        ref = oracle.qlinear(x, dg[0], gate.scales, gate.zeros, oracle.leading(k), oracle.leading(3584), rows=rows)
        check_output(y[rows], ref, "bf16", TOL["bf16"], "qwen gate keep %.2f M=%d" % (rate, M))
    del dg
    down = synth.random_qweight_fast(rng, 3584, 18944)
    dd = dev_weight(down)
    for rate in (1.0, 0.85, 0.65):
        k = synth.keep_count(rate, 18944)
        h = synth.draw_x(rng, M, k, "bf16")
        hd = dev_x(h, "bf16")
        y = torch.zeros((M, 3584), dtype=torch.bfloat16, device="cuda")
        B.qlinear_ex(hd, k, dd[1], dd[2], dd[3], None, M, 18944, 3584, None, k, None, 3584, y, 3584)
        torch.cuda.synchronize()
        rows = _sampled_rows(M)[::2]
        ref = oracle.qlinear(h, dd[0], down.scales, down.zeros, oracle.leading(3584), oracle.leading(k), rows=rows)
        check_output(y[rows], ref, "bf16", TOL["bf16"], "qwen down keep %.2f M=%d" % (rate, M))
    assert B.workspace_status() == 0


def test_llama_gate_few_split_tiles_full_grid(B):
    """Llama-3-8B gate projection at M = 1024 on the full grid: 448 tiles are three rounds of 148 plus 4 tiles
    whose k-blocks are spread over all blocks (about 37 blocks add their part to each of those tiles, ahead of
    their whole tiles).  Sampled token rows, all output columns, so the split tiles (the last ones) are covered;
    likewise the q|k projection with the rotary epilogue at M = 1024 (160 tiles: 12 split twelve ways)."""
    rng = np.random.default_rng(45)
    M, K, N = 1024, 4096, 14336
    w = synth.random_qweight_fast(rng, N, K)
    d = dev_weight(w)
    x = synth.draw_x(rng, M, K, "f16")
    xd = dev_x(x, "f16")
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    B.qlinear_ex(xd, K, d[1], d[2], d[3], None, M, K, N, None, K, None, N, y, N)
    torch.cuda.synchronize()
    rows = _sampled_rows(M)[::2] + [M - 300]
    ref = oracle.qlinear(x, d[0], w.scales, w.zeros, oracle.leading(N), oracle.leading(K), rows=rows)
    check_output(y[rows], ref, "f16", TOL["f16"], "llama gate M=1024, few split tiles")
    del d, w
    Hq, Hkv, D, keep, theta = 32, 8, 128, 128, 5e5
    wq, wk = synth.random_qweight_fast(rng, Hq * D, K), synth.random_qweight_fast(rng, Hkv * D, K)
    dq, dk = dev_weight(wq), dev_weight(wk)
    pos = synth.draw_pos(rng, M)
    idx = synth.draw_idx(rng, Hkv, D, keep)
    qo = torch.zeros((M, Hq * keep), dtype=torch.float16, device="cuda")
    ko = torch.zeros((M, Hkv * keep), dtype=torch.float16, device="cuda")
    B.qk_rope_proj(xd, K, dq[1], dq[2], dq[3], dk[1], dk[2], dk[3], None, None, M, K, Hq, Hkv, D, keep,
                   torch.from_numpy(idx).cuda(), torch.from_numpy(pos).cuda(), theta, None, qo, Hq * keep, ko, Hkv * keep)
    torch.cuda.synchronize()
    for (wt, dv, nh, g) in ((wq, dq, Hq, qo), (wk, dk, Hkv, ko)):
        O = oracle.expand_map(oracle.qk_halfhead_map(nh, D, keep))
        acc = oracle.qlinear(x, dv[0], wt.scales, wt.zeros, O, oracle.leading(K), rows=rows)
        ref = oracle.rope(acc, nh, Hkv, D, keep, idx, pos[rows], theta)
        check_output(g[rows], ref, "f16", TOL["f16"], "llama q/k rope M=1024, split tiles")
    assert B.workspace_status() == 0


def test_qwen_qk_rope_full_size_sampled(B):
    """Configuration 4's attention projections with the fused pruned RoPE at M = 512 (theta 1e6, 28 Q / 4 KV heads)."""
    rng = np.random.default_rng(44)
    M, K, Hq, Hkv, D, theta = 512, 3584, 28, 4, 128, 1e6
    wq, wk = synth.random_qweight_fast(rng, Hq * D, K), synth.random_qweight_fast(rng, Hkv * D, K)
    dq, dk = dev_weight(wq), dev_weight(wk)
    x = synth.draw_x(rng, M, K, "bf16")
    xd = dev_x(x, "bf16")
    pos = synth.draw_pos(rng, M)
    rows = _sampled_rows(M)
    for keep in (128, 84):
        idx = synth.draw_idx(rng, Hkv, D, keep)
        qo = torch.zeros((M, Hq * keep), dtype=torch.bfloat16, device="cuda")
        ko = torch.zeros((M, Hkv * keep), dtype=torch.bfloat16, device="cuda")
        B.qk_rope_proj(xd, K, dq[1], dq[2], dq[3], dk[1], dk[2], dk[3], None, None, M, K, Hq, Hkv, D, keep,
                       torch.from_numpy(idx).cuda(), torch.from_numpy(pos).cuda(), theta, None, qo, Hq * keep, ko,
                       Hkv * keep)
        torch.cuda.synchronize()
        for (w, d, nh, g) in ((wq, dq, Hq, qo), (wk, dk, Hkv, ko)):
            O = oracle.expand_map(oracle.qk_halfhead_map(nh, D, keep))
            acc = oracle.qlinear(x, d[0], w.scales, w.zeros, O, oracle.leading(K), rows=rows)
            ref = oracle.rope(acc, nh, Hkv, D, keep, idx, pos[rows], theta)
            check_output(g[rows], ref, "bf16", TOL["bf16"], "qwen q/k rope keep %d" % keep)


@pytest.mark.parametrize("M", [1, 1024])
def test_mamba2_full_size(B, M):
    """Configuration 5: Mamba2-2.7B in_proj [10576 x 2560] (z, x rows pruned per SSM head) and out_proj
    [2560 x 5120] (columns pruned per head), fp16; decode at M = 1, prefill / generic at M = 1024 (sampled rows)."""
    rng = np.random.default_rng(5)
    nheads, headdim, d_state, d_inner = 80, 64, 128, 5120
    qin = synth.random_qweight_fast(rng, 10576, 2560)
    qout = synth.random_qweight_fast(rng, 2560, d_inner)
    din, dout = dev_weight(qin), dev_weight(qout)
    rows = _sampled_rows(M)
    for keep in (64, 56, 48):
        om = synth.map_mamba_in_proj(d_inner, headdim, keep, d_state, 1, nheads)
        n_out = synth.map_size(om)
        x = synth.draw_x(rng, M, 2560, "f16")
        y = torch.zeros((M, n_out), dtype=torch.float16, device="cuda")
        B.qlinear_ex(dev_x(x, "f16"), 2560, din[1], din[2], din[3], None, M, 2560, 10576, None, 2560, om, 0, y, n_out)
        torch.cuda.synchronize()
        ref = oracle.qlinear(x, din[0], qin.scales, qin.zeros, oracle.expand_map(om), oracle.leading(2560), rows=rows)
        check_output(y[rows], ref, "f16", TOL["f16"], "mamba in_proj keep %d M=%d" % (keep, M))
        im = synth.map_per_head(nheads, headdim, keep)
        n_in = synth.map_size(im)
        h = synth.draw_x(rng, M, n_in, "f16")
        y2 = torch.zeros((M, 2560), dtype=torch.float16, device="cuda")
        B.qlinear_ex(dev_x(h, "f16"), n_in, dout[1], dout[2], dout[3], None, M, d_inner, 2560, im, 0, None, 2560, y2, 2560)
        torch.cuda.synchronize()
        ref2 = oracle.qlinear(h, dout[0], qout.scales, qout.zeros, oracle.leading(2560), oracle.expand_map(im), rows=rows)
        check_output(y2[rows], ref2, "f16", TOL["f16"], "mamba out_proj keep %d M=%d" % (keep, M))


@pytest.mark.parametrize("keep", [108, 96, 84])
def test_llama_attention_m512_pruned_heads(B, keep):
    """Configuration 3 at M = 512 with Llama-3-8B shapes and pruned heads: q|k|v in one launch with the rotary
    epilogue on q and k, then o_proj over the kept channels of every head (108 and 84 are multiples of 4 only: the
    activations are re-laid on 8-channel boundaries in front of the tensor-core kernel).  Sampled token rows."""
    rng = np.random.default_rng(46 + keep)
    M, K, Hq, Hkv, D, theta = 512, 4096, 32, 8, 128, 5e5
    wq, wk, wv = (synth.random_qweight_fast(rng, Hq * D, K), synth.random_qweight_fast(rng, Hkv * D, K),
                  synth.random_qweight_fast(rng, Hkv * D, K))
    dq, dk, dv = dev_weight(wq), dev_weight(wk), dev_weight(wv)
    x = synth.draw_x(rng, M, K, "f16")
    xd = dev_x(x, "f16")
    pos, idx = synth.draw_pos(rng, M), synth.draw_idx(rng, Hkv, D, keep)
    rows = _sampled_rows(M)
    qo = torch.zeros((M, Hq * keep), dtype=torch.float16, device="cuda")
    ko = torch.zeros((M, Hkv * keep), dtype=torch.float16, device="cuda")
    vo = torch.zeros((M, Hkv * keep), dtype=torch.float16, device="cuda")
    B.qkv_rope_proj(xd, K, dq[1], dq[2], dq[3], dk[1], dk[2], dk[3], dv[1], dv[2], dv[3], None, None, None, M, K, Hq, Hkv,
                    D, keep, keep, torch.from_numpy(idx).cuda(), torch.from_numpy(pos).cuda(), theta, None, qo, Hq * keep,
                    ko, Hkv * keep, vo, Hkv * keep)
    torch.cuda.synchronize()
    for (w, d, nh, g) in ((wq, dq, Hq, qo), (wk, dk, Hkv, ko)):
        O = oracle.expand_map(oracle.qk_halfhead_map(nh, D, keep))
        acc = oracle.qlinear(x, d[0], w.scales, w.zeros, O, oracle.leading(K), rows=rows)
        check_output(g[rows], oracle.rope(acc, nh, Hkv, D, keep, idx, pos[rows], theta), "f16", TOL["f16"],
                     "llama q/k rope keep %d M=512" % keep)
    Ov = oracle.expand_map(synth.map_per_head(Hkv, D, keep))
    check_output(vo[rows], oracle.qlinear(x, dv[0], wv.scales, wv.zeros, Ov, oracle.leading(K), rows=rows), "f16",
                 TOL["f16"], "llama v keep %d M=512" % keep)
    del dq, dk, dv
    wo = synth.random_qweight_fast(rng, K, Hq * D)
    do = dev_weight(wo)
    im = synth.map_per_head(Hq, D, keep)
    a = synth.draw_x(rng, M, Hq * keep, "f16")
    yo = torch.zeros((M, K), dtype=torch.float16, device="cuda")
    B.set_path(B.PATH_PREFILL)                      # the tensor-core kernel must take it
    B.qlinear_ex(dev_x(a, "f16"), Hq * keep, do[1], do[2], do[3], None, M, Hq * D, K, im, 0, None, K, yo, K)
    torch.cuda.synchronize()
    ref = oracle.qlinear(a, do[0], wo.scales, wo.zeros, oracle.leading(K), oracle.expand_map(im), rows=rows)
    check_output(yo[rows], ref, "f16", TOL["f16"], "llama o_proj keep %d M=512" % keep)
    assert B.workspace_status() == 0


def test_bf16_activations_outside_fp16_range(B):
    """The tensor cores run on an fp16 copy of bf16 activations.  Documented consequences: magnitudes above 65504
    saturate, magnitudes under 2^-14 keep fewer significand bits and those under 2^-24 become zero.  A small
    activation is therefore off by at most 2^-25 in absolute terms, and an output by at most sum |w| * 2^-25 (plus
    the usual tolerance); a saturated activation contributes w * 65504 instead of w * x."""
    B.set_path(B.PATH_PREFILL)
    rng = np.random.default_rng(47)
    qw = synth.draw_qweight(rng, 136, 512)
    dw = dev_weight(qw)
    M = 40
    x = (rng.standard_normal((M, 512)) * 1e-5).astype(np.float32)
    x = torch.from_numpy(x).to(torch.bfloat16).float().numpy()            # bf16 values, well under 2^-14
    y = torch.zeros((M, 136), dtype=torch.bfloat16, device="cuda")
    B.qlinear_ex(dev_x(x, "bf16"), 512, dw[1], dw[2], dw[3], None, M, 512, 136, None, 512, None, 136, y, 136)
    torch.cuda.synchronize()
    ref = oracle.qlinear(x, dw[0], qw.scales, qw.zeros, oracle.leading(136), oracle.leading(512))
    wabs = np.abs(oracle.dequant(dw[0], qw.scales, qw.zeros)).sum(axis=1)  # sum |w| per output row
    g = y.double().cpu().numpy()
    bound = wabs[None, :] * 2.0 ** -25 + 5e-4 * np.abs(ref).max() + np.abs(ref) * 2.0 ** -8
    assert np.isfinite(g).all() and (np.abs(g - ref) <= bound).all(), "small activations: beyond the flush bound"
    # saturation: one activation of 1e6 acts as 65504
    x2 = np.zeros((M, 512), dtype=np.float32)
    x2[:, 7] = 999424.0                                                   # a bf16 value near 1e6
    y2 = torch.zeros((M, 136), dtype=torch.bfloat16, device="cuda")
    B.qlinear_ex(dev_x(x2, "bf16"), 512, dw[1], dw[2], dw[3], None, M, 512, 136, None, 512, None, 136, y2, 136)
    torch.cuda.synchronize()
    x2s = x2.copy()
    x2s[:, 7] = 65504.0
    ref2 = oracle.qlinear(x2s, dw[0], qw.scales, qw.zeros, oracle.leading(136), oracle.leading(512))
    check_output(y2, ref2, "bf16", TOL["bf16"], "saturated activation")


def test_caller_workspace_smaller_than_the_header_is_refused(B):
    """The tensor-core kernel keeps its status word in the workspace header: a caller workspace that cannot even
    hold the header is turned down before anything is launched."""
    B.set_path(B.PATH_PREFILL)
    rng = np.random.default_rng(48)
    qw = synth.draw_qweight(rng, 64, 256)
    dw = dev_weight(qw)
    x = dev_x(synth.draw_x(rng, 32, 256, "f16"), "f16")
    y = torch.full((32, 64), -77.0, dtype=torch.float16, device="cuda")
    tiny = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.UniqlError) as e:
        B.qlinear_ex(x, 256, dw[1], dw[2], dw[3], None, 32, 256, 64, None, 256, None, 64, y, 64, workspace=tiny)
    assert e.value.status == 6
    torch.cuda.synchronize()
    assert (y == -77.0).all()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("streamk", [0, 1])
def test_chain_of_dependent_launches(B, dtype, streamk):
    """Launches whose input is the previous launch's output, enqueued back to back with no host synchronisation:
    with programmatic dependent launch the next kernel's blocks are set up (barriers, tensor memory, the first
    weight stages) while the previous one still runs, and only its activation loads, stores and workspace traffic
    wait for it.  The chain must give the same bits as with the attribute off, and its first link the oracle's
    values.  With split tiles every launch also re-uses the previous one's slots in the workspace."""
    B.set_path(B.PATH_PREFILL)
    B.set_option("prefill_streamk", streamk)
    if streamk:
        B.set_option("prefill_grid", 5)
    rng = np.random.default_rng(4242)
    n = 768
    qw = synth.draw_qweight(rng, n, n)
    dw = dev_weight(qw)
    M = 300
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    xd = (torch.from_numpy(synth.draw_x(rng, M, n, dtype)).cuda() * 2.0 ** -6).to(tdt)     # small, so that six links stay finite
    x0 = xd.float().cpu().numpy()

    def chain(pdl, links):
        B.set_option("pdl", pdl)
        bufs = [torch.zeros((M, n), dtype=tdt, device="cuda") for _ in range(2)]
        src = xd
        first = None
        for i in range(links):
            dst = bufs[i & 1]
            B.qlinear_ex(src, n, dw[1], dw[2], dw[3], None, M, n, n, None, n, None, n, dst, n)
            if i == 0:
                first = dst.clone()              # (enqueued on the same stream: ordered after the first launch)
            src = dst
        torch.cuda.synchronize()
        return first, src.clone()

    for rep in range(3):
        f_off, y_off = chain(0, 6)
        f_on, y_on = chain(1, 6)
        assert torch.isfinite(y_off.float()).all()
        assert torch.equal(f_on, f_off) and torch.equal(y_on, y_off), "repeat %d" % rep
    ref = oracle.qlinear(x0, dw[0], qw.scales, qw.zeros, oracle.leading(n), oracle.leading(n))
    check_output(f_on, ref, dtype, TOL[dtype], "first link of the chain")
    assert B.workspace_status() == 0


@pytest.mark.parametrize("grid", [2, 3, 4, 6, 7])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M", [513, 700, 1100])
def test_left_over_wide_tiles_as_half_tiles(B, M, dtype, grid):
    """Tiles of two boxes left over after the whole rounds run as half tiles (one box each, on two blocks, a block's
    last segment on the accumulator of its box).  Forced wherever the rule allows, on grids that leave one to three
    tiles over, against the oracle and bit for bit against tiles of 256 tokens (whole tiles either way: one block sums
    a tile's k-blocks in the same order); plain rows with bias, a per-head input map and the rotary epilogue."""
    B.set_path(B.PATH_PREFILL)
    B.set_option("prefill_grid", grid)
    B.set_option("prefill_streamk", 0)
    rng = np.random.default_rng(3300 + M + grid)
    qw = synth.draw_qweight(rng, 600, 512)                     # 5 weight tiles x 2 or 3 token tiles of 512
    dw = dev_weight(qw)
    bias = synth.to_dtype_values(rng.standard_normal(600).astype(np.float32), dtype)
    outs = {}
    for dual in (3, 0):
        B.set_option("prefill_dual", dual)
        for (k_in, k_out) in [(512, 600), (420, 388)]:
            x = synth.draw_x(np.random.default_rng(M + k_in), M, k_in, dtype)
            y, ref = run_ex(B, qw, dw, x, dtype, None, k_in, None, k_out, bias=bias, ldx_pad=8 - k_in % 8 if k_in % 8 else 0,
                            ldy_pad=5)
            check_output(y, ref, dtype, TOL[dtype], "half tiles=%d M=%d %s k=(%d,%d) grid %d" % (dual, M, dtype, k_in, k_out, grid))
            outs[(dual, k_in)] = y.clone()
    for k_in in (512, 420):
        assert torch.equal(outs[(3, k_in)], outs[(0, k_in)]), "half tiles changed the result"
    B.set_option("prefill_dual", 3)
    im = synth.map_per_head(4, 128, 104)
    x = synth.draw_x(rng, M, synth.map_size(im), dtype)
    y, ref = run_ex(B, qw, dw, x, dtype, im, 0, None, 600, ldx_pad=8)
    check_output(y, ref, dtype, TOL[dtype], "half tiles, per-head input map M=%d" % M)
    for (g, r) in run_rope(B, rng, M, 512, 6, 2, 128, 84, 5e5, dtype, bias=True):
        check_output(g, r, dtype, TOL[dtype], "half tiles, rope M=%d grid %d" % (M, grid))
    assert B.workspace_status() == 0


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M", [17, 64, 100, 200, 256])
def test_pairs_of_blocks_on_one_tile(B, M, dtype):
    """Few tiles: a cluster of two blocks per tile, half of the contraction each; the second block's fp32 sums go
    into the first one's shared memory and are added there (own + other, the same bits every run).  Forced, against
    the oracle, twice for the bits; plain rows with bias, pruned inputs and outputs, a per-head input map and the
    rotary epilogue; the library must come back clean."""
    B.set_path(B.PATH_PREFILL)
    B.set_option("prefill_streamk", 3)
    rng = np.random.default_rng(8800 + M)
    qw = synth.draw_qweight(rng, 300, 1024)
    dw = dev_weight(qw)
    bias = synth.to_dtype_values(rng.standard_normal(300).astype(np.float32), dtype)
    for (k_in, k_out) in [(1024, 300), (652, 132), (256, 40)]:
        x = synth.draw_x(np.random.default_rng(M + k_in), M, k_in, dtype)
        y, ref = run_ex(B, qw, dw, x, dtype, None, k_in, None, k_out, bias=bias, ldx_pad=8 - k_in % 8 if k_in % 8 else 0, ldy_pad=3)
        check_output(y, ref, dtype, TOL[dtype], "pairs M=%d %s k=(%d,%d)" % (M, dtype, k_in, k_out))
        y2, _ = run_ex(B, qw, dw, x, dtype, None, k_in, None, k_out, bias=bias, ldx_pad=8 - k_in % 8 if k_in % 8 else 0, ldy_pad=3)
        assert torch.equal(y, y2)
    im = synth.map_per_head(8, 128, 104)
    x = synth.draw_x(rng, M, synth.map_size(im), dtype)
    y, ref = run_ex(B, qw, dw, x, dtype, im, 0, None, 200, ldx_pad=8)
    check_output(y, ref, dtype, TOL[dtype], "pairs, per-head input map M=%d" % M)
    for (g, r) in run_rope(B, rng, M, 512, 6, 2, 128, 84, 5e5, dtype, bias=True):
        check_output(g, r, dtype, TOL[dtype], "pairs, rope M=%d" % M)
    assert B.workspace_status() == 0


def test_random_shapes_under_the_launcher_s_own_plan(B):
    """Seeded random shapes with nothing forced: whatever the launcher picks on the full grid (whole tiles of either
    width, pairs of blocks on a tile, split tiles in both forms, half tiles) must match the oracle, and launches
    whose plan is reproducible by construction must repeat bit for bit."""
    B.set_path(B.PATH_PREFILL)
    rng = np.random.default_rng(20261130)
    cases = []
    for _ in range(28):
        M = int(rng.choice([17, 40, 64, 100, 128, 200, 256, 257, 384, 512, 700, 1024, 1100]))
        N = int(rng.integers(1, 9)) * 128 - int(rng.choice([0, 0, 28, 96]))
        K = int(rng.integers(1, 9)) * 128
        cases.append((M, N, K, K - int(rng.choice([0, 0, 0, 52, 120]))))
    cases += [(4096, 2560, 256, 256), (2048, 9600, 128, 128), (1536, 2432, 384, 380)]   # more tiles than SMs: left-over rounds
    for (M, N, K, k_in) in cases:
        dtype = "bf16" if (M + N) % 3 == 0 else "f16"
        qw = synth.draw_qweight(rng, N, K)
        dw = dev_weight(qw)
        x = synth.draw_x(rng, M, k_in, dtype)
        y, ref = run_ex(B, qw, dw, x, dtype, None, k_in, None, N, ldx_pad=8 - k_in % 8 if k_in % 8 else 0)
        check_output(y, ref, dtype, TOL[dtype], "auto plan M=%d N=%d K=%d k_in=%d %s" % (M, N, K, k_in, dtype))
        assert B.workspace_status() == 0
