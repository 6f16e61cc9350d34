"""GPU parity of the 4-bit embedding gather (bit exact) and of the output layer (lm_head: the quantised linear
layer on a vocabulary-sized matrix) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_output, dev_weight, dev_x
from paper_2512_03383_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2512_03383_b200 import binding
    return binding


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("V,K", [(1000, 384), (37, 4096), (5, 128)])
def test_embedding_rows_bit_exact(B, V, K, dtype):
    rng = np.random.default_rng(V + K)
    qw = synth.draw_qweight(rng, V, K)
    packed, wp, ws, wz = dev_weight(qw)
    ids = np.concatenate([[0, V - 1, V - 1, 0], rng.integers(0, V, 29)]).astype(np.int32)
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    out = torch.full((len(ids), K + 8), -3.0, dtype=tdt, device="cuda")
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.embed_rows(wp, ws, wz, torch.from_numpy(ids).cuda(), out, bad_id=bad)
    torch.cuda.synchronize()
    assert int(bad) == 0
    assert (out[:, K:] == -3.0).all(), "wrote outside the row"
    W = oracle.dequant(packed, qw.scales, qw.zeros)[ids]                 # fp64; integer zero-points: one rounding
    ref = torch.from_numpy(W).to(tdt)
    assert torch.equal(out[:, :K].cpu().view(torch.int16), ref.view(torch.int16))
    # an unaligned output (odd leading dimension, offset start) takes the element-wise store
    buf = torch.full((len(ids) * (K + 3) + 1,), -3.0, dtype=tdt, device="cuda")
    out2 = buf[1:].view(len(ids), K + 3)
    B.embed_rows(wp, ws, wz, torch.from_numpy(ids).cuda(), out2)
    torch.cuda.synchronize()
    assert torch.equal(out2[:, :K].cpu().view(torch.int16), ref.view(torch.int16))
    assert (out2[:, K:] == -3.0).all()


def test_embedding_out_of_range_ids(B):
    rng = np.random.default_rng(4)
    qw = synth.draw_qweight(rng, 64, 256)
    packed, wp, ws, wz = dev_weight(qw)
    ids = np.array([3, -1, 64, 63, 2 ** 31 - 1], dtype=np.int32)
    out = torch.full((5, 256), 9.0, dtype=torch.float16, device="cuda")
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.embed_rows(wp, ws, wz, torch.from_numpy(ids).cuda(), out, bad_id=bad)
    torch.cuda.synchronize()
    assert int(bad) == 1
    W = oracle.dequant(packed, qw.scales, qw.zeros)
    for m, i in enumerate(ids):
        if 0 <= i < 64:
            assert torch.equal(out[m].cpu(), torch.from_numpy(W[i]).half())
        else:
            assert (out[m] == 0).all()
    with pytest.raises(RuntimeError):
        B.embed_rows(wp, ws, wz, torch.from_numpy(ids).cuda(), torch.zeros((5, 128), dtype=torch.float16, device="cuda"))


# ---------------------------------------------------------------- output layer at Llama-3 size
@pytest.fixture(scope="module")
def lm_head():
    rng = np.random.default_rng(9)
    qw = synth.random_qweight_fast(rng, 128256, 4096)
    return qw, dev_weight(qw)


@pytest.mark.parametrize("M", [1, 16, 128])
def test_lm_head_llama3_vocab(B, lm_head, M):
    """The largest single matrix of the model: every logit at M = 1, sampled logits above."""
    qw, (packed, wp, ws, wz) = lm_head
    rng = np.random.default_rng(90 + M)
    dtype = "f16" if M <= 16 else "bf16"
    x = synth.draw_x(rng, M, 4096, dtype, outlier_frac=0.005)
    xd = dev_x(x, dtype)
    y = torch.zeros((M, 128256), dtype=xd.dtype, device="cuda")
    B.qlinear_ex(xd, 4096, wp, ws, wz, None, M, 4096, 128256, None, 4096, None, 128256, y, 128256)
    torch.cuda.synchronize()
    assert B.workspace_status() == 0
    if M == 1:
        cols = np.arange(128256, dtype=np.int32)
    else:
        cols = np.unique(np.concatenate([[0, 63, 64, 128255, 128192], rng.integers(0, 128256, 300)])).astype(np.int32)
    ref = oracle.qlinear(x, packed, qw.scales, qw.zeros, cols, oracle.leading(4096))
    got = y[:, torch.from_numpy(cols.astype(np.int64)).cuda()]
    check_output(got, ref, dtype, 4e-4 if M <= 16 else 5e-4, "lm_head M=%d" % M)
