"""uniql_qlinear_noalloc through the C ABI, against the CPU oracle and against uniql_qlinear.

The entry point serves callers that may not allocate device memory (a serving loop whose memory pool is
fully handed out, a real-time callback, a sandbox without cudaMalloc): its scratch is a fixed array
inside the library.  The array is shared by all calls and keeps the last call's contents, so the check
is made on two calls in a row with different shapes: the second must not be disturbed by what the first
left behind.  This file sorts last on purpose: a run that stops at the first failure has then already
run every other test."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_output, dev_weight, dev_x
from paper_2512_03383_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 4e-4       # the tolerance of the other decode parity tests (fraction of the output scale)


def test_noalloc_matches_oracle_and_regular_entry_point_twice_in_a_row():
    from paper_2512_03383_b200 import binding as B
    rng = np.random.default_rng(123)
    qw = synth.draw_qweight(rng, 2048, 2048)
    packed, wp, ws, wz = dev_weight(qw)
    # first call: M = 4, keep 0.85 on both sides (split-K partial sums land in the scratch array);
    # second call: M = 1, full size (different tiling, reuses the same scratch); third: twelve rows in one launch
    try:
        B.set_path(B.PATH_DECODE)             # the regular entry point on the same kernel as the fixed-scratch one
        for (M, k) in ((4, synth.keep_count(0.85, 2048)), (1, 2048), (12, 2048)):
            x32 = synth.draw_x(rng, M, k, "f16")
            x = dev_x(x32, "f16")
            y_ref = torch.zeros((M, k), dtype=torch.float16, device="cuda")
            y_new = torch.full((M, k), -3.0, dtype=torch.float16, device="cuda")
            B.qlinear(x, wp, ws, wz, M, 2048, 2048, k, k, y_ref)
            B.qlinear_noalloc(x, wp, ws, wz, M, 2048, 2048, k, k, y_new)
            torch.cuda.synchronize()
            assert B.noalloc_status() == 0
            o = oracle.qlinear(x32, packed, qw.scales, qw.zeros, oracle.leading(k), oracle.leading(k))
            check_output(y_new, o, "f16", TOL, "noalloc M=%d k=%d" % (M, k))
            # the same kernel on the same plan: up to eight rows (larger batches: one launch here, two halves there)
            # and channels in multiples of 8 (otherwise the regular entry point re-lays the activations first)
            if M <= 8 and k % 8 == 0:
                assert torch.equal(y_new, y_ref), "M=%d k=%d: not bitwise equal to uniql_qlinear" % (M, k)
    finally:
        B.set_path(B.PATH_AUTO)


@pytest.mark.parametrize("rate", [1.0, 0.65])
def test_noalloc_llama_mlp_matrices_at_sixteen_rows(rate):
    """The header promises that the Llama-3-8B MLP matrices fit the fixed array for every M <= 16."""
    from paper_2512_03383_b200 import binding as B
    rng = np.random.default_rng(125)
    M, H, I = 16, 4096, 14336
    k = synth.keep_count(rate, I)
    rows = np.unique(np.concatenate([np.arange(0, 40), rng.integers(0, 4096, 40)]))
    for (N, K, k_in, k_out) in ((I, H, H, k), (H, I, k, H)):
        qw = synth.random_qweight_fast(rng, N, K)
        packed, wp, ws, wz = dev_weight(qw)
        x32 = synth.draw_x(rng, M, k_in, "f16")
        y = torch.full((M, k_out), -3.0, dtype=torch.float16, device="cuda")
        B.qlinear_noalloc(dev_x(x32, "f16"), wp, ws, wz, M, K, N, k_in, k_out, y)
        torch.cuda.synchronize()
        assert B.noalloc_status() == 0
        sel = rows[rows < k_out]
        o = oracle.qlinear(x32, packed, qw.scales, qw.zeros, sel.astype(np.int32), oracle.leading(k_in))
        check_output(y[:, torch.as_tensor(sel, device="cuda")], o, "f16", TOL, "noalloc %dx%d keep %.2f" % (N, K, rate))
        del wp, ws, wz


def test_noalloc_rejects_what_it_cannot_serve():
    from paper_2512_03383_b200 import binding as B
    rng = np.random.default_rng(124)
    qw = synth.draw_qweight(rng, 256, 256)
    packed, wp, ws, wz = dev_weight(qw)
    x = dev_x(synth.draw_x(rng, 32, 256, "f16"), "f16")
    y = torch.zeros((32, 256), dtype=torch.float16, device="cuda")
    with pytest.raises(B.UniqlError) as e:       # M > 16 is not a decode size: no kernel with scratch runs
        B.qlinear_noalloc(x, wp, ws, wz, 32, 256, 256, 256, 256, y)
    assert e.value.status == 5
    # a problem whose partial sums need more than the fixed array: turned down before anything is launched (the
    # buffers are therefore never touched and may be small)
    N, K, M = 1 << 20, 16384, 16
    small = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.UniqlError) as e:
        B.qlinear_noalloc(x, small, small, small, M, K, N, K, N, y)
    assert e.value.status == 6
    torch.cuda.synchronize()
    assert B.noalloc_status() == 0
