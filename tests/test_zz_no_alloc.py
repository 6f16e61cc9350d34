"""uniql_qlinear_noalloc against uniql_qlinear, through the C ABI.

The entry point serves callers that may not allocate device memory (a serving loop whose memory pool is
fully handed out, a real-time callback, a sandbox without cudaMalloc): its scratch is a fixed array
inside the library.  The array is shared by all calls and keeps the last call's contents, so the check
is made on two calls in a row with different shapes: the second must not be disturbed by what the first
left behind.  This file sorts last on purpose: a run that stops at the first failure has then already
run every other test."""
import numpy as np
import pytest
import torch

from helpers import dev_weight, dev_x
from paper_2512_03383_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 4e-4       # the tolerance of the other decode parity tests (fraction of the output scale)


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    from paper_2512_03383_b200 import binding as B
    rng = np.random.default_rng(123)
    qw = synth.draw_qweight(rng, 2048, 2048)
    packed, wp, ws, wz = dev_weight(qw)
    # first call: M = 4, keep 0.85 on both sides (split-K partial sums land in the scratch array);
    # second call: M = 1, full size (different tiling, reuses the same scratch)
    for (M, k) in ((4, synth.keep_count(0.85, 2048)), (1, 2048)):
        x = dev_x(synth.draw_x(rng, M, k, "f16"), "f16")
        y_ref = torch.zeros((M, k), dtype=torch.float16, device="cuda")
        y_new = torch.full((M, k), -3.0, dtype=torch.float16, device="cuda")
        B.qlinear(x, wp, ws, wz, M, 2048, 2048, k, k, y_ref)
        B.qlinear_noalloc(x, wp, ws, wz, M, 2048, 2048, k, k, y_new)
        torch.cuda.synchronize()
        a, b = y_ref.double().cpu().numpy(), y_new.double().cpu().numpy()
        assert np.isfinite(b).all()
        assert np.abs(a - b).max() <= TOL * np.abs(a).max(), "M=%d k=%d" % (M, k)


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
