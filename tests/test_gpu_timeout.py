"""A bounded device-side wait that runs out, without any fault: the barrier between the two phases of the
one-launch MLP polls a counter a limited number of times; with the limit cut to a single poll (option
"wait_shift") the blocks that reach the barrier before the others have finished their first phase give up, set
UNIQL_ERR_TIMEOUT in the status word of the workspace and return by their own logic.  The call itself returns, the
context stays usable, and after the workspace is prepared again the same call gives the oracle's result."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_output, dev_weight, dev_x
from paper_2512_03383_b200 import synth

pytestmark = pytest.mark.gpu


def test_grid_barrier_wait_runs_out_and_the_library_recovers():
    from paper_2512_03383_b200 import binding as B
    rng = np.random.default_rng(810)
    hidden, inter, M, k_int = 512, 1024, 2, 1024
    qg, qu, qd = (synth.draw_qweight(rng, inter, hidden), synth.draw_qweight(rng, inter, hidden),
                  synth.draw_qweight(rng, hidden, inter))
    (pg, wg, sg, zg), (pu, wu, su, zu), (pd, wd, sd, zd) = dev_weight(qg), dev_weight(qu), dev_weight(qd)
    x = synth.draw_x(rng, M, hidden, "f16")
    xd = dev_x(x, "f16")
    ws = torch.zeros(B.mlp_workspace_bytes(M, hidden, inter), dtype=torch.uint8, device="cuda")
    B.workspace_init(ws)

    def run():
        h = torch.zeros((M, k_int), dtype=torch.float16, device="cuda")
        y = torch.zeros((M, hidden), dtype=torch.float16, device="cuda")
        B.mlp_swiglu_decode(xd, hidden, wg, sg, zg, wu, su, zu, wd, sd, zd, M, hidden, inter, k_int, h, k_int, y, hidden,
                            fuse=1, workspace=ws)
        torch.cuda.synchronize()               # the kernel ends by itself
        return h, y

    try:
        B.set_option("wait_shift", 21)         # one poll: blocks without work in the first phase arrive too early
        run()
        assert B.workspace_status(ws) == 7, "the wait did not run out"
        assert B.status_string(7) == "device-side wait timed out"
    finally:
        B.set_option("wait_shift", 0)
    # the counters of the barrier and of shared tiles are left as the aborted launch had them: prepare again
    B.workspace_init(ws)
    h, y = run()
    assert B.workspace_status(ws) == 0
    h_ref, y_ref = oracle.mlp_swiglu(x, pg, qg.scales, qg.zeros, pu, qu.scales, qu.zeros, pd, qd.scales, qd.zeros, k_int)
    check_output(h, h_ref, "f16", 4e-4, "h after recovery")
    check_output(y, y_ref, "f16", 1e-3, "y after recovery")
