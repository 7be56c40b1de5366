"""A device-side wait that runs out ends in TSQ_ERR_TIMEOUT, quickly, and the buffers work again afterwards.

The failure is made on the host: after the workspace is initialised, its ticket counter is set to 1, so that
row 0 is never handed out and every other row's placement look-back waits for sizes that nobody publishes.  With
a wait limit of a few thousand polls every such wait gives up within milliseconds; nothing faults or spins
without bound, and the kernel returns the status."""
import time

import numpy as np
import pytest
import torch

from oracle import tsq_ref as R
from paper_2511_04002_b200 import binding as B
from paper_2511_04002_b200 import synth
from tests._parity import assert_blobs_equal, gpu_encode

pytestmark = pytest.mark.gpu
TIMEOUT = 7


@pytest.mark.parametrize("tokens,hidden", [(200, 512),     # one CTA per row, rows handed out by ticket (more rows than SMs)
                                           (700, 1024)])   # the persistent kernel for many rows
def test_wait_runs_out_into_timeout_status_and_workspace_recovers(tokens, hidden):
    g = torch.Generator().manual_seed(tokens)
    x_cpu = (torch.randn((tokens, hidden), generator=g) * 1.5).to(torch.float16).contiguous()
    plan = B.Plan(torch.float16, hidden, tokens, 6.0, [2, 4, 8], 0.2)
    blob, ws = plan.alloc(tokens)
    x = x_cpu.cuda()
    plan.workspace_set_wait_limit(ws, 3000)
    torch.cuda.synchronize()
    ws.view(torch.int32)[1] = 1                      # the ticket counter: row 0 will never be taken
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    plan.encode(x, blob, ws)
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    assert elapsed < 2.0, "the waits did not give up in time (%.2f s)" % elapsed
    assert plan.blob_info(blob).status == TIMEOUT
    assert plan.workspace_status(ws)[0] == TIMEOUT
    # the documented recovery: initialise the workspace again, then the same buffers encode correctly
    plan.workspace_init(ws)
    _, got, _ = gpu_encode(plan, x_cpu, ws=ws, blob=blob)
    assert_blobs_equal(got, R.encode(synth.raw_u16(x_cpu), R.F16, 6.0, [2, 4, 8], 0.2))
    assert plan.workspace_status(ws) == (0, 0)
