"""The bounded barrier wait that every persistent kernel relies on: a wait on a barrier nobody arrives on must give up
by itself and let the kernel return with a status the host can read (no fault, no trap, no endless loop)."""
import time

import pytest

from paper_2002_12418_b200 import binding as B

pytestmark = pytest.mark.gpu


def test_a_wait_that_nothing_satisfies_runs_out_and_reports():
    import torch
    assert torch.cuda.is_available()
    B.lib()
    word = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    t0 = time.time()
    B.mnn_wait_probe(word.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    waited = time.time() - t0
    assert int(word.item()) == 2, "the wait must give up (2), not complete (3) or never start (0/1)"
    assert 0.5 < waited < 10.0, waited          # the limit is one second of GPU wall time
    # the context is still usable afterwards
    assert float((torch.ones(8, device="cuda:0") * 2).sum().item()) == 16.0
