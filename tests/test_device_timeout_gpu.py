"""The bounded device-side wait: a wait that can never be satisfied gives up, the kernel returns
by itself, and the host reads MTLA_ERR_DEVICE_TIMEOUT from mtla_check.  The self-test kernel waits
on a barrier nobody arrives at with a budget of a millisecond; nothing traps and nothing spins
past the budget, so the context stays usable and the handle keeps working afterwards."""
import time

import numpy as np
import pytest
import torch

from oracle import mtla_oracle as O
from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    w = synth.WORKLOADS["tiny"].scaled(dtype="bf16", batch=2, n_heads=8, latent_rank=128,
                                       prefill_tokens=0, decode_steps=3)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    h = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        M.mtla_check(h)                                   # clean to start with
        t0 = time.perf_counter()
        M.mtla_selftest_wait_timeout(h, 1000)             # 1 ms budget
        with pytest.raises(M.MTLAError) as err:
            M.mtla_check(h)
        elapsed = time.perf_counter() - t0
        assert err.value.status == -8                     # MTLA_ERR_DEVICE_TIMEOUT
        assert elapsed < 1.0                              # it returned at the budget, not later
        with pytest.raises(M.MTLAError):                  # sticky until cleared
            M.mtla_check(h)
        M.mtla_clear_error(h)
        M.mtla_check(h)
        # The device and the handle are still good: decode against the oracle.
        states = [O.State() for _ in range(w.batch)]
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy())
                             for b in range(w.batch)])
            H.assert_close(y, want, "bf16", f"step {i}")
        M.mtla_check(h)
        with pytest.raises(M.MTLAError):
            M.mtla_selftest_wait_timeout(h, 0)            # budget out of range: argument error
        torch.cuda.synchronize()
    finally:
        M.mtla_destroy(h)
