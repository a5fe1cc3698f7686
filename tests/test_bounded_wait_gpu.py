"""The bounded device-side wait, made to run out on purpose in the one safe way: a probe kernel waits on an
mbarrier that nobody arrives at, with the limit shortened to a millisecond for that launch.  The wait gives up by
itself, the kernel returns normally (no trap, no fault), the status word reports the timeout once, and the library
goes on working."""
import numpy as np
import pytest
import torch

import nm_inputs as gen
import oracle
from gpu_util import assert_matmul_close, out_to_f64, to_dev

pytestmark = pytest.mark.gpu


def test_an_expired_wait_is_reported_once_and_the_library_keeps_working():
    import paper_2609_16009_b200 as nm
    nm.nm_check_status()                                           # clean before the probe
    elapsed = torch.zeros(2, dtype=torch.int64, device="cuda")
    nm.nm_debug_wait_probe(1_000_000, elapsed)                     # 1 ms
    with pytest.raises(nm.NmError) as e:
        nm.nm_check_status()
    assert e.value.status == -6                                    # NM_ERR_TIMEOUT
    nm.nm_check_status()                                           # reading the status cleared it
    ns, ok_mask = (int(x) for x in elapsed.cpu())
    assert ok_mask == 0                                            # neither wait claimed the barrier had completed
    assert 1_000_000 <= ns < 50_000_000, ns                        # gave up after the limit, and the second wait at once
    # the limit is back to its default and ordinary work is unaffected: a product with TMA ring, mbarriers and split-K
    M, K, N = 1, 7168, 576
    A, B = gen.narrow_bf16(M, K, N, seed=9500)
    ws = nm.new_workspace(nm.nm_matmul_workspace_bytes(M, N, K))
    C = torch.zeros(M * N, dtype=torch.int16, device="cuda")
    nm.nm_matmul_ws(to_dev(A), to_dev(B), C, M, N, K, nm.BF16, nm.ROW_MAJOR, ws)
    nm.nm_check_status()
    Cq, C64, bound = oracle.matmul(A, B, M, N, K, oracle.BF16, oracle.BF16)
    assert_matmul_close(out_to_f64(C, 1).reshape(M, N), Cq, C64, bound, 1, "product after the probe")


def test_the_probe_refuses_limits_outside_its_range():
    import paper_2609_16009_b200 as nm
    for bad in (0, 10, 2_000_000_000):
        with pytest.raises(nm.NmError):
            nm.nm_debug_wait_probe(bad)
    nm.nm_check_status()
