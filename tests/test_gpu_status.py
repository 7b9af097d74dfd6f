"""The give-up path of the bounded device-side waits: a wait that is known to run out sets the sticky status word, the
kernel ends normally, the status call reports the timeout, clears the word, and the device keeps working."""
import time

import pytest
import torch

import paper_2306_08162_b200 as ql
import qlora_inputs as qi
from test_gpu_layer import check_layer

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_cleared():
    assert ql.qlora_device_status() == 0
    t0 = time.perf_counter()
    ql.qlora_selftest_bounded_wait(1000)          # 1 ms
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0         # it ended by itself, promptly
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_device_status(clear=False)
    assert e.value.status == -6 and "gave up" in ql.qlora_status_string(-6)
    with pytest.raises(ql.QloraError):            # sticky until cleared
        ql.qlora_device_status(clear=True)
    assert ql.qlora_device_status() == 0
    # the context is intact: a layer runs and matches the oracle afterwards
    check_layer(qi.random_codes_layer(K=256, N=256, bits=4, group_size=128, r=8, alpha=16.0, M=300, seed=1))
    assert ql.qlora_device_status() == 0


def test_argument_range():
    for bad in (0, -5, 2_000_000):
        with pytest.raises(ql.QloraError) as e:
            ql.qlora_selftest_bounded_wait(bad)
        assert e.value.status == -1
