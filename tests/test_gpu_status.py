"""GPU: the failure path of the device-side waits, exercised without any fault.

A kernel of the library waits, with the same bounded wait the convolution kernels use on their staged tiles, on a
barrier at which nothing ever arrives; it gives up after a fixed number of polls, sets the device status word and
returns.  The host must see BS_ERR_TIMEOUT exactly once, and the device must go on working afterwards."""
import numpy as np
import pytest

import oracle
from paper_2207_08820_b200 import api, workloads as wl
from gpu_util import dev

pytestmark = pytest.mark.gpu


def test_wait_that_runs_out_is_reported_once_and_the_device_stays_usable():
    api.bs_check_status()                                   # clean start
    api.selftest_wait_timeout(polls=64)
    with pytest.raises(api.BitserialError) as err:
        api.bs_check_status()
    assert err.value.status == 5                            # BS_ERR_TIMEOUT
    api.bs_check_status()                                   # the word was cleared by the report
    # a normal launch right after: results still match the oracle
    c = wl.gemm_case(70, 40, 200, seed=9)
    ap = api.bs_pack_rows(dev(c["a"]), c["a_bits"], c["a_sign"])
    wp = api.bs_pack_rows(dev(c["w"]), c["w_bits"], c["w_sign"])
    out, _ = api.bitserial_gemm(ap, wp, c["K"], a_sign=c["a_sign"], w_sign=c["w_sign"])
    api.bs_check_status()
    assert np.array_equal(out.cpu().numpy(), oracle.gemm_i32(c["a"], c["w"]))
