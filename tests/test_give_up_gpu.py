"""The boundary's give-up path, exercised once in the permitted form.

Every wait inside the kernels is bounded; when one runs out the CTA records an error, raises its abort
flag, every role leaves its loop, tensor memory is freed and the kernel returns normally.  The host then
reads KLINEAGE_ERR_TIMEOUT through klineage_gemm_get_device_status.  A handle created with
KLINEAGE_FLAG_TEST_GIVE_UP makes its first suitable tcgen05-rung launch take that path (the producer stops,
the MMA issuer's wait for the next stage expires after about a millisecond): no trap, no fault, no
unbounded spin.  Checked here: the status and where it was raised, that C and every guard band are
untouched, and that the next call on the same handle computes the exact product again.
"""
import time

import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_bounded_wait_gives_up_and_the_handle_recovers(col):
    import torch
    from paper_2605_28213_b200 import binding as kb
    case = gen.make_case(256, 512, 512, seed=11, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=False,
                         name="give-up")
    C_ref, S = P.oracle_rows(case, np.arange(case.M))
    with kb.Gemm(0, b_col_major=col, test_give_up=True) as g:
        dev = P.DeviceCase(case)
        before = dev.c.download().copy()
        t0 = time.perf_counter()
        dev.run(g, kb.KLINEAGE_TCGEN05, check=False)          # returns after the synchronize: the kernel ended by itself
        elapsed = time.perf_counter() - t0
        code, kid = g.device_status()
        assert code == kb.KLINEAGE_ERR_TIMEOUT
        assert kid == 400, "the give-up hook belongs to the plain single-CTA kernel"
        block, where = g.last_give_up()
        assert where & 0xFF0 == 0x420 and (where & 0xF) == 2, hex(where)     # MMA issuer, third operand stage
        assert 0 <= block < 148
        assert elapsed < 5.0, "a give-up must come within the poll limit, not after a hang"
        assert np.array_equal(dev.c.download(), before), "a launch that gave up must not have written C"
        assert dev.a.guards_intact() and dev.b.guards_intact() and dev.c.guards_intact()
        # the status was cleared by the read; the same handle now computes the exact product
        assert g.device_status()[0] == kb.KLINEAGE_OK
        for _ in range(2):
            dev.run(g, kb.KLINEAGE_TCGEN05)
            vals, bits = dev.result()
            P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what="after the give-up")
        assert g.device_status() == (kb.KLINEAGE_OK, 400)
