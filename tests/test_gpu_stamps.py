"""Device time stamps (ETS_OPT_TIMING = 2): every kernel of a call records its start and end; the series are
ordered as the launch chain orders the kernels, and switching the option off stops the recording."""
import numpy as np
import pytest
import torch

import paper_2502_13575_b200 as ets
from workloads import make_workload
from workloads.loader import DecodeJob

pytestmark = pytest.mark.gpu


def test_stamps_follow_the_launch_order_and_outputs_do_not_change():
    wl = make_workload("cfg2")
    layers, tokens = 3, 4
    plain = DecodeJob(wl, headroom=tokens + 2, device=0, layers=layers, host_buffers=False, wide=33)
    stamped = DecodeJob(wl, headroom=tokens + 2, device=0, layers=layers, host_buffers=False, wide=33)
    stamped.ctx.set_option(ets.ETS_OPT_TIMING, 2)
    plain.decode_tokens(tokens)
    stamped.decode_tokens(tokens)
    torch.cuda.synchronize()
    assert torch.equal(plain.out.view(torch.int16), stamped.out.view(torch.int16))
    st = stamped.ctx.stamps_read()
    n = layers * tokens
    assert st["count"].tolist() == [n, n, n, n, n]      # append, narrow, wide, merge, "wait returned": one per call
    s, e = st["start_ns"], st["end_ns"]
    for i in range(n):
        assert s[0][i] <= e[0][i] and s[1][i] <= e[1][i] and s[2][i] <= e[2][i] and s[3][i] <= e[3][i]
        assert e[0][i] <= s[4][i] <= e[1][i]           # the narrow kernel's wait returns after the append has ended
        assert s[1][i] <= s[2][i]                      # the wide kernel starts behind the narrow one
        assert max(e[1][i], e[2][i]) <= e[3][i]        # the merge ends after both
        if i:
            assert e[3][i - 1] <= s[4][i]              # and nothing of the next call's attention before the merge ahead has ended
    stamped.ctx.poll_status()
    # the read cleared the table; with the option off nothing is recorded
    stamped.ctx.set_option(ets.ETS_OPT_TIMING, 0)
    stamped.decode_tokens(1)
    torch.cuda.synchronize()
    stamped.ctx.set_option(ets.ETS_OPT_TIMING, 2)
    assert stamped.ctx.stamps_read()["count"].tolist() == [0, 0, 0, 0, 0]
