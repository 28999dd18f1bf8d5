"""GPU parity of the paired-relay AllGather (Sections 3.1, 5.2) against the oracle, bit for bit."""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import workloads as wl

from gpu_util import Guarded, SENTINEL, torch_mod

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("flags", [0, mw.MW_FLAG_COPY_BULK])
@pytest.mark.parametrize("layout", [mw.MW_LAYOUT_MULTIWRITE, mw.MW_LAYOUT_UNICAST])
@pytest.mark.parametrize("R,S,direct", [(8, 64, 32), (8, 4112, 3072), (8, 64, 0), (8, 64, 64), (4, 48, 16), (2, 32, 16),
                                        (16, 160, 96), (8, 1 << 20, None), (8, 16 << 20, None), (80, 4096, 2048)])
def test_paired_allgather_parity(layout, R, S, direct, flags):
    torch = torch_mod()
    n = R // 2
    if direct is None:
        direct = mwo.balanced_direct_bytes(S, n, layout)
        assert direct == mw.mw_pair_balanced_direct_bytes(S, n, layout)
    sh = wl.make_allgather_shards(R, S, seed=4)
    want_relay, want_recv, want_tot, ret = mwo.paired_allgather(sh, direct, layout, fill=SENTINEL)
    assert ret == 0
    sh_d = torch.from_numpy(sh).cuda()
    relay, recv = Guarded(max(len(want_relay), 16)), Guarded(len(want_recv))
    with mw.Context(R, 8, 2, 16, 32, flags=flags) as ctx:
        rc, tot = ctx.mw_paired_allgather(sh_d, S, direct, layout, relay.ptr(), recv.ptr())
        torch.cuda.synchronize()
    assert tot == want_tot
    assert np.array_equal(recv.host(), want_recv)
    assert np.array_equal(relay.host()[:len(want_relay)], want_relay)
    assert relay.guards_intact() and recv.guards_intact()


def test_paired_allgather_errors():
    torch = torch_mod()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    with mw.Context(7, 8, 2, 16, 32) as ctx:
        assert ctx.mw_paired_allgather(buf, 64, 32, 0, buf, buf, check=False)[0] == mw.MW_ERR_INVALID_ARG   # odd R
    with mw.Context(8, 8, 2, 16, 32) as ctx:
        assert ctx.mw_paired_allgather(buf, 64, 80, 0, buf, buf, check=False)[0] == mw.MW_ERR_INVALID_ARG
        assert ctx.mw_paired_allgather(buf, 64, 24, 0, buf, buf, check=False)[0] == mw.MW_ERR_ALIGNMENT
        assert ctx.mw_paired_allgather(buf, 64, 32, 3, buf, buf, check=False)[0] == mw.MW_ERR_INVALID_ARG
        assert ctx.mw_paired_allgather(buf, 64, 32, 0, None, buf, check=False)[0] == mw.MW_ERR_INVALID_ARG
