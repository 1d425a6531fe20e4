"""The bounded device-side waits of the scoring kernel, exercised the only way that is safe on a
shared GPU: a wait is made to run out by a flag that nothing sets. A copy of the library built with
a test hook and a ~1.5 ms wait limit withholds the row statistics of one unit; the second sweep of
that unit then waits for them in vain, gives up, the whole kernel returns, the host reads
LAQ_ERR_TIMEOUT, and the next ordinary call on the same workspace works. Nothing traps or faults."""
import ctypes

import numpy as np
import pytest
import torch

from parity_util import SCORE_RTOL, score_rel_err

pytestmark = pytest.mark.gpu


def test_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    from paper_2505_20334_b200 import binding as laq
    from paper_2505_20334_b200 import build
    from oracle import laq_oracle as orc

    build.build_liblaq()
    hooked = laq.load_library(build.build_liblaq(
        defines=["-DLAQ_TEST_HOOKS", "-DLAQ_TIMEOUT_CYCLES=3000000LL"], variant="hooks"))
    hooked.laq_test_withhold_unit.argtypes = [ctypes.c_longlong]
    hooked.laq_test_withhold_unit.restype = None

    NL, Bt, Hq, Hkv, D, L, W, R, kernel, B = 1, 1, 8, 2, 128, 1024, 16, 16, 7, 100
    g = torch.Generator().manual_seed(9)
    q = torch.randn((NL, Bt, Hq, W, D), generator=g).to(torch.bfloat16).cuda()
    k = torch.randn((NL, Bt, Hkv, L, D), generator=g).to(torch.bfloat16).cuda()
    p = laq.params_for(q, k, R, kernel, B)
    ws = laq.alloc_workspace(p, "cuda")
    scores = torch.zeros((NL, Bt, Hkv, L - R), dtype=torch.float32, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def score(lib):
        return lib.laq_score(ctypes.byref(p), ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(k.data_ptr()),
                             ctypes.c_void_p(scores.data_ptr()), ctypes.c_void_p(ws.data_ptr()),
                             ws.numel(), stream)

    def status(lib):
        return lib.laq_last_device_status(ctypes.byref(p), ctypes.c_void_p(ws.data_ptr()), ws.numel(), stream)

    # unit 1 never publishes its statistics: the wait for them runs out
    hooked.laq_test_withhold_unit(1)
    try:
        assert score(hooked) == laq.LAQ_OK          # the call itself only enqueues
        assert status(hooked) == laq.LAQ_ERR_TIMEOUT
    finally:
        hooked.laq_test_withhold_unit(-1)
    assert torch.cuda.is_available() and torch.zeros(1, device="cuda").item() == 0  # context alive
    # the same build, hook off, same workspace: an ordinary run
    assert score(hooked) == laq.LAQ_OK
    assert status(hooked) == laq.LAQ_OK
    again = scores.clone()
    # and the shipped library gives the same bits
    scores.zero_()
    assert score(laq.lib) == laq.LAQ_OK and status(laq.lib) == laq.LAQ_OK
    assert torch.equal(again, scores)
    ref = orc.evict(q.cpu(), k.cpu(), None, R, kernel, B, want_idx=False)["scores"]
    assert score_rel_err(scores.cpu().numpy(), ref) <= SCORE_RTOL
