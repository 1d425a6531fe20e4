"""``laq_score_static`` -- the scoring entry point for hosts that may not allocate device memory
(a server whose own pool owns the GPU, a plugin handed only tensors and a stream) -- must give the
scores that ``laq_score`` gives with a caller-provided workspace. Its scratch is one fixed array
inside the library that every call reuses, so the check is made on two calls in a row with
different inputs: stale contents of the first call must not leak into the second. Collected last
(file name) so that a run which stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from parity_util import SCORE_RTOL, score_rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def laq():
    from paper_2505_20334_b200 import build
    build.build_liblaq()
    from paper_2505_20334_b200 import binding
    return binding


def _inputs(NL, Bt, Hq, Hkv, D, L, W, seed):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((NL, Bt, Hq, W, D), generator=g).to(torch.bfloat16).cuda()
    k = (torch.randn((NL, Bt, Hkv, L, D), generator=g) * 1.5).to(torch.bfloat16).cuda()
    return q, k


def _both(laq, q, k, R, kernel, B, expect_no_allocation=False):
    NL, Bt, Hkv, L = k.shape[0], k.shape[1], k.shape[2], k.shape[3]
    p = laq.params_for(q, k, R, kernel, B)
    want = torch.empty((NL, Bt, Hkv, L - R), dtype=torch.float32, device="cuda")
    ws = laq.alloc_workspace(p, "cuda")
    laq.laq_score(p, q, k, want, ws)
    # poison the output so that an entry point that enqueues nothing cannot pass
    got = torch.full_like(want, float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    laq.laq_score_static(p, q, k, got)
    torch.cuda.synchronize()
    if expect_no_allocation:
        # the property the entry point exists for: once the device is warmed up, a call takes no
        # device memory from the driver (torch's own pool is not involved: nothing is created here)
        assert torch.cuda.mem_get_info()[0] == free_before
    # both entry points run the same deterministic kernels: any difference is stale scratch
    assert torch.equal(got, want)
    return got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)


def _oracle_scores(q, k, R, kernel, B):
    from oracle import laq_oracle as orc
    out = orc.evict(q.cpu(), k.cpu(), None, R, kernel, B, want_idx=False)
    return np.asarray(out["scores"], np.float64)


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(laq):
    # first call: tensor-core path, several units and tasks, ragged last tile
    q, k = _inputs(2, 2, 8, 2, 128, 3000, 16, seed=101)
    got, want = _both(laq, q, k, 16, 7, 200)
    assert np.isfinite(got).all()
    assert score_rel_err(got, want) <= SCORE_RTOL
    # second call right after it: a smaller, differently shaped problem on the same scratch
    q, k = _inputs(1, 3, 4, 1, 128, 900, 8, seed=102)
    got, want = _both(laq, q, k, 8, 5, 64, expect_no_allocation=True)
    assert np.isfinite(got).all()
    assert score_rel_err(got, want) <= SCORE_RTOL
    # and against the CPU oracle, so that a mistake shared by both entry points cannot pass
    assert score_rel_err(got, _oracle_scores(q, k, 8, 5, 64).reshape(got.shape)) <= SCORE_RTOL
    # and the CUDA-core path (head_dim 64) shares the same scratch
    q, k = _inputs(1, 1, 8, 2, 64, 500, 8, seed=103)
    got, want = _both(laq, q, k, 8, 7, 90)  # first use of these kernels: they load here
    assert score_rel_err(got, want) <= SCORE_RTOL
    got, want = _both(laq, q, k, 8, 7, 90, expect_no_allocation=True)


def test_static_scratch_refuses_what_does_not_fit(laq):
    # 64 units of 65536 keys need 16 MiB of column sums alone: more than the fixed array holds
    p = laq.make_params(8, 1, 32, 8, 128, 65536, 32, 32, 7, 2048)
    q = torch.zeros((8, 1, 32, 32, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((1, 1, 1, 8, 128), dtype=torch.bfloat16, device="cuda")  # never read
    scores = torch.zeros(8, dtype=torch.float32, device="cuda")
    st = laq.laq_score_static(p, q, k, scores, check=False)
    assert st == laq.LAQ_ERR_WORKSPACE
    assert "workspace" in laq.status_string(st)
