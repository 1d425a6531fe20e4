"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs. Scores within 2e-3 relative; selection bit-exact on identical scores and equal to
the oracle's set outside the tie band; compaction bit-exact."""
import numpy as np
import pytest
import torch

from oracle import laq_oracle as orc
from paper_2505_20334_b200 import synth
from parity_util import SCORE_RTOL, bits, check_index_set, score_rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def laq():
    from paper_2505_20334_b200 import build
    build.build_liblaq()
    from paper_2505_20334_b200 import binding
    return binding


def rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed, kscale=1.0):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((NL, Bt, Hq, W, D), generator=g).to(torch.bfloat16)
    k = (torch.randn((NL, Bt, Hkv, L, D), generator=g) * kscale).to(torch.bfloat16)
    v = torch.randn((NL, Bt, Hkv, L, D), generator=g).to(torch.bfloat16)
    return q, k, v


def run_evict(laq, q, k, v, R, kernel, B, local_window=0, pool_mode=0, score_mode=0, seq_lens=None,
              group_mode=0):
    out = laq.evict(q.cuda(), k.cuda(), v.cuda(), B, pool_kernel=kernel, keep_tail=R,
                    want_scores=True, local_window=local_window, pool_mode=pool_mode,
                    score_mode=score_mode, seq_lens=seq_lens, group_mode=group_mode)
    assert laq.laq_last_device_status(out["params"], out["ws"]) == laq.LAQ_OK
    return out


def compare_all_units(laq, q, k, v, R, kernel, B, out=None, local_window=0, pool_mode=0,
                      seq_lens=None, group_mode=0):
    """Full comparison of every unit of a (small) problem against the oracle."""
    out = out or run_evict(laq, q, k, v, R, kernel, B, local_window, pool_mode, seq_lens=seq_lens,
                           group_mode=group_mode)
    ref = orc.evict(q, k, v, R, kernel, B, local_window=local_window, pool_mode=pool_mode,
                    seq_lens=seq_lens, group_mode=group_mode)
    NL, Bt, Hkv, L = k.shape[0], k.shape[1], k.shape[2], k.shape[3]
    if group_mode == 2:
        # every query head is a unit of its own and gathers from its KV head
        G = q.shape[2] // Hkv
        k, v, Hkv = k.repeat_interleave(G, dim=2), v.repeat_interleave(G, dim=2), q.shape[2]
    got_scores = out["scores"].cpu().numpy()
    err = score_rel_err(got_scores, ref["scores"])
    assert err <= SCORE_RTOL, f"score rel err {err:.3e}"
    got_idx = out["idx"].cpu().numpy()
    kb, vb = bits(k), bits(v)
    ko, vo = bits(out["k_out"]), bits(out["v_out"])
    differing = 0
    for n in range(NL):
        for b in range(Bt):
            Lb = L if seq_lens is None else int(seq_lens[b])   # this prompt's own length
            for h in range(Hkv):
                differing += check_index_set(got_idx[n, b, h], ref["idx"][n, b, h],
                                             ref["scores"][n, b, h][:Lb - R], Lb, R, B)
                assert (got_scores[n, b, h][Lb - R:] == 0).all()
                # selection is bit-exact on the GPU's own scores (tie-break included)
                want = orc.select(got_scores[n, b, h][:Lb - R], Lb, R, B, sorted_variant=True)
                assert (got_idx[n, b, h] == want).all()
                # compaction is bit-exact given the indices
                assert (ko[n, b, h] == kb[n, b, h][got_idx[n, b, h]]).all()
                assert (vo[n, b, h] == vb[n, b, h][got_idx[n, b, h]]).all()
    return err, differing


SHAPES = [
    # NL Bt Hq Hkv D    L     W  k  B     what
    (1, 1, 4, 1, 128, 1024, 8, 7, 128),    # config-1 geometry, M = 32
    (2, 1, 8, 2, 128, 1000, 16, 7, 100),   # M = 64, ragged last tile
    (1, 2, 8, 2, 128, 777, 32, 7, 200),    # M = 128
    (1, 1, 8, 1, 128, 1500, 32, 5, 64),    # M = 256
    (1, 2, 6, 1, 128, 2100, 16, 7, 150),   # M = 96: the two warpgroups of a pair take 2 and 1 row chunks
    (1, 1, 2, 2, 128, 300, 8, 3, 40),      # G = 1, M = 8
    (1, 1, 6, 2, 128, 640, 5, 3, 33),      # M = 15 (not a multiple of 16)
    (1, 1, 4, 2, 128, 50, 4, 7, 20),       # L smaller than one tile
    (1, 1, 8, 2, 64, 500, 8, 7, 90),       # head_dim 64: CUDA-core path
    (1, 1, 4, 1, 256, 260, 8, 5, 48),      # head_dim 256: CUDA-core path
    (2, 2, 8, 2, 128, 4500, 1, 7, 64),     # one lookahead step (Section 6.2): M = 4
    (1, 1, 8, 2, 128, 2500, 2, 5, 40),     # two lookahead steps: M = 8
    (1, 1, 16, 2, 128, 1100, 2, 3, 50),    # M = 16
]


@pytest.mark.parametrize("shape", SHAPES, ids=[f"L{s[5]}-M{s[2] // s[3] * s[6]}-D{s[4]}" for s in SHAPES])
def test_evict_matches_oracle_small(laq, shape):
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = shape
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=L + W, kscale=1.5)
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B)
    assert err < SCORE_RTOL


def test_score_select_compact_entry_points_agree_with_evict(laq):
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 2, 2, 8, 2, 128, 900, 8, 7, 150
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=5)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    fused = run_evict(laq, q, k, v, W, kernel, B)
    p = laq.params_for(qd, kd, W, kernel, B, v=vd)
    ws = laq.alloc_workspace(p, "cuda")
    scores = torch.empty((NL, Bt, Hkv, L - W), dtype=torch.float32, device="cuda")
    idx = torch.empty((NL, Bt, Hkv, B), dtype=torch.int32, device="cuda")
    k_out = torch.empty((NL, Bt, Hkv, B, D), dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)
    laq.laq_score(p, qd, kd, scores, ws)
    laq.laq_select(p, scores, idx)
    laq.laq_compact(p, kd, vd, idx, k_out, v_out)
    torch.cuda.synchronize()
    assert torch.equal(scores, fused["scores"])
    assert torch.equal(idx, fused["idx"])
    assert torch.equal(k_out, fused["k_out"]) and torch.equal(v_out, fused["v_out"])
    # evict without the optional outputs
    laq.laq_evict(p, qd, kd, vd, k_out.zero_(), v_out.zero_(), None, None, ws)
    torch.cuda.synchronize()
    assert torch.equal(k_out, fused["k_out"]) and torch.equal(v_out, fused["v_out"])


def test_select_bit_exact_on_ties_and_edges(laq):
    rng = np.random.default_rng(3)
    cases = []
    for Ls, R, Kb in [(1000, 8, 1), (1000, 0, 999), (5000, 16, 700), (37, 3, 10), (70000, 32, 2016),
                      (4096, 0, 128)]:
        for kind in ("ties", "const", "random", "tiny"):
            if kind == "ties":
                s = rng.integers(0, 5, Ls).astype(np.float32) * 0.25
            elif kind == "const":
                s = np.full(Ls, 0.125, np.float32)
            elif kind == "random":
                s = rng.random(Ls).astype(np.float32)
            else:
                s = (rng.random(Ls) * 1e-30).astype(np.float32)
                s[::7] = 0.0
            cases.append((Ls, R, Kb, s))
    for Ls, R, Kb, s in cases:
        L, B = Ls + R, Kb + R
        p = laq.make_params(1, 1, 1, 1, 128, L, 1, R, 1, B)
        sd = torch.from_numpy(s).cuda()
        idx = torch.empty(B, dtype=torch.int32, device="cuda")
        laq.laq_select(p, sd, idx)
        want = orc.select(s, L, R, B, sorted_variant=True)
        assert (idx.cpu().numpy() == want).all(), (Ls, R, Kb)


def test_compact_strided_layouts_bit_exact(laq):
    NL, Bt, Hkv, L, D, B = 2, 2, 3, 200, 128, 37
    g = torch.Generator().manual_seed(9)
    # K stored [NL][Bt][L][Hkv][D] (position-major), V dense; output with padded head stride
    k_store = torch.randn((NL, Bt, L, Hkv, D), generator=g).to(torch.bfloat16).cuda()
    k = k_store.permute(0, 1, 3, 2, 4)
    v = torch.randn((NL, Bt, Hkv, L, D), generator=g).to(torch.bfloat16).cuda()
    idx = torch.stack([torch.randperm(L, generator=g)[:B].sort().values
                       for _ in range(NL * Bt * Hkv)]).view(NL, Bt, Hkv, B).to(torch.int32).cuda()
    out_store = torch.zeros((NL, Bt, Hkv, B + 5, D), dtype=torch.bfloat16, device="cuda")
    k_out = out_store[:, :, :, :B]
    v_store = torch.zeros_like(out_store)
    v_out = v_store[:, :, :, :B]
    p = laq.make_params(NL, Bt, Hkv, Hkv, D, L, 4, 4, 1, B, k=k, v=v, out=k_out)
    laq.laq_compact(p, k, v, idx, k_out, v_out)
    torch.cuda.synchronize()
    gather = idx.long()[..., None].expand(-1, -1, -1, -1, D)
    assert torch.equal(k_out, torch.gather(k, 3, gather))
    assert torch.equal(v_out, torch.gather(v, 3, gather))
    assert (out_store[:, :, :, B:] == 0).all()


def test_strided_kv_cache_layout(laq):
    # K/V kept position-major ([NL][Bt][L][Hkv][D]) as many serving engines store them
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 1, 2, 8, 2, 128, 600, 8, 7, 64
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=77)
    ks = k.permute(0, 1, 3, 2, 4).contiguous().cuda().permute(0, 1, 3, 2, 4)
    vs = v.permute(0, 1, 3, 2, 4).contiguous().cuda().permute(0, 1, 3, 2, 4)
    assert not ks.is_contiguous()
    out = laq.evict(q.cuda(), ks, vs, B, pool_kernel=kernel, keep_tail=W, want_scores=True)
    compare_all_units(laq, q, k, v, W, kernel, B, out=out)


def test_edge_budgets_and_no_pooling(laq):
    q, k, v = rand_inputs(1, 1, 4, 2, 128, 400, 4, seed=13)
    compare_all_units(laq, q, k, v, 4, 1, 5)        # Kb = 1, no pooling
    compare_all_units(laq, q, k, v, 0, 7, 399)      # R = 0, keep all but one
    compare_all_units(laq, q, k, v, 4, 9, 399)      # Kb = Ls - 1
    q, k, v = rand_inputs(1, 1, 2, 1, 128, 12, 2, seed=14)
    compare_all_units(laq, q, k, v, 2, 15, 5)       # pool kernel wider than the scored range


def test_evict_identical_keys_ties_go_to_lower_positions(laq):
    # every key equal => all column sums equal; pooled interior equal, edges smaller: the kept
    # set is [k/2, k/2 + Kb) by the tie rule, through the fused pool + select kernel
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 1, 2, 4, 2, 128, 2500, 4, 7, 300
    g = torch.Generator().manual_seed(31)
    q = torch.randn((NL, Bt, Hq, W, D), generator=g).to(torch.bfloat16)
    row = torch.randn((D,), generator=g).to(torch.bfloat16)
    k = row.expand(NL, Bt, Hkv, L, D).contiguous()
    v = torch.randn((NL, Bt, Hkv, L, D), generator=g).to(torch.bfloat16)
    out = run_evict(laq, q, k, v, W, kernel, B)
    idx = out["idx"].cpu().numpy()
    Kb, Ls = B - W, L - W
    want = np.concatenate([np.arange(kernel // 2, kernel // 2 + Kb), np.arange(Ls, L)])
    got_scores = out["scores"].cpu().numpy()
    for b in range(Bt):
        for h in range(Hkv):
            # equal inputs give bit-equal interior scores on the GPU as well
            assert len(set(got_scores[0, b, h, kernel // 2: Ls - kernel // 2].tolist())) == 1
            assert (idx[0, b, h] == want).all()
            assert (idx[0, b, h] == orc.select(got_scores[0, b, h], L, W, B, sorted_variant=True)).all()


LOCAL_SHAPES = [
    # NL Bt Hq Hkv D    L     W  W_local k  B    what
    (1, 2, 8, 2, 128, 1028, 16, 8, 7, 120),   # 8 local + 8 lookahead; the window straddles two tiles
    (1, 1, 4, 1, 128, 777, 32, 16, 7, 200),   # M = 128, ragged last tile
    (1, 1, 8, 1, 128, 1536, 32, 32, 5, 64),   # M = 256, local queries only (SnapKV-style window)
    (1, 1, 4, 2, 128, 200, 6, 5, 3, 30),      # window length that is not a power of two
    (1, 1, 8, 2, 64, 500, 8, 4, 7, 90),       # head_dim 64: CUDA-core path
]


@pytest.mark.parametrize("shape", LOCAL_SHAPES, ids=[f"L{s[5]}-W{s[6]}-local{s[7]}-D{s[4]}" for s in LOCAL_SHAPES])
def test_unified_window_matches_oracle(laq, shape):
    NL, Bt, Hq, Hkv, D, L, W, Wl, kernel, B = shape
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=L + Wl, kscale=1.5)
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B, local_window=Wl)
    assert err < SCORE_RTOL
    # the causal mask matters: without it the scores differ
    plain = run_evict(laq, q, k, v, W, kernel, B)
    masked = run_evict(laq, q, k, v, W, kernel, B, local_window=Wl)
    assert not torch.allclose(plain["scores"], masked["scores"], rtol=1e-3, atol=0)


VARIANT_SHAPES = [
    # NL Bt Hq Hkv D    L     W  k  B
    (1, 2, 8, 2, 128, 1300, 16, 7, 150),   # M = 64, ragged last tile
    (1, 1, 4, 1, 128, 4500, 32, 5, 300),   # M = 128, several key chunks of the raw pass
    (1, 1, 8, 2, 64, 500, 8, 3, 90),       # head_dim 64
]


@pytest.mark.parametrize("shape", VARIANT_SHAPES, ids=[f"L{s[5]}-D{s[4]}-k{s[7]}" for s in VARIANT_SHAPES])
def test_max_pooling_matches_oracle(laq, shape):
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = shape
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=L + kernel, kscale=1.5)
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B, pool_mode=1)
    assert err < SCORE_RTOL
    avg = run_evict(laq, q, k, v, W, kernel, B)
    mx = run_evict(laq, q, k, v, W, kernel, B, pool_mode=1)
    assert (mx["scores"] >= avg["scores"]).all() and not torch.equal(mx["scores"], avg["scores"])


@pytest.mark.parametrize("shape", VARIANT_SHAPES, ids=[f"L{s[5]}-D{s[4]}-k{s[7]}" for s in VARIANT_SHAPES])
def test_raw_logit_mode_matches_oracle(laq, shape):
    # Eq. 4 read literally: sums of raw logits. The sums cancel, so the error is measured against
    # the sum of the absolute terms: fp32 accumulation of D products and of M query rows stays
    # below 2e-5 of it (D * 2^-24 = 7.6e-6 for the dot product, plus the query sum).
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = shape
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=3 * L + 1)
    R, G = W, Hq // Hkv
    out = run_evict(laq, q, k, v, R, kernel, B, score_mode=1)
    ref = orc.evict(q, k, v, R, kernel, B, score_mode=1)
    got_scores, got_idx = out["scores"].cpu().numpy(), out["idx"].cpu().numpy()
    kb, vb, ko, vo = bits(k), bits(v), bits(out["k_out"]), bits(out["v_out"])
    for n in range(NL):
        for b in range(Bt):
            for h in range(Hkv):
                qs = q[n, b, h * G:(h + 1) * G].double().reshape(-1, D).sum(0)
                mag = ((k[n, b, h].double().abs() @ qs.abs()) / np.sqrt(D)).numpy()
                tol = 2e-5 * orc.pool(mag, L - R, kernel)      # the pool averages the bounds too
                ref_p = ref["scores"][n, b, h]
                assert (np.abs(got_scores[n, b, h] - ref_p) <= tol).all()
                # kept set: equal to the oracle's except where the score is within the error of
                # the oracle's Kb-th largest
                theta = np.sort(ref_p)[::-1][B - R - 1]
                diff = sorted(set(got_idx[n, b, h, :B - R].tolist()) ^ set(ref["idx"][n, b, h, :B - R].tolist()))
                assert all(abs(ref_p[j] - theta) <= 2 * tol.max() for j in diff)
                assert got_idx[n, b, h, B - R:].tolist() == list(range(L - R, L))
                want = orc.select(got_scores[n, b, h], L, R, B, sorted_variant=True)
                assert (got_idx[n, b, h] == want).all()            # negative scores order correctly
                assert (ko[n, b, h] == kb[n, b, h][got_idx[n, b, h]]).all()
                assert (vo[n, b, h] == vb[n, b, h][got_idx[n, b, h]]).all()
    assert (got_scores < 0).any() and (got_scores > 0).any()


RAGGED_SHAPES = [
    # NL Bt Hq Hkv D    L     W  W_local k  B    lens
    (1, 3, 8, 2, 128, 1500, 16, 0, 7, 100, (1500, 333, 901)),    # second chunk of prompt 1 is empty
    (2, 2, 4, 1, 128, 3000, 32, 16, 5, 200, (2049, 3000)),       # M = 128, LAQ++ window at each prompt's own end
    (1, 2, 8, 1, 128, 1536, 32, 0, 7, 64, (700, 1536)),          # M = 256
    (1, 4, 4, 2, 128, 600, 8, 8, 3, 40, (41, 128, 129, 600)),    # shortest legal prompt, tile edges
    (1, 2, 8, 2, 64, 500, 8, 4, 7, 90, (500, 200)),              # head_dim 64: CUDA-core path
]


@pytest.mark.parametrize("shape", RAGGED_SHAPES, ids=[f"L{s[5]}-M{s[2] // s[3] * s[6]}-D{s[4]}" for s in RAGGED_SHAPES])
def test_prompts_of_different_lengths_match_oracle(laq, shape):
    NL, Bt, Hq, Hkv, D, L, W, Wl, kernel, B, lens = shape
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=L + sum(lens), kscale=1.5)
    # rows beyond a prompt's length may hold anything, NaN included
    for b, Lb in enumerate(lens):
        k[:, b, :, Lb:] = float("nan")
        v[:, b, :, Lb:] = float("nan")
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B, local_window=Wl, seq_lens=lens)
    assert err < SCORE_RTOL
    # the separate entry points take the lengths too
    qc, kc, vc = q.cuda(), k.cuda(), v.cuda()
    ref = laq.evict(qc, kc, vc, B, pool_kernel=kernel, keep_tail=W, want_scores=True,
                    local_window=Wl, seq_lens=lens)
    p = ref["params"]
    scores = torch.full_like(ref["scores"], -1.0)
    idx = torch.zeros_like(ref["idx"])
    laq.laq_score(p, qc, kc, scores, ref["ws"])
    laq.laq_select(p, scores, idx)
    assert torch.equal(scores, ref["scores"]) and torch.equal(idx, ref["idx"])
    # raw-logit mode on the same ragged batch
    raw = run_evict(laq, q, k, v, W, 1, B, score_mode=1, seq_lens=lens)
    want = orc.evict(q, k, v, W, 1, B, score_mode=1, seq_lens=lens)
    got = raw["scores"].cpu().numpy()
    assert np.isfinite(got).all()
    np.testing.assert_allclose(got, want["scores"], rtol=0, atol=2e-5 * np.abs(want["scores"]).max() * 8)
    for b, Lb in enumerate(lens):
        assert (got[:, b, :, Lb - W:] == 0).all()
        assert (raw["idx"][:, b, :, B - W:].cpu().numpy() == np.arange(Lb - W, Lb)).all()


def test_largest_ragged_batch_and_many_short_units(laq):
    # 512 prompts (the most the per-prompt lengths take) of one or two tiles each, and the same
    # geometry with equal lengths: many units with a single task each
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 1, 512, 2, 1, 128, 200, 4, 3, 24
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=77)
    rng = np.random.default_rng(77)
    lens = tuple(int(x) for x in rng.integers(B + 1, L + 1, size=Bt))
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B, seq_lens=lens)
    assert err < SCORE_RTOL
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B)
    assert err < SCORE_RTOL


def test_host_buffer_entry_point_equals_device_run(laq):
    # laq_evict_host: host tensors in, compressed cache out; same kernels, so the same bits
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 2, 2, 8, 2, 128, 1100, 16, 7, 90
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=88)
    for lens, Wl in ((None, 0), ((1100, 300), 8)):
        dev = laq.evict(q.cuda(), k.cuda(), v.cuda(), B, pool_kernel=kernel, local_window=Wl, seq_lens=lens)
        he = laq.HostEvictor(tuple(q.shape), tuple(k.shape), B, kernel, W, "cuda")
        he.params.local_window = Wl
        he.params.set_seq_lens(lens)
        # pinned V: its kept rows are gathered straight from host memory; pageable V: staged
        for v_host in (v.pin_memory(), v.clone()):
            hk, hv, hidx = he.run(q.pin_memory(), k.pin_memory(), v_host)
            torch.cuda.synchronize()
            assert laq.laq_last_device_status(he.params, he.ws) == laq.LAQ_OK
            assert torch.equal(hidx, dev["idx"].cpu())
            assert torch.equal(hk.view(torch.int16), dev["k_out"].cpu().view(torch.int16))
            assert torch.equal(hv.view(torch.int16), dev["v_out"].cpu().view(torch.int16))
            assert he.h2d_bytes == 2 * (q.numel() + k.numel()) + 2 * (
                hv.numel() if v_host.is_pinned() else v.numel())
            hk.zero_(); hv.zero_(); hidx.zero_()
        # pageable outputs are staged on the device and copied back
        pk, pv, pidx = torch.zeros_like(hk, pin_memory=False), torch.zeros_like(hv, pin_memory=False), \
            torch.zeros_like(hidx, pin_memory=False)
        assert not pk.is_pinned()
        laq.laq_evict_host(he.params, q.pin_memory(), k.pin_memory(), v.clone(), pk, pv, pidx,
                           he.staging, he.ws)
        torch.cuda.synchronize()
        assert torch.equal(pidx, dev["idx"].cpu())
        assert torch.equal(pk.view(torch.int16), dev["k_out"].cpu().view(torch.int16))
        assert torch.equal(pv.view(torch.int16), dev["v_out"].cpu().view(torch.int16))


def test_evict_can_be_captured_in_a_cuda_graph(laq):
    # laq_evict only enqueues stream work (a memset and kernels): after one eager call it can be
    # captured and replayed, and the replay gives the eager call's bits on new inputs
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 2, 2, 8, 2, 128, 1500, 16, 7, 100
    q, k, v = (t.cuda() for t in rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=91))
    eager = laq.evict(q, k, v, B, pool_kernel=kernel, want_scores=True)
    p, ws = eager["params"], eager["ws"]
    k_out, v_out = torch.empty_like(eager["k_out"]), torch.empty_like(eager["v_out"])
    idx, scores = torch.empty_like(eager["idx"]), torch.empty_like(eager["scores"])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        laq.laq_evict(p, q, k, v, k_out, v_out, idx, scores, ws)   # warm-up on the capture stream
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            laq.laq_evict(p, q, k, v, k_out, v_out, idx, scores, ws)
    torch.cuda.current_stream().wait_stream(side)
    for t in (k_out, v_out, idx, scores):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(idx, eager["idx"]) and torch.equal(scores, eager["scores"])
    assert torch.equal(k_out.view(torch.int16), eager["k_out"].view(torch.int16))
    # new contents in the same buffers: the replay follows them
    q2, k2, v2 = (t.cuda() for t in rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=92))
    q.copy_(q2); k.copy_(k2); v.copy_(v2)
    graph.replay()
    torch.cuda.synchronize()
    again = laq.evict(q, k, v, B, pool_kernel=kernel, want_scores=True)
    assert torch.equal(idx, again["idx"]) and torch.equal(scores, again["scores"])
    assert torch.equal(v_out.view(torch.int16), again["v_out"].view(torch.int16))
    assert laq.laq_last_device_status(p, ws) == laq.LAQ_OK


def test_seq_lens_argument_checks(laq):
    q, k, v = rand_inputs(1, 2, 4, 2, 128, 300, 8, seed=5)
    for bad in ((300, 40), (301, 100), (300,)):     # not longer than the budget / too long / too few
        with pytest.raises((laq.LaqError, ValueError)):
            laq.evict(q.cuda(), k.cuda(), v.cuda(), 40, seq_lens=bad)


def _random_case(seed):
    """A small random problem: geometry, options and per-prompt lengths drawn from a seeded stream."""
    rng = np.random.default_rng(9000 + seed)
    D = int(rng.choice([128, 128, 128, 64]))
    Hkv = int(rng.choice([1, 2, 3]))
    G = int(rng.choice([1, 2, 4, 8]))
    W = int(rng.choice([1, 3, 8, 16, 32]))
    while G * W > 256:
        W //= 2
    L = int(rng.integers(60, 2600))
    Bt = int(rng.choice([1, 2, 3]))
    NL = int(rng.choice([1, 2]))
    R = W
    B = int(rng.integers(R + 1, max(R + 2, min(L // 2, 300))))
    kernel = int(rng.choice([1, 3, 5, 7, 9]))
    Wl = int(rng.integers(0, W + 1)) if rng.random() < 0.5 else 0
    pool_mode = int(rng.random() < 0.3)
    lens = None
    if rng.random() < 0.5:
        lens = tuple(int(x) for x in rng.integers(B + 1, L + 1, size=Bt))
    return NL, Bt, Hkv * G, Hkv, D, L, W, Wl, kernel, B, pool_mode, lens


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_and_options_match_oracle(laq, seed):
    NL, Bt, Hq, Hkv, D, L, W, Wl, kernel, B, pool_mode, lens = _random_case(seed)
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=seed, kscale=1.0 + (seed % 3))
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B, local_window=Wl, pool_mode=pool_mode,
                               seq_lens=lens)
    assert err < SCORE_RTOL


def test_variant_argument_checks(laq):
    q, k, v = rand_inputs(1, 1, 4, 2, 128, 300, 8, seed=4)
    for kw in ({"pool_mode": 2}, {"pool_mode": -1}, {"score_mode": 2}):
        with pytest.raises(laq.LaqError):
            laq.evict(q.cuda(), k.cuda(), v.cuda(), 40, **kw)


def test_local_window_argument_checks(laq):
    q, k, v = rand_inputs(1, 1, 4, 2, 128, 300, 8, seed=3)
    for bad in (9, -1):          # longer than the window / negative
        with pytest.raises(laq.LaqError):
            laq.evict(q.cuda(), k.cuda(), v.cuda(), 40, keep_tail=8, local_window=bad)
    with pytest.raises(laq.LaqError):  # local queries must lie inside the retained tail
        laq.evict(q.cuda(), k.cuda(), v.cuda(), 40, keep_tail=4, local_window=6)


def test_recall_of_two_selections_matches_oracle(laq):
    # Eq. 1-3: the set chosen by a short window against the set chosen by a longer one
    NL, Bt, Hq, Hkv, D, L, kernel, B = 1, 2, 8, 2, 128, 1500, 7, 128
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, 32, seed=91)
    gold = run_evict(laq, q, k, v, 8, kernel, B)["idx"]                    # all 32 queries
    pred = run_evict(laq, q[:, :, :, :8].contiguous(), k, v, 8, kernel, B)["idx"]  # the first 8
    rec, common = laq.laq_recall(pred, gold)
    torch.cuda.synchronize()
    for b in range(Bt):
        for h in range(Hkv):
            r, n = orc.recall(pred[0, b, h].cpu().numpy(), gold[0, b, h].cpu().numpy())
            assert int(common[0, b, h]) == n
            assert float(rec[0, b, h]) == pytest.approx(r, rel=1e-6)
            assert 8 <= n < B          # the retained tail is always shared; the rest differs
    same, n_same = laq.laq_recall(gold, gold)
    assert (same == 1.0).all() and (n_same == B).all()
    # different set sizes
    small = gold[..., :40].contiguous()
    r2, n2 = laq.laq_recall(small, gold)
    assert (n2 == 40).all() and torch.allclose(r2, torch.full_like(r2, 40 / B))


def test_layer_wise_budgets_on_layer_slices(laq):
    # a pyramid of budgets, read back through the per-layer views of the ragged pool
    NL, Bt, Hq, Hkv, D, L, W, kernel = 4, 1, 4, 2, 128, 640, 8, 7
    budgets = [96, 96, 48, 24]
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=61)
    outs = laq.evict_layer_budgets(q.cuda(), k.cuda(), v.cuda(), budgets, pool_kernel=kernel)["layers"]
    torch.cuda.synchronize()
    for n, B in enumerate(budgets):
        ref = orc.evict(q[n:n + 1], k[n:n + 1], v[n:n + 1], W, kernel, B)
        got = outs[n]["idx"].cpu().numpy()
        for b in range(Bt):
            for h in range(Hkv):
                check_index_set(got[b, h], ref["idx"][0, b, h], ref["scores"][0, b, h], L, W, B)
                assert (bits(outs[n]["k_out"][b, h]) == bits(k[n, b, h])[got[b, h]]).all()
                assert (bits(outs[n]["v_out"][b, h]) == bits(v[n, b, h])[got[b, h]]).all()


def test_extreme_logits_and_late_maximum(laq):
    # logits of +-hundreds: the running reference of sweep 1 has to move several times, also in the
    # middle of a task, and sweep 2 sees probabilities far below the smallest fp32 normal
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 1, 1, 8, 2, 128, 2304, 16, 7, 150
    g = torch.Generator().manual_seed(404)
    q = torch.randn((NL, Bt, Hq, W, D), generator=g).to(torch.bfloat16)
    k = (torch.randn((NL, Bt, Hkv, L, D), generator=g) * 12.0).to(torch.bfloat16)
    v = torch.randn((NL, Bt, Hkv, L, D), generator=g).to(torch.bfloat16)
    # a key aligned with the mean query of each unit, very late in the prompt and very large
    for h in range(Hkv):
        qbar = q[0, 0, h * 4:(h + 1) * 4].float().mean(dim=(0, 1))
        k[0, 0, h, 2100] = (qbar * 60.0).to(torch.bfloat16)
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B)
    assert err < SCORE_RTOL


def test_extreme_logits_with_one_or_two_lookahead_steps(laq):
    # the same stress for the short windows of Section 6.2 (one or two lookahead steps, M = 8):
    # the large key arrives late, after many tiles of small logits
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 1, 1, 8, 2, 128, 4200, 2, 7, 90
    g = torch.Generator().manual_seed(405)
    q = torch.randn((NL, Bt, Hq, W, D), generator=g).to(torch.bfloat16)
    k = (torch.randn((NL, Bt, Hkv, L, D), generator=g) * 12.0).to(torch.bfloat16)
    v = torch.randn((NL, Bt, Hkv, L, D), generator=g).to(torch.bfloat16)
    for h in range(Hkv):
        qbar = q[0, 0, h * 4:(h + 1) * 4].float().mean(dim=(0, 1))
        k[0, 0, h, 3900] = (qbar * 60.0).to(torch.bfloat16)
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B)
    assert err < SCORE_RTOL
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B, local_window=1, seq_lens=None)
    assert err < SCORE_RTOL


def test_single_row_and_explicit_scale(laq):
    # M = 1 (one query head per KV head, one lookahead query) and a caller-chosen softmax scale
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 1, 2, 2, 2, 128, 700, 1, 3, 30
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=55)
    scale = 0.05
    out = laq.evict(q.cuda(), k.cuda(), v.cuda(), B, pool_kernel=kernel, keep_tail=W,
                    want_scores=True, softmax_scale=scale)
    ref = orc.evict(q, k, v, W, kernel, B, scale=scale)
    assert score_rel_err(out["scores"].cpu().numpy(), ref["scores"]) <= SCORE_RTOL
    # the default scale gives different scores, so the argument is really used
    out2 = laq.evict(q.cuda(), k.cuda(), v.cuda(), B, pool_kernel=kernel, keep_tail=W, want_scores=True)
    assert not torch.allclose(out["scores"], out2["scores"])


def test_workspace_reuse_back_to_back(laq):
    q, k, v = rand_inputs(2, 1, 8, 2, 128, 1300, 8, seed=21)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    a = laq.evict(qd, kd, vd, 100, want_scores=True)
    b = laq.evict(qd, kd, vd, 100, want_scores=True, ws=a["ws"])
    c = laq.evict(qd, kd, vd, 100, want_scores=True, ws=a["ws"])
    torch.cuda.synchronize()
    assert torch.equal(a["scores"], b["scores"]) and torch.equal(a["idx"], c["idx"])
    assert torch.equal(a["k_out"], c["k_out"])


# ---------------------------------------------------------------- the paper-shaped configs
def test_per_layer_budgets_write_one_ragged_pool(laq):
    # a pyramid of budgets; with and without per-prompt lengths; every layer against the oracle
    NL, Bt, Hq, Hkv, D, L, W, kernel = 4, 2, 8, 2, 128, 1100, 8, 7
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=71, kscale=1.5)
    for budgets, lens in (([160, 128, 96, 64], None), ([64, 300, 64, 65], [1100, 700])):
        out = laq.evict_layer_budgets(q.cuda(), k.cuda(), v.cuda(), budgets, pool_kernel=kernel,
                                      seq_lens=lens)
        assert laq.laq_last_device_status(out["params"], out["ws"]) == laq.LAQ_OK
        ref = orc.evict_layers(q, k, v, W, kernel, budgets, seq_lens=lens)
        got_idx = out["idx"].cpu().numpy()
        assert got_idx.shape == ref["idx"].shape
        kb, vb = bits(k), bits(v)
        ko, vo = bits(out["k_out"]), bits(out["v_out"])
        row = 0
        for n, B in enumerate(budgets):
            for b in range(Bt):
                Lb = L if lens is None else lens[b]
                for h in range(Hkv):
                    gi = got_idx[row:row + B]
                    check_index_set(gi, ref["idx"][row:row + B], ref["scores"][n, b, h][:Lb - W], Lb, W, B)
                    assert (ko[row:row + B] == kb[n, b, h][gi]).all()
                    assert (vo[row:row + B] == vb[n, b, h][gi]).all()
                    row += B
        assert row == got_idx.shape[0]
    # equal budgets give exactly what laq_evict gives
    uni = run_evict(laq, q, k, v, W, kernel, 100)
    same = laq.evict_layer_budgets(q.cuda(), k.cuda(), v.cuda(), [100] * NL, pool_kernel=kernel)
    assert torch.equal(same["idx"].view_as(uni["idx"]), uni["idx"])
    assert torch.equal(same["k_out"].view_as(uni["k_out"]), uni["k_out"])
    # host-side validation: the largest budget must be the one that sized the workspace
    p = laq.params_for(q.cuda(), k.cuda(), W, kernel, 100, v=v.cuda())
    assert laq.laq_layers_pool_entries(p, [100, 50, 120, 60]) == 0
    assert laq.laq_layers_pool_entries(p, [100, 50, W, 60]) == 0


def test_streaming_keep_set_and_its_compaction(laq):
    NL, Bt, Hq, Hkv, D, L, W, B, n_sink = 2, 3, 4, 2, 128, 500, 4, 48, 4
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=72)
    kd, vd = k.cuda(), v.cuda()
    for lens in (None, [500, 333, 49]):
        p = laq.params_for(q.cuda(), kd, W, 7, B, v=vd)
        p.set_seq_lens(lens)
        idx = torch.empty((NL, Bt, Hkv, B), dtype=torch.int32, device="cuda")
        laq.laq_streaming_indices(p, n_sink, idx)
        k_out = torch.empty((NL, Bt, Hkv, B, D), dtype=torch.bfloat16, device="cuda")
        v_out = torch.empty_like(k_out)
        laq.laq_compact(p, kd, vd, idx, k_out, v_out)
        got = idx.cpu().numpy()
        for b in range(Bt):
            want = orc.streaming_indices(L, B, n_sink, None if lens is None else lens[b])
            for n in range(NL):
                for h in range(Hkv):
                    assert (got[n, b, h] == want).all()
                    assert (bits(k_out[n, b, h]) == orc.compact(k[n, b, h], want)).all()
                    assert (bits(v_out[n, b, h]) == orc.compact(v[n, b, h], want)).all()
    p = laq.params_for(q.cuda(), kd, W, 7, B, v=vd)
    assert laq.laq_streaming_indices(p, B + 1, idx, check=False) == laq.LAQ_ERR_INVALID_ARG
    assert laq.laq_streaming_indices(p, -1, idx, check=False) == laq.LAQ_ERR_INVALID_ARG


GROUP_SHAPES = [
    # NL Bt Hq Hkv D    L     W  k  B
    (1, 2, 8, 2, 128, 1300, 32, 7, 120),   # one head per 32-row chunk (tensor-core path)
    (2, 1, 8, 2, 128, 900, 8, 5, 64),      # four heads per chunk, M = 32
    (1, 1, 8, 2, 128, 700, 16, 7, 90),     # two heads per chunk, M = 64
    (1, 1, 4, 1, 128, 640, 64, 7, 100),    # a head spans two chunks, M = 256
    (1, 1, 6, 2, 128, 500, 5, 3, 33),      # W = 5: heads straddle the groups of four -> CUDA-core path
    (1, 1, 8, 2, 64, 400, 8, 7, 60),       # head_dim 64: CUDA-core path
]


@pytest.mark.parametrize("mode", [1, 2], ids=["max-over-group", "per-query-head"])
@pytest.mark.parametrize("shape", GROUP_SHAPES, ids=[f"L{s[5]}-W{s[6]}-G{s[2] // s[3]}-D{s[4]}" for s in GROUP_SHAPES])
def test_group_modes_match_oracle(laq, shape, mode):
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = shape
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=300 + L + mode, kscale=1.5)
    err, _ = compare_all_units(laq, q, k, v, W, kernel, B, group_mode=mode)
    assert err < SCORE_RTOL


def test_group_modes_with_ragged_prompts_and_raw_mode_refusal(laq):
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 1, 3, 8, 2, 128, 1000, 16, 7, 80
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=311, kscale=1.5)
    k[:, 1, :, 600:] = float("nan")   # never read
    k[:, 2, :, 81:] = float("nan")
    for mode in (1, 2):
        compare_all_units(laq, q, k, v, W, kernel, B, seq_lens=[1000, 600, 81], group_mode=mode)
    p = laq.params_for(q.cuda(), k.cuda(), W, kernel, B)
    p.group_mode, p.score_mode = laq.LAQ_GROUP_MAX, laq.LAQ_SCORE_RAW
    assert laq.laq_workspace_bytes(p) == 0   # an unsupported combination has no workspace size


def test_per_layer_budgets_with_per_query_head_selection(laq):
    # the two options together: the ragged pool then holds [Bt][Hq][B_n] entries per layer
    NL, Bt, Hq, Hkv, D, L, W, kernel = 3, 1, 4, 2, 128, 900, 8, 5
    budgets = [40, 120, 64]
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=73, kscale=1.5)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    p = laq.params_for(qd, kd, W, kernel, max(budgets), v=vd)
    p.group_mode = laq.LAQ_GROUP_PER_HEAD
    entries = laq.laq_layers_pool_entries(p, budgets)
    assert entries == Bt * Hq * sum(budgets)
    idx = torch.empty(entries, dtype=torch.int32, device="cuda")
    k_out = torch.empty((entries, D), dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)
    ws = laq.alloc_workspace(p, "cuda")
    laq.laq_evict_layers(p, budgets, qd, kd, vd, k_out, v_out, idx, None, ws)
    assert laq.laq_last_device_status(p, ws) == laq.LAQ_OK
    ref = orc.evict_layers(q, k, v, W, kernel, budgets, group_mode=2)
    got = idx.cpu().numpy()
    G, row = Hq // Hkv, 0
    for n, B in enumerate(budgets):
        for hq in range(Hq):
            gi = got[row:row + B]
            check_index_set(gi, ref["idx"][row:row + B], ref["scores"][n, 0, hq], L, W, B)
            assert (bits(k_out[row:row + B]) == bits(k[n, 0, hq // G])[gi]).all()
            assert (bits(v_out[row:row + B]) == bits(v[n, 0, hq // G])[gi]).all()
            row += B


def test_gather_of_more_units_than_one_grid_dimension_holds(laq):
    # 70 000 units: the gather runs in slabs of 65 535 units
    NL, Bt, Hkv, D, L, B = 1, 8750, 8, 8, 16, 4
    g = torch.Generator().manual_seed(74)
    k = torch.randn((NL, Bt, Hkv, L, D), generator=g).to(torch.bfloat16).cuda()
    v = torch.randn((NL, Bt, Hkv, L, D), generator=g).to(torch.bfloat16).cuda()
    idx = torch.stack([torch.randperm(L, generator=g)[:B].sort().values for _ in range(64)])
    idx = idx.repeat(NL * Bt * Hkv // 64 + 1, 1)[:NL * Bt * Hkv].view(NL, Bt, Hkv, B).to(torch.int32).cuda()
    p = laq.make_params(NL, Bt, Hkv, Hkv, D, L, 1, 1, 1, B)
    k_out = torch.zeros((NL, Bt, Hkv, B, D), dtype=torch.bfloat16, device="cuda")
    v_out = torch.zeros_like(k_out)
    laq.laq_compact(p, k, v, idx, k_out, v_out)
    want_k = torch.gather(k, 3, idx.long()[..., None].expand(-1, -1, -1, -1, D))
    want_v = torch.gather(v, 3, idx.long()[..., None].expand(-1, -1, -1, -1, D))
    assert torch.equal(k_out, want_k) and torch.equal(v_out, want_v)


def test_long_units_select_in_a_pair_of_thread_blocks(laq):
    # 32768 < L - R <= 65536: two thread blocks share a unit's pooling and top-k
    D, W, kernel = 128, 1, 7
    # identical keys: every score ties; the kept set is [k/2, k/2 + Kb) and crosses the boundary
    # between the two blocks, so the tie-break has to be split between them
    for L, B in ((50000, 40000), (65536, 33000), (32800, 50)):
        q = torch.randn((1, 2, 1, W, D), generator=torch.Generator().manual_seed(L)).to(torch.bfloat16)
        k = torch.full((1, 2, 1, L, D), 0.25).to(torch.bfloat16)
        v = torch.randn((1, 2, 1, L, D), generator=torch.Generator().manual_seed(L + 1)).to(torch.bfloat16)
        out = run_evict(laq, q, k, v, W, kernel, B)
        want = list(range(kernel // 2, kernel // 2 + B - W)) + list(range(L - W, L))
        for b in range(2):
            assert out["idx"][0, b, 0].cpu().tolist() == want, (L, B, b)
            assert (bits(out["v_out"][0, b, 0]) == bits(v[0, b, 0])[np.array(want)]).all()
    # random keys: scores against the oracle, selection bit-exact on the GPU's own scores
    NL, Bt, Hq, Hkv, L, W, B = 1, 1, 4, 2, 60000, 4, 3000
    q, k, v = rand_inputs(NL, Bt, Hq, Hkv, D, L, W, seed=75, kscale=1.5)
    compare_all_units(laq, q, k, v, W, kernel, B)
    compare_all_units(laq, q, k, v, W, 5, 40000, seq_lens=[45000], pool_mode=1)


def test_config1_full_with_planted_key(laq):
    cfg = synth.CONFIGS[1]
    inp = synth.make_inputs(cfg, "cpu")
    B = cfg.budgets[0]
    out = run_evict(laq, inp["q"], inp["k"], inp["v"], cfg.keep_tail, cfg.pool_kernel, B)
    compare_all_units(laq, inp["q"], inp["k"], inp["v"], cfg.keep_tail, cfg.pool_kernel, B, out=out)
    assert int(inp["planted"]["one"][0, 0, 0]) in set(out["idx"][0, 0, 0].tolist())


def sampled_parity(laq, cfg, budgets, units, device="cuda"):
    """Runs the full-size problem on the GPU, in the launch configuration the benchmark times, and
    checks the listed units against the oracle. The scores do not depend on the budget, so the
    oracle scores every sampled unit once (all of them in one call, spread over its OpenMP
    threads) and only re-selects per budget."""
    inp = synth.make_inputs(cfg, device)
    q, k, v = inp["q"], inp["k"], inp["v"]
    R, L, D = cfg.keep_tail, cfg.prompt_len, cfg.head_dim
    NL, Bt, Hkv = cfg.n_layers, cfg.batch, cfg.n_kv_heads
    units = sorted(set(int(u) for u in units))
    slices = [synth.unit_slices(cfg, inp, u) for u in units]
    qs = torch.stack([x[0][0] for x in slices])   # [n, 1, G, W, D]
    ks = torch.stack([x[1][0] for x in slices])   # [n, 1, 1, L, D]
    ref_scores = orc.evict(qs, ks, None, R, cfg.pool_kernel, max(budgets), want_idx=False)["scores"]
    worst = 0.0
    ws = None
    for B in budgets:
        k_out = torch.empty((NL, Bt, Hkv, B, D), dtype=torch.bfloat16, device=k.device)
        v_out = torch.empty_like(k_out)
        idx = torch.empty((NL, Bt, Hkv, B), dtype=torch.int32, device=k.device)
        scores = torch.empty((NL, Bt, Hkv, L - R), dtype=torch.float32, device=k.device)
        p = laq.params_for(q, k, R, cfg.pool_kernel, B, v=v, out=k_out)
        if ws is None or ws.numel() < laq.laq_workspace_bytes(p):
            ws = laq.alloc_workspace(p, k.device)
        laq.laq_evict(p, q, k, v, k_out, v_out, idx, scores, ws)
        assert laq.laq_last_device_status(p, ws) == laq.LAQ_OK
        # a second run hands the tasks to other SMs in another order; the bits must not change
        scores2, idx2 = torch.empty_like(scores), torch.empty_like(idx)
        laq.laq_evict(p, q, k, v, k_out, v_out, idx2, scores2, ws)
        assert torch.equal(scores, scores2) and torch.equal(idx, idx2)
        del scores2, idx2
        for j, u in enumerate(units):
            h, b, n = u % Hkv, (u // Hkv) % Bt, u // (Hkv * Bt)
            ku, vu = slices[j][1], slices[j][2]
            ref_s = ref_scores[j, 0, 0]
            ref_idx = orc.select(ref_s, L, R, B, sorted_variant=True)
            got_s = scores[n, b, h].cpu().numpy()
            err = score_rel_err(got_s, ref_s)
            worst = max(worst, err)
            assert err <= SCORE_RTOL, f"unit {u} B {B}: score rel err {err:.3e}"
            gi = idx[n, b, h].cpu().numpy()
            check_index_set(gi, ref_idx, ref_s, L, R, B)
            assert (gi == orc.select(got_s, L, R, B, sorted_variant=True)).all()
            assert (bits(k_out[n, b, h]) == bits(ku[0, 0, 0])[gi]).all()
            assert (bits(v_out[n, b, h]) == bits(vu[0, 0, 0])[gi]).all()
            if "sink" in inp["planted"]:
                assert 0 in set(gi.tolist())
            if "needles" in inp["planted"] and B - R >= (cfg.n_needles + 1) * cfg.pool_kernel:
                assert set(inp["planted"]["needles"][n, b, h].tolist()) <= set(gi.tolist())
    return worst


def spread_units(cfg, n_random):
    """First and last layer, every batch item and KV head at least once, plus seeded random units."""
    Hkv, Bt, NL = cfg.n_kv_heads, cfg.batch, cfg.n_layers
    units = set(synth.sample_units(cfg, n_random))
    for b in range(Bt):  # every batch item, in the first and in the last layer, rotating the head
        units.add((0 * Bt + b) * Hkv + b % Hkv)
        units.add(((NL - 1) * Bt + b) * Hkv + (b + 1) % Hkv)
    units.add(cfg.units - 1)
    return sorted(units)


def test_config2_full_size_sampled_units(laq):
    cfg = synth.CONFIGS[2]
    sampled_parity(laq, cfg, cfg.budgets, spread_units(cfg, 8))


def test_config3_full_size_sampled_units(laq):
    cfg = synth.CONFIGS[3]
    units = spread_units(cfg, 6)
    assert len(units) >= 16
    sampled_parity(laq, cfg, cfg.budgets, units)   # 128, 256, 512, 1024, 2048


def test_config4_full_size_sampled_units(laq):
    cfg = synth.CONFIGS[4]
    units = spread_units(cfg, 4)
    assert len(units) >= 16
    sampled_parity(laq, cfg, cfg.budgets, units)


def test_config5_full_size_one_pool(laq):
    cfg = synth.CONFIGS[5]
    units = spread_units(cfg, 4)  # the last unit's keys lie beyond 2^32 bytes from the base
    assert len(units) >= 16 and units[-1] == cfg.units - 1
    sampled_parity(laq, cfg, cfg.budgets, units)   # 256 and 2048
