"""Pins for the fp64 CPU oracle: each test checks it against something other than itself -- a
hand-derived example, brute force, an independent library routine (torch fp64 on CPU), a closed
form or an invariant -- chosen so that a dropped term, a wrong sign or index or a transposed
operand fails at least one of them. No GPU needed."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import laq_oracle as orc
from paper_2505_20334_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(t):
    return t.to(torch.bfloat16)


def rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return bf16(torch.randn(shape, generator=g) * scale)


def torch_colsum(q, k, scale):
    """Independent statement with library routines: softmax over keys, summed over rows."""
    G, W, D = q.shape
    s = (q.double().reshape(G * W, D) @ k.double().T) * scale
    return torch.softmax(s, dim=-1).sum(0).numpy(), s


# ---------------------------------------------------------------- hand-derived example
def test_hand_example_exact_rationals():
    vals = {}
    with open(os.path.join(GOLDEN, "hand_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *nums = line.split()
            vals[key] = [int(x) for x in nums]
    q = bf16(torch.tensor([[[1.0], [2.0]]]))  # G=1, W=2, D=1
    k = bf16(torch.tensor([[0.0], [1.0], [2.0]]))
    c, m, l = orc.unit_colsum(q, k, scale=math.log(2.0))
    want_c = [Fraction(n, vals["c_den"][0]) for n in vals["c_num"]]
    np.testing.assert_allclose(c, [float(x) for x in want_c], rtol=1e-14)
    np.testing.assert_allclose(m, [2 * math.log(2), 4 * math.log(2)], rtol=1e-15)
    want_l = [Fraction(n, d) for n, d in zip(vals["l_num"], vals["l_den"])]
    np.testing.assert_allclose(l, [float(x) for x in want_l], rtol=1e-14)
    p = orc.pool(c, 3, 3)
    want_p = [Fraction(n, vals["p_den"][0]) for n in vals["p_num"]]
    np.testing.assert_allclose(p, [float(x) for x in want_p], rtol=1e-14)
    idx = orc.select(p, L=3, R=0, B=2)
    assert idx.tolist() == [1, 2]


# ---------------------------------------------------------------- softmax / column sums
@pytest.mark.parametrize("G,W,D,L", [(1, 1, 2, 3), (2, 3, 4, 7), (3, 2, 8, 16)])
def test_bruteforce_softmax_tiny(G, W, D, L):
    q = rand_bf16((G, W, D), 1)
    k = rand_bf16((L, D), 2)
    scale = 1.0 / math.sqrt(D)
    c, m, l = orc.unit_colsum(q, k)
    ql = q.double().reshape(G * W, D).tolist()
    kl = k.double().tolist()
    want = [0.0] * L
    for r in range(G * W):
        e = [math.exp(scale * sum(ql[r][d] * kl[j][d] for d in range(D))) for j in range(L)]
        z = math.fsum(e)  # naive exp / sum(exp): no max subtraction
        for j in range(L):
            want[j] += e[j] / z
        smax = max(scale * sum(ql[r][d] * kl[j][d] for d in range(D)) for j in range(L))
        assert m[r] == pytest.approx(smax, rel=1e-14, abs=1e-15)
        assert m[r] + math.log(l[r]) == pytest.approx(math.log(z), rel=1e-13, abs=1e-13)
    np.testing.assert_allclose(c, want, rtol=1e-13)


@pytest.mark.parametrize("G,W,D,L,seed", [(4, 8, 128, 300, 3), (1, 5, 64, 77, 4), (8, 2, 32, 129, 5)])
def test_against_torch_softmax_fp64(G, W, D, L, seed):
    q = rand_bf16((G, W, D), seed)
    k = rand_bf16((L, D), seed + 100, scale=1.5)
    scale = 1.0 / math.sqrt(D)
    c, m, l = orc.unit_colsum(q, k)
    want, s = torch_colsum(q, k, scale)
    np.testing.assert_allclose(c, want, rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(m, s.max(dim=-1).values.numpy(), rtol=1e-14)
    np.testing.assert_allclose(m + np.log(l), torch.logsumexp(s, dim=-1).numpy(), rtol=1e-13)
    # each query's probabilities sum to one, so the column sums add up to M = G*W
    assert c.sum() == pytest.approx(G * W, rel=1e-12)
    assert (c > 0).all()


def test_explicit_scale_argument_is_used():
    q = rand_bf16((2, 2, 16), 11)
    k = rand_bf16((40, 16), 12)
    c, _, _ = orc.unit_colsum(q, k, scale=0.37)
    want, _ = torch_colsum(q, k, 0.37)
    np.testing.assert_allclose(c, want, rtol=1e-12)
    c0, _, _ = orc.unit_colsum(q, k)
    assert not np.allclose(c, c0, rtol=1e-3)


def test_zero_queries_give_uniform_attention():
    G, W, D, L = 2, 3, 16, 50
    q = bf16(torch.zeros((G, W, D)))
    k = rand_bf16((L, D), 7)
    c, m, l = orc.unit_colsum(q, k)
    np.testing.assert_allclose(c, np.full(L, G * W / L), rtol=1e-14)
    np.testing.assert_allclose(l, np.full(G * W, L), rtol=1e-14)


def test_key_shift_invariance_exact_inputs():
    # integers are exact in bf16, so shifting every key by the same vector changes each row's
    # logits by a constant and leaves the softmax untouched
    g = torch.Generator().manual_seed(21)
    q = bf16(torch.randint(-2, 3, (2, 2, 8), generator=g).float())
    k = torch.randint(-4, 5, (33, 8), generator=g).float()
    delta = torch.randint(-3, 4, (8,), generator=g).float()
    c1, _, _ = orc.unit_colsum(q, bf16(k))
    c2, _, _ = orc.unit_colsum(q, bf16(k + delta))
    np.testing.assert_allclose(c1, c2, rtol=1e-12)


def test_additivity_over_heads_and_queries():
    G, W, D, L = 3, 4, 32, 90
    q = rand_bf16((G, W, D), 31)
    k = rand_bf16((L, D), 32)
    c, _, _ = orc.unit_colsum(q, k)
    by_head = sum(orc.unit_colsum(q[g:g + 1], k)[0] for g in range(G))
    by_query = sum(orc.unit_colsum(q[:, i:i + 1], k)[0] for i in range(W))
    np.testing.assert_allclose(c, by_head, rtol=1e-12)
    np.testing.assert_allclose(c, by_query, rtol=1e-12)


# ---------------------------------------------------------------- pooling
@pytest.mark.parametrize("kernel", [1, 3, 5, 7])
def test_pool_matches_library_avg_pool(kernel):
    g = torch.Generator().manual_seed(41)
    c = torch.rand(57, generator=g, dtype=torch.float64)
    p = orc.pool(c.numpy(), 57, kernel)
    want = torch.nn.functional.avg_pool1d(c[None, None], kernel, stride=1, padding=kernel // 2,
                                          count_include_pad=True)[0, 0].numpy()
    np.testing.assert_allclose(p, want, rtol=1e-13)
    if kernel == 1:
        assert (p == c.numpy()).all()


def test_pool_ignores_tail_positions():
    # positions >= Ls (the retained tail) are invisible to the pool
    c = np.arange(1.0, 21.0)
    p_a = orc.pool(c, 15, 5)
    c2 = c.copy()
    c2[15:] = 1e9
    p_b = orc.pool(c2, 15, 5)
    assert (p_a == p_b).all()
    assert p_a[14] == pytest.approx((13 + 14 + 15) / 5.0)


def test_pool_closed_forms():
    kernel, Ls, val = 7, 40, 0.125
    p = orc.pool(np.full(Ls, val), Ls, kernel)
    h = kernel // 2
    for j in range(Ls):
        cover = min(j, h) + 1 + min(Ls - 1 - j, h)
        assert p[j] == pytest.approx(val * cover / kernel, rel=1e-15)
    c = np.random.default_rng(5).random(Ls)
    p = orc.pool(c, Ls, kernel)
    cover = np.array([min(j, h) + 1 + min(Ls - 1 - j, h) for j in range(Ls)])
    assert p.sum() == pytest.approx((c * cover).sum() / kernel, rel=1e-13)


# ---------------------------------------------------------------- selection
def test_select_identical_keys_closed_form():
    # identical keys: c_j = M/L everywhere, so only the pool's edge attenuation and the tie-break
    # decide: the kept set is [k/2, k/2 + Kb) followed by the tail
    G, W, D, L, R, kernel, B = 2, 4, 16, 64, 4, 7, 20
    q = rand_bf16((1, 1, G, W, D), 51)
    k = bf16(torch.ones((1, 1, 1, L, D)) * 0.5)
    out = orc.evict(q, k, k, R, kernel, B, fast_select=False)
    want = list(range(kernel // 2, kernel // 2 + (B - R))) + list(range(L - R, L))
    assert out["idx"][0, 0, 0].tolist() == want
    out2 = orc.evict(q, k, k, R, kernel, B, fast_select=True)
    assert out2["idx"][0, 0, 0].tolist() == want
    np.testing.assert_allclose(out["scores"][0, 0, 0, 10], G * W / L, rtol=1e-13)


def test_select_reduces_to_topk_of_raw_logits():
    # W = G = k = 1, R = 0: softmax is monotone, so the kept set is the top-B of q.k
    D, L, B = 32, 200, 17
    q = rand_bf16((1, 1, 1, 1, D), 61)
    k = rand_bf16((1, 1, 1, L, D), 62)
    out = orc.evict(q, k, k, 0, 1, B)
    logits = k[0, 0, 0].double() @ q[0, 0, 0, 0].double()
    want = sorted(torch.topk(logits, B).indices.tolist())
    assert out["idx"][0, 0, 0].tolist() == want


def test_select_structure_ties_and_variants_agree():
    rng = np.random.default_rng(71)
    for L, R, B in [(50, 4, 12), (33, 0, 33), (40, 8, 9), (17, 3, 16)]:
        p = rng.integers(0, 6, L - R).astype(np.float64)  # many ties
        a = orc.select(p, L, R, B)
        b = orc.select(p, L, R, B, sorted_variant=True)
        assert (a == b).all()
        Kb = B - R
        assert a.shape == (B,) and len(set(a.tolist())) == B
        assert (np.diff(a[:Kb]) > 0).all() and (a[:Kb] < L - R).all() if Kb > 1 else True
        assert a[Kb:].tolist() == list(range(L - R, L))
        # independent statement: stable argsort of -p (ties keep the lower position first)
        want = np.sort(np.argsort(-p, kind="stable")[:Kb])
        assert (a[:Kb] == want).all()
        thr = np.sort(p)[::-1][Kb - 1]
        assert (p[a[:Kb]] >= thr).all()


def test_select_budget_nestedness():
    p = np.random.default_rng(81).random(300)
    prev = set()
    for B in [8, 16, 64, 200]:
        cur = set(orc.select(p, 304, 4, B).tolist())
        assert prev <= cur
        prev = cur


# ---------------------------------------------------------------- compaction, GQA mapping, whole step
def test_compact_is_row_gather():
    src = rand_bf16((30, 16), 91)
    idx = np.array([3, 4, 9, 29, 0], np.int32)
    got = orc.compact(src, idx)
    want = src.view(torch.int16).numpy().view(np.uint16)[idx]
    assert (got == want).all()


def test_evict_gqa_mapping_and_dense_layout():
    NL, Bt, Hq, Hkv, D, L, W, R, kernel, B = 2, 2, 6, 2, 16, 48, 3, 3, 3, 11
    G = Hq // Hkv
    q = rand_bf16((NL, Bt, Hq, W, D), 101)
    k = rand_bf16((NL, Bt, Hkv, L, D), 102)
    v = rand_bf16((NL, Bt, Hkv, L, D), 103)
    out = orc.evict(q, k, v, R, kernel, B, want_colsum=True, fast_select=False)
    # library statement of GQA: repeat each KV head G times, attend per query head, then sum the
    # G heads of a group
    kr = k.double().repeat_interleave(G, dim=2)  # [NL,Bt,Hq,L,D]
    s = torch.einsum("nbhwd,nbhld->nbhwl", q.double(), kr) / math.sqrt(D)
    c = torch.softmax(s, dim=-1).sum(3).view(NL, Bt, Hkv, G, L).sum(3)
    np.testing.assert_allclose(out["colsum"], c.numpy(), rtol=1e-12)
    pooled = torch.nn.functional.avg_pool1d(c[..., :L - R].reshape(-1, 1, L - R), kernel, 1,
                                            kernel // 2).view(NL, Bt, Hkv, L - R)
    np.testing.assert_allclose(out["scores"], pooled.numpy(), rtol=1e-12)
    kb = k.view(torch.int16).numpy().view(np.uint16)
    vb = v.view(torch.int16).numpy().view(np.uint16)
    for n in range(NL):
        for b in range(Bt):
            for h in range(Hkv):
                idx = out["idx"][n, b, h]
                want = np.sort(np.argsort(-out["scores"][n, b, h], kind="stable")[:B - R])
                assert (idx[:B - R] == want).all()
                assert idx[B - R:].tolist() == list(range(L - R, L))
                assert (out["k_out"][n, b, h] == kb[n, b, h][idx]).all()
                assert (out["v_out"][n, b, h] == vb[n, b, h][idx]).all()


def test_evict_unit_list_matches_full_run():
    q = rand_bf16((2, 1, 4, 2, 16), 111)
    k = rand_bf16((2, 1, 2, 40, 16), 112)
    full = orc.evict(q, k, k, 2, 3, 10)
    part = orc.evict(q, k, k, 2, 3, 10, units=[1, 2])
    for u in (1, 2):
        n, h = divmod(u, 2)
        assert (part["idx"][n, 0, h] == full["idx"][n, 0, h]).all()
        assert (part["scores"][n, 0, h] == full["scores"][n, 0, h]).all()
    assert (part["idx"][0, 0, 0] == 0).all()


def test_config1_planted_key_is_kept():
    cfg = synth.CONFIGS[1]
    inp = synth.make_inputs(cfg, "cpu")
    out = orc.evict(inp["q"], inp["k"], inp["v"], cfg.keep_tail, cfg.pool_kernel, cfg.budgets[0])
    idx = out["idx"][0, 0, 0]
    B, R, L = cfg.budgets[0], cfg.keep_tail, cfg.prompt_len
    assert idx.shape == (B,) and len(set(idx.tolist())) == B
    assert idx[B - R:].tolist() == list(range(L - R, L))
    assert int(inp["planted"]["one"][0, 0, 0]) in set(idx.tolist())
    assert out["scores"].sum() <= cfg.rows + 1e-9


def test_sink_and_needles_kept_when_budget_allows():
    cfg = synth.CONFIGS[3].scaled(n_layers=1, batch=1, n_kv_heads=2, n_q_heads=8, prompt_len=2048,
                                  window_len=8)
    inp = synth.make_inputs(cfg, "cpu")
    B = 8 + (cfg.n_needles + 1) * cfg.pool_kernel + 64
    out = orc.evict(inp["q"], inp["k"], inp["v"], cfg.keep_tail, cfg.pool_kernel, B)
    for h in range(cfg.n_kv_heads):
        kept = set(out["idx"][0, 0, h].tolist())
        assert 0 in kept
        assert set(inp["planted"]["needles"][0, 0, h].tolist()) <= kept


# ---------------------------------------------------------------- LAQ++ unified window (Eq. 5)
def _visible(i, W_local, L):
    return L - W_local + i + 1 if i < W_local else L


@pytest.mark.parametrize("G,W,Wl,D,L", [(1, 2, 1, 2, 4), (2, 4, 2, 4, 9), (2, 5, 5, 8, 12)])
def test_local_window_bruteforce_causal_softmax(G, W, Wl, D, L):
    q = rand_bf16((G, W, D), 900 + L)
    k = rand_bf16((L, D), 901 + L)
    scale = 0.37
    c, m, l = orc.unit_colsum(q, k, scale=scale, local_window=Wl)
    qf, kf = q.double().numpy(), k.double().numpy()
    want = np.zeros(L)
    for g in range(G):
        for i in range(W):
            vis = _visible(i, Wl, L)
            logits = [scale * sum(qf[g, i, d] * kf[j, d] for d in range(D)) for j in range(vis)]
            den = sum(math.exp(x) for x in logits)
            for j in range(vis):
                want[j] += math.exp(logits[j]) / den
            r = g * W + i
            assert m[r] == pytest.approx(max(logits), rel=1e-14, abs=1e-14)
            assert l[r] == pytest.approx(sum(math.exp(x - max(logits)) for x in logits), rel=1e-13)
    np.testing.assert_allclose(c, want, rtol=1e-13, atol=1e-15)


def test_local_window_against_torch_masked_softmax():
    G, W, Wl, D, L = 4, 16, 8, 32, 300
    q, k = rand_bf16((G, W, D), 77), rand_bf16((L, D), 78)
    scale = 1.0 / math.sqrt(D)
    c, _, _ = orc.unit_colsum(q, k, local_window=Wl)
    s = (q.double().reshape(G * W, D) @ k.double().T) * scale
    mask = torch.zeros_like(s, dtype=torch.bool)
    for r in range(G * W):
        mask[r, _visible(r % W, Wl, L):] = True
    want = torch.softmax(s.masked_fill(mask, -float("inf")), dim=-1).sum(0).numpy()
    np.testing.assert_allclose(c, want, rtol=1e-12, atol=1e-15)
    assert c.sum() == pytest.approx(G * W, rel=1e-12)       # every row still sums to one
    # the last key is seen by the lookahead rows and by the last local query of each head only
    assert c[L - 1] < (W - Wl + 1) * G


def test_local_window_zero_is_the_plain_window_and_identical_keys_closed_form():
    G, W, D, L = 2, 6, 16, 40
    q, k = rand_bf16((G, W, D), 5), rand_bf16((L, D), 6)
    a, _, _ = orc.unit_colsum(q, k)
    b, _, _ = orc.unit_colsum(q, k, local_window=0)
    assert (a == b).all()
    # identical keys: a row spreads its weight evenly over the keys it sees
    Wl = 4
    kk = k[:1].expand(L, D).contiguous()
    c, _, _ = orc.unit_colsum(q, kk, local_window=Wl)
    want = np.zeros(L)
    for i in range(W):
        vis = _visible(i, Wl, L)
        want[:vis] += G / vis
    np.testing.assert_allclose(c, want, rtol=1e-13)


def test_local_window_evict_scores_and_tail():
    NL, Bt, Hq, Hkv, D, L, W, Wl, kernel, B = 1, 2, 4, 2, 16, 64, 6, 3, 3, 20
    g = torch.Generator().manual_seed(12)
    q = bf16(torch.randn((NL, Bt, Hq, W, D), generator=g))
    k = bf16(torch.randn((NL, Bt, Hkv, L, D), generator=g))
    v = bf16(torch.randn((NL, Bt, Hkv, L, D), generator=g))
    R = W
    out = orc.evict(q, k, v, R, kernel, B, local_window=Wl, want_colsum=True)
    G = Hq // Hkv
    for b in range(Bt):
        for h in range(Hkv):
            c, _, _ = orc.unit_colsum(q[0, b, h * G:(h + 1) * G], k[0, b, h], local_window=Wl)
            np.testing.assert_allclose(out["colsum"][0, b, h], c, rtol=1e-14)
            np.testing.assert_allclose(out["scores"][0, b, h], orc.pool(c, L - R, kernel), rtol=1e-14)
            assert out["idx"][0, b, h][B - R:].tolist() == list(range(L - R, L))


# ---------------------------------------------------------------- recall of two index sets (Eq. 1-3)
def test_recall_hand_cases_and_numpy_intersection():
    assert orc.recall([1, 2, 3], [4, 5, 6]) == (0.0, 0)
    assert orc.recall([7, 3, 5], [3, 5, 7]) == (1.0, 3)
    r, n = orc.recall([0, 2, 4, 6, 8], [1, 2, 3, 4])
    assert n == 2 and r == pytest.approx(0.5)
    rng = np.random.default_rng(8)
    for B, L in ((16, 40), (300, 1000), (64, 64)):
        a = rng.permutation(L)[:B]
        b = rng.permutation(L)[:B]
        r, n = orc.recall(a, b)
        assert n == len(np.intersect1d(a, b)) and r == pytest.approx(n / B)
    # selections from the same scores at nested budgets: the smaller set is recalled in full
    p = rng.random(500)
    small, big = orc.select(p, 500, 0, 50), orc.select(p, 500, 0, 200)
    assert orc.recall(big, small) == (1.0, 50)
    assert orc.recall(small, big)[1] == 50


# ---------------------------------------------------------------- maximum pooling
@pytest.mark.parametrize("kernel", [1, 3, 5, 7])
def test_max_pool_matches_library_max_pool(kernel):
    g = torch.Generator().manual_seed(43)
    c = torch.rand(61, generator=g, dtype=torch.float64) - 0.3     # some negative values too
    p = orc.pool(c.numpy(), 61, kernel, mode=1)
    want = torch.nn.functional.max_pool1d(c[None, None], kernel, stride=1,
                                          padding=kernel // 2)[0, 0].numpy()
    assert (p == want).all()
    if kernel == 1:
        assert (p == c.numpy()).all()


def test_max_pool_closed_forms_and_tail():
    # a single spike becomes a plateau of width k; an increasing ramp is shifted by k/2
    Ls, kernel = 30, 5
    c = np.zeros(Ls)
    c[11] = 2.5
    p = orc.pool(c, Ls, kernel, mode=1)
    assert p.tolist() == [2.5 if 9 <= j <= 13 else 0.0 for j in range(Ls)]
    ramp = np.arange(Ls, dtype=np.float64)
    p = orc.pool(ramp, Ls, kernel, mode=1)
    assert p.tolist() == [float(min(j + 2, Ls - 1)) for j in range(Ls)]
    # all values negative: padding must not contribute a zero
    p = orc.pool(-1.0 - ramp, Ls, kernel, mode=1)
    assert p.tolist() == [-1.0 - max(j - 2, 0) for j in range(Ls)]
    # the retained tail is invisible to the pool
    c2 = np.concatenate([ramp, np.full(6, 1e9)])
    assert (orc.pool(c2, Ls, kernel, mode=1) == orc.pool(ramp, Ls, kernel, mode=1)).all()


# ---------------------------------------------------------------- Eq. 4 read literally (raw logit sums)
def test_rawsum_is_the_summed_query_times_keys():
    G, W, D, L = 3, 5, 16, 37
    q, k = rand_bf16((G, W, D), 51), rand_bf16((L, D), 52)
    c = orc.unit_rawsum(q, k)
    # another route: add the queries first, then one matrix-vector product
    want = (k.double() @ q.double().reshape(-1, D).sum(0)).numpy() / math.sqrt(D)
    np.testing.assert_allclose(c, want, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(orc.unit_rawsum(q, k, scale=0.5), want * 0.5 * math.sqrt(D),
                               rtol=1e-12, atol=1e-13)
    # odd in K, additive over query heads
    np.testing.assert_allclose(orc.unit_rawsum(q, -k), -c, rtol=1e-15)
    parts = sum(orc.unit_rawsum(q[g:g + 1], k) for g in range(G))
    np.testing.assert_allclose(parts, c, rtol=1e-12, atol=1e-13)


def test_rawsum_hand_example_small_integers():
    # q rows (1,2) and (3,-1); keys (1,0), (0,1), (2,2): row sums of Q K^T = 4, 1, 10; scale 1/2
    q = bf16(torch.tensor([[[1.0, 2.0], [3.0, -1.0]]]))
    k = bf16(torch.tensor([[1.0, 0.0], [0.0, 1.0], [2.0, 2.0]]))
    assert orc.unit_rawsum(q, k, scale=0.5).tolist() == [2.0, 0.5, 5.0]


def test_evict_variants_raw_mode_and_max_pool():
    NL, Bt, Hq, Hkv, D, L, W, kernel, B = 1, 2, 4, 2, 16, 80, 4, 3, 24
    g = torch.Generator().manual_seed(14)
    q = bf16(torch.randn((NL, Bt, Hq, W, D), generator=g))
    k = bf16(torch.randn((NL, Bt, Hkv, L, D), generator=g))
    v = bf16(torch.randn((NL, Bt, Hkv, L, D), generator=g))
    R, G = W, Hq // Hkv
    raw = orc.evict(q, k, v, R, 1, B, score_mode=1)
    mx = orc.evict(q, k, v, R, kernel, B, pool_mode=1, want_colsum=True)
    for b in range(Bt):
        for h in range(Hkv):
            s = (k[0, b, h].double() @ q[0, b, h * G:(h + 1) * G].double().reshape(-1, D).sum(0)) / math.sqrt(D)
            np.testing.assert_allclose(raw["scores"][0, b, h], s[:L - R].numpy(), rtol=1e-12, atol=1e-13)
            top = torch.topk(s[:L - R], B - R).indices.sort().values.tolist()
            assert raw["idx"][0, b, h].tolist() == top + list(range(L - R, L))
            want = torch.nn.functional.max_pool1d(torch.from_numpy(mx["colsum"][0, b, h][None, None, :L - R]),
                                                  kernel, stride=1, padding=kernel // 2)[0, 0].numpy()
            assert (mx["scores"][0, b, h] == want).all()
            assert (mx["idx"][0, b, h] == orc.select(want, L, R, B)).all()


# ---------------------------------------------------------------- prompts of different lengths
def test_seq_lens_equal_separate_runs_on_truncated_prompts():
    NL, Bt, Hq, Hkv, D, L, W, Wl, kernel, B = 2, 3, 4, 2, 16, 96, 6, 2, 5, 20
    g = torch.Generator().manual_seed(15)
    q = bf16(torch.randn((NL, Bt, Hq, W, D), generator=g))
    k = bf16(torch.randn((NL, Bt, Hkv, L, D), generator=g))
    v = bf16(torch.randn((NL, Bt, Hkv, L, D), generator=g))
    lens = np.array([96, 41, 70], np.int32)
    R = W
    # rows beyond a prompt's length hold garbage that must never be read
    k2, v2 = k.clone(), v.clone()
    for b in range(Bt):
        k2[:, b, :, lens[b]:] = float("nan")
        v2[:, b, :, lens[b]:] = float("nan")
    out = orc.evict(q, k2, v2, R, kernel, B, local_window=Wl, seq_lens=lens, want_colsum=True)
    for b in range(Bt):
        Lb = int(lens[b])
        ref = orc.evict(q[:, b:b + 1], k[:, b:b + 1, :, :Lb], v[:, b:b + 1, :, :Lb], R, kernel, B,
                        local_window=Wl, want_colsum=True)
        assert (out["scores"][:, b, :, :Lb - R] == ref["scores"][:, 0]).all()
        assert (out["scores"][:, b, :, Lb - R:] == 0).all()
        assert (out["colsum"][:, b, :, :Lb] == ref["colsum"][:, 0]).all()
        assert (out["colsum"][:, b, :, Lb:] == 0).all()
        assert (out["idx"][:, b] == ref["idx"][:, 0]).all()
        assert (out["idx"][:, b, :, B - R:] == np.arange(Lb - R, Lb)).all()
        assert (out["k_out"][:, b] == ref["k_out"][:, 0]).all()
        assert (out["v_out"][:, b] == ref["v_out"][:, 0]).all()


# ---------------------------------------------------------------- per-layer budgets, streaming keep-set
def test_layer_budgets_identical_keys_closed_form_and_pool_layout():
    # identical keys in every layer: layer n keeps [k/2, k/2 + B_n - R) and the tail, whatever its
    # queries are; the ragged pool holds the layers end to end, [Bt][Hkv][B_n] entries each
    NL, Bt, Hq, Hkv, W, D, L, R, kernel = 3, 2, 4, 2, 4, 16, 64, 4, 7
    budgets = [20, 9, 33]
    q = rand_bf16((NL, Bt, Hq, W, D), 61)
    k = bf16(torch.ones((NL, Bt, Hkv, L, D)) * 0.25)
    v = rand_bf16((NL, Bt, Hkv, L, D), 62)
    out = orc.evict_layers(q, k, v, R, kernel, budgets)
    assert out["idx"].shape == (Bt * Hkv * sum(budgets),)
    row = 0
    vb = v.view(torch.int16).numpy().view(np.uint16)
    for n, B in enumerate(budgets):
        want = list(range(kernel // 2, kernel // 2 + (B - R))) + list(range(L - R, L))
        for b in range(Bt):
            for h in range(Hkv):
                got = out["idx"][row:row + B]
                assert got.tolist() == want, (n, b, h)
                assert (out["v_out"][row:row + B] == vb[n, b, h][got]).all()
                row += B
    assert row == out["idx"].shape[0]


def test_layer_budgets_nest_when_layers_hold_the_same_cache():
    # the same queries and keys in every layer: a smaller budget keeps a subset of a larger one,
    # and each layer equals a uniform run with its own budget
    NL, W, D, L, R, kernel = 3, 4, 32, 200, 4, 5
    q1, k1 = rand_bf16((1, 1, 2, W, D), 63), rand_bf16((1, 1, 1, L, D), 64, 1.5)
    q, k = q1.repeat(NL, 1, 1, 1, 1), k1.repeat(NL, 1, 1, 1, 1)
    budgets = [12, 40, 25]
    out = orc.evict_layers(q, k, None, R, kernel, budgets, fast_select=False)
    sets, row = [], 0
    for B in budgets:
        sets.append(set(out["idx"][row:row + B].tolist()))
        assert len(sets[-1]) == B
        row += B
    assert sets[0] < sets[2] < sets[1]
    uni = orc.evict(q1, k1, None, R, kernel, 25, fast_select=False)
    assert sets[2] == set(uni["idx"][0, 0, 0].tolist())


def test_streaming_keep_set_structure():
    for L, B, ns, Lb in [(100, 10, 4, None), (100, 10, 0, None), (100, 10, 10, None), (100, 30, 4, 57)]:
        idx = orc.streaming_indices(L, B, ns, Lb)
        end = L if Lb is None else Lb
        assert idx.shape == (B,) and (np.diff(idx) > 0).all()
        assert idx[:ns].tolist() == list(range(ns))
        if ns < B:
            assert idx[-1] == end - 1 and idx[ns] == end - (B - ns)
        assert set(idx.tolist()) == set(range(ns)) | set(range(end - (B - ns), end))


# ---------------------------------------------------------------- how the heads of a GQA group combine
def test_per_head_column_sums_against_library_softmax_and_the_group_sum():
    G, W, D, L = 4, 3, 32, 150
    q, k = rand_bf16((G, W, D), 81), rand_bf16((L, D), 82, 1.5)
    ch = orc.unit_colsum_heads(q, k)
    assert ch.shape == (G, L)
    s = (q.double().reshape(G, W, D) @ k.double().T) / math.sqrt(D)   # [G, W, L]
    want = torch.softmax(s, dim=-1).sum(1).numpy()
    np.testing.assert_allclose(ch, want, rtol=1e-12)
    np.testing.assert_allclose(ch.sum(1), W, rtol=1e-12)           # W probability rows per head
    c_all, _, _ = orc.unit_colsum(q, k)                               # the G-head statement
    np.testing.assert_allclose(orc.group_reduce(ch, 0), c_all, rtol=1e-12)
    np.testing.assert_allclose(orc.group_reduce(ch, 1), want.max(0), rtol=1e-12)
    # max <= sum <= G * max, and one head alone is both
    mx, sm = orc.group_reduce(ch, 1), orc.group_reduce(ch, 0)
    assert (mx <= sm).all() and (sm <= G * mx * (1 + 1e-12)).all()
    one = orc.unit_colsum_heads(q[:1], k)
    np.testing.assert_array_equal(orc.group_reduce(one, 1), orc.group_reduce(one, 0))


def test_group_max_mode_selects_on_the_largest_head():
    NL, Bt, Hq, Hkv, W, D, L, R, kernel, B = 1, 2, 6, 2, 4, 32, 120, 4, 5, 30
    q, k, v = rand_bf16((NL, Bt, Hq, W, D), 83), rand_bf16((NL, Bt, Hkv, L, D), 84, 1.5), rand_bf16((NL, Bt, Hkv, L, D), 85)
    out = orc.evict(q, k, v, R, kernel, B, group_mode=1, want_colsum=True, fast_select=False)
    G = Hq // Hkv
    for b in range(Bt):
        for h in range(Hkv):
            s = (q[0, b, h * G:(h + 1) * G].double() @ k[0, b, h].double().T) / math.sqrt(D)
            c = torch.softmax(s, dim=-1).sum(1).max(0).values          # [L]
            np.testing.assert_allclose(out["colsum"][0, b, h], c.numpy(), rtol=1e-12)
            p = torch.nn.functional.avg_pool1d(c[None, None, :L - R], kernel, 1, kernel // 2,
                                               count_include_pad=True)[0, 0]
            np.testing.assert_allclose(out["scores"][0, b, h], p.numpy(), rtol=1e-12)
            order = np.argsort(-out["scores"][0, b, h], kind="stable")[:B - R]
            assert out["idx"][0, b, h].tolist() == sorted(order.tolist()) + list(range(L - R, L))


def test_per_query_head_selection_is_the_step_with_every_head_as_its_own_group():
    # replicate each KV head for its G query heads: the per-head mode on the GQA problem must give
    # what the plain step gives on that expanded problem
    NL, Bt, Hq, Hkv, W, D, L, R, kernel, B = 2, 1, 4, 2, 3, 16, 90, 3, 3, 25
    G = Hq // Hkv
    q, k, v = rand_bf16((NL, Bt, Hq, W, D), 86), rand_bf16((NL, Bt, Hkv, L, D), 87, 2.0), rand_bf16((NL, Bt, Hkv, L, D), 88)
    got = orc.evict(q, k, v, R, kernel, B, group_mode=2, fast_select=False)
    k_rep, v_rep = k.repeat_interleave(G, dim=2), v.repeat_interleave(G, dim=2)
    want = orc.evict(q, k_rep, v_rep, R, kernel, B, fast_select=False)
    assert got["idx"].shape == (NL, Bt, Hq, B)
    np.testing.assert_array_equal(got["idx"], want["idx"])
    np.testing.assert_array_equal(got["scores"], want["scores"])
    np.testing.assert_array_equal(got["k_out"], want["k_out"])
    np.testing.assert_array_equal(got["v_out"], want["v_out"])
    # with per-prompt lengths too
    got = orc.evict(q, k, v, R, kernel, B, group_mode=2, seq_lens=[70])
    want = orc.evict(q, k_rep, v_rep, R, kernel, B, seq_lens=[70])
    np.testing.assert_array_equal(got["idx"], want["idx"])
