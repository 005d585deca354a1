"""Pins for the CPU oracle: every check here compares the oracle with something that is
not the oracle -- a pure-Python brute force of the definition on tiny inputs, a closed
form, a textbook/library routine on a special case, or an invariant of the mathematics
(row-softmax sums, the softmax Lipschitz lemma, permutation equivariance)."""
import math

import numpy as np
import pytest
import torch


def bf16_bits(x: torch.Tensor) -> np.ndarray:
    return x.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def bf16_round(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.bfloat16).double()


def make(n_seq=1, L=1, Hq=2, Hkv=1, R=3, d=4, n=8, seed=0, kscale=1.0):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(n_seq, L, Hq, R, d, generator=g)
    k = torch.randn(L, Hkv, n_seq * n, d, generator=g) * kscale
    return q, k


def brute_scores(q, k, cu, scale, mode="sum", weights=None, causal_window=0, n_window=0):
    """Definition of the importance score, written with Python loops and math.exp only."""
    q = bf16_round(q)
    k = bf16_round(k)
    n_seq, L, Hq, R, d = q.shape
    _, Hkv, T, _ = k.shape
    G = Hq // Hkv
    out = [[[0.0] * T for _ in range(Hkv)] for _ in range(L)]
    for s in range(n_seq):
        b, e = cu[s], cu[s + 1]
        n = e - b
        for l in range(L):
            for g in range(Hq):
                h = g // G
                for r in range(R):
                    vis = n
                    if causal_window and r < n_window:
                        vis = min(n, max(0, n - n_window + r) + 1)
                    logits = []
                    for j in range(vis):
                        acc = 0.0
                        for c in range(d):
                            acc += float(q[s, l, g, r, c]) * float(k[l, h, b + j, c])
                        logits.append(scale * acc)
                    m = max(logits)
                    ex = [math.exp(x - m) for x in logits]
                    Z = sum(ex)
                    w = 1.0 if weights is None else weights[r]
                    for j in range(vis):
                        p = w * ex[j] / Z
                        if mode == "sum":
                            out[l][h][b + j] += p
                        else:
                            out[l][h][b + j] = max(out[l][h][b + j], p)
    return np.array(out)


# ---------------------------------------------------------------- scoring ------------

def test_score_brute_force_tiny(oracle):
    q, k = make(n_seq=2, L=2, Hq=4, Hkv=2, R=3, d=4, n=7, seed=1)
    cu = [0, 7, 14]
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k), cu, n_lookahead=2, n_window=1, scale=0.5)
    want = brute_scores(q, k, cu, 0.5)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)


def test_score_brute_force_ragged_and_max_and_weights(oracle):
    q, k = make(n_seq=3, L=1, Hq=2, Hkv=2, R=4, d=3, n=6, seed=2)
    cu = [0, 5, 6, 16]   # lengths 5, 1, 10 ; two tokens of the packed axis unused
    w = [0.25, 0.5, 1.0, 1.0]
    for mode, omode in (("sum", 0), ("max", 1)):
        got = oracle.spec_score(bf16_bits(q), bf16_bits(k), cu, 2, 2, 0.7,
                                row_weight=np.array(w), mode=omode)
        want = brute_scores(q, k, cu, 0.7, mode=mode, weights=w)
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
        assert np.all(got[:, :, 16:] == 0)


def test_score_causal_window_brute(oracle):
    q, k = make(n_seq=1, L=1, Hq=2, Hkv=1, R=5, d=4, n=9, seed=3)
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 9], n_lookahead=2, n_window=3, scale=1.0,
                            causal_window=True)
    want = brute_scores(q, k, [0, 9], 1.0, causal_window=1, n_window=3)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
    # the first window row sits at prompt position n-3 and must not see the last two keys
    plain = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 9], 2, 3, 1.0)
    assert not np.allclose(got, plain)


def test_score_matches_library_softmax(oracle):
    """Special case that is a library routine: softmax(Q K^T * scale).sum(rows) per KV head."""
    q, k = make(n_seq=1, L=2, Hq=6, Hkv=2, R=5, d=16, n=37, seed=4)
    scale = 1 / math.sqrt(16)
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 37], 3, 2, scale)
    qd, kd = bf16_round(q), bf16_round(k)
    for l in range(2):
        for h in range(2):
            rows = qd[0, l, 3 * h:3 * h + 3].reshape(15, 16)          # the 3 query heads of KV head h
            want = torch.softmax(rows @ kd[l, h].T * scale, dim=-1).sum(0).numpy()
            np.testing.assert_allclose(got[l, h], want, rtol=1e-12)
            wmax = torch.softmax(rows @ kd[l, h].T * scale, dim=-1).max(0).values.numpy()
            gmax = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 37], 3, 2, scale, mode=oracle.MAX)
            np.testing.assert_allclose(gmax[l, h], wmax, rtol=1e-12)


def test_score_two_key_sigmoid_closed_form(oracle):
    """n = 2, d = 1, one row: p0 = 1 / (1 + exp(scale*q*(k1-k0)))."""
    q = torch.tensor([[[[[2.0]]]]])
    k = torch.tensor([[[[0.5], [-1.5]]]])
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 2], 1, 0, 0.75)
    p0 = 1.0 / (1.0 + math.exp(0.75 * 2.0 * (-1.5 - 0.5)))
    np.testing.assert_allclose(got[0, 0], [p0, 1 - p0], rtol=1e-14)


def test_score_closed_forms(oracle):
    q, k = make(L=1, Hq=4, Hkv=2, R=3, d=8, n=10, seed=5)
    M = 2 * 3
    # identical keys -> uniform rows -> M/n everywhere
    k_same = k[:, :, :1].expand(-1, -1, 10, -1).clone()
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k_same), [0, 10], 2, 1, 0.3)
    np.testing.assert_allclose(got, M / 10, rtol=1e-13)
    # zero queries -> uniform
    got = oracle.spec_score(bf16_bits(q * 0), bf16_bits(k), [0, 10], 2, 1, 0.3)
    np.testing.assert_allclose(got, M / 10, rtol=1e-13)
    # single key (degenerate case used in the paper's proofs: A = [1]) -> score = M
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k[:, :, :1]), [0, 1], 2, 1, 0.3)
    np.testing.assert_allclose(got, M, rtol=1e-14)
    # n_lookahead = 0 (the SnapKV special case) is accepted
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 10], 0, 3, 0.3)
    np.testing.assert_allclose(got.sum(-1), M, rtol=1e-13)


def test_score_dominant_key_takes_all_mass(oracle):
    d, n, R = 8, 32, 4
    g = torch.Generator().manual_seed(6)
    q = torch.randn(1, 1, 1, R, d, generator=g)
    q[..., 0] = 4.0
    k = torch.randn(1, 1, n, d, generator=g) * 0.1
    k[0, 0, 17] = 0
    k[0, 0, 17, 0] = 64.0          # logit margin ~ 256 over anything else
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, n], R, 0, 1.0)[0, 0]
    assert abs(got[17] - R) < 1e-12 and got.sum() - got[17] < 1e-12


def test_score_row_sum_invariant_and_weights(oracle):
    """Each softmax row sums to 1, so a KV head's aggregate sums to G * sum(w)."""
    q, k = make(n_seq=2, L=2, Hq=8, Hkv=2, R=6, d=16, n=50, seed=7)
    cu = [0, 50, 100]
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k), cu, 4, 2, 0.25)
    np.testing.assert_allclose(got[:, :, :50].sum(-1), 4 * 6, rtol=1e-13)
    np.testing.assert_allclose(got[:, :, 50:].sum(-1), 4 * 6, rtol=1e-13)
    w = np.array([0.5, 1.0, 1, 1, 1, 1])      # window weights j / n_window of the SpecPC algorithm
    got = oracle.spec_score(bf16_bits(q), bf16_bits(k), cu, 4, 2, 0.25, row_weight=w)
    np.testing.assert_allclose(got[:, :, :50].sum(-1), 4 * w.sum(), rtol=1e-13)


def test_score_scale_invariance_and_key_permutation(oracle):
    q, k = make(L=1, Hq=2, Hkv=1, R=4, d=8, n=20, seed=8)
    base = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 20], 3, 1, 0.5)
    # (4Q, scale/4): exact in bf16 (power of two)
    alt = oracle.spec_score(bf16_bits(q * 4), bf16_bits(k), [0, 20], 3, 1, 0.125)
    np.testing.assert_allclose(alt, base, rtol=1e-13)
    perm = torch.randperm(20, generator=torch.Generator().manual_seed(1))
    alt = oracle.spec_score(bf16_bits(q), bf16_bits(k[:, :, perm]), [0, 20], 3, 1, 0.5)
    np.testing.assert_allclose(alt[0, 0], base[0, 0][perm.numpy()], rtol=1e-12)


def test_score_gqa_is_sum_over_group_heads(oracle):
    """Stacking a group's query heads = adding the single-head scores; also pins head g -> KV head g // G."""
    q, k = make(L=1, Hq=6, Hkv=3, R=3, d=8, n=12, seed=9)
    full = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 12], 2, 1, 0.4)
    for h in range(3):
        acc = 0
        for g in (2 * h, 2 * h + 1):
            acc = acc + oracle.spec_score(bf16_bits(q[:, :, g:g + 1]), bf16_bits(k[:, h:h + 1]),
                                          [0, 12], 2, 1, 0.4)[0, 0]
        np.testing.assert_allclose(full[0, h], acc, rtol=1e-13)


def test_score_ragged_equals_separate_calls(oracle):
    q, k = make(n_seq=3, L=2, Hq=2, Hkv=2, R=2, d=4, n=9, seed=10)
    cu = [0, 4, 13, 27]
    full = oracle.spec_score(bf16_bits(q), bf16_bits(k), cu, 1, 1, 1.0)
    for s in range(3):
        part = oracle.spec_score(bf16_bits(q[s:s + 1]), bf16_bits(k[:, :, cu[s]:cu[s + 1]]),
                                 [0, cu[s + 1] - cu[s]], 1, 1, 1.0)
        np.testing.assert_array_equal(full[:, :, cu[s]:cu[s + 1]], part)


def test_softmax_lipschitz_lemma(oracle):
    """Lemma 1: ||softmax(x) - softmax(y)||_2 <= ||x - y||_inf, checked on the oracle's rows
    (d = 1, q = 1, keys = logits; values on a bf16-exact grid)."""
    g = torch.Generator().manual_seed(11)
    one = torch.ones(1, 1, 1, 1, 1)
    for _ in range(50):
        n = int(torch.randint(2, 40, (1,), generator=g))
        x = (torch.randint(-64, 64, (n,), generator=g).float() / 8).view(1, 1, n, 1)
        y = x + (torch.randint(-8, 9, (n,), generator=g).float() / 16).view(1, 1, n, 1)
        px = oracle.spec_score(bf16_bits(one), bf16_bits(x), [0, n], 1, 0, 1.0)[0, 0]
        py = oracle.spec_score(bf16_bits(one), bf16_bits(y), [0, n], 1, 0, 1.0)[0, 0]
        assert np.linalg.norm(px - py) <= float((x - y).abs().max()) + 1e-12


def test_importance_error_bound_theorem1(oracle):
    """Theorem 1 in its proof's intermediate form: for the mean score s = score / rows,
    ||s - s_hat||_2 <= max_i ||logits_i - logits_hat_i||_inf under a perturbation of the queries."""
    g = torch.Generator().manual_seed(12)
    d, n, R = 8, 24, 5
    q = torch.randn(1, 1, 1, R, d, generator=g)
    dq = torch.randn(1, 1, 1, R, d, generator=g) * 0.05
    k = torch.randn(1, 1, n, d, generator=g)
    scale = 1 / math.sqrt(d)
    s = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, n], R, 0, scale)[0, 0] / R
    sh = oracle.spec_score(bf16_bits(q + dq), bf16_bits(k), [0, n], R, 0, scale)[0, 0] / R
    lg = bf16_round(q)[0, 0, 0] @ bf16_round(k)[0, 0].T * scale
    lgh = bf16_round(q + dq)[0, 0, 0] @ bf16_round(k)[0, 0].T * scale
    bound = float((lg - lgh).abs().max(dim=1).values.max())
    assert np.linalg.norm(s - sh) <= bound + 1e-12


def test_score_strided_keys(oracle):
    """Token-major key layout [L, T, Hkv, d] passed through strides gives the same scores."""
    import ctypes
    q, k = make(L=2, Hq=4, Hkv=2, R=2, d=4, n=6, seed=13)
    base = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, 6], 1, 1, 1.0)
    kt = bf16_bits(k.permute(0, 2, 1, 3).contiguous())       # [L, T, Hkv, d]
    qb = bf16_bits(q)
    cu = np.array([0, 6], dtype=np.int32)
    out = np.zeros((2, 2, 6))
    lib = oracle._load()
    p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    rc = lib.oracle_spec_score(p(qb), p(kt), 6 * 2 * 4, 4, 2 * 4, 1, p(cu), 2, 4, 2, 4, 1, 1, 1.0,
                               None, 0, 0, 6, p(out))
    assert rc == 0
    np.testing.assert_array_equal(out, base)


# ---------------------------------------------------------------- pooling ------------

@pytest.mark.parametrize("k", [1, 3, 7, 13])
def test_pool_matches_library(oracle, k):
    g = torch.Generator().manual_seed(20 + k)
    for n in (1, 2, 5, 64, 101):
        x = torch.rand(n, generator=g, dtype=torch.float64)
        mx = torch.nn.functional.max_pool1d(x.view(1, 1, n), k, 1, k // 2).view(-1).numpy()
        np.testing.assert_array_equal(oracle.pool(x.numpy(), k, oracle.POOL_MAX), mx)
        av = torch.nn.functional.avg_pool1d(x.view(1, 1, n), k, 1, k // 2, count_include_pad=True)
        np.testing.assert_allclose(oracle.pool(x.numpy(), k, oracle.POOL_AVG), av.view(-1).numpy(), rtol=1e-13)
    x = torch.rand(33, generator=g, dtype=torch.float64).numpy()
    if k == 1:
        np.testing.assert_array_equal(oracle.pool(x, 1, oracle.POOL_MAX), x)
    assert np.all(oracle.pool(x, k, oracle.POOL_MAX) >= x)


@pytest.mark.parametrize("k", [2, 4, 8, 32, 64])
def test_pool_even_width_matches_library_first_n_outputs(oracle, k):
    """An even width has no centre: the library's pooling with padding k // 2 and stride 1 yields n + 1
    outputs, and its first n are the windows [j - k/2, j + k/2 - 1] the oracle uses (zero padding and
    divisor k for the average, -inf padding for the maximum)."""
    g = torch.Generator().manual_seed(40 + k)
    for n in (1, 3, k - 1, k, k + 1, 200):
        x = torch.rand(n, generator=g, dtype=torch.float64) - 0.3
        mx = torch.nn.functional.max_pool1d(x.view(1, 1, n), k, 1, k // 2).view(-1)[:n].numpy()
        np.testing.assert_array_equal(oracle.pool(x.numpy(), k, oracle.POOL_MAX), mx)
        av = torch.nn.functional.avg_pool1d(x.view(1, 1, n), k, 1, k // 2, count_include_pad=True).view(-1)[:n].numpy()
        np.testing.assert_allclose(oracle.pool(x.numpy(), k, oracle.POOL_AVG), av, rtol=1e-12, atol=1e-15)


def test_pool_brute_window(oracle):
    x = np.array([0.1, 0.9, 0.2, 0.3, 0.0, 0.0, 0.0, 0.0, 0.5, 0.4])
    got = oracle.pool(x, 7, oracle.POOL_MAX)
    want = [max(x[max(0, j - 3):j + 4]) for j in range(10)]
    np.testing.assert_array_equal(got, want)
    assert got[4] == 0.9 and got[5] == 0.5 and got[9] == 0.5     # reach is exactly 3 on each side


# ---------------------------------------------------------------- selection ----------

def brute_topk(pooled, c):
    order = sorted(range(len(pooled)), key=lambda j: (-pooled[j], j))
    return sorted(order[:c])


def test_topk_brute_force_with_ties(oracle):
    g = np.random.default_rng(30)
    L, H, n, C = 2, 3, 40, 9
    scores = g.integers(0, 6, size=(L, H, n)).astype(np.float64) / 4     # many exact ties
    idx, cnt, pooled, th = oracle.pool_topk(scores, [0, n], oracle.POOL_MAX, 3, C)
    for l in range(L):
        for h in range(H):
            pv = [max(scores[l, h, max(0, j - 1):j + 2]) for j in range(n)]
            assert list(idx[0, l, h]) == brute_topk(pv, C)
            assert cnt[0, l, h] == C
            assert th[0, l, h] == sorted(pv, reverse=True)[C - 1]
            sel = set(idx[0, l, h])
            assert min(pv[j] for j in sel) >= max(pv[j] for j in range(n) if j not in sel)


def test_topk_lower_index_wins_ties(oracle):
    scores = np.zeros((1, 1, 10))
    scores[0, 0, [2, 5, 8]] = 1.0
    idx, cnt, _, _ = oracle.pool_topk(scores, [0, 10], oracle.POOL_MAX, 1, 2)
    assert list(idx[0, 0, 0]) == [2, 5]
    idx, _, _, _ = oracle.pool_topk(scores, [0, 10], oracle.POOL_MAX, 1, 5)
    assert list(idx[0, 0, 0]) == [0, 1, 2, 5, 8]


def test_topk_forced_tail_and_short_sequences(oracle):
    g = np.random.default_rng(31)
    scores = g.random((1, 1, 30))
    cu = [0, 20, 23, 30]
    idx, cnt, pooled, _ = oracle.pool_topk(scores, cu, oracle.POOL_MAX, 3, 8, n_forced_tail=4)
    # sequence 0: 16 eligible, 4 best of them + forced {16..19}
    pv = [max(scores[0, 0, max(0, j - 1):min(16, j + 2)]) for j in range(16)]     # pooling never reads the tail
    assert list(idx[0, 0, 0]) == brute_topk(pv, 4) + [16, 17, 18, 19]
    # sequence 1: 3 tokens, all forced, padded with -1
    assert list(idx[1, 0, 0]) == [0, 1, 2, -1, -1, -1, -1, -1] and cnt[1, 0, 0] == 3
    # sequence 2: 7 tokens: 3 eligible (all kept) + 4 forced
    assert list(idx[2, 0, 0]) == [0, 1, 2, 3, 4, 5, 6, -1] and cnt[2, 0, 0] == 7


def test_topk_planted_heavy_hitters_selected(oracle):
    """Planted heavy keys dominate the attention mass and must be in the keep set."""
    from paper_2506_08373_b200 import workloads as W
    w = W.CONFIGS[0]
    q, k, _ = W.gen_layers(w, [0], want_v=False)
    sc = oracle.spec_score(bf16_bits(q), bf16_bits(k), W.cu_seqlens(w), w.n_lookahead, w.n_window, w.scale)
    idx, cnt, pooled, th = oracle.pool_topk(sc, W.cu_seqlens(w), oracle.POOL_MAX, w.pool_k, w.c_max)
    pos = W.planted_positions(w, 0, 0, w.n_in).numpy()
    for h in range(w.n_kv_heads):
        sel = set(idx[0, 0, h])
        assert 0 in sel                                   # attention sink
        assert set(pos[h]).issubset(sel)
        assert pooled[0, h, pos[h]].min() > 4 * th[0, 0, h]
    np.testing.assert_allclose(sc.sum(-1), w.group * w.rows, rtol=1e-12)


# ---------------------------------------------------------------- compaction ---------

def test_compact_is_fancy_indexing(oracle):
    g = np.random.default_rng(40)
    L, H, T, d, C = 2, 2, 25, 8, 6
    src = g.integers(0, 65536, size=(L, H, T, d)).astype(np.uint16)
    cu = [0, 10, 25]
    idx = np.full((2, L, H, C), -1, dtype=np.int32)
    for s, n in enumerate((10, 15)):
        for l in range(L):
            for h in range(H):
                idx[s, l, h, :5] = np.sort(g.choice(n, 5, replace=False))
    out = oracle.compact(src, cu, idx)
    for s in range(2):
        for l in range(L):
            for h in range(H):
                np.testing.assert_array_equal(out[s, l, h, :5], src[l, h, cu[s] + idx[s, l, h, :5]])
                assert np.all(out[s, l, h, 5] == 0)
    bt = np.array([[3, 0], [1, 2]], dtype=np.int32)
    paged = oracle.compact(src, cu, idx, block_table=bt, page_size=4, n_pages=4)
    for s in range(2):
        for c in range(C):
            np.testing.assert_array_equal(paged[:, bt[s, c // 4], :, c % 4], out[s, :, :, c])
    assert np.all(paged[:, bt[0, 1], :, 2:] == 0xFFFF)     # slots past c_max are untouched


# ---------------------------------------------------------------- SpecPC -------------

def brute_keep(scores, n, c, nb, k, forced=0, reduce="sum"):
    e = n - forced
    t = scores[:, :, :e].sum((0, 1)) if reduce == "sum" else scores[:, :, :e].max((0, 1))
    pv = [max(t[max(0, j - k // 2):min(e, j + k // 2 + 1)]) for j in range(e)]
    top = brute_topk(pv, min(c, e))
    keep = set(range(e, n))
    for i in top:
        keep.update(range(max(0, i - nb), min(e - 1, i + nb) + 1))
    return sorted(keep), top


def test_specpc_brute_force(oracle):
    g = np.random.default_rng(50)
    L, H, n = 3, 2, 60
    scores = g.random((L, H, n)) ** 4
    for red, rname in ((oracle.SUM, "sum"), (oracle.MAX, "max")):
        for nb, forced in ((0, 0), (2, 0), (3, 5)):
            keep, n_keep, tok, th = oracle.specpc_select(scores, [0, n], red, oracle.POOL_MAX, 3, 6, nb, forced)
            want, top = brute_keep(scores, n, 6, nb, 3, forced, rname)
            got = list(keep[0, :n_keep[0]])
            assert got == want
            assert np.all(keep[0, n_keep[0]:] == -1)
            if nb == 0 and forced == 0:
                assert got == top                                    # no neighbours: exactly the top-C set
            assert set(top).issubset(got)
            assert all(any(abs(j - i) <= nb for i in top) or j >= n - forced for j in got)


def test_specpc_planted_neighbourhoods_kept(oracle):
    from paper_2506_08373_b200 import workloads as W
    w = W.CONFIGS[3].replace(n_layers=2, n_in=4096, c_max=512, n_planted=8)
    q, k, _ = W.gen_layers(w, [0, 1], want_v=False)
    sc = oracle.spec_score(bf16_bits(q), bf16_bits(k), [0, w.n_in], w.n_lookahead, w.n_window, w.scale)
    keep, n_keep, _, _ = oracle.specpc_select(sc, [0, w.n_in], oracle.SUM, oracle.POOL_MAX, w.pool_k,
                                              w.c_max, w.n_neighbor)
    got = set(keep[0, :n_keep[0]])
    assert list(keep[0, :n_keep[0]]) == sorted(got)
    for p in W.planted_positions(w, 0, 0, w.n_in)[0].tolist():
        assert set(range(max(0, p - 8), min(w.n_in - 1, p + 8) + 1)).issubset(got)


# ---------------------------------------------------------------- geometry -----------

def test_config_geometry_matches_paper_constants():
    import os
    from paper_2506_08373_b200 import workloads as W
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                a, b = line.split("=")
                vals[a.strip()] = b.strip()
    w = W.CONFIGS[2]
    kv_bytes = w.n_in * w.n_layers * w.n_kv_heads * w.head_dim * 2 * 2
    assert kv_bytes == 16 * 2 ** 30 and kv_bytes > int(vals["kv_cache_bytes_llama31_8b_128k_min"])
    for c in (W.CONFIGS[1], W.CONFIGS[2], W.CONFIGS[4]):
        assert c.n_window == int(vals["speckv_n_window"]) and c.pool_k == int(vals["speckv_pool_k"])
    assert W.CONFIGS[1].n_lookahead == int(vals["latency_n_lookahead"])
    assert W.CONFIGS[3].n_window == int(vals["specpc_n_window"])
    lens = W.seq_lens(W.CONFIGS[4])
    assert len(lens) == 16 and min(lens) >= 4096 and max(lens) <= 65536


def test_gather_tokens_is_fancy_indexing_packed(oracle):
    """Prompt compression (Section 4.3): kept rows of every sequence, packed back to back."""
    rng = np.random.default_rng(21)
    L, H, d = 2, 3, 8
    cu = [0, 5, 5, 17]
    src = rng.integers(0, 65535, size=(L, H, 17, d)).astype(np.uint16)
    keep = np.array([[0, 2, 4, -1], [-1, -1, -1, -1], [1, 3, 10, 11]], dtype=np.int32)
    n_keep = np.array([3, 0, 4], dtype=np.int32)
    dst, cu_out = oracle.gather_tokens(src, cu, keep, n_keep, 9)
    assert list(cu_out) == [0, 3, 3, 7]
    want = np.concatenate([src[:, :, [0, 2, 4], :], src[:, :, [6, 8, 15, 16], :]], axis=2)
    np.testing.assert_array_equal(dst[:, :, :7], want)
    assert (dst[:, :, 7:] == 0xFFFF).all()


def test_specpc_printed_order_two_stage_pool(oracle):
    """Algorithm 2 lines 8-10 as printed: AvgPool1D(k), MaxPool1D(n_neighbor), top-C_max union window, so
    exactly C_max + n_window tokens survive; checked against the two pooling steps done by hand."""
    rng = np.random.default_rng(33)
    L, H, n, k, nb, c_max, win = 3, 2, 200, 5, 7, 20, 6
    scores = rng.random((L, H, n))
    keep, n_keep, tok, th = oracle.specpc_select(scores, [0, n], oracle.MAX, oracle.POOL_AVG_THEN_MAX, k, c_max, nb, win)
    e = n - win
    t = scores.max(axis=(0, 1))[:e]
    avg = np.array([t[max(0, j - k // 2): min(e, j - k // 2 + k)].sum() / k for j in range(e)])
    mx = np.array([avg[max(0, j - nb // 2): min(e, j - nb // 2 + nb)].max() for j in range(e)])
    np.testing.assert_allclose(tok[:e], mx, rtol=1e-12)
    order = sorted(range(e), key=lambda j: (-mx[j], j))[:c_max]
    want = sorted(order) + list(range(e, n))
    assert n_keep[0] == c_max + win
    assert keep[0, :n_keep[0]].tolist() == want
    # widths of one reduce it to the plain selection
    k1, n1, _, _ = oracle.specpc_select(scores, [0, n], oracle.MAX, oracle.POOL_AVG_THEN_MAX, 1, c_max, 1, win)
    k2, n2, _, _ = oracle.specpc_select(scores, [0, n], oracle.MAX, oracle.POOL_MAX, 1, c_max, 0, win)
    np.testing.assert_array_equal(k1, k2)
