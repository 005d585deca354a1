"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Scores within 2e-3 relative + 1e-6 absolute; index sets identical outside the
tolerance band around the weakest selected score; index work on given scores and the gather
bit-exact."""
import numpy as np
import pytest
import torch

from util import Gpu, assert_index_sets_match, assert_scores_close, bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2506_08373_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


@pytest.fixture(scope="module")
def W():
    from paper_2506_08373_b200 import workloads
    return workloads


def small(W, **kw):
    base = W.CONFIGS[1].replace(n_layers=2, n_in=1000, c_max=64, seed=11)
    return base.replace(**kw)


SCORE_CASES = {
    "c0_tiny": lambda W: (W.CONFIGS[0], [0]),
    "d128_M384_ragged_tail": lambda W: (small(W), [0, 1]),
    "d128_M640": lambda W: (small(W, n_lookahead=128, n_in=2500, seed=12), [0]),
    "d64_M512": lambda W: (W.CONFIGS[3].replace(n_in=3000, n_layers=2, c_max=300, n_planted=8), [0, 1]),
    "d64_M5_one_head": lambda W: (small(W, head_dim=64, n_q_heads=2, n_kv_heads=2, n_lookahead=3, n_window=2,
                                        zipf_bias=False, n_in=777), [0]),
    "d128_M21": lambda W: (small(W, n_q_heads=6, n_kv_heads=2, n_lookahead=4, n_window=3, n_in=300), [0, 1]),
    # more query rows than stay resident in shared memory: scored in several groups of rows
    "d128_M800_two_row_groups": lambda W: (small(W, n_lookahead=168, n_in=1500), [0]),
    "d128_G8_M1536_three_row_groups": lambda W: (small(W, n_q_heads=16, n_kv_heads=2, n_lookahead=160, n_in=700), [0, 1]),
    "d64_M1400_two_row_groups": lambda W: (small(W, head_dim=64, n_lookahead=318, n_in=900), [0]),
    "snapkv_no_lookahead": lambda W: (small(W, n_lookahead=0, n_in=513), [0]),
    "single_key": lambda W: (small(W, n_in=1, zipf_bias=False, planted="singletons", n_planted=0), [0]),
    "ragged_batch": lambda W: (W.CONFIGS[4].replace(n_layers=2, n_seq=7, len_lo=1, len_hi=900, c_max=64), [0, 1]),
}


@pytest.mark.parametrize("case", sorted(SCORE_CASES))
def test_score_parity(B, W, oracle, case):
    w, layers = SCORE_CASES[case](W)
    g = Gpu(B, W, w, layers)
    got = g.score().cpu().numpy()
    ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale)
    assert_scores_close(got, ref, g.cu)
    # each softmax row sums to one: the aggregate of a KV head sums to the number of stacked rows
    for s in range(w.n_seq):
        if g.cu[s + 1] > g.cu[s]:
            np.testing.assert_allclose(got[:, :, g.cu[s]:g.cu[s + 1]].astype(np.float64).sum(-1),
                                       w.group * w.rows, rtol=1e-4)


def test_score_ragged_with_empty_and_tile_edge_lengths(B, W, oracle):
    w = W.CONFIGS[4].replace(n_layers=1, n_seq=8, c_max=32)
    lens = [1, 127, 128, 129, 0, 700, 256, 5]
    g = Gpu.__new__(Gpu)
    g.B, g.w, g.L = B, w, 1
    T = sum(lens)
    gen = torch.Generator().manual_seed(5)
    g.q = torch.randn(8, 1, w.n_q_heads, w.rows, w.head_dim, generator=gen).to(torch.bfloat16).cuda()
    g.k = torch.randn(1, w.n_kv_heads, T, w.head_dim, generator=gen).to(torch.bfloat16).cuda()
    g.v = None
    g.cu = [0] + list(np.cumsum(lens))
    g.T = T
    g.cu_t = torch.tensor(g.cu, dtype=torch.int32, device="cuda")
    g.pr = B.make_problem(n_layers=1, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                          n_lookahead=w.n_lookahead, n_window=w.n_window, softmax_scale=w.scale, total_tokens=T,
                          n_in=max(lens), n_seq=8, cu_seqlens=g.cu_t, k=g.k)
    g.ws = torch.empty(B.spec_workspace_bytes(g.pr), dtype=torch.uint8, device="cuda")
    g.status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = g.score().cpu().numpy()
    ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale)
    assert_scores_close(got, ref, g.cu)
    idx, cnt = g.topk(torch.from_numpy(got).cuda(), B.POOL_MAX, 7, 32)
    oidx, ocnt, _, _ = oracle.pool_topk(got.astype(np.float64), g.cu, oracle.POOL_MAX, 7, 32)
    np.testing.assert_array_equal(idx.cpu().numpy(), oidx)
    np.testing.assert_array_equal(cnt.cpu().numpy(), ocnt)
    assert list(ocnt[:, 0, 0]) == [1, 32, 32, 32, 0, 32, 32, 5]


def test_score_max_reduce_and_row_weights(B, W, oracle):
    w = small(W, n_in=600)
    g = Gpu(B, W, w, [0])
    rw = torch.linspace(1.0 / w.rows, 1.0, w.rows)
    rw[3] = 0.0
    for reduce in (B.REDUCE_SUM, B.REDUCE_MAX):
        got = g.score(reduce=reduce, row_weight=rw.cuda()).cpu().numpy()
        ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale,
                                row_weight=rw.double().numpy(), mode=reduce)
        assert_scores_close(got, ref, g.cu)
    got = g.score(reduce=B.REDUCE_MAX).cpu().numpy()
    ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale, mode=oracle.MAX)
    assert_scores_close(got, ref, g.cu)
    assert got.max() <= 1.0 + 1e-5
    # the same over several groups of rows (G * R = 840 > 640): weights and the causal window follow the row index
    w = small(W, n_in=700, n_lookahead=170, n_window=40)
    g = Gpu(B, W, w, [0])
    rw = torch.linspace(1.0 / w.rows, 1.0, w.rows)
    for reduce in (B.REDUCE_SUM, B.REDUCE_MAX):
        got = g.score(reduce=reduce, row_weight=rw.cuda(), causal_window=1).cpu().numpy()
        ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale,
                                row_weight=rw.double().numpy(), mode=reduce, causal_window=True)
        assert_scores_close(got, ref, g.cu)


def test_score_causal_window(B, W, oracle):
    """Window row r sees keys up to its own prompt position only (the model's causal mask)."""
    cases = [small(W, n_in=600), small(W, n_in=257, n_window=40, n_lookahead=3),
             small(W, n_in=20, n_window=32, n_lookahead=5),            # window longer than the prompt
             W.CONFIGS[4].replace(n_layers=1, n_seq=5, len_lo=1, len_hi=700, c_max=16)]
    for w in cases:
        g = Gpu(B, W, w, [0])
        for reduce in (B.REDUCE_SUM, B.REDUCE_MAX):
            got = g.score(reduce=reduce, causal_window=1).cpu().numpy()
            ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale, mode=reduce,
                                    causal_window=True)
            assert_scores_close(got, ref, g.cu)
    # the mask changes the result where it should
    w = cases[0]
    g = Gpu(B, W, w, [0])
    a, b = g.score(causal_window=0), g.score(causal_window=1)
    assert not torch.equal(a[..., -w.n_window:], b[..., -w.n_window:])
    assert torch.allclose(a.sum(-1), b.sum(-1), rtol=1e-4)              # rows still sum to one


def test_score_seeded_random_geometry(B, W, oracle):
    """Seeded sweep over GQA group sizes, row counts, head sizes, single and ragged batches, both
    reductions, the causal window and row weights, each against the oracle."""
    rng = np.random.default_rng(77)
    for case in range(16):
        hkv = int(rng.choice([1, 2]))
        group = int(rng.choice([1, 2, 3, 4, 7]))
        kw = dict(head_dim=int(rng.choice([64, 128])), n_kv_heads=hkv, n_q_heads=hkv * group,
                  n_lookahead=int(rng.integers(0, 41)), n_window=int(rng.integers(1, 41)), seed=100 + case,
                  zipf_bias=bool(case % 2), n_planted=4)
        if case % 3 == 0:
            w = W.CONFIGS[4].replace(n_layers=1, n_seq=int(rng.integers(2, 5)), len_lo=0, len_hi=int(rng.integers(1, 700)),
                                     c_max=8, **kw)
        else:
            w = small(W, n_layers=1, n_in=int(rng.choice([1, 5, 127, 128, 129, 255, 257, 700, 1500])), **kw)
        g = Gpu(B, W, w, [0])
        reduce = int(case % 2)
        causal = bool((case // 2) % 2)
        rw = None
        if case % 4 == 3:
            rw = torch.from_numpy(rng.random(w.rows).astype(np.float32) + 0.05)
        got = g.score(reduce=reduce, causal_window=int(causal), row_weight=None if rw is None else rw.cuda()).cpu().numpy()
        ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale, mode=reduce,
                                causal_window=causal, row_weight=None if rw is None else rw.double().numpy())
        assert_scores_close(got, ref, g.cu)


def test_score_token_major_key_layout_and_reproducibility(B, W, oracle):
    w = small(W, n_in=900)
    g = Gpu(B, W, w, [0, 1])
    base = g.score()
    again = g.score()
    assert torch.equal(base, again), "scores must be bit-reproducible run to run"
    kt = g.k.permute(0, 2, 1, 3).contiguous()               # memory order [L, T, Hkv, d]
    view = kt.permute(0, 2, 1, 3)                           # logical [L, Hkv, T, d] with token-major strides
    g.pr = B.make_problem(n_layers=2, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                          n_lookahead=w.n_lookahead, n_window=w.n_window, softmax_scale=w.scale,
                          total_tokens=g.T, n_in=w.n_in, k=view)
    g.k = view
    assert torch.equal(g.score(), base)


def test_score_wide_gqa_group_in_five_row_groups(B, W, oracle):
    w = small(W, n_q_heads=64, n_kv_heads=2, n_in=400)     # 32 * 96 = 3072 query rows per KV head
    g = Gpu(B, W, w, [0])
    got = g.score().cpu().numpy()
    ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale)
    assert_scores_close(got, ref, g.cu)
    np.testing.assert_allclose(got.astype(np.float64).sum(-1), w.group * w.rows, rtol=1e-4)


# ------------------------------------------------------------------ selection ---------

def run_topk_case(B, W, oracle, scores, cu, pool, k, c_max, forced, exact=True):
    """spec_pool_topk on given scores against the oracle, twice: without a workspace (the selection that keeps
    a unit resident in a thread-block cluster) and with one (the streaming selection, where it applies)."""
    L, H, T = scores.shape
    cu_t = torch.tensor(cu, dtype=torch.int32, device="cuda") if len(cu) > 2 else None   # must outlive the call
    pr = B.make_problem(n_layers=L, n_q_heads=H, n_kv_heads=H, head_dim=128, n_lookahead=1, n_window=0,
                        softmax_scale=1.0, total_tokens=T, n_in=int(max(np.diff(cu))), n_seq=len(cu) - 1,
                        cu_seqlens=cu_t)
    oidx, ocnt, pooled, th = oracle.pool_topk(scores.astype(np.float64), cu, pool, k, c_max, forced)
    scores_t = torch.from_numpy(scores).cuda()
    ws = torch.empty(max(B.spec_workspace_bytes(pr), 16), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for workspace in (None, ws):
        idx = torch.full((len(cu) - 1, L, H, c_max), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((len(cu) - 1, L, H), -7, dtype=torch.int32, device="cuda")
        B.spec_pool_topk(pr, scores_t, pool, k, c_max, forced, idx, cnt, workspace=workspace, status_word=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        np.testing.assert_array_equal(cnt.cpu().numpy(), ocnt)
        if exact:
            np.testing.assert_array_equal(idx.cpu().numpy(), oidx)
        else:
            gi = idx.cpu().numpy()
            for s in range(len(cu) - 1):
                for l in range(L):
                    for h in range(H):
                        nf = min(forced, cu[s + 1] - cu[s])
                        e = cu[s + 1] - cu[s] - nf
                        ge, oe = gi[s, l, h], oidx[s, l, h]
                        assert_index_sets_match(ge[(ge >= 0) & (ge < e)], oe[(oe >= 0) & (oe < e)],
                                                pooled[l, h, cu[s]:cu[s + 1]], th[s, l, h])


def test_topk_exact_with_ties_runs_and_forced_tail(B, W, oracle):
    rng = np.random.default_rng(1)
    # heavy ties: few distinct values, max-pool makes runs of equal keys
    scores = (rng.integers(0, 5, size=(2, 3, 5000)) / 8).astype(np.float32)
    run_topk_case(B, W, oracle, scores, [0, 5000], 0, 7, 256, 0)
    run_topk_case(B, W, oracle, scores, [0, 5000], 0, 7, 256, 32)
    run_topk_case(B, W, oracle, scores, [0, 1200, 1200, 1210, 5000], 0, 7, 100, 16)
    run_topk_case(B, W, oracle, np.zeros((1, 1, 3000), np.float32), [0, 3000], 0, 7, 500, 0)   # all equal
    scores = rng.random((2, 2, 4097)).astype(np.float32) ** 8
    for k in (1, 3, 7, 13):
        run_topk_case(B, W, oracle, scores, [0, 4097], 0, k, 1024, 0)
    run_topk_case(B, W, oracle, scores, [0, 4097], 0, 7, 4096, 0)       # one position dropped
    run_topk_case(B, W, oracle, scores, [0, 4097], 0, 7, 4097, 0)       # keep all
    run_topk_case(B, W, oracle, scores, [0, 4097], 0, 7, 5000, 7)       # c_max > n : -1 padding
    run_topk_case(B, W, oracle, scores, [0, 4097], 0, 7, 1, 0)
    run_topk_case(B, W, oracle, scores, [0, 4097], 0, 7, 64, 64)        # nothing but the forced tail


def test_topk_streaming_regime_long_sequence(B, W, oracle):
    rng = np.random.default_rng(2)
    scores = rng.random((1, 2, 70001)).astype(np.float32) ** 6
    scores[0, 0, ::1000] = 0.75                                          # ties at the top
    run_topk_case(B, W, oracle, scores, [0, 70001], 0, 7, 2048, 0)
    run_topk_case(B, W, oracle, scores, [0, 70001], 0, 7, 2048, 32)


def test_topk_clustered_keys_large_budget_and_odd_offsets(B, W, oracle):
    rng = np.random.default_rng(7)
    # every heavy key inside the range one warp streams: its candidate list overflows and is re-filtered
    scores = (rng.random((1, 2, 100000)).astype(np.float32) * 0.01)
    scores[:, :, 1000:4000] += rng.random((1, 2, 3000)).astype(np.float32) + 1.0
    run_topk_case(B, W, oracle, scores, [0, 100000], 0, 7, 2048, 0)
    # ascending scores: every new position is a new maximum
    ramp = np.linspace(0.0, 1.0, 60000, dtype=np.float32)[None, None, :].repeat(2, axis=1)
    run_topk_case(B, W, oracle, ramp, [0, 60000], 0, 7, 1024, 0)
    # a budget beyond the candidate lists: generic selection
    scores = rng.random((1, 2, 50000)).astype(np.float32) ** 3
    run_topk_case(B, W, oracle, scores, [0, 50000], 0, 7, 6000, 0)
    # sequence starts that are not multiples of four elements (16-byte loads need realignment)
    scores = rng.random((2, 2, 4099 + 33333 + 12345)).astype(np.float32) ** 5
    run_topk_case(B, W, oracle, scores, [0, 4099, 4099 + 33333, 4099 + 33333 + 12345], 0, 7, 512, 0)
    run_topk_case(B, W, oracle, scores, [0, 4099, 4099 + 33333, 4099 + 33333 + 12345], 0, 7, 512, 40)


def test_topk_large_keys_crowded_into_the_part_swept_first(B, W, oracle):
    """The sweep raises its floor early from the part of the unit seen so far.  Here that part (the first
    256 positions of each of the 16 ranges the warps stream) holds a third of the large keys, so the early
    floor lands above the final threshold and most winners, met later, fall under it: the kernel must
    notice and still return the exact set."""
    rng = np.random.default_rng(11)
    n, c_max = 100000, 2048
    x = (rng.random((1, 2, n)) * 0.01).astype(np.float32)
    span = 6400                                               # ceil(n / 16 / 256) * 256
    first = np.concatenate([np.arange(w * span, w * span + 256) for w in range(16)])
    first = first[first < n]
    early = rng.choice(first, 1000, replace=False)
    late = rng.choice(np.setdiff1d(np.arange(n), first), 3000, replace=False)
    for h in range(2):
        x[0, h, early] = (10.0 * 2.0 ** (3.0 * rng.random(early.size))).astype(np.float32)
        x[0, h, late] = (10.0 * 2.0 ** (3.0 * rng.random(late.size))).astype(np.float32)
    for k in (1, 7):
        run_topk_case(B, W, oracle, x, [0, n], 0, k, c_max, 0)
    run_topk_case(B, W, oracle, x, [0, n], 0, 7, 512, 0)


def test_topk_seeded_random_shapes_and_special_values(B, W, oracle):
    """Many small seeded cases: lengths around tile and vector edges, budgets from 1 to beyond n, odd
    and even pooling widths, forced tails, and score vectors with negatives, signed zeros, infinities and
    long runs of equal values.  Max-pool selection is exact, ties to the lower position."""
    rng = np.random.default_rng(2024)
    for case in range(48):
        n_seq = int(rng.integers(1, 4))
        lens = [int(rng.choice([0, 1, 2, 7, 31, 127, 128, 129, 1000, int(rng.integers(1, 6000))])) for _ in range(n_seq)]
        if sum(lens) == 0:
            lens[0] = 5
        cu = [0] + list(np.cumsum(lens))
        T = cu[-1] + int(rng.integers(0, 5))                   # a few tokens no sequence covers
        kind = case % 4
        if kind == 0:
            x = rng.standard_normal((2, 2, T)).astype(np.float32)
        elif kind == 1:
            x = (rng.integers(0, 4, size=(2, 2, T)) * 0.25).astype(np.float32)          # long runs of ties
        elif kind == 2:
            x = rng.random((2, 2, T)).astype(np.float32) ** 10
            x[rng.random(x.shape) < 0.02] = np.inf
            x[rng.random(x.shape) < 0.02] = -np.inf
        else:
            x = np.where(rng.random((2, 2, T)) < 0.5, np.float32(0.0), np.float32(-0.0)).astype(np.float32)
            x[rng.random(x.shape) < 0.1] = 1e-30
        k = int(rng.choice([1, 2, 3, 4, 5, 7, 9, 31, 64]))        # even widths: window [j - k/2, j + k/2 - 1]
        c_max = int(rng.choice([1, 2, 16, 100, 1024, max(lens) + 3]))
        forced = int(rng.integers(0, min(c_max, 20) + 1)) if case % 3 == 0 else 0
        run_topk_case(B, W, oracle, x, cu, 0, k, c_max, forced)


def test_topk_avg_pool_within_band(B, W, oracle):
    rng = np.random.default_rng(3)
    scores = rng.random((1, 2, 3000)).astype(np.float32) ** 4
    run_topk_case(B, W, oracle, scores, [0, 3000], 1, 7, 128, 0, exact=False)
    run_topk_case(B, W, oracle, scores, [0, 3000], 1, 13, 128, 8, exact=False)


# ------------------------------------------------------------------ compaction --------

@pytest.mark.parametrize("d", [64, 128])
def test_compact_bit_exact_contiguous_and_paged(B, W, oracle, d):
    rng = np.random.default_rng(4)
    L, H, C = 2, 3, 70
    cu = [0, 300, 300, 1000]
    T = 1000
    def raw():                       # arbitrary bit patterns (NaNs included), except the oracle's 0xFFFF "untouched" mark
        a = rng.integers(-32768, 32767, size=(L, H, T, d)).astype(np.int16)
        a[a == -1] = 7
        return torch.from_numpy(a).view(torch.bfloat16).cuda()
    k, v = raw(), raw()
    idx = np.full((3, L, H, C), -1, dtype=np.int32)
    for s, n in enumerate((300, 0, 700)):
        for l in range(L):
            for h in range(H):
                m = min(n, C - 3)
                idx[s, l, h, :m] = np.sort(rng.choice(n, m, replace=False)) if n else []
    cu_t = torch.tensor(cu, dtype=torch.int32, device="cuda")
    pr = B.make_problem(n_layers=L, n_q_heads=H, n_kv_heads=H, head_dim=d, n_lookahead=1, n_window=0,
                        softmax_scale=1.0, total_tokens=T, n_in=700, n_seq=3, cu_seqlens=cu_t, k=k, v=v)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    idx_t = torch.from_numpy(idx).cuda()
    ko = torch.full((3, L, H, C, d), 1.0, dtype=torch.bfloat16, device="cuda")
    vo = torch.full_like(ko, 1.0)
    B.spec_compact_kv(pr, k, v, idx_t, C, ko, vo, status_word=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    np.testing.assert_array_equal(bits(ko), oracle.compact(bits(k), cu, idx))
    np.testing.assert_array_equal(bits(vo), oracle.compact(bits(v), cu, idx))
    # V left in page-locked host memory: only the selected rows cross the bus
    v_host = v.cpu().pin_memory()
    vo.fill_(1.0)
    B.spec_compact_kv(pr, k, v_host, idx_t, C, ko, vo, status_word=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    np.testing.assert_array_equal(bits(vo), oracle.compact(bits(v), cu, idx))
    # K only
    ko.fill_(1.0)
    B.spec_compact_kv(pr, k, None, idx_t, C, ko, None, status_word=status)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(bits(ko), oracle.compact(bits(k), cu, idx))
    # paged, pages deliberately scattered
    ps, pps = 16, (C + 15) // 16
    n_pages = 3 * pps + 2
    bt = rng.permutation(n_pages)[: 3 * pps].astype(np.int32).reshape(3, pps)
    kp = torch.from_numpy(np.full((L, n_pages, H, ps, d), 0x7FFF, np.int16)).view(torch.bfloat16).cuda()
    vp = kp.clone()
    B.spec_compact_kv(pr, k, v, idx_t, C, kp, vp, block_table=torch.from_numpy(bt).cuda(), page_size=ps,
                      n_pages=n_pages, status_word=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for src, pool in ((k, kp), (v, vp)):
        want = oracle.compact(bits(src), cu, idx, block_table=bt, page_size=ps, n_pages=n_pages)
        want[want == 0xFFFF] = 0x7FFF                               # slots the call must not touch keep their fill
        np.testing.assert_array_equal(bits(pool), want)
    # a page id out of range is skipped and reported, not written
    bad = bt.copy()
    bad[0, 0] = n_pages
    B.spec_compact_kv(pr, k, v, idx_t, C, kp, vp, block_table=torch.from_numpy(bad).cuda(), page_size=ps,
                      n_pages=n_pages, status_word=status)
    torch.cuda.synchronize()
    assert status.item() == B.ERR_BAD_ARG


# ------------------------------------------------------------------ whole path --------

def check_pipeline(B, W, oracle, w, layers, units=None):
    """score -> pool/top-C -> gather on the GPU against the oracle; `units` restricts the oracle to
    sampled (layer, kv head) pairs."""
    g = Gpu(B, W, w, layers)
    scores = g.score()
    idx, cnt = g.topk(scores, B.POOL_MAX, w.pool_k, w.c_max)
    ko = torch.empty((w.n_seq, g.L, w.n_kv_heads, w.c_max, w.head_dim), dtype=torch.bfloat16, device="cuda")
    vo = torch.empty_like(ko)
    bt = None
    if w.page_size:
        bt = W.block_table(w, "cuda")
        n_pages = bt.numel()
        ko = torch.zeros((g.L, n_pages, w.n_kv_heads, w.page_size, w.head_dim), dtype=torch.bfloat16, device="cuda")
        vo = torch.zeros_like(ko)
        B.spec_compact_kv(g.pr, g.k, g.v, idx, w.c_max, ko, vo, block_table=bt, page_size=w.page_size,
                          n_pages=n_pages, status_word=g.status)
    else:
        B.spec_compact_kv(g.pr, g.k, g.v, idx, w.c_max, ko, vo, status_word=g.status)
    torch.cuda.synchronize()
    assert g.status.item() == 0
    G = w.group
    units = units or [(l, h) for l in range(g.L) for h in range(w.n_kv_heads)]
    idx_np, tot_in, tot_out = idx.cpu().numpy(), 0, 0
    for (l, h) in units:
        qs = g.q[:, l:l + 1, h * G:(h + 1) * G]
        ks = g.k[l:l + 1, h:h + 1]
        ref = oracle.spec_score(bits(qs), bits(ks), g.cu, w.n_lookahead, w.n_window, w.scale)
        assert_scores_close(scores[l:l + 1, h:h + 1].cpu().numpy(), ref, g.cu)
        oidx, ocnt, pooled, th = oracle.pool_topk(ref, g.cu, oracle.POOL_MAX, w.pool_k, w.c_max)
        for s in range(w.n_seq):
            a, b = assert_index_sets_match(idx_np[s, l, h], oidx[s, 0, 0], pooled[0, 0, g.cu[s]:g.cu[s + 1]], th[s, 0, 0])
            tot_out += a
            tot_in += b
            n = g.cu[s + 1] - g.cu[s]
            if w.planted != "token" and n >= w.c_max * 4:
                pos = W.planted_positions(w, layers[l], s, n)[h].numpy()
                assert set(pos).issubset(set(idx_np[s, l, h])), "planted heavy hitters must be selected"
        # gather is bit-exact given the GPU's own indices
        gk = oracle.compact(bits(ks), g.cu, idx_np[:, l:l + 1, h:h + 1], None if bt is None else bt.cpu().numpy(),
                            w.page_size, 0 if bt is None else bt.numel())
        gv = oracle.compact(bits(g.v[l:l + 1, h:h + 1]), g.cu, idx_np[:, l:l + 1, h:h + 1],
                            None if bt is None else bt.cpu().numpy(), w.page_size, 0 if bt is None else bt.numel())
        if bt is None:
            np.testing.assert_array_equal(bits(ko[:, l:l + 1, h:h + 1]), gk)
            np.testing.assert_array_equal(bits(vo[:, l:l + 1, h:h + 1]), gv)
        else:
            np.testing.assert_array_equal(bits(ko[l:l + 1, :, h:h + 1]), gk)
            np.testing.assert_array_equal(bits(vo[l:l + 1, :, h:h + 1]), gv)
    return tot_out, tot_in


def test_pipeline_config0_full(B, W, oracle):
    out, inside = check_pipeline(B, W, oracle, W.CONFIGS[0], [0])
    assert out > 0


def test_pipeline_config1_full_size_sampled_units(B, W, oracle):
    w = W.CONFIGS[1]
    check_pipeline(B, W, oracle, w, list(range(w.n_layers)), units=[(0, 0), (13, 5), (31, 7)])


def test_pipeline_config2_full_size_sampled_units(B, W, oracle):
    w = W.CONFIGS[2]
    free, _ = torch.cuda.mem_get_info()
    layers = list(range(w.n_layers)) if free > 40e9 else list(range(4))
    check_pipeline(B, W, oracle, w, layers, units=[(0, 3), (len(layers) - 1, 6)])


def test_pipeline_config4_ragged_paged_sampled_units(B, W, oracle):
    w = W.CONFIGS[4]
    # layers spread over the model (first, middle, last), one sampled KV head of each
    check_pipeline(B, W, oracle, w, [0, 15, 31], units=[(0, 2), (1, 7), (2, 4)])


# ------------------------------------------------------------------ SpecPC ------------

def run_keep(B, pr, scores_t, reduce, pool, k, c_max, nb, forced, cap, n_seq):
    keep = torch.full((n_seq, cap), -7, dtype=torch.int32, device="cuda")
    n_keep = torch.full((n_seq,), -7, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.spec_workspace_bytes(pr), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.specpc_token_select(pr, scores_t, reduce, pool, k, c_max, nb, forced, keep, cap, n_keep, ws, status_word=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return keep.cpu().numpy(), n_keep.cpu().numpy()


def test_specpc_exact_on_dyadic_scores(B, W, oracle):
    """Scores on a dyadic grid sum exactly in fp32, so the keep list must equal the oracle's."""
    rng = np.random.default_rng(6)
    L, H = 4, 2
    cu = [0, 900, 905, 905, 3000]
    scores = (rng.integers(0, 64, size=(L, H, 3000)) / 64).astype(np.float32)
    cu_t = torch.tensor(cu, dtype=torch.int32, device="cuda")
    pr = B.make_problem(n_layers=L, n_q_heads=H, n_kv_heads=H, head_dim=64, n_lookahead=1, n_window=0,
                        softmax_scale=1.0, total_tokens=3000, n_in=2095, n_seq=4, cu_seqlens=cu_t)
    st = torch.from_numpy(scores).cuda()
    for reduce in (0, 1):
        for (c_max, nb, forced, k) in ((64, 8, 0, 7), (64, 0, 0, 7), (50, 3, 16, 3), (2000, 2, 0, 7), (10, 64, 4, 1)):
            cap = 2095
            keep, n_keep = run_keep(B, pr, st, reduce, 0, k, c_max, nb, forced, cap, 4)
            ok, on, _, _ = oracle.specpc_select(scores.astype(np.float64), cu, reduce, 0, k, c_max, nb, forced, cap)
            np.testing.assert_array_equal(n_keep, on)
            np.testing.assert_array_equal(keep, ok)
        # Algorithm 2 lines 8-9 in the printed order (average pool, max pool, then select): power-of-two
        # pool widths keep the fp32 averages exact
        for (c_max, nb, forced, k) in ((64, 8, 0, 4), (100, 1, 16, 8), (30, 5, 64, 1), (2000, 16, 0, 2)):
            cap = 2095
            keep, n_keep = run_keep(B, pr, st, reduce, B.POOL_AVG_THEN_MAX, k, c_max, nb, forced, cap, 4)
            ok, on, _, _ = oracle.specpc_select(scores.astype(np.float64), cu, reduce, oracle.POOL_AVG_THEN_MAX, k,
                                                c_max, nb, forced, cap)
            np.testing.assert_array_equal(n_keep, on)
            np.testing.assert_array_equal(keep, ok)
            lens = np.diff(cu)
            np.testing.assert_array_equal(n_keep, np.minimum(lens, np.minimum(c_max, np.maximum(lens - forced, 0))
                                                             + np.minimum(forced, lens)))


def test_specpc_seeded_random_shapes(B, W, oracle):
    """Seeded sweep of the keep set: ragged batches with empty sequences, both reductions, max pooling
    and the printed average-then-max order, neighbour widths, forced tails; dyadic scores keep the
    fp32 sums and power-of-two averages exact, so the lists must be identical."""
    rng = np.random.default_rng(99)
    for case in range(24):
        L, H = int(rng.integers(1, 5)), int(rng.integers(1, 4))
        n_seq = int(rng.integers(1, 5))
        lens = [int(rng.choice([0, 1, 3, 64, 129, 1000, int(rng.integers(1, 4000))])) for _ in range(n_seq)]
        if sum(lens) == 0:
            lens[-1] = 17
        cu = [0] + list(np.cumsum(lens))
        T = cu[-1]
        scores = (rng.integers(0, 64, size=(L, H, T)) / 64).astype(np.float32)
        cu_t = torch.tensor(cu, dtype=torch.int32, device="cuda")
        pr = B.make_problem(n_layers=L, n_q_heads=H, n_kv_heads=H, head_dim=64, n_lookahead=1, n_window=0,
                            softmax_scale=1.0, total_tokens=T, n_in=max(lens), n_seq=n_seq, cu_seqlens=cu_t)
        reduce = case % 2
        two_stage = case % 3 == 0
        k = int(rng.choice([1, 2, 4, 8])) if two_stage else int(rng.choice([1, 3, 7, 9]))
        c_max = int(rng.choice([1, 5, 64, 300, 5000]))
        nb = int(rng.choice([0, 1, 2, 8, 33]))
        forced = int(rng.integers(0, 40)) if case % 4 == 1 or two_stage else 0
        pool = B.POOL_AVG_THEN_MAX if two_stage else 0
        cap = max(lens)
        keep, n_keep = run_keep(B, pr, torch.from_numpy(scores).cuda(), reduce, pool, k, c_max, nb, forced, cap, n_seq)
        ok, on, _, _ = oracle.specpc_select(scores.astype(np.float64), cu, reduce, oracle.POOL_AVG_THEN_MAX if two_stage else 0,
                                            k, c_max, nb, forced, cap)
        np.testing.assert_array_equal(n_keep, on, err_msg="case %d" % case)
        np.testing.assert_array_equal(keep, ok, err_msg="case %d" % case)


def test_specpc_config3_full(B, W, oracle):
    w = W.CONFIGS[3]
    g = Gpu(B, W, w, list(range(w.n_layers)))
    scores = g.score()
    cap = min(w.n_in, w.c_max * (2 * w.n_neighbor + 1))
    keep, n_keep = run_keep(B, g.pr, scores, B.REDUCE_SUM, B.POOL_MAX, w.pool_k, w.c_max, w.n_neighbor, 0, cap, 1)
    got = keep[0, :n_keep[0]]
    assert np.all(np.diff(got) > 0) and np.all(keep[0, n_keep[0]:] == -1)
    ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale)
    assert_scores_close(scores.cpu().numpy(), ref, g.cu)
    okeep, on, tok, th = oracle.specpc_select(ref, g.cu, oracle.SUM, oracle.POOL_MAX, w.pool_k, w.c_max,
                                              w.n_neighbor, 0, cap)
    ref_keep = set(okeep[0, :on[0]])
    # planted token positions and their +-8 neighbourhoods are kept
    for p in W.planted_positions(w, 0, 0, w.n_in)[0].tolist():
        assert set(range(max(0, p - 8), min(w.n_in - 1, p + 8) + 1)).issubset(set(got))
    # every disagreement with the oracle is explained by a top-C candidate inside the tolerance band
    band = 2e-3 * abs(th[0]) + 1e-6
    near = np.flatnonzero(np.abs(tok - th[0]) <= band)
    for j in set(got) ^ ref_keep:
        assert np.any(np.abs(near - j) <= w.n_neighbor), "keep-list difference at %d outside the band" % j


def test_specpc_paper_settings_from_real_scores(B, W, oracle):
    """Algorithm 2 at the hyper-parameter table's SpecPC column, from the scoring call's own output on a
    draft-shaped problem: max reduction over query rows, window rows weighted j / n_window, the first l_skip = 8
    layers skipped by pointer offset, max over layers and heads, AvgPool(k) then MaxPool(n_neighbor) before the
    selection, the window always kept.  Lists equal the oracle's except for positions whose pooled value lies
    within the score tolerance of the threshold."""
    n_window, l_skip, c_max = 64, 8, 1024
    w = W.CONFIGS[3].replace(n_in=12000, n_layers=12, n_lookahead=1, n_window=n_window, n_planted=32, seed=17)
    g = Gpu(B, W, w, list(range(w.n_layers)))
    rw = torch.cat([torch.arange(1, n_window + 1, dtype=torch.float32) / n_window, torch.ones(w.n_lookahead)])
    scores = g.score(reduce=B.REDUCE_MAX, row_weight=rw.cuda())
    ref = oracle.spec_score(bits(g.q), bits(g.k), g.cu, w.n_lookahead, w.n_window, w.scale,
                            row_weight=rw.double().numpy(), mode=oracle.MAX)
    assert_scores_close(scores.cpu().numpy(), ref, g.cu)
    used = scores[l_skip:]                                       # a view: the call sees layers l_skip.. only
    pr = B.make_problem(n_layers=w.n_layers - l_skip, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                        n_lookahead=w.n_lookahead, n_window=w.n_window, softmax_scale=w.scale, total_tokens=w.n_in, n_in=w.n_in)
    cap = c_max + n_window
    for k, nb in ((64, 64), (32, 32)):
        keep, n_keep = run_keep(B, pr, used, B.REDUCE_MAX, B.POOL_AVG_THEN_MAX, k, c_max, nb, n_window, cap, 1)
        okeep, on, pooled, th = oracle.specpc_select(ref[l_skip:], g.cu, oracle.MAX, oracle.POOL_AVG_THEN_MAX, k, c_max, nb,
                                                     n_window, cap)
        assert n_keep[0] == on[0] == c_max + n_window            # exactly C_max tokens plus the window
        got, want = keep[0, :n_keep[0]], okeep[0, :on[0]]
        assert np.all(np.diff(got) > 0)
        np.testing.assert_array_equal(got[-n_window:], np.arange(w.n_in - n_window, w.n_in))
        band = 2e-3 * abs(th[0]) + 1e-6
        for j in np.setxor1d(got, want):
            assert abs(pooled[j] - th[0]) <= band, "k=%d: position %d decided outside the tolerance band" % (k, j)
    # the single-stage average pool of Algorithm 1 line 10 as printed, on the same real scores
    sc = scores.cpu().numpy()[:2]
    run_topk_case(B, W, oracle, sc, g.cu, oracle.POOL_AVG, 7, 512, n_window, exact=False)
    run_topk_case(B, W, oracle, sc, g.cu, oracle.POOL_AVG, 64, 512, 0, exact=False)
    run_topk_case(B, W, oracle, sc, g.cu, oracle.POOL_MAX, 32, 512, 0)


def test_score_zero_length_prompt_clears_the_output(B, W):
    """n_in = 0 with a non-empty token axis: nothing to score, and the whole output buffer reads as zero."""
    pr = B.make_problem(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=2, n_window=2, softmax_scale=0.125,
                        total_tokens=300, n_in=0)
    q = torch.randn(1, 2, 4, 4, 64, device="cuda").to(torch.bfloat16)
    k = torch.randn(2, 2, 300, 64, device="cuda").to(torch.bfloat16)
    out = torch.full((2, 2, 300), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(B.spec_workspace_bytes(pr), 16), dtype=torch.uint8, device="cuda")
    B.spec_score(pr, q, k, out, ws)
    torch.cuda.synchronize()
    assert torch.count_nonzero(out).item() == 0


# ------------------------------------------------------------------ widening rows -----

def run_vert_case(B, oracle, scores, cu, k, c_max, forced, n_vert):
    """spec_pool_topk_vert against two oracle selections on the same pooled scores."""
    L, H, T = scores.shape
    n_seq = len(cu) - 1
    cu_t = torch.tensor(cu, dtype=torch.int32, device="cuda") if n_seq > 1 else None
    pr = B.make_problem(n_layers=L, n_q_heads=H, n_kv_heads=H, head_dim=128, n_lookahead=1, n_window=0,
                        softmax_scale=1.0, total_tokens=T, n_in=int(max(np.diff(cu))), n_seq=n_seq, cu_seqlens=cu_t)
    s64 = scores.astype(np.float64)
    o_cache, o_cnt, _, _ = oracle.pool_topk(s64, cu, oracle.POOL_MAX, k, c_max, forced)
    # i_vert is the plain top-n_vert of the positions before the forced tail: the oracle gets them as
    # sequences cut at the tail, with the same pooling clipped to that range
    o_vert = np.full((n_seq, L, H, n_vert), -1, dtype=np.int32)
    o_vcnt = np.zeros((n_seq, L, H), dtype=np.int32)
    for s in range(n_seq):
        n = cu[s + 1] - cu[s]
        e = n - min(forced, n)
        if e > 0:
            oi, oc, _, _ = oracle.pool_topk(s64[:, :, cu[s]:cu[s] + e].copy(), [0, e], oracle.POOL_MAX, k, n_vert, 0)
            o_vert[s], o_vcnt[s] = oi[0], oc[0]
    ws = torch.empty(max(B.spec_workspace_bytes(pr), 16), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for workspace in (None, ws):                       # cluster-resident and streaming selection
        idx = torch.full((n_seq, L, H, c_max), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((n_seq, L, H), -7, dtype=torch.int32, device="cuda")
        vidx = torch.full((n_seq, L, H, n_vert), -7, dtype=torch.int32, device="cuda")
        vcnt = torch.full((n_seq, L, H), -7, dtype=torch.int32, device="cuda")
        B.spec_pool_topk_vert(pr, torch.from_numpy(scores).cuda(), B.POOL_MAX, k, c_max, forced, idx, cnt, n_vert, vidx, vcnt,
                              workspace=workspace, status_word=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        np.testing.assert_array_equal(idx.cpu().numpy(), o_cache)
        np.testing.assert_array_equal(cnt.cpu().numpy(), o_cnt)
        np.testing.assert_array_equal(vidx.cpu().numpy(), o_vert)
        np.testing.assert_array_equal(vcnt.cpu().numpy(), o_vcnt)


def test_vertical_and_cache_indices_from_one_sweep(B, W, oracle):
    """Algorithm 1 lines 11 and 13: i_vert = topk(s, n_vert) and i_cache = topk(s, C_max - n_window) + window
    from the same pooled scores, in one call that reads the scores once."""
    rng = np.random.default_rng(21)
    x = rng.random((2, 2, 20000)).astype(np.float32) ** 6
    run_vert_case(B, oracle, x, [0, 20000], 7, 256, 32, 2048)            # the paper's n_vert and window
    run_vert_case(B, oracle, x, [0, 20000], 7, 2048, 0, 256)             # vertical budget below the cache budget
    run_vert_case(B, oracle, x, [0, 20000], 7, 256, 32, 30000)           # n_vert beyond the sequence: all, -1 padded
    ties = (rng.integers(0, 6, size=(1, 3, 9000)) / 4).astype(np.float32)  # long runs of equal pooled values
    run_vert_case(B, oracle, ties, [0, 9000], 7, 300, 16, 1000)
    run_vert_case(B, oracle, ties, [0, 2000, 2000, 2003, 9000], 5, 64, 8, 100)   # ragged, an empty and a tiny sequence
    # from real scores of the scoring call, long enough for a cluster of several CTAs
    w = small(W, n_in=40000, c_max=256)
    g = Gpu(B, W, w, [0])
    sc = g.score().cpu().numpy()
    run_vert_case(B, oracle, sc, g.cu, w.pool_k, 256, w.n_window, 2048)


STRUCTURED = {
    "random": lambda rng, n: rng.random(n) ** 6,
    "rising": lambda rng, n: np.linspace(0.0, 1.0, n),
    "falling": lambda rng, n: np.linspace(1.0, 0.0, n),
    "recency_decay": lambda rng, n: np.exp(-(n - 1 - np.arange(n)) / (n / 12.0)) * (0.5 + rng.random(n)),
    "winners_in_one_sixteenth": lambda rng, n: np.where((np.arange(n) >= 5 * (n // 16)) & (np.arange(n) < 6 * (n // 16)),
                                                         1.0 + rng.random(n), 0.01 * rng.random(n)),
    "few_distinct_values": lambda rng, n: rng.integers(0, 5, n) / 8.0,
}


def test_topk_structured_score_vectors_exact_and_not_slow(B, W, oracle):
    """Score vectors with the shapes real attention mass takes (recency-biased, trending, concentrated) and
    large budgets, at the 128K unit size: exact lists, and no input shape may cost more than a small
    multiple of random scores."""
    rng = np.random.default_rng(31)
    n, H = 131072, 8
    pr = B.make_problem(n_layers=1, n_q_heads=H, n_kv_heads=H, head_dim=128, n_lookahead=1, n_window=0,
                        softmax_scale=1.0, total_tokens=n, n_in=n)
    ws = torch.empty(B.spec_workspace_bytes(pr), dtype=torch.uint8, device="cuda")
    times = {}
    for name, fn in STRUCTURED.items():
        for c_max in (2048, 4096, 8192):
            if name not in ("random", "recency_decay") and c_max != 2048:
                continue
            x = np.stack([fn(rng, n) for _ in range(H)])[None].astype(np.float32)
            xt = torch.from_numpy(x).cuda()
            idx = torch.full((1, 1, H, c_max), -7, dtype=torch.int32, device="cuda")
            B.spec_pool_topk(pr, xt, B.POOL_MAX, 7, c_max, 0, idx, None, workspace=ws)
            torch.cuda.synchronize()
            oidx, _, _, _ = oracle.pool_topk(x.astype(np.float64), [0, n], oracle.POOL_MAX, 7, c_max, 0)
            np.testing.assert_array_equal(idx.cpu().numpy(), oidx, err_msg="%s c_max=%d" % (name, c_max))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                B.spec_pool_topk(pr, xt, B.POOL_MAX, 7, c_max, 0, idx, None, workspace=ws)
            e1.record()
            torch.cuda.synchronize()
            times[(name, c_max)] = e0.elapsed_time(e1) / 10
    print("select ms per call (8 units of 131072):", {"%s/%d" % k: round(v, 4) for k, v in times.items()})
    base = times[("random", 2048)]
    for key, t in times.items():
        if key[0] == "few_distinct_values":        # thousands of positions tie at the threshold: the generic path, exact but slow
            continue
        assert t <= 3.0 * base + 0.02, "%s takes %.3f ms against %.3f ms for random scores" % (key, t, base)


def test_topk_short_units_in_one_cta_and_streamed(B, W, oracle):
    """Units of up to 16381 positions are selected by one CTA each (scores, floor sample, candidates and the
    finishing step all in shared memory); many hundreds of such units with a workspace are streamed
    instead.  Both against the oracle: sizes at the one-CTA limit, odd offsets of the units in memory,
    empty and tiny sequences, a forced tail, structured scores, heavy ties, a second budget."""
    rng = np.random.default_rng(61)
    for n in (16381, 16382, 16384, 9001):                     # 16384 (units on 16-byte boundaries) and 16381 (anywhere) are the longest
        x = (rng.random((1, 2, n)) ** 6).astype(np.float32)
        run_topk_case(B, W, oracle, x, [0, n], 0, 7, 1024, 0)
    # sequences at odd offsets (a unit's first score on any 4-byte boundary), one empty, one tiny
    cu = [0, 16381, 16381, 16384, 27003, 39990]
    x = (rng.random((2, 3, cu[-1])) ** 5).astype(np.float32)
    run_topk_case(B, W, oracle, x, cu, 0, 7, 1500, 0)
    run_topk_case(B, W, oracle, x, cu, 0, 7, 1500, 32)
    run_vert_case(B, oracle, x, cu, 7, 1024, 32, 2048)
    for name, fn in STRUCTURED.items():
        y = np.stack([fn(rng, 12000) for _ in range(3)])[None].astype(np.float32)
        run_topk_case(B, W, oracle, y, [0, 12000], 0, 7, 2000, 0)
        run_vert_case(B, oracle, y, [0, 5000, 12000], 7, 300, 16, 700)
    y = np.zeros((1, 2, 8000), np.float32)                        # every key equal: the generic selection
    run_topk_case(B, W, oracle, y, [0, 8000], 0, 7, 1000, 0)
    # 640 units of 3000 with a workspace: more units than the one-CTA kernel is given, so they are streamed
    z = (rng.random((40, 16, 3000)) ** 4).astype(np.float32)
    z[:, :, 100:140] = 0.75                                          # a run of ties around the threshold of some units
    run_topk_case(B, W, oracle, z, [0, 3000], 0, 7, 256, 0)
    run_vert_case(B, oracle, z, [0, 1000, 3000], 7, 128, 8, 150)


def test_topk_unit_too_long_for_a_cluster_takes_the_generic_path(B, W, oracle):
    rng = np.random.default_rng(41)
    n = 2_000_003
    x = (rng.random((1, 1, n)) ** 4).astype(np.float32)
    x[0, 0, ::50000] = 0.9                                           # ties at the top
    run_topk_case(B, W, oracle, x, [0, n], 0, 7, 1000, 32)


def test_selection_skips_a_sequence_longer_than_the_given_bound(B, W, oracle):
    """With cu_seqlens the lengths live on the device and n_in is only the caller's bound.  A sequence longer
    than the bound is reported and skipped: no write outside the shared memory sized from the bound."""
    rng = np.random.default_rng(51)
    cu = [0, 3000, 3100]
    x = rng.random((1, 2, 3100)).astype(np.float32)
    cu_t = torch.tensor(cu, dtype=torch.int32, device="cuda")
    pr = B.make_problem(n_layers=1, n_q_heads=2, n_kv_heads=2, head_dim=64, n_lookahead=1, n_window=0, softmax_scale=1.0,
                        total_tokens=3100, n_in=200, n_seq=2, cu_seqlens=cu_t)            # 200 < 3000: too small a bound
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    idx = torch.full((2, 1, 2, 16), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((2, 1, 2), -7, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.spec_workspace_bytes(pr), dtype=torch.uint8, device="cuda")
    o, _, _, _ = oracle.pool_topk(x.astype(np.float64), cu, oracle.POOL_MAX, 7, 16, 0)
    for workspace in (None, ws):                                                 # both selection paths
        B.spec_pool_topk(pr, torch.from_numpy(x).cuda(), B.POOL_MAX, 7, 16, 0, idx, cnt, workspace=workspace, status_word=status)
        torch.cuda.synchronize()
        assert status.item() == B.ERR_BAD_ARG
        assert cnt[0].tolist() == [[0, 0]] and cnt[1].tolist() == [[16, 16]]     # the short sequence is still served
        np.testing.assert_array_equal(idx[1].cpu().numpy(), o[1])
        assert (idx[0] == -1).all()
        status.zero_()
    keep = torch.full((2, 200), -7, dtype=torch.int32, device="cuda")
    n_keep = torch.full((2,), -7, dtype=torch.int32, device="cuda")
    B.specpc_token_select(pr, torch.from_numpy(x).cuda(), B.REDUCE_SUM, B.POOL_MAX, 7, 8, 2, 0, keep, 200, n_keep, ws,
                          status_word=status)
    torch.cuda.synchronize()
    assert status.item() == B.ERR_BAD_ARG
    assert n_keep[0].item() == 0 and 8 <= n_keep[1].item() <= 40


def test_gather_tokens_bit_exact(B, W, oracle):
    rng = np.random.default_rng(9)
    L, H, d, cap = 2, 3, 128, 50
    cu = [0, 300, 300, 1000]
    T = 1000
    k = torch.from_numpy(rng.integers(-32768, 32767, size=(L, H, T, d)).astype(np.int16)).view(torch.bfloat16).cuda()
    v = torch.from_numpy(rng.integers(-32768, 32767, size=(L, H, T, d)).astype(np.int16)).view(torch.bfloat16).cuda()
    n_keep = np.array([37, 0, 50], dtype=np.int32)
    keep = np.full((3, cap), -1, dtype=np.int32)
    for s, n in enumerate((300, 0, 700)):
        keep[s, :n_keep[s]] = np.sort(rng.choice(max(n, 1), n_keep[s], replace=False)) if n_keep[s] else []
    cu_t = torch.tensor(cu, dtype=torch.int32, device="cuda")
    pr = B.make_problem(n_layers=L, n_q_heads=H, n_kv_heads=H, head_dim=d, n_lookahead=1, n_window=0,
                        softmax_scale=1.0, total_tokens=T, n_in=700, n_seq=3, cu_seqlens=cu_t, k=k, v=v)
    out_tokens = 100
    ko = torch.from_numpy(np.full((L, H, out_tokens, d), -1, np.int16)).view(torch.bfloat16).cuda()
    vo = ko.clone()
    cu_out = torch.full((4,), -9, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.spec_gather_tokens(pr, k, v, torch.from_numpy(keep).cuda(), cap, torch.from_numpy(n_keep).cuda(), ko, vo,
                         out_tokens, cu_out, status_word=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for src, got in ((k, ko), (v, vo)):
        want, want_cu = oracle.gather_tokens(bits(src), cu, keep, n_keep, out_tokens)
        np.testing.assert_array_equal(bits(got), want)
        np.testing.assert_array_equal(cu_out.cpu().numpy(), want_cu)
    # a packed total beyond out_tokens is reported, nothing is written out of bounds
    B.spec_gather_tokens(pr, k, None, torch.from_numpy(keep).cuda(), cap, torch.from_numpy(n_keep).cuda(), ko, None,
                         60, cu_out, status_word=status)
    torch.cuda.synchronize()
    assert status.item() == B.ERR_BAD_ARG


def test_speckv_pc_cascade_without_host_sync(B, W, oracle):
    """Section 4.3: SpecPC keep set from draft scores -> compressed target K/V -> SpecKV on the compressed
    prompt, every length staying on the device.  Checked against the same chain of oracle functions."""
    wd = W.CONFIGS[3].replace(n_in=3000, n_layers=2, c_max=200, n_planted=8)          # draft model
    wt = small(W, n_in=3000, n_layers=2, c_max=64, seed=31)                              # target model
    gd, gt = Gpu(B, W, wd, [0, 1]), Gpu(B, W, wt, [0, 1])
    n, cap = 3000, 200 * 17
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # 1. SpecPC on the draft
    sd = gd.score()
    keep = torch.empty((1, cap), dtype=torch.int32, device="cuda")
    n_keep = torch.empty((1,), dtype=torch.int32, device="cuda")
    B.specpc_token_select(gd.pr, sd, B.REDUCE_SUM, B.POOL_MAX, 7, 200, 8, wd.n_window, keep, cap, n_keep, gd.ws,
                          status_word=status)
    # 2. compress the target's K/V (lengths stay on the device)
    v = torch.randn(gt.k.shape, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16).cuda()
    gt.pr = B.make_problem(n_layers=2, n_q_heads=wt.n_q_heads, n_kv_heads=wt.n_kv_heads, head_dim=wt.head_dim,
                           n_lookahead=wt.n_lookahead, n_window=wt.n_window, softmax_scale=wt.scale,
                           total_tokens=n, n_in=n, k=gt.k, v=v)
    kc = torch.zeros((2, wt.n_kv_heads, cap, wt.head_dim), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    cu2 = torch.empty((2,), dtype=torch.int32, device="cuda")
    B.spec_gather_tokens(gt.pr, gt.k, v, keep, cap, n_keep, kc, vc, cap, cu2, status_word=status)
    # 3. SpecKV on the compressed prompt
    pr2 = B.make_problem(n_layers=2, n_q_heads=wt.n_q_heads, n_kv_heads=wt.n_kv_heads, head_dim=wt.head_dim,
                         n_lookahead=wt.n_lookahead, n_window=wt.n_window, softmax_scale=wt.scale,
                         total_tokens=cap, n_in=cap, n_seq=1, cu_seqlens=cu2, k=kc, v=vc)
    ws2 = torch.empty(B.spec_workspace_bytes(pr2), dtype=torch.uint8, device="cuda")
    s2 = torch.empty((2, wt.n_kv_heads, cap), dtype=torch.float32, device="cuda")
    idx = torch.empty((1, 2, wt.n_kv_heads, 64), dtype=torch.int32, device="cuda")
    ko = torch.empty((1, 2, wt.n_kv_heads, 64, wt.head_dim), dtype=torch.bfloat16, device="cuda")
    vo = torch.empty_like(ko)
    B.spec_score(pr2, gt.q, kc, s2, ws2, status_word=status)
    B.spec_pool_topk(pr2, s2, B.POOL_MAX, 7, 64, wt.n_window, idx, None, status_word=status)
    B.spec_compact_kv(pr2, kc, vc, idx, 64, ko, vo, status_word=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    # oracle chain on the GPU's keep list (the keep list itself is covered by the SpecPC parity test)
    nk = int(n_keep.item())
    keep_h, cu2_h = keep.cpu().numpy(), [0, nk]
    assert cu2.cpu().tolist() == cu2_h and wd.n_window <= nk <= cap
    okc, _ = oracle.gather_tokens(bits(gt.k), [0, n], keep_h, np.array([nk], np.int32), cap)
    np.testing.assert_array_equal(bits(kc)[:, :, :nk], okc[:, :, :nk])
    ref = oracle.spec_score(bits(gt.q), okc[:, :, :nk].copy(), cu2_h, wt.n_lookahead, wt.n_window, wt.scale)
    got = s2.cpu().numpy()[:, :, :nk]
    assert_scores_close(got, ref, cu2_h)
    oidx, _, _, _ = oracle.pool_topk(got.astype(np.float64), cu2_h, oracle.POOL_MAX, 7, 64, wt.n_window)
    np.testing.assert_array_equal(idx.cpu().numpy(), oidx)
    np.testing.assert_array_equal(bits(ko), oracle.compact(okc[:, :, :nk].copy(), cu2_h, oidx))
