"""The workspace-free SpecPC entry point, for callers that cannot allocate device memory (for
example code running inside a serving engine whose pool already owns the GPU): its scratch is an
array inside the library.  It must give exactly what the workspace-taking entry point gives, and
what the CPU oracle gives, on consecutive calls that reuse (and must not depend on) the array's
old contents.  Scores sit on a dyadic grid, so that fp32 sums and power-of-two averages are exact
and the lists must be identical.  Collected last on purpose, so that a failure here cannot hide
any other test."""
import ctypes

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _problem(B, cu, L, H):
    cu_t = torch.tensor(cu, dtype=torch.int32, device="cuda")
    return B.make_problem(n_layers=L, n_q_heads=H, n_kv_heads=H, head_dim=64, n_lookahead=1, n_window=0,
                          softmax_scale=1.0, total_tokens=cu[-1], n_in=int(max(np.diff(cu))), n_seq=len(cu) - 1,
                          cu_seqlens=cu_t)


def _both(B, pr, scores, n_seq, cap, args):
    outs = []
    for static in (False, True):
        keep = torch.full((n_seq, cap), -7, dtype=torch.int32, device="cuda")
        n_keep = torch.full((n_seq,), -7, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if static:
            B.specpc_token_select_static(pr, scores, *args, keep, cap, n_keep, status_word=status)
        else:
            ws = torch.empty(B.spec_workspace_bytes(pr), dtype=torch.uint8, device="cuda")
            B.specpc_token_select(pr, scores, *args, keep, cap, n_keep, ws, status_word=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        outs.append((keep.cpu().numpy(), n_keep.cpu().numpy()))
    return outs


def _oracle_keep(oracle, scores, cu, cap, args):
    reduce, pool, k, c_max, nb, forced = args
    keep, n_keep, _, _ = oracle.specpc_select(scores.astype(np.float64), cu, reduce, pool, k, c_max, nb, forced, cap)
    return keep, n_keep


def test_static_scratch_entry_point_matches_workspace_entry_point_and_oracle_twice(oracle):
    from paper_2506_08373_b200 import binding as B
    B.lib()
    rng = np.random.default_rng(77)
    # first call: long packed axis, so the array is left full of large token scores
    cu1, L1, H1 = [0, 3000, 3007, 9000], 4, 2
    s1 = (rng.integers(0, 256, size=(L1, H1, 9000)) / 32 + 5.0).astype(np.float32)
    args1 = (B.REDUCE_SUM, B.POOL_MAX, 7, 256, 8, 0)
    (k_ws, n_ws), (k_st, n_st) = _both(B, _problem(B, cu1, L1, H1), torch.from_numpy(s1).cuda(), 3, 5993, args1)
    k_or, n_or = _oracle_keep(oracle, s1, cu1, 5993, args1)
    np.testing.assert_array_equal(n_st, n_or)
    np.testing.assert_array_equal(k_st, k_or)
    np.testing.assert_array_equal(n_ws, n_or)
    np.testing.assert_array_equal(k_ws, k_or)
    assert n_or.min() > 0
    # second call, right after: other shapes, smaller scores, other options; stale contents must not matter
    cu2, L2, H2 = [0, 500, 2100], 3, 4
    s2 = (rng.integers(0, 64, size=(L2, H2, 2100)) / 64).astype(np.float32)
    args2 = (B.REDUCE_MAX, B.POOL_AVG, 4, 100, 3, 16)
    (k_ws, n_ws), (k_st, n_st) = _both(B, _problem(B, cu2, L2, H2), torch.from_numpy(s2).cuda(), 2, 1600, args2)
    k_or, n_or = _oracle_keep(oracle, s2, cu2, 1600, args2)
    np.testing.assert_array_equal(n_st, n_or)
    np.testing.assert_array_equal(k_st, k_or)
    np.testing.assert_array_equal(n_ws, n_or)
    np.testing.assert_array_equal(k_ws, k_or)


def test_static_scratch_entry_point_rejects_more_tokens_than_its_array():
    from paper_2506_08373_b200 import binding as B
    too_many = B.STATIC_MAX_TOKENS + 1
    pr = B.make_problem(n_layers=1, n_q_heads=1, n_kv_heads=1, head_dim=64, n_lookahead=1, n_window=0,
                        softmax_scale=1.0, total_tokens=too_many, n_in=too_many)
    one = ctypes.c_void_p(256)          # never dereferenced: the size check comes first
    rc = B.lib().specpc_token_select_static(ctypes.byref(pr), one, 0, 0, 7, 16, 0, 0, one, too_many, one, None, None)
    assert rc == B.ERR_UNSUPPORTED
    assert str(B.STATIC_MAX_TOKENS) in B.spec_last_error()
