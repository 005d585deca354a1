"""Helpers shared by the GPU parity tests: problem set-up through the C-ABI binding and the
comparison rules (score tolerance, index sets outside the tolerance band, bit-exact gather)."""
from __future__ import annotations

import numpy as np
import torch

REL_TOL = 2e-3      # score tolerance: |gpu - oracle| <= REL_TOL*|oracle| + ABS_TOL
ABS_TOL = 1e-6


def bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class Gpu:
    """One problem instance on cuda:0 with its workspace and status word."""

    def __init__(self, B, W, w, layers):
        self.B, self.w = B, w
        dev = "cuda"
        self.q, self.k, self.v = W.gen_layers(w, layers, dev)
        self.cu = W.cu_seqlens(w)
        self.T = self.cu[-1]
        self.L = len(layers)
        self.cu_t = torch.tensor(self.cu, dtype=torch.int32, device=dev) if w.n_seq > 1 else None
        self.pr = B.make_problem(n_layers=self.L, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                                 head_dim=w.head_dim, n_lookahead=w.n_lookahead, n_window=w.n_window,
                                 softmax_scale=w.scale, total_tokens=self.T,
                                 n_in=(w.n_in if w.n_in is not None else max(W.seq_lens(w))),
                                 n_seq=w.n_seq, cu_seqlens=self.cu_t, k=self.k, v=self.v)
        self.ws = torch.empty(max(B.spec_workspace_bytes(self.pr), 16), dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)

    def score(self, reduce=0, row_weight=None, causal_window=0):
        scores = torch.full((self.L, self.w.n_kv_heads, self.T), float("nan"), dtype=torch.float32, device="cuda")
        self.B.spec_score(self.pr, self.q, self.k, scores, self.ws, row_weight=row_weight, reduce=reduce,
                          causal_window=causal_window, status_word=self.status)
        torch.cuda.synchronize()
        assert self.status.item() == 0
        return scores

    def topk(self, scores, pool, pool_k, c_max, forced=0):
        idx = torch.full((self.w.n_seq, self.L, self.w.n_kv_heads, c_max), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((self.w.n_seq, self.L, self.w.n_kv_heads), -7, dtype=torch.int32, device="cuda")
        self.B.spec_pool_topk(self.pr, scores, pool, pool_k, c_max, forced, idx, cnt, workspace=self.ws, status_word=self.status)
        torch.cuda.synchronize()
        assert self.status.item() == 0
        return idx, cnt


def assert_scores_close(got: np.ndarray, ref: np.ndarray, cu):
    """Element-wise score parity on the tokens the sequences cover."""
    hi = cu[-1]
    g, r = got[..., :hi].astype(np.float64), ref[..., :hi]
    err = np.abs(g - r)
    tol = REL_TOL * np.abs(r) + ABS_TOL
    assert np.all(np.isfinite(g))
    worst = float((err / tol).max()) if err.size else 0.0
    assert worst <= 1.0, "score error %.3g x tolerance" % worst


def assert_index_sets_match(gpu_idx: np.ndarray, ora_idx: np.ndarray, pooled: np.ndarray, thresh: float):
    """Selected sets must be identical except for positions whose oracle pooled score lies within
    the score tolerance of the oracle's weakest selected score.  Returns (#outside, #inside band)."""
    g = gpu_idx[gpu_idx >= 0]
    o = ora_idx[ora_idx >= 0]
    assert len(g) == len(o), "selection sizes differ"
    assert np.all(np.diff(g) > 0), "indices must be ascending and unique"
    diff = np.setxor1d(g, o)
    band = REL_TOL * abs(thresh) + ABS_TOL
    for j in diff:
        assert abs(pooled[j] - thresh) <= band, "position %d decided outside the tolerance band" % j
    return len(o) - len(diff) // 2, len(diff) // 2
