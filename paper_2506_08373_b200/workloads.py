"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers and lays them out; it contains none of the
method's arithmetic (no softmax, pooling, selection or gather).  Both the CUDA
path and the CPU oracle consume the bf16 tensors produced here, so that the two
sides see bit-identical inputs without sharing any other code.

The recipe stands in for real long-context prompts pushed through Llama-shaped
models (the paper's RULER / LongBench runs need weights and data that are not
available): Q/K/V are i.i.d. N(0,1); a reserved feature channel gives every key
an additive, power-law ("Zipf 1.1") logit bias so attention mass is
approximately sparse; a small set of planted heavy-hitter keys aligned with the
mean query direction plays the role of retrieval needles.

All tensors are generated per layer from an independent seeded stream, so any
layer can be regenerated alone on either device type.  CPU and CUDA generators
give different values for the same seed; a comparison always moves the bytes,
never regenerates them on the other device.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and distribution parameters of one synthetic workload."""

    name: str
    seed: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_lookahead: int
    n_window: int
    pool_k: int
    c_max: int
    # Either a single length (n_seq == 1) or None with (n_seq, len_lo, len_hi).
    n_in: Optional[int] = None
    n_seq: int = 1
    len_lo: int = 0
    len_hi: int = 0
    # Distribution controls.
    key_scale: float = 1.0          # multiplies background keys
    softmax_scale: Optional[float] = None  # None -> 1/sqrt(head_dim)
    zipf_bias: bool = False         # reserve last feature as logit-bias channel
    planted: str = "runs"           # "runs" (1% in runs of 16), "singletons", "token" (same positions everywhere)
    n_planted: int = 0              # count for "singletons"/"token"
    planted_gain: Optional[float] = None   # None -> row-mean logit 4..4.5; else key = gain * unit mean-query direction
    sink_gain: float = 0.0          # >0: key 0 is planted with this gain
    n_neighbor: int = 0             # SpecPC neighbour radius
    page_size: int = 0              # >0: paged destination cache
    l_skip: int = 0                 # SpecPC: draft layers left out of the token scores
    paper_specpc: bool = False      # SpecPC run with the paper's own settings (max reductions, window row weights,
                                    # average pool then max pool before the selection, window always kept)

    @property
    def rows(self) -> int:
        return self.n_lookahead + self.n_window

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def scale(self) -> float:
        return self.softmax_scale if self.softmax_scale is not None else 1.0 / math.sqrt(self.head_dim)

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five benchmark workloads (index = configuration number).
CONFIGS: List[Workload] = [
    Workload(name="c0_tiny", seed=0, n_layers=1, n_q_heads=8, n_kv_heads=2, head_dim=64,
             n_in=2048, n_lookahead=32, n_window=16, pool_k=7, c_max=256,
             key_scale=0.125, softmax_scale=1.0, planted="singletons", n_planted=16,
             planted_gain=4.0, sink_gain=6.0),
    Workload(name="c1_llama8b_16k", seed=1, n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128,
             n_in=16384, n_lookahead=64, n_window=32, pool_k=7, c_max=1024, zipf_bias=True),
    Workload(name="c2_llama8b_128k", seed=2, n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128,
             n_in=131072, n_lookahead=128, n_window=32, pool_k=7, c_max=2048, zipf_bias=True),
    Workload(name="c3_specpc_1b_32k", seed=3, n_layers=16, n_q_heads=32, n_kv_heads=8, head_dim=64,
             n_in=32768, n_lookahead=64, n_window=64, pool_k=7, c_max=4096, planted="token",
             n_planted=64, n_neighbor=8),
    Workload(name="c4_ragged_16seq", seed=4, n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128,
             n_seq=16, len_lo=4096, len_hi=65536, n_lookahead=64, n_window=32, pool_k=7, c_max=1024,
             zipf_bias=True, page_size=16),
    # not one of the five benchmark workloads: the SpecPC column of the paper's hyper-parameter table on the
    # draft shape of workload 3 (n_window 64, n_lookahead 1, Pool Avg k = 64, n_neighbor 64, l_skip 8, C_max 1024)
    Workload(name="c5_specpc_paper_settings", seed=5, n_layers=16, n_q_heads=32, n_kv_heads=8, head_dim=64,
             n_in=32768, n_lookahead=1, n_window=64, pool_k=64, c_max=1024, planted="token",
             n_planted=64, n_neighbor=64, l_skip=8, paper_specpc=True),
]


def _gen(device, *parts: int) -> torch.Generator:
    """Independent stream per (seed, layer, tensor, ...) tuple."""
    s = 0x9E3779B97F4A7C15
    for p in parts:
        s = (s * 6364136223846793005 + (int(p) + 1) * 1442695040888963407) & ((1 << 63) - 1)
    g = torch.Generator(device=device)
    g.manual_seed(s)
    return g


def seq_lens(w: Workload) -> List[int]:
    """Prompt length of every sequence (seeded for ragged workloads)."""
    if w.n_in is not None:
        return [int(w.n_in)] * w.n_seq
    g = _gen("cpu", w.seed, 0xA11CE)
    lens = torch.randint(w.len_lo, w.len_hi + 1, (w.n_seq,), generator=g)
    return [int(x) for x in lens]


def cu_seqlens(w: Workload) -> List[int]:
    out = [0]
    for n in seq_lens(w):
        out.append(out[-1] + n)
    return out


def block_table(w: Workload, device="cpu") -> torch.Tensor:
    """Caller-assigned page ids for the paged destination: a seeded permutation, so
    that pages of one sequence are deliberately non-contiguous."""
    assert w.page_size > 0
    pages_per_seq = (w.c_max + w.page_size - 1) // w.page_size
    g = _gen("cpu", w.seed, 0xB10C)
    perm = torch.randperm(w.n_seq * pages_per_seq, generator=g).to(torch.int32)
    return perm.view(w.n_seq, pages_per_seq).to(device)


def planted_positions(w: Workload, layer: int, seq: int, n: int) -> torch.Tensor:
    """int64 [n_kv_heads, P] planted key positions of one (layer, sequence).  CPU tensor."""
    H = w.n_kv_heads
    if w.planted == "token":
        g = _gen("cpu", w.seed, 0x9A, seq)
        pos = torch.randperm(n, generator=g)[: min(w.n_planted, n)]
        return pos.sort().values.unsqueeze(0).repeat(H, 1)
    out = []
    for h in range(H):
        g = _gen("cpu", w.seed, 0x9B, layer, seq, h)
        if w.planted == "singletons":
            lo = 1 if w.sink_gain > 0 else 0
            pos = torch.randperm(n - lo, generator=g)[: min(w.n_planted, n - lo)] + lo
        else:  # runs of 16 covering ~1% of the positions
            run = 16
            n_runs = max(1, int(round(0.01 * n / run))) if n >= run else 0
            slots = torch.randperm(max(n // run, 1), generator=g)[:n_runs]
            pos = (slots.unsqueeze(1) * run + torch.arange(run).unsqueeze(0)).reshape(-1)
            pos = pos[pos < n]
        out.append(pos.sort().values)
    P = min(len(p) for p in out)
    return torch.stack([p[:P] for p in out])


def gen_layer(w: Workload, layer: int, device="cpu", want_v: bool = True):
    """Generate one layer.

    Returns (q, k, v): q [n_seq, n_q_heads, R, d], k and v [n_kv_heads, T, d], bf16, on
    `device`.  T is the packed token axis (sum of sequence lengths).  v is None when
    want_v is False (the scoring step never reads V).
    """
    dev = torch.device(device)
    lens = seq_lens(w)
    cu = cu_seqlens(w)
    T = cu[-1]
    d, R, G, Hk = w.head_dim, w.rows, w.group, w.n_kv_heads
    scale = w.scale

    q = torch.randn((w.n_seq, w.n_q_heads, R, d), generator=_gen(dev.type, w.seed, layer, 1),
                    device=dev, dtype=torch.float32)
    k = torch.randn((Hk, T, d), generator=_gen(dev.type, w.seed, layer, 2),
                    device=dev, dtype=torch.float32)
    if w.key_scale != 1.0:
        k *= w.key_scale
    feat = d - 1 if w.zipf_bias else d
    if w.zipf_bias:
        # Exact additive per-key logit bias through a reserved feature channel.
        qb = torch.tensor(1.0 / scale, dtype=torch.float32).to(torch.bfloat16).float().item()
        q[..., d - 1] = qb
        for s, n in enumerate(lens):
            u = torch.rand((Hk, n), generator=_gen(dev.type, w.seed, layer, 3, s), device=dev)
            rank = u.argsort(dim=1).argsort(dim=1).float() + 1.0
            k[:, cu[s]:cu[s + 1], d - 1] = -1.1 * torch.log(rank)
    q = q.to(torch.bfloat16)

    # Heavy hitters: keys aligned with the mean of the M stacked bf16 query rows.
    for s, n in enumerate(lens):
        if n == 0:
            continue
        pos = planted_positions(w, layer, s, n).to(dev)          # [Hk, P]
        P = pos.shape[1]
        qm = q[s].float().view(Hk, G * R, d)[:, :, :feat].mean(dim=1)   # [Hk, feat]
        nrm = qm.norm(dim=1, keepdim=True).clamp_min(1e-6)
        unit = qm / nrm
        if w.planted_gain is not None:
            gain = torch.full((Hk, P), float(w.planted_gain), device=dev)
        else:
            u = torch.rand((Hk, P), generator=_gen(dev.type, w.seed, layer, 4, s), device=dev)
            gain = (4.0 + 0.5 * u) / (scale * nrm)
        rows = torch.zeros((Hk, P, d), device=dev)
        rows[:, :, :feat] = gain.unsqueeze(2) * unit.unsqueeze(1)
        k[torch.arange(Hk, device=dev).unsqueeze(1), cu[s] + pos] = rows
        if w.sink_gain > 0:
            k[:, cu[s], :] = 0
            k[:, cu[s], :feat] = w.sink_gain * unit
    k = k.to(torch.bfloat16)

    v = None
    if want_v:
        v = torch.randn((Hk, T, d), generator=_gen(dev.type, w.seed, layer, 5),
                        device=dev, dtype=torch.float32).to(torch.bfloat16)
    return q, k, v


def gen_layers(w: Workload, layers: Sequence[int], device="cpu", want_v: bool = True):
    """Stack several layers: q [n_seq, L', Hq, R, d], k/v [L', Hkv, T, d] (contiguous bf16)."""
    lens = seq_lens(w)
    T = sum(lens)
    Lp = len(layers)
    dev = torch.device(device)
    q = torch.empty((w.n_seq, Lp, w.n_q_heads, w.rows, w.head_dim), dtype=torch.bfloat16, device=dev)
    k = torch.empty((Lp, w.n_kv_heads, T, w.head_dim), dtype=torch.bfloat16, device=dev)
    v = torch.empty_like(k) if want_v else None
    for i, l in enumerate(layers):
        ql, kl, vl = gen_layer(w, l, device, want_v)
        q[:, i] = ql
        k[i] = kl
        if want_v:
            v[i] = vl
    return q, k, v
