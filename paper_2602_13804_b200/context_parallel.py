"""Exchange steps of the sequence-sharded (context-parallel) variant of the decode step.

The decode step shards without communication across sequences and KV heads.  When ONE sequence's
pages are spread over several ranks instead, three small exchanges make the ranks agree with what a
single rank would compute (paper Sec. 7: the routed page set, the candidate set and the readout are
functions of per-page / per-token scores that do not depend on where a page lives):

1. page routing: every rank scores the summaries of its own pages and proposes its local top-P;
   one all-gather of the (score, logical page) pairs and a merge under the library's total order
   (score descending, page ascending, -0 = +0) yields the global top-P on every rank;
2. token routing: the same merge on (score, token position) pairs with each rank's local
   top-(K_c + 1) of the routed pages it owns yields the global candidate set and the best rejected
   score (the gap statistic);
3. readout: every rank's partial softmax readout over its own members of the set, with its
   log-sum-exp, is combined by weights exp(lse_r - lse).

The functions below are those exchanges and nothing else: they take what the per-rank kernels produce
(tensors on the rank's device), call torch.distributed collectives (NCCL over NVLink on GPUs, gloo on
CPU) and return identical results on every rank.  Messages are a few hundred KB at most:
batch * heads * P (or K_c + 1) pairs, and batch * heads * (d + 1) floats.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def page_range(n_pages: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous logical pages [lo, hi) of a sequence of n_pages pages that `rank` holds."""
    return (n_pages * rank) // world, (n_pages * (rank + 1)) // world


def _all_gather_cat(t: torch.Tensor, group=None) -> torch.Tensor:
    """[..., n] on every rank -> [..., world * n], rank-major."""
    world = dist.get_world_size(group)
    parts = [torch.empty_like(t) for _ in range(world)]
    dist.all_gather(parts, t.contiguous(), group=group)
    return torch.cat(parts, dim=-1)


def merge_top(scores: torch.Tensor, index: torch.Tensor, k: int, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Global top-k of the ranks' proposals under (score descending, index ascending).

    scores fp32 [..., n], index int32/int64 [..., n] (global page or token ids; -1 marks an unused slot,
    whose score is ignored).  Every rank must propose at least its local top-k for the result to be the
    top-k of the union.  Returns (scores [..., k], index [..., k]), unused slots (-inf, -1), identical on
    every rank.
    """
    s = _all_gather_cat(scores.to(torch.float32), group)
    i = _all_gather_cat(index.to(torch.int64), group)
    unused = i < 0
    s = s + 0.0                                   # -0 and +0 are one key
    s = torch.where(unused, torch.full_like(s, float("-inf")), s)
    big = torch.iinfo(torch.int64).max
    i_key = torch.where(unused, torch.full_like(i, big), i)
    # two stable sorts: by index ascending, then by score descending (ties keep the index order)
    order = torch.sort(i_key, dim=-1, stable=True).indices
    s1, i1 = torch.gather(s, -1, order), torch.gather(i_key, -1, order)
    order = torch.sort(s1, dim=-1, descending=True, stable=True).indices
    s2, i2 = torch.gather(s1, -1, order)[..., :k], torch.gather(i1, -1, order)[..., :k]
    if s2.shape[-1] < k:      # fewer proposals than k: the tail is unused
        extra = k - s2.shape[-1]
        s2 = torch.cat([s2, torch.full(s2.shape[:-1] + (extra,), float("-inf"), dtype=s2.dtype, device=s2.device)], -1)
        i2 = torch.cat([i2, torch.full(i2.shape[:-1] + (extra,), big, dtype=i2.dtype, device=i2.device)], -1)
    pad = i2 == big
    return torch.where(pad, torch.full_like(s2, float("-inf")), s2), torch.where(pad, torch.full_like(i2, -1), i2)


def combine_partials(out: torch.Tensor, lse: torch.Tensor, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Readout over the union of the ranks' token sets from each rank's partial readout.

    out [..., d] is the rank's softmax-weighted value sum normalised over its OWN tokens, lse [...] the
    log-sum-exp of their logits (-inf for a rank that holds none of them).  Returns (out, lse) of the
    union: lse = log sum_r exp(lse_r), out = sum_r exp(lse_r - lse) out_r.
    """
    world = dist.get_world_size(group)
    outs = [torch.empty_like(out) for _ in range(world)]
    lses = [torch.empty_like(lse) for _ in range(world)]
    dist.all_gather(outs, out.contiguous(), group=group)
    dist.all_gather(lses, lse.contiguous(), group=group)
    L = torch.stack(lses, dim=0)
    total = torch.logsumexp(L, dim=0)
    w = torch.exp(L - total.unsqueeze(0))
    w = torch.where(torch.isfinite(L), w, torch.zeros_like(w))
    O = torch.stack(outs, dim=0)
    O = torch.where(torch.isfinite(L).unsqueeze(-1), O, torch.zeros_like(O))
    return (w.unsqueeze(-1) * O).sum(dim=0), total


def gap_from_merged(scores: torch.Tensor, index: torch.Tensor, k_c: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """From the merged top-(K_c + 1) tokens: the candidate ids [..., K_c] and the gap statistic
    s(1) - best rejected (+inf when fewer than K_c + 1 tokens were scored anywhere)."""
    cand = index[..., :k_c]
    has_rejected = index[..., k_c] >= 0 if index.shape[-1] > k_c else torch.zeros_like(index[..., 0], dtype=torch.bool)
    s1 = scores[..., 0]
    rej = scores[..., k_c] if index.shape[-1] > k_c else torch.full_like(s1, float("-inf"))
    delta = torch.where(has_rejected, s1 - rej, torch.full_like(s1, float("inf")))
    return cand, delta
