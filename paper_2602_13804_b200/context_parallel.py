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


def merge_lists(s: torch.Tensor, i: torch.Tensor, k: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """Top-k of concatenated proposals under (score descending, index ascending); no communication.

    s fp32 [..., n], i int [..., n] (global page or token ids; -1 marks an unused slot, whose score is
    ignored).  Returns (scores [..., k], index [..., k]), unused slots (-inf, -1).
    """
    s = s.to(torch.float32)
    i = i.to(torch.int64)
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


def merge_top(scores: torch.Tensor, index: torch.Tensor, k: int, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Global top-k of the ranks' proposals under (score descending, index ascending).

    scores fp32 [..., n], index int32/int64 [..., n] (global page or token ids; -1 marks an unused slot,
    whose score is ignored).  Every rank must propose at least its local top-k for the result to be the
    top-k of the union.  Returns (scores [..., k], index [..., k]), unused slots (-inf, -1), identical on
    every rank.
    """
    s = _all_gather_cat(scores.to(torch.float32), group)
    i = _all_gather_cat(index.to(torch.int64), group)
    return merge_lists(s, i, k)


def combine_lists(outs: torch.Tensor, lses: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """Readout over the union from stacked partial readouts; no communication.
    outs [R, ..., d], lses [R, ...] (-inf where a rank holds no token)."""
    total = torch.logsumexp(lses, dim=0)
    w = torch.exp(lses - total.unsqueeze(0))
    w = torch.where(torch.isfinite(lses), w, torch.zeros_like(w))
    O = torch.where(torch.isfinite(lses).unsqueeze(-1), outs, torch.zeros_like(outs))
    return (w.unsqueeze(-1) * O).sum(dim=0), total


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
    return combine_lists(torch.stack(outs, dim=0), torch.stack(lses, dim=0))


def gap_from_merged(scores: torch.Tensor, index: torch.Tensor, k_c: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """From the merged top-(K_c + 1) tokens: the candidate ids [..., K_c] and the gap statistic
    s(1) - best rejected (+inf when fewer than K_c + 1 tokens were scored anywhere)."""
    cand = index[..., :k_c]
    has_rejected = index[..., k_c] >= 0 if index.shape[-1] > k_c else torch.zeros_like(index[..., 0], dtype=torch.bool)
    s1 = scores[..., 0]
    rej = scores[..., k_c] if index.shape[-1] > k_c else torch.full_like(s1, float("-inf"))
    delta = torch.where(has_rejected, s1 - rej, torch.full_like(s1, float("inf")))
    return cand, delta


class RankKernels:
    """The per-rank GPU steps of the sequence-sharded decode step (one instance per rank and shape): thin
    calls into the C ABI on this rank's shard.  `block_table` has the full width, with negative entries for
    the pages other ranks hold; `seq_lens` are the global lengths."""

    def __init__(self, shape, P: int, K_c: int, device):
        from . import binding as B
        self.B, self.shape, self.P, self.K_c, self.device = B, shape, P, K_c, device
        bh = (shape.batch, shape.n_q_heads)
        self.ws_route = B.alloc_workspace(shape, P, K_c, B.VSA_WS_ROUTE, device)
        self.pages = torch.empty(bh + (P,), dtype=torch.int32, device=device)
        self.page_scores = torch.empty(bh + (P,), dtype=torch.float32, device=device)
        self.cand_pos = torch.empty(bh + (K_c + 1,), dtype=torch.int32, device=device)
        self.cand_score = torch.empty(bh + (K_c + 1,), dtype=torch.float32, device=device)
        self.out = torch.empty(bh + (shape.head_dim,), dtype=torch.float32, device=device)
        self.lse = torch.empty(bh, dtype=torch.float32, device=device)

    def propose_pages(self, q, summaries, block_table, seq_lens):
        """local top-P (score, logical page); pages this rank does not hold (score -inf) are dropped"""
        self.B.vsa_route_pages(self.shape, q, summaries, block_table, seq_lens, self.P, self.pages, self.page_scores,
                               self.ws_route)
        held = self.page_scores > float("-inf")
        return self.page_scores, torch.where(held, self.pages, torch.full_like(self.pages, -1))

    def propose_tokens(self, q, k_cache, block_table, seq_lens, routed_pages):
        """local top-(K_c + 1) tokens (score, position) of the globally routed pages this rank holds"""
        self.B.vsa_cp_token_candidates(self.shape, q, k_cache, block_table, seq_lens, routed_pages.to(torch.int32).contiguous(),
                                       self.P, self.K_c + 1, self.cand_pos, self.cand_score)
        return self.cand_score, self.cand_pos

    def partial_readout(self, v_cache, block_table, seq_lens, cand_pos, cand_score, epsilon: float):
        """(out, lse) over this rank's own members of the global candidate set"""
        self.B.vsa_cp_partial_readout(self.shape, v_cache, block_table, seq_lens, cand_pos.to(torch.int32).contiguous(),
                                      cand_score.to(torch.float32).contiguous(), self.K_c, epsilon, self.out, self.lse)
        return self.out, self.lse


def decode_step(rank: RankKernels, q, summaries, k_cache, v_cache, block_table, seq_lens, epsilon: float, group=None):
    """The whole sequence-sharded step on one rank: three kernels, three exchanges.  Returns
    (out [B, H, d], lse [B, H], delta [B, H], routed_pages [B, H, P], cand_pos [B, H, K_c]), identical on
    every rank."""
    ps, pi = rank.propose_pages(q, summaries, block_table, seq_lens)
    _, routed = merge_top(ps, pi, rank.P, group)
    ts, ti = rank.propose_tokens(q, k_cache, block_table, seq_lens, routed)
    ms, mi = merge_top(ts, ti, rank.K_c + 1, group)
    cand, delta = gap_from_merged(ms, mi, rank.K_c)
    o, l = rank.partial_readout(v_cache, block_table, seq_lens, cand, ms[..., :rank.K_c], epsilon)
    out, lse = combine_partials(o, l, group)
    return out, lse, delta, routed, cand
