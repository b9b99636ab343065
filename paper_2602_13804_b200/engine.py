"""Buffer owner around the C-ABI calls: allocates outputs and scratch once, then every call is a
single library call on the current CUDA stream.  No arithmetic happens here."""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as B


class SparsePagedDecoder:
    """Device buffers for decode steps of one fixed shape (batch, heads, block-table width, P, K_c)."""

    def __init__(self, shape: B.vsa_shape_t, P: int, K_c: int, epsilon: float, gap_threshold: float,
                 device="cuda:0", host_io: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("SparsePagedDecoder needs a CUDA device; there is no CPU path")
        B.lib()
        self.shape, self.P, self.K_c = shape, int(P), int(K_c)
        self.epsilon, self.gap_threshold = float(epsilon), float(gap_threshold)
        self.device = torch.device(device)
        units = shape.batch * shape.n_q_heads
        self.units = units
        dev = self.device
        self.out = torch.empty((shape.batch, shape.n_q_heads, shape.head_dim), dtype=torch.float32, device=dev)
        self.diag = B.alloc_diag(units, dev)
        self.routed_pages = torch.empty((shape.batch, shape.n_q_heads, self.P), dtype=torch.int32, device=dev)
        self.fallback_list = torch.empty(units, dtype=torch.int32, device=dev)
        self.fallback_count = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ws = B.alloc_workspace(shape, self.P, self.K_c, B.VSA_WS_STEP, dev)
        self.summaries: Optional[torch.Tensor] = None
        if host_io:
            self.q_dev = torch.empty((shape.batch, shape.n_q_heads, shape.head_dim), dtype=torch.bfloat16, device=dev)
            self.out_host = torch.empty(self.out.shape, dtype=torch.float32).pin_memory()
            self.diag_host = torch.empty((units, B.DIAG_BYTES // 4), dtype=torch.int32).pin_memory()

    def build_summaries(self, k_cache, block_table, seq_lens, first_page=None, summaries=None) -> torch.Tensor:
        if summaries is None:
            summaries = torch.zeros((self.shape.num_pool_pages, self.shape.n_kv_heads, self.shape.head_dim),
                                    dtype=torch.bfloat16, device=self.device)
        B.vsa_build_page_summaries(self.shape, k_cache, block_table, seq_lens, first_page, summaries)
        self.summaries = summaries
        return summaries

    def step(self, q, summaries, k_cache, v_cache, block_table, seq_lens) -> torch.Tensor:
        """One decode step with device-resident q; returns the (device) output buffer."""
        B.vsa_decode_step(self.shape, q, summaries, k_cache, v_cache, block_table, seq_lens, self.P, self.K_c,
                          self.epsilon, self.gap_threshold, self.out, self.diag, self.routed_pages,
                          self.fallback_list, self.fallback_count, self.ws)
        return self.out

    def step_host(self, q_host, summaries, k_cache, v_cache, block_table, seq_lens) -> torch.Tensor:
        """One decode step with q in (pinned) host memory; results land in self.out_host / self.diag_host
        once the current stream has been synchronised."""
        B.vsa_decode_step_host(self.shape, q_host, self.q_dev, summaries, k_cache, v_cache, block_table, seq_lens,
                               self.P, self.K_c, self.epsilon, self.gap_threshold, self.out_host, self.out,
                               self.diag_host, self.diag, self.routed_pages, self.fallback_list,
                               self.fallback_count, self.ws)
        return self.out_host

    # ---- variants of the step ---------------------------------------------------------------------

    def step_entropic(self, q, summaries, k_cache, v_cache, block_table, seq_lens, solver_iters: int) -> torch.Tensor:
        """The step with the candidate weights taken from `solver_iters` entropic mirror-descent
        iterations; the per-unit certificate and objective land in self.solve ([units, 4] float32)."""
        if not hasattr(self, "solve"):
            self.solve = B.alloc_solve(self.units, self.device)
        B.vsa_decode_step_entropic(self.shape, q, summaries, k_cache, v_cache, block_table, seq_lens, self.P,
                                   self.K_c, self.epsilon, self.gap_threshold, int(solver_iters), self.out,
                                   self.diag, self.solve, self.routed_pages, self.fallback_list,
                                   self.fallback_count, self.ws)
        return self.out

    def build_radii(self, k_cache, summaries, block_table, seq_lens, first_page=None, radii=None) -> torch.Tensor:
        if radii is None:
            radii = torch.zeros((self.shape.num_pool_pages, self.shape.n_kv_heads), dtype=torch.float32,
                                device=self.device)
        B.vsa_build_page_radii(self.shape, k_cache, summaries, block_table, seq_lens, first_page, radii)
        return radii

    def step_certified(self, q, summaries, radii, k_cache, v_cache, block_table, seq_lens) -> torch.Tensor:
        """The step with the routing certificate: the certified gap (self.cert, [units, 4] int32 view of
        vsa_cert_t, see binding.cert_to_dict) decides which units fall back to the dense pass."""
        if not hasattr(self, "cert"):
            self.cert = B.alloc_cert(self.units, self.device)
        if not hasattr(self, "ws_cert"):
            self.ws_cert = B.alloc_workspace(self.shape, self.P, self.K_c, B.VSA_WS_STEP_CERTIFIED, self.device)
        B.vsa_decode_step_certified(self.shape, q, summaries, radii, k_cache, v_cache, block_table, seq_lens, self.P,
                                    self.K_c, self.epsilon, self.gap_threshold, self.out, self.diag, self.cert,
                                    self.routed_pages, self.fallback_list, self.fallback_count, self.ws_cert)
        return self.out

    def build_super_summaries(self, summaries, block_table, seq_lens, first_super=None) -> torch.Tensor:
        """Representative summary per 16 logical pages (cache maintenance for step_two_level)."""
        if not hasattr(self, "super_summaries"):
            self.super_summaries = torch.zeros((self.shape.batch, B.n_super_pages(self.shape), self.shape.n_kv_heads,
                                                self.shape.head_dim), dtype=torch.bfloat16, device=self.device)
        B.vsa_build_super_summaries(self.shape, summaries, block_table, seq_lens, first_super, self.super_summaries)
        return self.super_summaries

    def step_two_level(self, q, summaries, super_summaries, k_cache, v_cache, block_table, seq_lens,
                       P_super: int) -> torch.Tensor:
        """The step with two-level routing: only the pages of the P_super best super-pages are scored."""
        if getattr(self, "_P_super", None) != int(P_super):
            self._P_super = int(P_super)
            self.ws_two_level = B.alloc_workspace(self.shape, self._P_super, self.K_c, B.VSA_WS_STEP_TWO_LEVEL,
                                                  self.device)
        B.vsa_decode_step_two_level(self.shape, q, summaries, super_summaries, k_cache, v_cache, block_table,
                                    seq_lens, self._P_super, self.P, self.K_c, self.epsilon, self.gap_threshold,
                                    self.out, self.diag, self.routed_pages, self.fallback_list,
                                    self.fallback_count, self.ws_two_level)
        return self.out

    def append(self, k_new, v_new, k_cache, v_cache, block_table, seq_lens_after, summaries, radii=None) -> None:
        """Append one token per sequence (lengths AFTER the append) and refresh its page's summary / radius."""
        B.vsa_append_kv(self.shape, k_new, v_new, k_cache, v_cache, block_table, seq_lens_after, summaries, radii)

    def step_frank_wolfe(self, q, summaries, k_cache, v_cache, block_table, seq_lens, solver_iters: int) -> torch.Tensor:
        """The step with the candidate weights taken from `solver_iters` Frank-Wolfe iterations (exact line
        search, unregularised problem); certificate and objective land in self.solve."""
        if not hasattr(self, "solve"):
            self.solve = B.alloc_solve(self.units, self.device)
        B.vsa_decode_step_frank_wolfe(self.shape, q, summaries, k_cache, v_cache, block_table, seq_lens, self.P,
                                      self.K_c, self.epsilon, self.gap_threshold, int(solver_iters), self.out,
                                      self.diag, self.solve, self.routed_pages, self.fallback_list,
                                      self.fallback_count, self.ws)
        return self.out

    def step_certified_expand(self, q, summaries, radii, k_cache, v_cache, block_table, seq_lens,
                              P_expand: int) -> torch.Tensor:
        """The certified step with one expansion round: refused units are retried with `P_expand` pages
        before the dense pass.  self.routed_pages_expand ([batch, heads, P_expand]) holds each unit's
        pages of its last pass."""
        if not hasattr(self, "cert"):
            self.cert = B.alloc_cert(self.units, self.device)
        if getattr(self, "_expand_P", None) != int(P_expand):
            self._expand_P = int(P_expand)
            self.ws_expand = B.alloc_workspace(self.shape, self._expand_P, self.K_c, B.VSA_WS_STEP_EXPAND, self.device)
            self.routed_pages_expand = torch.empty((self.shape.batch, self.shape.n_q_heads, self._expand_P),
                                                   dtype=torch.int32, device=self.device)
        B.vsa_decode_step_certified_expand(self.shape, q, summaries, radii, k_cache, v_cache, block_table, seq_lens,
                                           self.P, self._expand_P, self.K_c, self.epsilon, self.gap_threshold,
                                           self.out, self.diag, self.cert, self.routed_pages_expand,
                                           self.fallback_list, self.fallback_count, self.ws_expand)
        return self.out
