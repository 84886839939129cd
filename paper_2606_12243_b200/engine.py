"""Device-side set-up of a synthetic workload: weights, caches and step inputs in HBM.

Memory management only (torch allocations and host->device copies of generated tensors);
every step of the verification path runs in the CUDA library through `binding`.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

from synth import workloads as W
from . import binding as vb


def to_device(a: np.ndarray, device="cuda") -> torch.Tensor:
    """Generated tensor (fp32, int32, or bf16 as raw uint16 words) -> CUDA tensor of the right dtype."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


class Engine:
    GUARD = 8192                         # bytes of poisoned memory kept on either side of the workspace

    def guards_intact(self) -> bool:
        off = self.workspace.data_ptr() - self._ws_block.data_ptr()
        before, after = self._ws_block[:off], self._ws_block[off + self.workspace.numel():]
        return bool((before == 0xFF).all().item()) and bool((after == 0xFF).all().item())

    def __init__(self, wl: W.Workload, device="cuda", max_query: Optional[int] = None,
                 extra_ctx: int = 0, fill_context=True, weights_from: Optional["Engine"] = None,
                 state_from: Optional["Engine"] = None):
        """fill_context: True = the generator's committed context (what the parity tests compare against);
        "device" = values of the same distribution drawn on the device (timing sweeps over caches of tens of
        GB, where only the shape matters); False = leave the caches empty.
        weights_from: another engine of the same model shape and seed whose weight tensors are reused.
        state_from: a handle for one more slim verifier of the same model (an n-tier step): the full verifier's
        cache, lengths, pending tokens and token list are the other engine's; only the slim cache and the workspace
        are this engine's own."""
        self.wl, self.device = wl, device
        s = wl.shape
        self.tdtype = torch.float32 if s.dtype == "f32" else torch.bfloat16
        self.max_query = max_query or wl.rows
        self.max_ctx = wl.ctx + max(self.max_query, wl.rows) + extra_ctx
        self.cfg = vb.make_config(s.n_layers, s.d_model, s.n_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.vocab,
                                  s.dtype, wl.batch, self.max_ctx, self.max_query, s.rms_eps, s.rope_theta)
        if weights_from is not None:
            o = weights_from.wl
            assert (o.shape, o.seed, o.weight_sigma, o.gain_jitter) == (s, wl.seed, wl.weight_sigma, wl.gain_jitter)
            self.embed, self.lm_head, self.final_norm = weights_from.embed, weights_from.lm_head, weights_from.final_norm
            self.layers: List[Dict[str, torch.Tensor]] = weights_from.layers
        else:
            gen = W.Model(wl)
            self.embed = to_device(gen.tensor(-1, "embed"), device)
            self.lm_head = to_device(gen.tensor(-1, "lm_head"), device)
            self.final_norm = to_device(gen.tensor(-1, "final_norm"), device)
            self.layers = []
            for l in range(s.n_layers):
                self.layers.append({k: to_device(v, device) for k, v in gen.layer(l).items()})
        self.routed = wl.routed
        mask = [1 if l in set(self.routed) else 0 for l in range(s.n_layers)]
        nbytes = vb.workspace_bytes(self.cfg, len(self.routed))
        assert nbytes > 0, "configuration rejected by viasd_workspace_bytes"
        # Poisoned on purpose (every float a NaN, every counter -1): the library has to initialise what it relies on,
        # and recycled device memory is not zero.
        # The library gets exactly the bytes it asked for, cut out of the middle of a larger block whose two ends
        # serve as guard zones: anything written outside the workspace shows in guards_intact().
        self._ws_block = torch.full((nbytes + 2 * self.GUARD,), 0xFF, dtype=torch.uint8, device=device)
        off = (-self._ws_block.data_ptr()) % 256 + self.GUARD // 2
        self.workspace = self._ws_block[off:off + nbytes]
        self.model = vb.init_model(self.cfg, self.embed, self.lm_head, self.final_norm, self.layers, mask,
                                   self.workspace)
        kv = lambda nl: torch.zeros((nl, wl.batch, s.n_kv_heads, self.max_ctx, s.head_dim), dtype=self.tdtype,
                                    device=device)
        self.k_slim, self.v_slim = kv(len(self.routed)), kv(len(self.routed))
        if state_from is not None:
            o = state_from
            assert o.max_ctx == self.max_ctx and o.wl.batch == wl.batch and o.wl.shape == s
            self.k_full, self.v_full, self.len, self.pending = o.k_full, o.v_full, o.len, o.pending
            self.tokens, self.len_full = o.tokens, o.len_full
        else:
            self.k_full, self.v_full = kv(s.n_layers), kv(s.n_layers)
            self.len = torch.zeros(wl.batch, dtype=torch.int32, device=device)
            self.pending = torch.zeros(wl.batch, dtype=torch.int32, device=device)
            self.tokens = torch.zeros((wl.batch, self.max_ctx), dtype=torch.int32, device=device)
            self.len_full = torch.zeros(wl.batch, dtype=torch.int32, device=device)
        self.cache = vb.make_cache(self.k_full, self.v_full, self.k_slim, self.v_slim, self.len, self.pending,
                                   self.tokens, self.len_full)
        if fill_context == "device" and wl.ctx > 0:
            self.fill_random_context()
        elif fill_context and not wl.real_prefill and wl.ctx > 0:
            self.fill_synthetic_context(slim_only=state_from is not None)
        self.draft = None
        self.inputs = None

    # -- committed context ---------------------------------------------------------------
    def fill_synthetic_context(self, slim_only: bool = False) -> None:
        wl = self.wl
        for cache_id, (kc, vc, nl) in enumerate(((self.k_full, self.v_full, wl.shape.n_layers),
                                                 (self.k_slim, self.v_slim, len(self.routed)))):
            if slim_only and cache_id == 0:
                continue
            for o in range(nl):
                kc[o, :, :, :wl.ctx] = to_device(W.context_kv(wl, cache_id, o, 0), self.device)
                vc[o, :, :, :wl.ctx] = to_device(W.context_kv(wl, cache_id, o, 1), self.device)
        self.len.fill_(wl.ctx)
        self.len_full.fill_(wl.ctx)

    def fill_random_context(self) -> None:
        """Committed context drawn on the device, N(0, kv_sigma) like the generator's: for timing only."""
        g = torch.Generator(device=self.device)
        g.manual_seed(self.wl.seed)
        sigma = W.kv_sigma(self.wl)
        for t in (self.k_full, self.v_full, self.k_slim, self.v_slim):
            for o in range(t.shape[0]):
                t[o, :, :, :self.wl.ctx].normal_(0.0, sigma, generator=g)
        self.len.fill_(self.wl.ctx)
        self.len_full.fill_(self.wl.ctx)

    def prefill(self, prompt: np.ndarray) -> None:
        """Push a prompt [B, T] through both models with the library's own forward + commit calls."""
        B, T = prompt.shape
        V = self.wl.shape.vocab
        self.pending.copy_(torch.from_numpy(prompt[:, 0].astype(np.int32)))
        pos = 1
        while pos < T:
            n = min(self.max_query - 1, T - pos)
            tok = torch.from_numpy(prompt[:, pos:pos + n].astype(np.int32)).to(self.device).contiguous()
            parent = torch.arange(-1, n - 1, dtype=torch.int32, device=self.device)
            d = vb.make_draft(tok, parent, parent, 0, None)
            logits = torch.empty((B, n + 1, V), dtype=torch.float32, device=self.device)
            vb.full_forward(self.model, self.cache, d, logits)
            vb.slim_forward(self.model, self.cache, d, logits)
            res = vb.alloc_result(B, n, self.device)
            res.n_acc.fill_(n)
            res.n_emit.fill_(n)
            res.path.copy_(torch.arange(n, dtype=torch.int32, device=self.device).expand(B, n))
            res.out_tok[:, :n] = tok
            vb.kv_commit(self.model, self.cache, d, res)
            pos += n

    # -- step inputs -------------------------------------------------------------------------
    def set_inputs(self, si: W.StepInputs, set_pending: bool = True) -> None:
        dev = self.device
        self.inputs = si
        self.draft_tok = torch.from_numpy(si.draft_tok.astype(np.int32)).to(dev).contiguous()
        self.parent = torch.from_numpy(si.parent.astype(np.int32)).to(dev)
        self.prow = torch.from_numpy(si.prow.astype(np.int32)).to(dev)
        self.drafter_logits = torch.from_numpy(si.drafter_logits).to(dev)
        if set_pending:
            self.pending.copy_(torch.from_numpy(si.pending.astype(np.int32)))
        self.draft = vb.make_draft(self.draft_tok, self.parent, self.prow, si.n_prows, self.drafter_logits)

    def logits_buffer(self) -> torch.Tensor:
        return torch.empty((self.wl.batch, self.wl.rows, self.wl.shape.vocab), dtype=torch.float32,
                           device=self.device)

    def params(self, step: int = 0, **kw) -> vb.Params:
        lo, hi = W.thresholds(self.wl)
        kw.setdefault("mode", 1 if self.wl.mode == "sampling" else 0)
        kw.setdefault("temperature", self.wl.temperature)
        kw.setdefault("seed", self.wl.seed)
        return vb.make_params(kw.pop("log_tau_lo", lo), kw.pop("log_tau_hi", hi), step=step, **kw)
