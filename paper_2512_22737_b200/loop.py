"""Streaming Parallel Decoding (Algorithm 1) as a loop around the library's step calls.

Harness for the end-to-end configuration: a random-init pre-norm decoder (RMSNorm, GQA attention,
SwiGLU) whose dense projections are plain library GEMMs (torch.matmul), while every step of the
decoding hot path runs in this package's kernels: wedlm_reorder, wedlm_window_attn (RoPE at the
logical ids, staging into the paged cache, causal window attention), wedlm_confidence_commit
(confidence, Eq. 11 selection, commit / refill) and wedlm_window_refill (prefill commit).

Window state, block tables and caches stay on the device for the whole generation; the host reads
back only the committed tokens of each step.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as w


def _dev(x: np.ndarray) -> torch.Tensor:
    return w.to_device(x)


class StreamingDecoder:
    def __init__(self, mcfg, weights: Dict[str, np.ndarray], *, batch: int, window: int, max_total_len: int,
                 conf_mode: str = "entropy", tau: float = 0.3, lam: float = 0.1, maxprob_thr: float = 0.9,
                 tilt: float = 0.0, target: Optional[np.ndarray] = None, page_size: int = 16,
                 attn_impl: str = "auto", seed: int = 0, commit_mode: str = "streaming",
                 fused_lm_head: bool = False, temperature: float = 0.0, sample_seed: int = 0):
        self.m = mcfg
        self.B, self.W = batch, window
        self.dtype = torch.bfloat16 if mcfg.dtype == "bf16" else torch.float32
        self.wt = {k: _dev(v) for k, v in weights.items()}
        self.tilt = tilt
        self.target = None if target is None else torch.from_numpy(target.astype(np.int64)).cuda()
        # paged caches, one pair per layer, sharing one block table (scattered pages)
        pages_per_seq = (max_total_len + window + page_size - 1) // page_size
        self.num_pages = batch * pages_per_seq + 3
        g = np.random.default_rng(seed)
        order = g.permutation(self.num_pages).astype(np.int32)
        self.block_table = torch.from_numpy(order[: batch * pages_per_seq].reshape(batch, pages_per_seq).copy()).cuda()
        shape = (self.num_pages, mcfg.n_kv_heads, page_size, mcfg.head_dim)
        self.k_cache = [torch.zeros(shape, dtype=self.dtype, device="cuda") for _ in range(mcfg.n_layers)]
        self.v_cache = [torch.zeros(shape, dtype=self.dtype, device="cuda") for _ in range(mcfg.n_layers)]
        self.cfg = w.make_config(
            batch=batch, window=window, n_q_heads=mcfg.n_q_heads, n_kv_heads=mcfg.n_kv_heads, head_dim=mcfg.head_dim,
            page_size=page_size, max_pages_per_seq=pages_per_seq, num_pages=self.num_pages, vocab=mcfg.vocab,
            dtype=mcfg.dtype, rope_theta=mcfg.rope_theta, conf_mode=conf_mode, tau=tau, lam=lam,
            maxprob_thr=maxprob_thr, mask_token_id=mcfg.mask_token_id, max_prefix_len=max_total_len,
            attn_impl=attn_impl, commit_mode=commit_mode, sample_temperature=temperature, sample_seed=sample_seed)
        if fused_lm_head and temperature > 0.0:
            raise ValueError("the fused LM head keeps no logits to sample from; use fused_lm_head=False with a temperature")
        self.step_bufs = w.DecodeStep(self.cfg)
        # fused LM head: logits are never materialised; the output embedding is kept as [V, H]
        self.fused_lm_head = fused_lm_head
        self.lm_head_vh = None
        self.lm_ws = None
        if fused_lm_head:
            if "lm_head" in self.wt:
                self.lm_head_vh = self.wt["lm_head"].t().contiguous()
            self.lm_ws = torch.empty(w.wedlm_lmhead_confidence_workspace_bytes(self.cfg, int(mcfg.hidden)), dtype=torch.uint8, device="cuda")
        i32 = dict(dtype=torch.int32, device="cuda")
        self.window_tokens = torch.full((batch, window), mcfg.mask_token_id, **i32)
        self.filled = torch.zeros(batch, window, dtype=torch.uint8, device="cuda")
        self.prefix_len = torch.zeros(batch, **i32)
        self.window_len = torch.zeros(batch, **i32)
        self.budget = torch.zeros(batch, **i32)
        self.n_fwd = 0
        self.steps = 0

    # ------------------------------------------------------------------ dense parts (library GEMMs)
    def _rms(self, x: torch.Tensor, gain: torch.Tensor) -> torch.Tensor:
        return torch.nn.functional.rms_norm(x, (x.shape[-1],), gain, self.m.rms_eps)     # one library kernel

    def _fused(self, l: int):
        """[wq | wk | wv] and [wg | wu] of layer l as single matrices, so that each pair of projections is one GEMM."""
        key = f"l{l}.wqkv"
        if key not in self.wt:
            self.wt[key] = torch.cat([self.wt[f"l{l}.wq"], self.wt[f"l{l}.wk"], self.wt[f"l{l}.wv"]], dim=1).contiguous()
            self.wt[f"l{l}.wgu"] = torch.cat([self.wt[f"l{l}.wg"], self.wt[f"l{l}.wu"]], dim=1).contiguous()
        return self.wt[key], self.wt[f"l{l}.wgu"]

    def forward(self, capture_layer: Optional[int] = None, want_logits: bool = True):
        """Causal forward of the reordered window on top of the cache -> logits [B, W, V] (or, with
        want_logits=False, the normalised hidden states [B, W, H] that feed the LM head)."""
        s, m = self.step_bufs, self.m
        B, W = self.B, self.W
        s.reorder(self.filled, self.window_tokens, self.prefix_len, self.window_len)
        h = self.wt["embed"][s.tokens_phys.long()]                       # [B, W, H]
        cap = None
        for l in range(m.n_layers):
            wqkv, wgu = self._fused(l)
            a = self._rms(h, self.wt[f"l{l}.norm1"])
            nq, nkv = m.n_q_heads * m.head_dim, m.n_kv_heads * m.head_dim
            qkv = a @ wqkv
            q = qkv[..., :nq].reshape(B, W, m.n_q_heads, m.head_dim).contiguous()
            k = qkv[..., nq:nq + nkv].reshape(B, W, m.n_kv_heads, m.head_dim).contiguous()
            v = qkv[..., nq + nkv:].reshape(B, W, m.n_kv_heads, m.head_dim).contiguous()
            if capture_layer == l:
                cap = dict(q=q.clone(), k=k.clone(), v=v.clone(), k_cache=self.k_cache[l].clone(),
                           v_cache=self.v_cache[l].clone())
            s.attention(q, k, v, self.k_cache[l], self.v_cache[l], self.block_table, self.prefix_len)
            if capture_layer == l:
                cap["out"] = s.out.clone()
                cap["kv_slot_idx"] = s.kv_slot_idx.clone()
            h = h + s.out.view(B, W, -1) @ self.wt[f"l{l}.wo"]
            mm = self._rms(h, self.wt[f"l{l}.norm2"])
            gu = mm @ wgu
            h = h + (torch.nn.functional.silu(gu[..., :m.ffn]) * gu[..., m.ffn:]) @ self.wt[f"l{l}.wd"]
        hn = self._rms(h, self.wt["norm_f"])
        if not want_logits:
            return hn.contiguous(), cap
        logits = hn @ self.wt["lm_head"]
        if self.tilt != 0.0 and self.target is not None:
            pos = s.pos_ids.long().clamp_(max=self.target.shape[1] - 1)
            idx = self.target.gather(1, pos)                                 # [B, W] target id at each row's position
            logits.scatter_add_(2, idx.unsqueeze(-1), torch.full((B, W, 1), self.tilt, dtype=self.dtype, device="cuda"))
        return logits.contiguous(), cap

    # ------------------------------------------------------------------ Algorithm 1
    def prefill(self, prompt: np.ndarray) -> None:
        """Push the prompt through the layers W tokens at a time (windows of filled slots); each
        window is committed whole, which is just prefix_len += n."""
        B, W = self.B, self.W
        P = prompt.shape[1]
        prompt_dev = torch.from_numpy(prompt.astype(np.int32)).cuda()
        zero_budget = torch.zeros(B, dtype=torch.int32, device="cuda")
        for at in range(0, P, W):
            n = min(W, P - at)
            self.window_tokens.fill_(self.m.mask_token_id)
            self.window_tokens[:, :n] = prompt_dev[:, at:at + n]
            self.filled.zero_()
            self.filled[:, :n] = 1
            self.window_len.fill_(n)
            self.forward()
            zero_budget.zero_()
            w.wedlm_window_refill(self.cfg, self.step_bufs.n_commit, self.window_tokens, self.filled, self.prefix_len,
                                  self.window_len, zero_budget, None, None)

    def start(self, max_new_tokens: int) -> None:
        n0 = min(self.W, max_new_tokens)
        self.window_tokens.fill_(self.m.mask_token_id)
        self.filled.zero_()
        self.window_len.fill_(n0)
        self.budget.fill_(max_new_tokens - n0)
        self.n_fwd = 0
        self.steps = 0

    def step(self, capture_layer: Optional[int] = None):
        """One iteration of Algorithm 1.  Returns (committed_count, committed_tokens) device tensors
        (and the captured tensors of one layer when asked)."""
        s = self.step_bufs
        active = int(self.window_len.sum().item()) if capture_layer is not None else None
        snap = None
        if capture_layer is not None:
            snap = dict(filled=self.filled.clone(), window_tokens=self.window_tokens.clone(),
                        prefix_len=self.prefix_len.clone(), window_len=self.window_len.clone(),
                        budget=self.budget.clone())
        if self.fused_lm_head and capture_layer is None:
            hn, cap = self.forward(None, want_logits=False)
            tilt_ids = None
            if self.tilt != 0.0 and self.target is not None:
                pos = s.pos_ids.long().clamp_(max=self.target.shape[1] - 1)
                tilt_ids = self.target.gather(1, pos).to(torch.int32)
            if self.lm_head_vh is None:
                self.lm_head_vh = self.wt["lm_head"].t().contiguous()
            w.wedlm_lmhead_confidence_commit(self.cfg, hn, self.lm_head_vh, tilt_ids, float(self.tilt), s.perm, s.n_filled,
                                             s.n_commit, self.window_tokens, self.filled, self.prefix_len, self.window_len,
                                             self.budget, s.argmax, s.maxprob, s.entropy, s.lse, s.committed_tokens,
                                             s.committed_count, s.filled_count, self.lm_ws)
            self.steps += 1
            return s.committed_count, s.committed_tokens
        logits, cap = self.forward(capture_layer)
        s.confidence_commit(logits, self.window_tokens, self.filled, self.prefix_len, self.window_len, self.budget)
        self.steps += 1
        if capture_layer is not None:
            cap.update(snap)
            cap["logits"] = logits
            cap["active"] = active
            return s.committed_count, s.committed_tokens, cap
        return s.committed_count, s.committed_tokens

    def _state(self):
        return (self.window_tokens, self.filled, self.prefix_len, self.window_len, self.budget)

    def capture_step(self) -> "torch.cuda.CUDAGraph":
        """One step of Algorithm 1 (all layers, LM head, confidence / commit / refill) as a CUDA graph.  Every
        size the step depends on lives in device memory, so one capture serves the whole generation.  One eager
        step runs first (library and GEMM set-up); the window state is put back afterwards, and what that step
        staged into the caches lies beyond the committed prefix, where the next step overwrites it."""
        saved = [t.clone() for t in self._state()]
        self.step()
        torch.cuda.synchronize()
        for t, s0 in zip(self._state(), saved):
            t.copy_(s0)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.step()
        for t, s0 in zip(self._state(), saved):
            t.copy_(s0)
        self.steps = 0
        return graph

    def generate(self, max_new_tokens: int, max_steps: int = 1_000_000, use_graph: bool = False) -> Dict[str, object]:
        """Runs until every window is empty.  Returns the committed text per sequence, the number of
        steps and the prefix cacheability p_cache = N_gen / N_fwd (Eq. 4).  With use_graph the step is
        captured once and replayed; the host still reads the commits of every step."""
        if use_graph:
            return self._generate_graph(max_new_tokens, max_steps)
        self.start(max_new_tokens)
        ys: List[List[int]] = [[] for _ in range(self.B)]
        commits_per_step = []
        while self.steps < max_steps:
            wl = self.window_len.cpu()
            if int(wl.sum()) == 0:
                break
            self.n_fwd += int(wl.sum())
            cc, ct = self.step()
            cc_h, ct_h = cc.cpu().numpy(), ct.cpu().numpy()
            for b in range(self.B):
                ys[b].extend(ct_h[b, : cc_h[b]].tolist())
            commits_per_step.append(int(cc_h.sum()))
        n_gen = sum(len(y) for y in ys)
        return dict(y=ys, steps=self.steps, n_fwd=self.n_fwd, p_cache=(n_gen / self.n_fwd if self.n_fwd else 0.0),
                    commits_per_step=commits_per_step)

    def _generate_graph(self, max_new_tokens: int, max_steps: int) -> Dict[str, object]:
        import time
        self.start(max_new_tokens)
        t_capture = time.perf_counter()
        graph = self.capture_step()
        torch.cuda.synchronize()
        t_decode = time.perf_counter()
        t_capture = t_decode - t_capture
        s = self.step_bufs
        B, W = self.B, self.W
        # one pinned buffer receives everything the host needs from a step: window_len | count | tokens
        host = torch.empty(B * (2 + W), dtype=torch.int32).pin_memory()
        dev = torch.empty(B * (2 + W), dtype=torch.int32, device="cuda")
        ys: List[List[int]] = [[] for _ in range(B)]
        commits_per_step = []
        wl = self.window_len.cpu().numpy()
        while self.steps < max_steps and int(wl.sum()) > 0:
            self.n_fwd += int(wl.sum())
            graph.replay()
            self.steps += 1
            dev[:B].copy_(self.window_len)
            dev[B:2 * B].copy_(s.committed_count)
            dev[2 * B:].copy_(s.committed_tokens.view(-1))
            host.copy_(dev, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            h = host.numpy()
            wl = h[:B].copy()
            cc_h, ct_h = h[B:2 * B], h[2 * B:].reshape(B, W)
            for b in range(B):
                ys[b].extend(ct_h[b, : cc_h[b]].tolist())
            commits_per_step.append(int(cc_h.sum()))
        n_gen = sum(len(y) for y in ys)
        t_decode = time.perf_counter() - t_decode
        # capture_s: capturing the step once; decode_s: the replay loop with its per-step read-back (host wall clock)
        return dict(y=ys, steps=self.steps, n_fwd=self.n_fwd, p_cache=(n_gen / self.n_fwd if self.n_fwd else 0.0),
                    commits_per_step=commits_per_step, capture_s=t_capture, decode_s=t_decode)
