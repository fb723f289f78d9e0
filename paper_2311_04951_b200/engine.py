"""Generation loops on top of the C ABI: orchestration only (which call comes next, where its
buffers live).  No arithmetic of the method happens here; every number is produced by the
library's kernels.

One speculative iteration (Section "Speculative Sampling", Figure 2; cache handling of Section
"So, what's the problem?") is:  K x draft_step  ->  target_verify  ->  spec_advance,
all queued on one stream, wired through device buffers so that nothing returns to the host:
draft_step writes its token straight into the verification row block and its q row straight
into the q block; spec_advance writes the next pending token and the draft's catch-up rows.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional

import numpy as np
import torch

from . import binding as B


def expected_tokens(alpha: float, k: int) -> float:
    """Tokens emitted per iteration with k draft tokens when each is accepted independently with
    probability alpha: 1 + alpha + ... + alpha^k."""
    return float(k + 1) if alpha >= 1.0 else (1.0 - alpha ** (k + 1)) / (1.0 - alpha)


class AdaptiveK:
    """Number of draft tokens per iteration from the running acceptance rate (Section "Speculative
    Sampling": drafting pays off while the draft's tokens keep being accepted).  The rate is estimated as
    accepted / tested over the iterations reported so far (exponentially forgotten), and the next k maximises
    tokens per unit of time, expected_tokens(alpha, k) / (1 + k * cost), where cost = time of a draft step /
    time of a verification pass.  Host-side policy only: no arithmetic of the method."""

    def __init__(self, k_max: int, cost: float, k_min: int = 1, forget: float = 0.9, alpha0: float = 0.5):
        assert 1 <= k_min <= k_max and cost >= 0.0 and 0.0 <= forget <= 1.0
        self.k_max, self.k_min, self.cost, self.forget = k_max, k_min, float(cost), float(forget)
        self.acc, self.tested = alpha0, 1.0          # one pseudo-observation at alpha0

    @property
    def alpha(self) -> float:
        return self.acc / self.tested if self.tested > 0 else 0.0

    def update(self, accepted, k: int) -> None:
        """accepted: the iteration's accepted counts (one per sequence) with k draft tokens each."""
        for a in accepted:
            a = int(a)
            self.acc = self.forget * self.acc + a
            self.tested = self.forget * self.tested + min(a + 1, k)   # the tests up to and including the first refusal

    def choose(self) -> int:
        a = self.alpha
        return max(range(self.k_min, self.k_max + 1), key=lambda k: (expected_tokens(a, k) / (1.0 + k * self.cost), -k))


class Engine:
    def __init__(self, target: B.Model, draft: Optional[B.Model], batch: int, max_len: int, K: int,
                 temperature: float, out_cap: int):
        self.target, self.draft = target, draft
        self.batch, self.max_len, self.K, self.T = batch, max_len, K, float(temperature)
        self.K_max = K
        # Draft loop as ONE draft_steps call (one launch that ends every step inside the kernel) or as one
        # draft_step call per token.  Measured on B200 the two are within a few per cent of each other (the
        # in-kernel tail costs grid barriers where the other path costs two small launches); the per-token form
        # is the default because it is the faster one at batch 1.
        self.fused_draft = False
        self.prompt_ws_cap = 4 << 30      # bytes of temporary workspace the prompt pass may take
        V = target.arch.vocab
        dev = "cuda"
        self.tkv = B.KV(target, batch, max_len)
        self.ws_t = target.new_workspace(batch, K + 1, max_len)
        self.rows = torch.zeros(batch, K + 1, dtype=torch.int32, device=dev)
        self._rows_of = {K: self.rows}    # row blocks of iterations that draft fewer than K tokens (stride k + 1)
        # accepted counts of the last `log_cap` iterations, one row each: target_verify writes row it % log_cap
        # (a pointer, not a copy), so acceptance statistics can be read after a run without touching the loop
        self.log_cap = max(1, out_cap // (K + 1) + 1)
        self.n_acc_log = torch.zeros(self.log_cap, batch, dtype=torch.int32, device=dev)
        self.it = 0
        self.next_tok = torch.zeros(batch, dtype=torch.int32, device=dev)
        self.out_cap = out_cap
        self.out_tokens = torch.zeros(batch, out_cap, dtype=torch.int32, device=dev)
        self.out_count = torch.zeros(batch, dtype=torch.int32, device=dev)
        self.chunk = min(B.MAX_ROWS_PER_SEQ, B.MAX_ROWS // batch)   # rows per sequence of a prompt-pass forward
        self.ws_pre_t = target.new_workspace(batch, self.chunk, max_len)
        if draft is not None and K > 0:
            self.dkv = B.KV(draft, batch, max_len)
            self.ws_d = draft.new_workspace(batch, 2, max_len)
            self.ws_pre_d = draft.new_workspace(batch, self.chunk, max_len)
            self.q_full = torch.zeros(batch * K * V, dtype=torch.float32, device=dev)
            self.q = self.q_full.view(batch, K, V)
            self.draft_in = torch.zeros(batch, 2, dtype=torch.int32, device=dev)
            self.draft_n_in = torch.ones(batch, dtype=torch.int32, device=dev)
        else:
            self.dkv = None
            self.q = None

    @property
    def n_acc(self) -> torch.Tensor:
        """int32 [batch]: where the current iteration's accepted counts are written and read."""
        return self.n_acc_log[self.it % self.log_cap]

    def refresh_bounds(self) -> None:
        """Make the host-side length bounds (from which attention splits are planned) exact; synchronises."""
        self.tkv.lengths()
        if self.dkv is not None:
            self.dkv.lengths()

    def copy_cache_from(self, other: "Engine") -> None:
        """Take over the target cache contents, lengths and pending tokens of an engine of the same shape."""
        assert self.tkv.buf.numel() == other.tkv.buf.numel() and self.batch == other.batch
        self.tkv.buf.copy_(other.tkv.buf)
        self.rows[:, 0] = other.rows[:, 0]
        self.tkv.lengths()

    # ---- prompt pass (functional, untimed) ----
    def prefill(self, prompts: torch.Tensor) -> None:
        """prompts int32 [batch, P] on the device: all but the last token are fed to both caches; the
        last one becomes the pending token."""
        P = prompts.shape[1]
        if P > 1:
            body = prompts[:, :P - 1].contiguous()
            n = torch.full((self.batch,), P - 1, dtype=torch.int32, device=prompts.device)
            B.kv_prefill(self.target, self.tkv, body, n, self._prompt_workspace(self.target, P - 1, self.ws_pre_t))
            if self.dkv is not None:
                B.kv_prefill(self.draft, self.dkv, body, n, self._prompt_workspace(self.draft, P - 1, self.ws_pre_d))
        self.rows[:, 0] = prompts[:, P - 1]
        if self.dkv is not None:
            self.draft_in[:, 0] = prompts[:, P - 1]
            self.draft_n_in.fill_(1)
        self.out_count.zero_()

    def _prompt_workspace(self, model: "B.Model", n_tokens: int, small: torch.Tensor) -> torch.Tensor:
        """Workspace for the prompt pass: from 256 rows per pass a temporary block for the many-row form (up to
        `prompt_ws_cap` bytes, released after the pass), else the few-row workspace."""
        rows = min(n_tokens, 8192 // self.batch)
        while rows * self.batch >= 256:
            nbytes = model.prefill_workspace_bytes(self.batch, rows)
            if nbytes == 0:
                break
            if nbytes <= self.prompt_ws_cap:
                return B.device_buffer(nbytes)
            rows //= 2
        return small

    def set_k(self, k: int) -> None:
        """Draft k <= K tokens in the following iterations: the row block and the q block become [batch, k + 1]
        and [batch, k, V] (views of the buffers sized for K); the pending token moves along."""
        assert 1 <= k <= self.K_max and self.dkv is not None
        if k == self.K:
            return
        if k not in self._rows_of:
            self._rows_of[k] = torch.zeros(self.batch, k + 1, dtype=torch.int32, device=self.rows.device)
        new = self._rows_of[k]
        new[:, 0] = self.rows[:, 0]
        self.rows, self.K = new, k
        self.q = self.q_full[:self.batch * k * self.target.arch.vocab].view(self.batch, k, self.target.arch.vocab)

    # ---- one iteration; u_draft [batch, >= K] (row stride = its width), u_verify [batch, K+1] contiguous, on the device ----
    def spec_iteration(self, u_draft: torch.Tensor, u_verify: torch.Tensor, p_debug: Optional[torch.Tensor] = None):
        K, V = self.K, self.target.arch.vocab
        us = u_draft.stride(0)
        if self.fused_draft:  # the K draft steps as one call: tokens into columns 1.. of the row block, q rows into the q block
            B.draft_steps(self.draft, self.dkv, K, self.draft_in, 2, 2, self.draft_n_in, self.T, u_draft, us,
                          self.rows[:, 1:], K + 1, self.q, K * V, self.ws_d)
        for i in ([] if self.fused_draft else range(K)):
            if i == 0:
                tok_in, stride, rows_in, n_in = self.draft_in, 2, 2, self.draft_n_in
            else:
                tok_in, stride, rows_in, n_in = self.rows[:, i:], K + 1, 1, None
            B.draft_step(self.draft, self.dkv, tok_in, stride, rows_in, n_in, self.T, u_draft[:, i:], us,
                         self.rows[:, i + 1:], K + 1, self.q[:, i], K * V, self.ws_d)
        B.target_verify(self.target, self.tkv, self.rows, K, self.q, u_verify, self.T, self.n_acc, self.next_tok, 1,
                        p_debug, self.ws_t)

    def advance(self) -> None:
        B.spec_advance(self.tkv, self.dkv, self.rows, self.K, self.n_acc, self.next_tok, 1, self.out_tokens,
                       self.out_cap, self.out_count, self.draft_in if self.dkv is not None else None,
                       self.draft_n_in if self.dkv is not None else None)
        self.it += 1

    def ar_step(self, u: torch.Tensor, p_debug: Optional[torch.Tensor] = None) -> None:
        """Plain autoregressive decode step (Eq. 1): one row per sequence, token drawn with u [batch, 1]."""
        assert self.K == 0
        B.target_verify(self.target, self.tkv, self.rows, 0, None, u, self.T, self.n_acc, self.next_tok, 1, p_debug,
                        self.ws_t)
        self.advance()

    # ---- whole generations ----
    def generate(self, prompts: np.ndarray, n_new: int, uniforms: Callable[[int, int], np.ndarray],
                 check_every: int = 4, max_iters: Optional[int] = None, policy: Optional[AdaptiveK] = None) -> Dict:
        """uniforms(seq, iteration) -> fp32 [2K+1] (speculative) or [>=1] (autoregressive, K == 0).
        Runs until every sequence has >= n_new tokens; the host only polls the counters.
        With a policy, the number of draft tokens follows it from iteration to iteration (the accepted counts
        are read back every iteration); the block of uniforms keeps the layout of the largest K: draft draws
        u[0:k], accept tests u[K:K+k], the target's draw u[2K]."""
        if policy is not None:
            return self._generate_adaptive(prompts, n_new, uniforms, policy, max_iters)
        dev = "cuda"
        K = self.K
        self.prefill(torch.from_numpy(np.ascontiguousarray(prompts, np.int32)).to(dev))
        iters = 0
        limit = max_iters if max_iters is not None else n_new
        while iters < limit:
            for _ in range(check_every):
                if iters >= limit:
                    break
                u = np.stack([uniforms(s, iters) for s in range(self.batch)]).astype(np.float32)
                if K == 0:
                    self.ar_step(torch.from_numpy(u[:, :1].copy()).to(dev))
                else:
                    ud = torch.from_numpy(u[:, :K].copy()).to(dev)
                    uv = torch.from_numpy(u[:, K:2 * K + 1].copy()).to(dev)
                    self.spec_iteration(ud, uv)
                    self.advance()
                iters += 1
            if int(self.out_count.min().item()) >= n_new:
                break
        counts = self.out_count.cpu().numpy()
        toks = self.out_tokens.cpu().numpy()
        return {"tokens": [toks[b, :min(n_new, counts[b])].tolist() for b in range(self.batch)],
                "counts": counts, "iterations": iters, "status": self.tkv.status()}

    def _generate_adaptive(self, prompts, n_new, uniforms, policy: AdaptiveK, max_iters) -> Dict:
        dev = "cuda"
        Km = self.K_max
        self.prefill(torch.from_numpy(np.ascontiguousarray(prompts, np.int32)).to(dev))
        iters, ks = 0, []
        limit = max_iters if max_iters is not None else n_new
        while iters < limit:
            k = policy.choose()
            self.set_k(k)
            u = np.stack([uniforms(s, iters) for s in range(self.batch)]).astype(np.float32)
            ud = torch.from_numpy(u[:, :k].copy()).to(dev)
            uv = torch.from_numpy(np.concatenate([u[:, Km:Km + k], u[:, 2 * Km:2 * Km + 1]], axis=1).copy()).to(dev)
            self.spec_iteration(ud, uv)
            acc = self.n_acc.cpu().numpy()
            self.advance()
            policy.update(acc, k)
            ks.append(k)
            iters += 1
            if int(self.out_count.min().item()) >= n_new:
                break
        counts = self.out_count.cpu().numpy()
        toks = self.out_tokens.cpu().numpy()
        return {"tokens": [toks[b, :min(n_new, counts[b])].tolist() for b in range(self.batch)],
                "counts": counts, "iterations": iters, "status": self.tkv.status(), "ks": ks}
