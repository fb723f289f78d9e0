"""Helpers of the GPU parity tests: tolerances and the lock-step trajectory comparison.

Comparison scheme (one flipped decision changes everything after it, so three layers):
  A. distributions: while the GPU and the oracle have seen the same tokens, the p and q rows agree
     within P_ATOL (logits within LOGIT_ATOL + LOGIT_RTOL |ref|);
  B. decisions: the oracle's rule applied to the GPU's OWN rows reproduces the GPU's accepted
     count and tokens exactly, except when u*S sits within 1e-6 S of a CDF step (fp64 sums in a
     different order);
  C. trajectory: tokens agree with the oracle's for as long as they do; after the first
     difference (a decision within tolerance of its threshold) only B continues.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import sampling as osamp

LOGIT_ATOL, LOGIT_RTOL = 2e-2, 1e-2
P_ATOL = 1e-4
# A logit error d moves a probability by a factor e^(+-2d) at most (numerator and normaliser).  On
# models whose weights are scaled up to make the rows peaky, a bf16-weight logit error well inside
# LOGIT_ATOL therefore exceeds 1e-4 absolute on a large p; those comparisons add this relative term.
P_RTOL_PEAKY = 5e-2


class GuardedAllocator:
    """Stand-in for binding.device_buffer: each block sits between two bands of BAND bytes filled with a
    pattern; check() compares every band with the pattern (on the device, one number back per block)."""
    BAND = 8192
    PATTERN = 0xA5

    def __init__(self):
        self.blocks = []

    def alloc(self, nbytes: int) -> torch.Tensor:
        n = max(int(nbytes), 1)
        n_pad = (n + 255) // 256 * 256
        big = torch.empty(n_pad + 2 * self.BAND, dtype=torch.uint8, device="cuda")
        big[:self.BAND] = self.PATTERN
        big[self.BAND + n:] = self.PATTERN
        self.blocks.append((big, n))
        return big[self.BAND:self.BAND + n]

    def check(self) -> None:
        for i, (big, n) in enumerate(self.blocks):
            lo = int((big[:self.BAND] != self.PATTERN).sum().item())
            hi = int((big[self.BAND + n:] != self.PATTERN).sum().item())
            assert lo == 0 and hi == 0, f"block {i} ({n} bytes): {lo} bytes written below it, {hi} above it"


def guarded_like(reg: GuardedAllocator, shape, dtype) -> torch.Tensor:
    """An output tensor of `shape` carved from a guarded block (for arrays the tests allocate themselves)."""
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    return reg.alloc(n).view(dtype).view(*shape)


def assert_probs_close(got, ref, peaky, what=""):
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    bound = P_ATOL + (P_RTOL_PEAKY * ref if peaky else 0.0)
    worst = int(np.argmax(err - bound))
    assert (err <= bound).all(), f"{what}: |dp| {err.flat[worst]:.3e} at p = {ref.flat[worst]:.3e}"


def scaled_weights(synth, arch, seed, scale):
    """Weights scaled up so that attention and logits are far from uniform (every term matters)."""
    out = []
    for w, name in zip(synth.gen_weights(arch, seed), synth.tensor_names(arch)):
        if w is None or name.endswith("_g") or scale == 1.0:
            out.append(w)
        elif w.dtype == np.uint16:
            out.append(synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(w) * scale))
        else:
            out.append(w * np.float32(scale))
    return out


def assert_logits_close(got, ref):
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    bound = LOGIT_ATOL + LOGIT_RTOL * np.abs(ref)
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert (err <= bound).all(), f"logit err {err[worst]:.3e} > bound {bound[worst]:.3e} at {worst}"


def cdf_boundary_near(weights, u, rel=1e-6):
    c = np.cumsum(np.asarray(weights, np.float64))
    S = c[-1]
    if S <= 0:
        return True
    t = float(np.float32(u)) * S
    return bool(np.min(np.abs(c - t)) <= rel * S)


def check_decisions_on_own_rows(p_rows, q_rows, drafts, u_acc, u_res, a_got, y_got):
    """Layer B for one verification.  Returns True if checked exactly, False if excused."""
    K = len(drafts)
    a_ref, y_ref = osamp.accept_resample(p_rows, q_rows, drafts, u_acc, u_res)
    assert a_ref == a_got, f"accepted count {a_got} != rule on the same rows {a_ref}"
    if y_ref == y_got:
        return True
    row = p_rows[a_ref]
    w = osamp.residual(row, q_rows[a_ref]) if a_ref < K else row
    if float(w.astype(np.float64).sum()) <= 0:
        w = row
    assert cdf_boundary_near(w, u_res), f"token {y_got} != rule on the same rows {y_ref}, not at a CDF step"
    return False


def check_draw_on_own_row(q_row, u, tok_got):
    ref = osamp.inv_cdf(q_row, u)
    if ref == tok_got:
        return True
    assert cdf_boundary_near(q_row, u), f"draft token {tok_got} != inverse CDF of its own row {ref}"
    return False


def cdf_flip_excusable(w_gpu, w_ref, u, j_gpu, j_ref):
    """Two inverse-CDF draws with the same uniform picked different indices from two weight rows that
    agree within the row tolerance.  Excusable iff the perturbation of the normalised CDF between the two
    rows (delta = max_j |C_gpu(j) - C_ref(j)|) can carry a CDF step lying between the picks across u."""
    cg = np.cumsum(np.asarray(w_gpu, np.float64))
    cr = np.cumsum(np.asarray(w_ref, np.float64))
    if cg[-1] <= 0 or cr[-1] <= 0:
        return True
    cg, cr = cg / cg[-1], cr / cr[-1]
    delta = float(np.max(np.abs(cg - cr))) + 1e-6
    lo, hi = min(j_gpu, j_ref), max(j_gpu, j_ref)
    uu = float(np.float32(u))
    return bool(np.min(np.abs(cr[lo:hi] - uu)) <= delta)


def accept_flip_excusable(p_x, q_x, u):
    """The accept test u*q(x) < p(x) came out differently: excusable iff the oracle's margin is within the
    probability tolerance (absolute 1e-4 plus 4 % of p for the bf16 logit tolerance)."""
    return abs(float(p_x) - float(np.float32(u) * np.float32(q_x))) <= 1e-4 + 4e-2 * float(p_x)


def resync(engine, x_ref, n_prev, d_prev, n0, t_len, d_len):
    """Bring a batch-1 engine to the oracle's state after an excusable difference: both caches are cut
    back (kv_rollback) to what they held before the iteration (n_prev - 1 target rows, d_prev draft rows),
    the oracle's tokens are fed again (kv_prefill), and the pending token, the draft's catch-up rows and
    the output list are set to the oracle's.  x_ref: all committed tokens of the oracle after the
    iteration; t_len / d_len: its cache lengths."""
    dev = "cuda"
    i32 = lambda v: torch.tensor(v, dtype=torch.int32, device=dev)
    from paper_2311_04951_b200 import binding as B
    B.kv_rollback(engine.tkv, i32([n_prev - 1]))
    B.kv_rollback(engine.dkv, i32([d_prev]))
    for model, kv, ws, a, b in ((engine.target, engine.tkv, engine.ws_pre_t, n_prev - 1, t_len),
                                (engine.draft, engine.dkv, engine.ws_pre_d, d_prev, d_len)):
        if b > a:
            B.kv_prefill(model, kv, i32([x_ref[a:b]]), i32([b - a]), ws)
    n = len(x_ref)
    assert t_len == n - 1 and d_len in (n - 1, n - 2)
    engine.rows[:, 0] = int(x_ref[-1])
    feed = x_ref[d_len:n]
    engine.draft_in[0, :len(feed)] = i32(feed)
    engine.draft_n_in.fill_(len(feed))
    engine.out_count.fill_(n - n0)
    engine.out_tokens[0, :n - n0] = i32(x_ref[n0:n])
    assert engine.tkv.lengths().tolist() == [t_len] and engine.dkv.lengths().tolist() == [d_len]


def lockstep(engine, synth, prompt, n_iters, K, seed_u, oracle_trace, seq=0, peaky=False):
    """Run the oracle's iterations on the GPU engine (batch 1, T > 0) in lock step:
      A. distributions: q rows up to the first differing draft token and p rows conditioned on equal
         drafts agree with the oracle's within the probability tolerance;
      B. decisions: the oracle's rule on the GPU's own rows reproduces the GPU's decisions;
      C. trajectory: every decision (K draft draws, the accept tests up to the first refusal, one draw by
         the target) equals the oracle's, or differs excusably (within tolerance of its threshold); after
         an excusable difference the engine is resynchronised to the oracle's tokens and cache lengths
         (kv_rollback + re-feed) and the comparison goes on to the last iteration.
    Returns {"iterations", "identical", "excused", "decisions"}; any other difference fails."""
    V = engine.target.arch.vocab
    dev = "cuda"
    engine.prefill(torch.from_numpy(np.ascontiguousarray(prompt[None], np.int32)).to(dev))
    p_dbg = torch.zeros(1, K + 1, V, dtype=torch.float32, device=dev)
    n0 = len(prompt)
    x_ref = [int(t) for t in prompt]
    identical = excused = decisions = 0
    for it in range(min(n_iters, len(oracle_trace))):
        t = oracle_trace[it]
        n_prev = len(x_ref)
        assert t["n"] == n_prev
        d_prev = int(engine.dkv.lengths()[0])
        u = synth.gen_uniforms(seed_u, seq, it, 2 * K + 1)
        ud = torch.from_numpy(u[None, :K].copy()).to(dev)
        uv = torch.from_numpy(u[None, K:].copy()).to(dev)
        engine.spec_iteration(ud, uv, p_dbg)
        rows = engine.rows.cpu().numpy()[0]
        a = int(engine.n_acc.cpu().numpy()[0])
        y = int(engine.next_tok.cpu().numpy()[0])
        p = p_dbg.cpu().numpy()[0]
        q = engine.q.cpu().numpy()[0]
        drafts = rows[1:].tolist()
        engine.advance()
        # B: decisions on the GPU's own rows
        for i in range(K):
            check_draw_on_own_row(q[i], u[i], drafts[i])
        check_decisions_on_own_rows(p, q, drafts, u[K:2 * K], u[2 * K], a, y)
        # A + C against the oracle's record of this iteration
        a_ref, y_ref = t["a"], t["y"]
        decisions += K + min(a_ref + 1, K) + 1
        diverged = False
        same_drafts = 0
        for i in range(K):
            assert_probs_close(q[i], t["q"][i], peaky, f"q row {i} of iteration {it}")
            if drafts[i] != t["drafts"][i]:
                assert cdf_flip_excusable(q[i], t["q"][i], u[i], drafts[i], t["drafts"][i]), \
                    f"iteration {it}: draft token {i} is {drafts[i]}, oracle {t['drafts'][i]}: not at a CDF step"
                diverged = True
                break
            same_drafts += 1
        for i in range(same_drafts + 1):      # p row i is conditioned on drafts[:i]
            assert_probs_close(p[i], t["p"][i], peaky, f"p row {i} of iteration {it}")
        if not diverged and a != a_ref:
            i = min(a, a_ref)
            x = t["drafts"][i]
            assert accept_flip_excusable(t["p"][i][x], t["q"][i][x], u[K + i]), \
                f"iteration {it}: accept test {i} differs from the oracle away from its threshold"
            diverged = True
        if not diverged and y != y_ref:
            w_ref = t["p"][a_ref]
            w_gpu = p[a_ref]
            if a_ref < K:
                r_ref = osamp.residual(t["p"][a_ref], t["q"][a_ref])
                if float(r_ref.astype(np.float64).sum()) > 0:
                    w_ref, w_gpu = r_ref, osamp.residual(p[a_ref], q[a_ref])
            assert cdf_flip_excusable(w_gpu, w_ref, u[2 * K], y, y_ref), \
                f"iteration {it}: the target's token is {y}, oracle {y_ref}: not at a CDF step"
            diverged = True
        x_ref.extend(t["drafts"][:a_ref] + [y_ref])
        if diverged:
            excused += 1
            n = len(x_ref)
            resync(engine, x_ref, n_prev, d_prev, n0, n - 1, min(n_prev + a_ref, n_prev + K - 1))
        else:
            identical += 1
    return {"iterations": min(n_iters, len(oracle_trace)), "identical": identical, "excused": excused,
            "decisions": decisions}
