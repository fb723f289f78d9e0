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


def lockstep(engine, synth, prompt, n_iters, K, seed_u, oracle_trace, seq=0, peaky=False):
    """Run n_iters speculative iterations on the GPU engine (batch 1), checking layers A-C against
    the oracle's per-iteration records.  Returns (#iterations in sync, #iterations run)."""
    V = engine.target.arch.vocab
    dev = "cuda"
    engine.prefill(torch.from_numpy(np.ascontiguousarray(prompt[None], np.int32)).to(dev))
    p_dbg = torch.zeros(1, K + 1, V, dtype=torch.float32, device=dev)
    synced, in_sync = 0, True
    for it in range(n_iters):
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
        # A + C while the contexts coincide
        if in_sync and it < len(oracle_trace):
            t = oracle_trace[it]
            same_drafts = 0
            for i in range(K):
                assert_probs_close(q[i], t["q"][i], peaky, f"q row {i} of iteration {it}")
                if drafts[i] != t["drafts"][i]:
                    break
                same_drafts += 1
            # p row i is conditioned on drafts[:i]: comparable while those coincide
            for i in range(same_drafts + 1):
                assert_probs_close(p[i], t["p"][i], peaky, f"p row {i} of iteration {it}")
            if same_drafts == K and a == t["a"] and y == t["y"]:
                synced += 1
            else:
                in_sync = False
    return synced, n_iters
