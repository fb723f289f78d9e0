"""Pins for the oracle's generation loops.

What the paper fixes (Section "Autoregressive vs Speculative Sampling"): speculative sampling
gives "the same sampling quality as autoregressive sampling on the target itself".  With
greedy selection that is an exact statement about tokens: speculative greedy output equals
autoregressive greedy output, for any K and ANY draft model, however bad.  The cache protocol
(Section "So, what's the problem?") is pinned by its invariant: after every iteration both
caches equal those of a fresh pass over the committed tokens, the target is fed exactly K+1
rows per iteration, and the draft catches up with 1 or 2 rows.
"""
import numpy as np
import pytest

from oracle import decoder as od
from oracle import sampling, spec
from paper_2311_04951_b200 import synth

TGT = synth.gpt2_like(2, 32, 4, 64, 40, 96)
FAMS = {
    "gpt2": TGT,
    "neox_bf16": synth.neox_like(2, 48, 4, 96, 40),
    "llama_bf16": synth.llama_like(2, 40, 4, 64, 40),
}


def _w(arch, seed, scale=12.0):
    out = []
    for w, name in zip(synth.gen_weights(arch, seed), synth.tensor_names(arch)):
        if w is None or name.endswith("_g"):
            out.append(w)
        elif w.dtype == np.uint16:
            out.append(synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(w) * scale))
        else:
            out.append(w * np.float32(scale))
    return out


def _uniforms(seed, K):
    return lambda it: synth.gen_uniforms(seed, 0, it, 2 * K + 1)


@pytest.mark.parametrize("K", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("draft_kind", ["prefix", "unrelated"])
def test_greedy_speculative_equals_greedy_autoregressive(K, draft_kind):
    ws = _w(TGT, 1)
    target = od.Model(TGT, ws)
    if draft_kind == "prefix":
        d_arch, d_ws = synth.prefix_draft(TGT, ws, 1)
        draft = od.Model(d_arch, d_ws)
    else:  # an adversarial draft: different random weights, shares nothing but the vocabulary
        d_arch = synth.gpt2_like(1, 16, 2, 32, 40, 96)
        draft = od.Model(d_arch, _w(d_arch, 99))
    prompt = synth.gen_prompt(2, 1, 7, TGT.vocab)[0]
    n_new = 30
    ar = spec.autoregressive_generate(target, prompt, n_new, 0.0, _uniforms(3, K), 96)
    sp = spec.speculative_generate(target, draft, prompt, n_new, K, 0.0, _uniforms(3, K), 96)
    assert sp["tokens"] == ar["tokens"]
    assert len(set(ar["tokens"])) > 3            # not a degenerate constant string
    if draft_kind == "prefix":
        assert sum(sp["accepted"]) > 0           # some drafts really are accepted ...
    assert any(a < K for a in sp["accepted"])    # ... and some rejected


@pytest.mark.parametrize("fam", list(FAMS))
def test_cache_protocol_invariants(fam):
    arch = FAMS[fam]
    ws = _w(arch, 4)
    target = od.Model(arch, ws)
    d_arch, d_ws = synth.prefix_draft(arch, ws, 1)
    draft = od.Model(d_arch, d_ws)
    K, n_new, s_max = 3, 24, 64
    prompt = synth.gen_prompt(5, 1, 6, arch.vocab)[0]
    out = spec.speculative_generate(target, draft, prompt, n_new, K, 0.7, _uniforms(6, K), s_max, keep_trace=True)
    x = out["all_tokens"]
    # exactly K+1 target rows per iteration, no more (nothing is recomputed)
    assert out["target_rows"] == out["iterations"] * (K + 1)
    assert set(out["catchups"]) <= {1, 2}
    assert all((c == 2) == (i > 0 and out["accepted"][i - 1] == K) for i, c in enumerate(out["catchups"]))
    # both caches equal a fresh pass over the committed tokens
    tc, dc = out["target_cache"], out["draft_cache"]
    assert tc.len == len(x) - 1 and dc.len in (len(x) - 1, len(x) - 2)
    fresh_t = target.new_cache(s_max)
    fresh_t.feed(x[:tc.len], want_logits=False)
    assert np.array_equal(fresh_t.kv[:, :, :, :tc.len], tc.kv[:, :, :, :tc.len])
    fresh_d = draft.new_cache(s_max)
    fresh_d.feed(x[:dc.len], want_logits=False)
    assert np.array_equal(fresh_d.kv[:, :, :, :dc.len], dc.kv[:, :, :, :dc.len])
    # the emitted string is consistent with the per-iteration records
    rebuilt = list(prompt)
    for t in out["trace"]:
        assert t["n"] == len(rebuilt)
        rebuilt += t["drafts"][:t["a"]] + [t["y"]]
    assert rebuilt == x and out["tokens"] == x[len(prompt):len(prompt) + n_new]
    # each verification row i is the target's next-token distribution after the accepted prefix:
    # check against a full recompute (no cache at all) at one iteration
    t = out["trace"][min(2, len(out["trace"]) - 1)]
    seq = x[:t["n"]] + t["drafts"]
    full = target.forward_full(np.array(seq, np.int32))
    np.testing.assert_allclose(t["logits"], full[t["n"] - 1:], atol=1e-5)


def test_sampled_speculative_is_lockstep_deterministic_and_uses_its_uniform_blocks():
    arch = TGT
    ws = _w(arch, 8)
    target = od.Model(arch, ws)
    d_arch, d_ws = synth.prefix_draft(arch, ws, 1)
    draft = od.Model(d_arch, d_ws)
    prompt = synth.gen_prompt(9, 1, 5, arch.vocab)[0]
    a = spec.speculative_generate(target, draft, prompt, 20, 4, 1.0, _uniforms(10, 4), 64, keep_trace=True)
    b = spec.speculative_generate(target, draft, prompt, 20, 4, 1.0, _uniforms(10, 4), 64)
    assert a["tokens"] == b["tokens"] and len(a["tokens"]) == 20
    for it, t in enumerate(a["trace"]):
        assert np.array_equal(t["u"], synth.gen_uniforms(10, 0, it, 9))
        # the recorded decision is what the rule gives on the recorded rows
        assert sampling.accept_resample(t["p"], t["q"], t["drafts"], t["u"][4:8], t["u"][8]) == (t["a"], t["y"])
    # mean tokens per iteration lies in [1, K+1]
    tpi = (len(a["all_tokens"]) - len(prompt)) / a["iterations"]
    assert 1.0 <= tpi <= 5.0


def test_autoregressive_sampling_distribution_on_a_tiny_vocabulary():
    """AR sampling draws token j from softmax(logits/T): empirical first-token frequencies over a
    grid of uniforms equal the softmax of the model's own logits (Eq. 1 + temperature)."""
    arch = synth.gpt2_like(1, 8, 2, 16, 5, 16)
    ws = _w(arch, 3, scale=30.0)
    target = od.Model(arch, ws)
    prompt = [1, 3]
    logits = target.forward_full(np.array(prompt, np.int32))[-1].astype(np.float64)
    T = 0.7
    ref = np.exp(logits / T - (logits / T).max())
    ref /= ref.sum()
    G = 2000
    counts = np.zeros(arch.vocab)
    for k in range(G):
        u = np.array([(k + 0.5) / G], np.float32)
        counts[spec.autoregressive_generate(target, prompt, 1, T, lambda j: u, 8)["tokens"][0]] += 1
    np.testing.assert_allclose(counts / G, ref, atol=2.0 / G)
