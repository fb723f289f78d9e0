"""Pins for the oracle's decoder forward.

 * GPT-2-like family, whole model: equals torch's own ``nn.TransformerEncoderLayer``
   (norm_first, erf-GELU, causal mask) + embeddings + tied LM head in float64 -- a library
   routine, not a restatement.
 * NeoX / Llama families: reduce to the pinned sequential block when one branch is switched
   off; parallel residual is additive in its branches; SwiGLU / RMSNorm / rotary enter through
   primitives pinned on their own plus the structural invariants below.
 * What the paper fixes: KV caching changes nothing ("poses no risk to accuracy") -- cached
   logits equal full-recompute logits at every position, in any chunking, also after a
   rollback; and position n's logits depend on tokens 1..n only (Eq. 1).
"""
import numpy as np
import pytest
import torch
import torch.nn as nn
import torch.nn.functional as F

from oracle import decoder as od
from paper_2311_04951_b200 import synth

SMALL = {
    "gpt2": synth.gpt2_like(2, 32, 4, 64, 50, 40),
    "neox": synth.neox_like(2, 48, 4, 96, 60, dtype=synth.DT_F32),
    "neox_bf16": synth.neox_like(2, 48, 4, 96, 60),
    "llama": synth.llama_like(2, 40, 4, 64, 55, dtype=synth.DT_F32),
    "llama_bf16": synth.llama_like(2, 40, 4, 64, 55),
    "neox_partial_rotary": synth.neox_like(1, 64, 4, 64, 30, dtype=synth.DT_F32).replace(rotary_dim=8),
}


def big_weights(arch, seed):
    """Weights with std 0.02 give near-zero attention logits; scale them up so that every term
    of the block matters in the comparisons."""
    ws = synth.gen_weights(arch, seed)
    out = []
    for w, name in zip(ws, synth.tensor_names(arch)):
        if w is None:
            out.append(None)
            continue
        if name.endswith("_g"):
            out.append(w)
        elif w.dtype == np.uint16:
            out.append(synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(w) * 8))
        else:
            out.append(w * np.float32(8))
    return out


def tokens(n, vocab, seed=5):
    return np.random.default_rng(seed).integers(0, vocab, n).astype(np.int32)


def test_gpt2_family_matches_torch_transformer_layers():
    a = SMALL["gpt2"]
    ws = big_weights(a, 3)
    names = synth.tensor_names(a)
    W = {n: (None if w is None else torch.from_numpy(w).double()) for n, w in zip(names, ws)}
    layers = []
    for l in range(a.n_layers):
        lay = nn.TransformerEncoderLayer(a.d_model, a.n_heads, a.d_ff, dropout=0.0, activation=F.gelu,
                                         layer_norm_eps=a.norm_eps, batch_first=True, norm_first=True).double()
        sd = {"self_attn.in_proj_weight": W[f"l{l}.w_qkv"], "self_attn.in_proj_bias": W[f"l{l}.b_qkv"],
              "self_attn.out_proj.weight": W[f"l{l}.w_o"], "self_attn.out_proj.bias": W[f"l{l}.b_o"],
              "linear1.weight": W[f"l{l}.w_in"], "linear1.bias": W[f"l{l}.b_in"],
              "linear2.weight": W[f"l{l}.w_out"], "linear2.bias": W[f"l{l}.b_out"],
              "norm1.weight": W[f"l{l}.ln1_g"], "norm1.bias": W[f"l{l}.ln1_b"],
              "norm2.weight": W[f"l{l}.ln2_g"], "norm2.bias": W[f"l{l}.ln2_b"]}
        lay.load_state_dict(sd)
        lay.train()  # dropout is 0; train mode keeps torch on its plain (non-fused) path
        layers.append(lay)
    n = 11
    tok = tokens(n, a.vocab)
    x = F.embedding(torch.from_numpy(tok).long(), W["tok_emb"]) + W["pos_emb"][:n]
    mask = nn.Transformer.generate_square_subsequent_mask(n, dtype=torch.float64)
    x = x[None]
    with torch.no_grad():
        for lay in layers:
            x = lay(x, src_mask=mask, is_causal=True)
        x = F.layer_norm(x[0], (a.d_model,), W["lnf_g"], W["lnf_b"], a.norm_eps)
        ref = (x @ W["tok_emb"].T).numpy()
    got = od.Model(a, ws).forward_full(tok)
    assert np.abs(ref).max() > 0.5          # the comparison is not vacuous
    np.testing.assert_allclose(got, ref, atol=5e-5, rtol=0)


def test_hand_case_one_layer_two_dims():
    """d=2, one head, all matrices zero except the embedding: attention and MLP output their
    biases, so logits = LN(e + b_o + b_out) E^T, computed by hand below."""
    a = synth.gpt2_like(1, 2, 1, 2, 3, 4)
    ws = [None if s is None else np.zeros(s, np.float32)
          for s in (synth.tensor_shape(a, n) for n in synth.tensor_names(a))]
    names = synth.tensor_names(a)
    ix = {n: i for i, n in enumerate(names)}
    ws[ix["tok_emb"]] = np.array([[1, 0], [0, 2], [3, 3]], np.float32)
    ws[ix["l0.b_o"]] = np.array([0.5, 0.0], np.float32)
    ws[ix["l0.b_out"]] = np.array([0.0, -1.0], np.float32)
    for g in ("l0.ln1_g", "l0.ln2_g", "lnf_g"):
        ws[ix[g]] = np.ones(2, np.float32)
    got = od.Model(a.replace(norm_eps=0.0), ws).forward_full(np.array([1], np.int32))
    # x = e_1 + (0.5, 0) + (0, -1) = (0.5, 1): LayerNorm of two numbers with eps 0 is (-1, +1)
    # logits = (-1, 1) . rows of E = (-1, 2, 0)
    np.testing.assert_allclose(got[0], [-1.0, 2.0, 0.0], atol=1e-6)


@pytest.mark.parametrize("fam", list(SMALL))
def test_cached_equals_full_recompute_in_any_chunking(fam):
    a = SMALL[fam]
    ws = big_weights(a, 7)
    m = od.Model(a, ws)
    n = 14
    tok = tokens(n, a.vocab, 9)
    full = m.forward_full(tok)
    assert np.abs(full).max() > 0.3
    for chunks in ([1] * n, [5, 1, 4, 4], [n], [2, 12]):
        c = m.new_cache(20)
        rows, p = [], 0
        for k in chunks:
            rows.append(c.feed(tok[p:p + k]))
            p += k
        got = np.concatenate(rows)
        np.testing.assert_allclose(got, full, atol=1e-5, rtol=0)


@pytest.mark.parametrize("fam", ["gpt2", "neox_bf16", "llama_bf16"])
def test_rollback_then_refeed_equals_fresh_prefill(fam):
    """Rejected rows are dropped by length only; what is fed afterwards overwrites them, and the
    committed part of the cache equals that of a fresh pass over the committed tokens."""
    a = SMALL[fam]
    m = od.Model(a, big_weights(a, 8))
    tok = tokens(12, a.vocab, 4)
    other = tokens(5, a.vocab, 6)
    c = m.new_cache(24)
    c.feed(tok[:6])
    c.feed(other, advance=False)        # tentative rows, never committed
    c.feed(other[:2])                   # 2 committed, then cut them again
    c.rollback(6)
    late = c.feed(tok[6:])
    ref = m.new_cache(24)
    ref_logits = ref.feed(tok)
    np.testing.assert_allclose(late, ref_logits[6:], atol=1e-6, rtol=0)
    assert np.array_equal(c.kv[:, :, :, :12], ref.kv[:, :, :, :12])


@pytest.mark.parametrize("fam", ["gpt2", "neox", "llama"])
def test_logits_depend_on_the_prefix_only(fam):
    a = SMALL[fam]
    m = od.Model(a, big_weights(a, 2))
    tok = tokens(10, a.vocab, 1)
    base = m.forward_full(tok)
    tok2 = tok.copy()
    tok2[6] = (tok2[6] + 1) % a.vocab
    alt = m.forward_full(tok2)
    assert np.array_equal(base[:6], alt[:6])
    assert np.abs(base[6:] - alt[6:]).max() > 1e-3


def _zeroed(arch, ws, which):
    names = synth.tensor_names(arch)
    out = list(ws)
    for i, n in enumerate(names):
        if n.split(".")[-1] in which and out[i] is not None:
            out[i] = np.zeros_like(out[i])
    return out


def test_parallel_residual_is_the_sum_of_its_branches():
    """With one branch's output projection zeroed the parallel block and the (torch-pinned)
    sequential block coincide; with both on, the parallel block adds the two branch outputs
    computed from the SAME input."""
    par = SMALL["neox"].replace(n_layers=1)
    seq = par.replace(parallel_residual=0)
    ws = big_weights(par, 5)
    tok = tokens(9, par.vocab, 3)
    attn_only = _zeroed(par, ws, ("w_out", "b_out"))
    mlp_only = _zeroed(par, ws, ("w_o", "b_o"))
    a_par = od.Model(par, attn_only).forward_full(tok)
    a_seq = od.Model(seq, attn_only).forward_full(tok)
    np.testing.assert_allclose(a_par, a_seq, atol=1e-6)
    m_par = od.Model(par, mlp_only).forward_full(tok)
    m_seq = od.Model(seq, mlp_only).forward_full(tok)
    np.testing.assert_allclose(m_par, m_seq, atol=1e-6)
    # and the two wirings do differ when both branches are on
    assert np.abs(od.Model(par, ws).forward_full(tok) - od.Model(seq, ws).forward_full(tok)).max() > 1e-3


def test_swiglu_mlp_against_torch_silu_and_matmul():
    """Llama family, one layer, attention switched off: logits = RMS(x + W_d(silu(W_g h) * (W_u h)))
    W_lm^T with h = RMS(x): assembled from torch library calls in float64."""
    a = SMALL["llama"].replace(n_layers=1)
    ws = _zeroed(a, big_weights(a, 12), ("w_o",))
    names = synth.tensor_names(a)
    W = {n: (None if w is None else torch.from_numpy(w).double()) for n, w in zip(names, ws)}
    tok = tokens(6, a.vocab, 2)
    x = F.embedding(torch.from_numpy(tok).long(), W["tok_emb"])
    h = F.rms_norm(x, (a.d_model,), W["l0.ln2_g"], a.norm_eps)
    gu = h @ W["l0.w_in"].T
    gate, up = gu[:, :a.d_ff], gu[:, a.d_ff:]
    x = x + (F.silu(gate) * up) @ W["l0.w_out"].T
    ref = (F.rms_norm(x, (a.d_model,), W["lnf_g"], a.norm_eps) @ W["w_lm"].T).numpy()
    got = od.Model(a, ws).forward_full(tok)
    np.testing.assert_allclose(got, ref, atol=5e-5)


def test_rotary_attention_block_against_sdpa():
    """NeoX family, one layer, MLP switched off, rotary positions: q and k turned by the pinned
    rotary primitive, then torch's scaled_dot_product_attention with a causal mask."""
    a = SMALL["neox"].replace(n_layers=1)
    ws = _zeroed(a, big_weights(a, 13), ("w_out", "b_out"))
    names = synth.tensor_names(a)
    W = {n: (None if w is None else torch.from_numpy(w).double()) for n, w in zip(names, ws)}
    n, d, H, Dh = 8, a.d_model, a.n_heads, a.head_dim
    tok = tokens(n, a.vocab, 7)
    x = F.embedding(torch.from_numpy(tok).long(), W["tok_emb"])
    h = F.layer_norm(x, (d,), W["l0.ln1_g"], W["l0.ln1_b"], a.norm_eps)
    qkv = h @ W["l0.w_qkv"].T + W["l0.b_qkv"]
    q, k, v = [t.reshape(n, H, Dh).clone() for t in (qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:])]
    for r in range(n):
        for hh in range(H):
            q[r, hh] = torch.from_numpy(od.rotary(q[r, hh].float().numpy(), a.rotary_dim, r)).double()
            k[r, hh] = torch.from_numpy(od.rotary(k[r, hh].float().numpy(), a.rotary_dim, r)).double()
    o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                       v.transpose(0, 1)[None], is_causal=True)[0].transpose(0, 1).reshape(n, d)
    x = x + o @ W["l0.w_o"].T + W["l0.b_o"]
    ref = (F.layer_norm(x, (d,), W["lnf_g"], W["lnf_b"], a.norm_eps) @ W["w_lm"].T).numpy()
    got = od.Model(a, ws).forward_full(tok)
    np.testing.assert_allclose(got, ref, atol=2e-4)   # q,k pass through fp32 in the rotary primitive


def test_bf16_cache_rounding_is_applied_to_k_and_v_only():
    a = SMALL["llama_bf16"]
    m = od.Model(a, big_weights(a, 4))
    c = m.new_cache(8)
    c.feed(tokens(5, a.vocab, 1))
    kv = c.kv[:, :, :, :5]
    rounded = torch.from_numpy(kv).bfloat16().float().numpy()
    assert np.array_equal(kv, rounded) and np.abs(kv).max() > 0


@pytest.mark.parametrize("fam", ["gpt2", "llama"])
def test_bf16_embedding_and_lm_head_reads(fam):
    """bf16 matrices reach the oracle as uint16 bit patterns.  With every layer matrix and bias zeroed the
    residual stream is the embedding row (+ learned position row), so the logits are
    norm(E[tok] (+ P[pos])) . W_lm^T: written out here in float64 from the widened bit patterns, which pins the
    bf16 branch of the embedding read, of the position table and of the LM head (tied and untied)."""
    arch = synth.gpt2_like(2, 64, 4, 128, 97, 16, dtype=synth.DT_BF16) if fam == "gpt2" else synth.llama_like(2, 64, 2, 96, 97)
    ws = synth.gen_weights(arch, 5)
    for i, n in enumerate(synth.tensor_names(arch)):
        base = n.split(".")[-1]
        if "." in n and ws[i] is not None and not base.endswith("_g"):
            ws[i] = np.zeros_like(ws[i])          # all layer matrices and biases (bf16 zero is the zero pattern)
    toks = np.array([3, 96, 0, 41, 3], np.int32)
    got = od.Model(arch, ws).forward_full(toks)
    names = synth.tensor_names(arch)
    f = lambda n: None if ws[names.index(n)] is None else (
        synth.bf16_bits_to_f32(ws[names.index(n)]).astype(np.float64) if ws[names.index(n)].dtype == np.uint16
        else ws[names.index(n)].astype(np.float64))
    E, P, g, b = f("tok_emb"), f("pos_emb"), f("lnf_g"), f("lnf_b")
    W = E if arch.tie_lm_head else f("w_lm")
    for i, t in enumerate(toks):
        x = E[t] + (P[i] if P is not None else 0.0)
        x = x.astype(np.float32).astype(np.float64)            # the residual stream is stored in fp32
        if arch.norm == synth.NORM_LAYERNORM:
            y = (x - x.mean()) / np.sqrt(x.var() + arch.norm_eps) * g + b
        else:
            y = x / np.sqrt((x * x).mean() + arch.norm_eps) * g
        ref = W @ y.astype(np.float32).astype(np.float64)
        assert np.abs(got[i] - ref).max() <= 1e-5 * max(1.0, np.abs(ref).max()), (fam, i)
    assert np.abs(got).max() > 1e-3
