"""GPU parity of the decoder forward against the KV cache: logits of the verification rows,
cache contents, chunked prompt pass, for every block family and both dtypes, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import decoder as od
from paper_2311_04951_b200 import binding as B, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

ARCHS = {
    "gpt2_f32": synth.gpt2_like(2, 128, 4, 256, 300, 96),
    "neox_f32": synth.neox_like(2, 128, 4, 256, 300, dtype=synth.DT_F32),
    "llama_f32": synth.llama_like(2, 128, 2, 192, 300, dtype=synth.DT_F32),
    "gpt2_bf16": synth.gpt2_like(2, 128, 4, 256, 300, 96, dtype=synth.DT_BF16),
    "neox_bf16": synth.neox_like(3, 256, 4, 512, 1000),             # head 64, several 128-row tiles
    "neox_bf16_h80": synth.neox_like(2, 320, 4, 640, 520),          # head 80, ragged vocab tile
    "neox_partial_rotary": synth.neox_like(2, 256, 2, 384, 300).replace(rotary_dim=32),
    "llama_bf16": synth.llama_like(3, 256, 2, 704, 1000),           # head 128, d_ff = 11 x 64
}


def gpu_logits(model, kv, ws, rows_np, K):
    dev = "cuda"
    Bn = rows_np.shape[0]
    rows = torch.from_numpy(rows_np).to(dev)
    V = model.arch.vocab
    q = torch.full((Bn, max(K, 1), V), 1.0 / V, device=dev)
    u = torch.full((Bn, K + 1), 0.5, device=dev)
    n_acc = torch.zeros(Bn, dtype=torch.int32, device=dev)
    nxt = torch.zeros(Bn, dtype=torch.int32, device=dev)
    B.target_verify(model, kv, rows, K, q if K else None, u, 1.0, n_acc, nxt, 1, None, ws)
    out = B.last_logits(model, Bn, K + 1, ws)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("name", list(ARCHS))
def test_verify_rows_logits_and_cache_match_oracle(name):
    arch = ARCHS[name]
    ws_np = gu.scaled_weights(synth, arch, 3, 6.0)
    omodel = od.Model(arch, ws_np)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    Bn, S, P, K = 2, 48, 11, 4
    prompts = synth.gen_prompt(4, Bn, P, arch.vocab)
    lens = np.array([P, P - 4], np.int32)                         # ragged prompt lengths
    kv = B.KV(model, Bn, S)
    ws = model.new_workspace(Bn, 8, S)
    dev = "cuda"
    B.kv_prefill(model, kv, torch.from_numpy(prompts).to(dev), torch.from_numpy(lens).to(dev), ws)
    assert kv.lengths().tolist() == lens.tolist()
    rows = synth.gen_prompt(5, Bn, K + 1, arch.vocab)
    got = gpu_logits(model, kv, ws, rows, K)
    assert kv.status() == 0
    assert kv.lengths().tolist() == lens.tolist()                 # verify does not commit
    cache = kv.cache_view().float().cpu().numpy()
    for b in range(Bn):
        oc = omodel.new_cache(S)
        oc.feed(prompts[b, :lens[b]], want_logits=False)
        ref = oc.feed(rows[b], advance=False)
        assert np.abs(ref).max() > 0.5
        gu.assert_logits_close(got[b], ref)
        n = lens[b] + K + 1
        # keys/values: same numbers up to fp32 summation order (one bf16 step where rounding flips)
        g, r = cache[:, b, :, :, :n], oc.kv[:, :, :, :n]
        tol = gu.LOGIT_RTOL * np.abs(r) + gu.LOGIT_ATOL if arch.dtype else 1e-4
        assert (np.abs(g - r) <= tol).all()
        if arch.dtype:
            assert (g == r).mean() > 0.9
    # commit 3 rows of sequence 0 and 1 of sequence 1, then feed one more row: positions follow
    B.kv_commit(kv, torch.tensor([3, 1], dtype=torch.int32, device=dev))
    assert kv.lengths().tolist() == (lens + np.array([3, 1])).tolist()
    rows2 = synth.gen_prompt(6, Bn, 1, arch.vocab)
    got2 = gpu_logits(model, kv, ws_single(model, Bn, S), rows2, 0)
    for b, keep in enumerate((3, 1)):
        oc = omodel.new_cache(S)
        oc.feed(np.concatenate([prompts[b, :lens[b]], rows[b, :keep]]), want_logits=False)
        gu.assert_logits_close(got2[b], oc.feed(rows2[b], advance=False))


def ws_single(model, Bn, S):
    return model.new_workspace(Bn, 1, S)


def test_row_results_do_not_depend_on_how_many_rows_are_fed():
    """K candidate rows in one pass give the same logits as feeding them one at a time (the claim
    that lets verification replace K decode steps)."""
    arch = ARCHS["llama_bf16"]
    ws_np = gu.scaled_weights(synth, arch, 9, 6.0)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    S, K = 32, 5
    rows = synth.gen_prompt(7, 1, K + 1, arch.vocab)
    kv = B.KV(model, 1, S)
    together = gpu_logits(model, kv, model.new_workspace(1, K + 1, S), rows, K)[0]
    kv2 = B.KV(model, 1, S)
    ws1 = model.new_workspace(1, 1, S)
    one = torch.ones(1, dtype=torch.int32, device="cuda")
    for i in range(K + 1):
        single = gpu_logits(model, kv2, ws1, rows[:, i:i + 1], 0)[0, 0]
        B.kv_commit(kv2, one)
        assert np.abs(single - together[i]).max() <= 5e-3       # same math, fp32 reduction order only


def test_capacity_and_argument_errors():
    arch = ARCHS["gpt2_f32"]
    model = B.Model(arch, B.upload_weights(arch, synth.gen_weights(arch, 1)))
    dev = "cuda"
    kv = B.KV(model, 1, 8)
    ws = model.new_workspace(1, 8, 8)
    # prompt longer than the cache: refused on the host
    with pytest.raises(B.SsdError) as e:
        B.kv_prefill(model, kv, torch.zeros(1, 9, dtype=torch.int32, device=dev),
                     torch.tensor([9], dtype=torch.int32, device=dev), ws)
    assert e.value.code == -3
    B.kv_prefill(model, kv, torch.zeros(1, 6, dtype=torch.int32, device=dev),
                 torch.tensor([6], dtype=torch.int32, device=dev), ws)
    # 4 more rows do not fit 8: the device records it, feeds nothing and the lengths stay
    rows = torch.zeros(1, 4, dtype=torch.int32, device=dev)
    z = torch.zeros(4, dtype=torch.int32, device=dev)
    f = torch.full((1, 3, arch.vocab), 1.0 / arch.vocab, device=dev)
    B.target_verify(model, kv, rows, 3, f, torch.zeros(1, 4, device=dev), 1.0, z, z[1:], 1, None, ws)
    assert kv.status() == -3 and kv.lengths().tolist() == [6]
    # workspace too small / rows beyond the limits
    with pytest.raises(B.SsdError):
        B.target_verify(model, kv, rows, 3, f, torch.zeros(1, 4, device=dev), 1.0, z, z, 1, None, ws[:1024])
    assert model.workspace_bytes(8, 9, 8) == 0 and model.workspace_bytes(1, 33, 8) == 0
    # unsupported architectures are refused at creation
    bad = arch.replace(n_heads=3)
    with pytest.raises(B.SsdError) as e:
        B.Model(bad, B.upload_weights(arch, synth.gen_weights(arch, 1)))
    assert e.value.code == -2


@pytest.mark.parametrize("name", ["neox_bf16", "llama_bf16", "gpt2_bf16", "neox_bf16_h80"])
def test_single_kernel_forward_equals_stepwise_forward(name):
    """The whole-forward cooperative kernel and the one-launch-per-step path compute the same
    logits and cache rows (same arithmetic; only the fp32 reduction order differs)."""
    arch = ARCHS[name]
    ws_np = gu.scaled_weights(synth, arch, 3, 6.0)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    Bn, S, K = 2, 64, 4
    prompts = synth.gen_prompt(4, Bn, 20, arch.vocab)
    rows = synth.gen_prompt(5, Bn, K + 1, arch.vocab)
    res = []
    for persistent in (True, False):
        B.set_persistent(persistent)
        try:
            kv = B.KV(model, Bn, S)
            ws = model.new_workspace(Bn, 8, S)
            B.kv_prefill(model, kv, torch.from_numpy(prompts).to("cuda"),
                         torch.tensor([20, 13], dtype=torch.int32, device="cuda"), ws)
            lg = gpu_logits(model, kv, ws, rows, K)
            assert kv.status() == 0
            res.append((lg, kv.cache_view().float().cpu().numpy()))
        finally:
            B.set_persistent(True)
    assert np.abs(res[0][0] - res[1][0]).max() < 1e-2
    for b, n in enumerate((20 + K + 1, 13 + K + 1)):
        a, c = res[0][1][:, b, :, :, :n], res[1][1][:, b, :, :, :n]
        assert (np.abs(a - c) <= gu.LOGIT_RTOL * np.abs(c) + gu.LOGIT_ATOL).all()


@pytest.mark.parametrize("Bn,M", [(1, 9), (1, 17), (3, 11), (8, 5), (2, 32), (8, 8)])
def test_row_counts_of_the_single_kernel_gemms(Bn, M):
    """The forward kernel is instantiated per padded row count (8, 16, 24, 32, 40, 64 rows: operand tiles of
    1-8 blocks, MMA M = 64 up to 32 rows and 128 beyond, ring stages of 34-48 KB).  One verification pass of
    Bn x M rows per variant, logits against the oracle."""
    arch = ARCHS["neox_bf16"]
    ws_np = gu.scaled_weights(synth, arch, 21, 6.0)
    omodel = od.Model(arch, ws_np)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    S, P = 64, 7
    prompts = synth.gen_prompt(22, Bn, P, arch.vocab)
    kv = B.KV(model, Bn, S)
    ws = model.new_workspace(Bn, max(M, 8), S)
    dev = "cuda"
    B.kv_prefill(model, kv, torch.from_numpy(prompts).to(dev), torch.full((Bn,), P, dtype=torch.int32, device=dev), ws)
    rows = synth.gen_prompt(23, Bn, M, arch.vocab)
    got = gpu_logits(model, kv, ws, rows, M - 1)
    assert kv.status() == 0
    for b in range(Bn):
        oc = omodel.new_cache(S)
        oc.feed(prompts[b], want_logits=False)
        gu.assert_logits_close(got[b], oc.feed(rows[b], advance=False))


@pytest.mark.parametrize("name,Bn", [("llama_bf16", 2), ("neox_bf16", 1), ("gpt2_f32", 3)])
def test_prompt_pass_in_large_chunks_matches_oracle(name, Bn):
    """kv_prefill with a workspace for 32 (or 64 / batch) rows per sequence: chunks of up to 32 rows, two 16-row
    attention tiles, ragged prompt lengths that end inside a chunk; cache rows and a following verification pass
    against the oracle."""
    arch = ARCHS[name]
    ws_np = gu.scaled_weights(synth, arch, 3, 6.0)
    omodel = od.Model(arch, ws_np)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    S, P = 96, 70
    if arch.pos == 0:
        S = P = min(S, arch.max_pos) - 8
        S += 8
    lens = np.array([P, P - 33, 5][:Bn], np.int32)
    prompts = synth.gen_prompt(14, Bn, P, arch.vocab)
    C = min(B.MAX_ROWS_PER_SEQ, B.MAX_ROWS // Bn)
    kv = B.KV(model, Bn, S)
    dev = "cuda"
    B.kv_prefill(model, kv, torch.from_numpy(prompts).to(dev), torch.from_numpy(lens).to(dev), model.new_workspace(Bn, C, S))
    assert kv.status() == 0 and kv.lengths().tolist() == lens.tolist()
    rows = synth.gen_prompt(15, Bn, 3, arch.vocab)
    got = gpu_logits(model, kv, model.new_workspace(Bn, 3, S), rows, 2)
    cache = kv.cache_view().float().cpu().numpy()
    for b in range(Bn):
        oc = omodel.new_cache(S)
        oc.feed(prompts[b, :lens[b]], want_logits=False)
        gu.assert_logits_close(got[b], oc.feed(rows[b], advance=False))
        n = int(lens[b])
        g, r = cache[:, b, :, :, :n], oc.kv[:, :, :, :n]
        # (layer-2 rows of these scaled-up models carry the bf16 roundings of two layers of cached keys / values, which
        #  differ between 32-row and 1-row passes: the relative term is taken against the row's largest entry)
        tol = gu.LOGIT_RTOL * np.abs(r).max(axis=-1, keepdims=True) + gu.LOGIT_ATOL if arch.dtype else 1e-4
        bad = np.argwhere(np.abs(g - r) > tol)
        assert bad.shape[0] == 0, (b, bad[:8].tolist(), [(float(g[tuple(i)]), float(r[tuple(i)])) for i in bad[:8]])
