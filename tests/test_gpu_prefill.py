"""Many-row prompt pass (tiled tcgen05 GEMMs + causal attention over the cache) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import decoder as od
from paper_2311_04951_b200 import binding as B, synth
from tests import gpu_util as gu
from tests.test_gpu_forward import ARCHS, gpu_logits

pytestmark = pytest.mark.gpu

BF16 = [n for n, a in ARCHS.items() if a.dtype == synth.DT_BF16]


@pytest.fixture(params=[2, 3], ids=["tc-attention-where-it-applies", "mma-attention"])
def many_row_mode(request):
    B.set_prefill_mode(request.param)
    yield
    B.set_prefill_mode(0)


def _cache_close(arch, got, ref):
    tol = gu.LOGIT_RTOL * np.abs(ref).max(axis=-1, keepdims=True) + gu.LOGIT_ATOL
    bad = np.argwhere(np.abs(got - ref) > tol)
    assert bad.shape[0] == 0, (bad[:8].tolist(), [(float(got[tuple(i)]), float(ref[tuple(i)])) for i in bad[:8]])


def _check_against_oracle(arch, omodel, model, kv, prompts, lens, S):
    Bn = prompts.shape[0]
    assert kv.status() == 0 and kv.lengths().tolist() == lens.tolist()
    rows = synth.gen_prompt(15, Bn, 3, arch.vocab)
    got = gpu_logits(model, kv, model.new_workspace(Bn, 3, S), rows, 2)
    cache = kv.cache_view().float().cpu().numpy()
    for b in range(Bn):
        oc = omodel.new_cache(S)
        oc.feed(prompts[b, :lens[b]], want_logits=False)
        gu.assert_logits_close(got[b], oc.feed(rows[b], advance=False))
        n = int(lens[b])
        _cache_close(arch, cache[:, b, :, :, :n], oc.kv[:, :, :, :n])


@pytest.mark.parametrize("name", BF16)
def test_many_row_prompt_pass_matches_oracle(name, many_row_mode):
    """One pass over ragged prompts: several 128-row GEMM tiles with a ragged last one, several 64-row attention
    tiles per sequence, a sequence that ends inside a tile, one that feeds a single token."""
    arch = ARCHS[name]
    ws_np = gu.scaled_weights(synth, arch, 3, 6.0)
    omodel = od.Model(arch, ws_np)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    P = 150
    if arch.pos == 0:
        P = arch.max_pos - 8
    S = P + 8
    Bn = 3
    lens = np.array([P, P - 67, 1], np.int32)
    prompts = synth.gen_prompt(31, Bn, P, arch.vocab)
    nbytes = model.prefill_workspace_bytes(Bn, P)
    assert nbytes > 0
    kv = B.KV(model, Bn, S)
    n0 = B.launch_count()
    B.kv_prefill(model, kv, torch.from_numpy(prompts).cuda(), torch.from_numpy(lens).cuda(), B.device_buffer(nbytes))
    # one pass: set-up, embedding, and per layer 4 GEMMs + norm(s) + append + attention + activation
    per_layer = 8 if arch.parallel_residual else 9
    assert B.launch_count() - n0 == 1 + 2 + per_layer * arch.n_layers + 1
    _check_against_oracle(arch, omodel, model, kv, prompts, lens, S)


@pytest.mark.parametrize("name", ["llama_bf16", "neox_bf16"])
def test_many_row_prompt_pass_in_several_passes_and_on_a_filled_cache(name, many_row_mode):
    """A workspace that holds only part of the prompt: equal passes, the later ones attending to what the earlier
    ones stored; then a second prompt call that continues the same sequences."""
    arch = ARCHS[name]
    ws_np = gu.scaled_weights(synth, arch, 3, 6.0)
    omodel = od.Model(arch, ws_np)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    Bn, P1, P2 = 2, 200, 45
    S = P1 + P2 + 8
    prompts = synth.gen_prompt(32, Bn, P1 + P2, arch.vocab)
    lens1 = np.array([P1, P1 - 90], np.int32)
    ws = B.device_buffer(model.prefill_workspace_bytes(Bn, 80))      # 200 tokens -> the largest power-of-two share that fits: four passes of 64 rows
    kv = B.KV(model, Bn, S)
    first = np.ascontiguousarray(prompts[:, :P1])
    B.kv_prefill(model, kv, torch.from_numpy(first).cuda(), torch.from_numpy(lens1).cuda(), ws)
    assert kv.status() == 0 and kv.lengths().tolist() == lens1.tolist()
    lens2 = np.array([P2, P2 - 4], np.int32)
    second = np.stack([prompts[b, lens1[b]:lens1[b] + P2] for b in range(Bn)])
    B.kv_prefill(model, kv, torch.from_numpy(np.ascontiguousarray(second)).cuda(), torch.from_numpy(lens2).cuda(), ws)
    total = lens1 + lens2
    _check_against_oracle(arch, omodel, model, kv, prompts, total, S)


def test_many_row_form_is_taken_from_256_rows_and_equals_the_chunked_form():
    """Default mode: 2 x 130 rows take the many-row form (fewer launches than chunks), 2 x 100 do not; both forms
    leave the same cache up to rounding."""
    arch = ARCHS["llama_bf16"]
    ws_np = gu.scaled_weights(synth, arch, 3, 6.0)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    Bn, S = 2, 160
    C = min(B.MAX_ROWS_PER_SEQ, B.MAX_ROWS // Bn)
    caches = {}
    for P in (130, 100):
        prompts = torch.from_numpy(synth.gen_prompt(33, Bn, P, arch.vocab)).cuda()
        lens = torch.full((Bn,), P, dtype=torch.int32, device="cuda")
        big = B.device_buffer(max(model.prefill_workspace_bytes(Bn, P), model.workspace_bytes(Bn, C, S)))
        for mode in (0, 1):
            B.set_prefill_mode(mode)
            try:
                kv = B.KV(model, Bn, S)
                n0 = B.launch_count()
                B.kv_prefill(model, kv, prompts, lens, big)
                caches[(P, mode)] = (kv.cache_view().float().cpu().numpy()[..., :P, :], B.launch_count() - n0)
                assert kv.status() == 0 and kv.lengths().tolist() == [P] * Bn
            finally:
                B.set_prefill_mode(0)
    chunks = lambda P: -(-P // C)
    assert caches[(130, 1)][1] == 3 * chunks(130) and caches[(100, 0)][1] == 3 * chunks(100)
    assert caches[(130, 0)][1] == 1 + 2 + 9 * arch.n_layers + 1
    _cache_close(arch, caches[(130, 0)][0], caches[(130, 1)][0])


def test_prompt_longer_than_the_cache_is_refused(many_row_mode):
    arch = ARCHS["neox_bf16"]
    model = B.Model(arch, B.upload_weights(arch, gu.scaled_weights(synth, arch, 3, 6.0)))
    kv = B.KV(model, 2, 64)
    prompts = torch.from_numpy(synth.gen_prompt(34, 2, 80, arch.vocab)).cuda()
    lens = torch.full((2,), 80, dtype=torch.int32, device="cuda")
    with pytest.raises(B.SsdError):
        B.kv_prefill(model, kv, prompts, lens, B.device_buffer(model.prefill_workspace_bytes(2, 80)))
    assert kv.lengths().tolist() == [0, 0]
