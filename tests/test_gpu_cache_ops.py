"""GPU tests of the cache bookkeeping calls through the C ABI: kv_rollback (cut back, feed other tokens,
compare with the oracle and with a fresh prompt pass), the capacity clamp of kv_commit, the host-side
length bound that follows the device without a synchronisation, and the failure-detection probe."""
import numpy as np
import pytest
import torch

from oracle import decoder as od
from paper_2311_04951_b200 import binding as B, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _i32(v):
    return torch.tensor(v, dtype=torch.int32, device="cuda")


def _verify(model, kv, ws, rows_np, K):
    Bn, V = rows_np.shape[0], model.arch.vocab
    q = torch.full((Bn, max(K, 1), V), 1.0 / V, device="cuda")
    u = torch.full((Bn, K + 1), 0.5, device="cuda")
    n_acc, nxt = _i32([0] * Bn), _i32([0] * Bn)
    B.target_verify(model, kv, torch.from_numpy(rows_np).cuda(), K, q if K else None, u, 1.0, n_acc, nxt, 1, None, ws)
    return B.last_logits(model, Bn, K + 1, ws).cpu().numpy()


@pytest.mark.parametrize("name,arch", [
    ("llama_bf16", synth.llama_like(3, 256, 2, 704, 640)),
    ("neox_bf16", synth.neox_like(2, 256, 4, 512, 640)),
    ("gpt2_f32", synth.gpt2_like(2, 128, 4, 256, 400, 96)),
])
def test_rollback_then_refeed_matches_oracle_and_fresh_prompt_pass(name, arch):
    """Three sequences with ragged prompts: a verification pass, some rows committed, then kv_rollback to
    an earlier length per sequence (one of them below its prompt, one unchanged because the new length is
    larger), other tokens fed, another verification pass.  Logits and cache rows must equal the oracle's
    rollback + feed, and the committed rows must equal those of a fresh prompt pass over the same tokens
    (the cache invariant: what lies below the length is the cache of the committed tokens)."""
    ws_np = gu.scaled_weights(synth, arch, 61, 6.0)
    model, omodel = B.Model(arch, B.upload_weights(arch, ws_np)), od.Model(arch, ws_np)
    Bn, S, K = 3, 64, 4
    P = [13, 9, 11]
    prompts = synth.gen_prompt(62, Bn, max(P), arch.vocab)
    kv = B.KV(model, Bn, S)
    ws = model.new_workspace(Bn, 8, S)
    B.kv_prefill(model, kv, torch.from_numpy(prompts).cuda(), _i32(P), ws)
    rows1 = synth.gen_prompt(63, Bn, K + 1, arch.vocab)
    _verify(model, kv, ws, rows1, K)
    keep = [3, 5, 1]
    B.kv_commit(kv, _i32(keep))
    assert kv.lengths().tolist() == [p + k for p, k in zip(P, keep)]
    new_len = [14, 6, 40]                 # cut into the committed rows / into the prompt / no cut (beyond the length)
    B.kv_rollback(kv, _i32(new_len))
    after = [min(p + k, n) for p, k, n in zip(P, keep, new_len)]
    assert kv.lengths().tolist() == after
    other = synth.gen_prompt(64, Bn, 6, arch.vocab)
    n_other = [6, 2, 4]
    B.kv_prefill(model, kv, torch.from_numpy(other).cuda(), _i32(n_other), ws)
    final = [a + n for a, n in zip(after, n_other)]
    assert kv.lengths().tolist() == final
    rows2 = synth.gen_prompt(65, Bn, K + 1, arch.vocab)
    got = _verify(model, kv, ws, rows2, K)
    assert kv.status() == 0
    cache = kv.cache_view().float().cpu().numpy()
    # the same cache from a fresh prompt pass over the committed tokens
    committed = []
    for b in range(Bn):
        seq = np.concatenate([prompts[b, :P[b]], rows1[b, :keep[b]]])[:after[b]]
        committed.append(np.concatenate([seq, other[b, :n_other[b]]]).astype(np.int32))
    kv2 = B.KV(model, Bn, S)
    toks = np.zeros((Bn, max(final)), np.int32)
    for b in range(Bn):
        toks[b, :final[b]] = committed[b]
    B.kv_prefill(model, kv2, torch.from_numpy(toks).cuda(), _i32(final), ws)
    cache2 = kv2.cache_view().float().cpu().numpy()
    tol_c = (lambda r: gu.LOGIT_RTOL * np.abs(r) + gu.LOGIT_ATOL) if arch.dtype else (lambda r: 1e-4)
    for b in range(Bn):
        oc = omodel.new_cache(S)
        oc.feed(np.concatenate([prompts[b, :P[b]], rows1[b, :keep[b]]]), want_logits=False)
        oc.rollback(after[b])
        oc.feed(other[b, :n_other[b]], want_logits=False)
        assert oc.len == final[b]
        ref = oc.feed(rows2[b], advance=False)
        gu.assert_logits_close(got[b], ref)
        n = final[b]
        g, r, f = cache[:, b, :, :, :n], oc.kv[:, :, :, :n], cache2[:, b, :, :, :n]
        assert (np.abs(g - r) <= tol_c(r)).all()
        # cut + re-feed versus fresh pass: the same kernels on the same tokens (rows may sit in other chunks)
        assert (np.abs(g - f) <= tol_c(f)).all()
        assert (g == f).mean() > 0.9


def test_commit_beyond_the_capacity_is_clamped_and_reported():
    arch = synth.llama_like(1, 128, 1, 128, 128)
    model = B.Model(arch, B.upload_weights(arch, synth.gen_weights(arch, 1)))
    kv = B.KV(model, 2, 32)
    B.kv_commit(kv, _i32([10, 31]))
    assert kv.status() == 0 and kv.lengths().tolist() == [10, 31]
    B.kv_commit(kv, _i32([1, 5]))              # sequence 1 would reach 36 > 32
    assert kv.lengths().tolist() == [11, 32]
    assert kv.status() == -3


def test_length_bound_follows_rejections_without_a_synchronisation():
    """Twenty iterations in which every draft is refused (q puts all its mass on the draft token, the
    target far less): the lengths grow by one per iteration although each pass appends K + 1 = 8 rows.
    The host never reads the lengths back, only lets the stream drain; a prompt pass of 40 more tokens
    must then be admitted (20 + 40 <= 96), which a bound advanced by 8 per iteration would refuse."""
    arch = synth.llama_like(2, 256, 2, 512, 512)
    model = B.Model(arch, B.upload_weights(arch, gu.scaled_weights(synth, arch, 3, 6.0)))
    K, S, iters = 7, 96, 20
    kv = B.KV(model, 1, S)
    ws = model.new_workspace(1, K + 1, S)
    V = arch.vocab
    rows = _i32([[1, 2, 3, 4, 5, 6, 7, 8]])
    q = torch.zeros(1, K, V, device="cuda")
    for i in range(K):
        q[0, i, i + 2] = 1.0                    # one-hot on draft token i: accepted only if p(x) > 0.999
    u = torch.full((1, K + 1), 0.999, device="cuda")
    n_acc, nxt, out_count = _i32([0]), _i32([0]), _i32([0])
    for _ in range(iters):
        B.target_verify(model, kv, rows, K, q, u, 1.0, n_acc, nxt, 1, None, ws)
        B.spec_advance(kv, None, rows, K, n_acc, nxt, 1, None, 0, out_count, None, None)
    torch.cuda.synchronize()                    # (no length read-back)
    more = synth.gen_prompt(9, 1, 40, V)
    B.kv_prefill(model, kv, torch.from_numpy(more).cuda(), _i32([40]), model.new_workspace(1, 8, S))
    assert kv.status() == 0
    assert int(out_count.cpu()[0]) == iters
    assert kv.lengths().tolist() == [iters + 40]


def test_wait_that_nobody_satisfies_times_out_and_leaves_the_context_usable():
    """Failure detection without a fault: with a short wait limit, a probe kernel waits on a barrier that
    nothing ever arrives at; the wait gives up, SSD_E_TIMEOUT lands in the status word, the kernel returns,
    and an ordinary verification pass on fresh handles afterwards is correct."""
    arch = synth.llama_like(2, 256, 2, 512, 512)
    ws_np = gu.scaled_weights(synth, arch, 7, 6.0)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    kv = B.KV(model, 1, 32)
    assert kv.status() == 0
    B.set_wait_limit(2_000_000)                 # about a millisecond
    try:
        B.wait_probe(kv)
        assert kv.status() == -5
    finally:
        B.set_wait_limit(0)
    # the status word is sticky for that cache; fresh handles work as before
    kv2 = B.KV(model, 1, 32)
    ws = model.new_workspace(1, 4, 32)
    rows = synth.gen_prompt(8, 1, 4, arch.vocab)
    got = _verify(model, kv2, ws, rows, 3)
    assert kv2.status() == 0
    ref = od.Model(arch, ws_np).new_cache(32).feed(rows[0], advance=False)
    gu.assert_logits_close(got[0], ref)
