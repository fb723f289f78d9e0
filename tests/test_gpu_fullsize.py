"""Parity at a full benchmark size, in the launch configuration bench.py times: the 1.4B NeoX-shape
target (24 layers, d 2048, vocab 50304, bf16), batch 1, K = 5 -> one verification pass over 6 rows
through the single forward kernel, compared with the oracle on the same seeded weights."""
import numpy as np
import pytest
import torch

from oracle import decoder as od
from oracle import sampling as osamp
from paper_2311_04951_b200 import binding as B, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_verify_pass_at_the_1p4b_shape_matches_the_oracle():
    cfg = synth.PRESETS["neox-1.4b"]
    arch, K, T = cfg["target"], cfg["K"], cfg["temperature"]
    ws_np = synth.gen_weights(arch, cfg["seeds"]["w"])          # natural N(0, 0.02) init, bf16 matrices
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    P, S = 24, 64
    prompt = synth.gen_prompt(cfg["seeds"]["prompt"], 1, P, arch.vocab)
    rows_np = synth.gen_prompt(77, 1, K + 1, arch.vocab)
    dev = "cuda"
    kv = B.KV(model, 1, S)
    ws = model.new_workspace(1, 8, S)
    B.kv_prefill(model, kv, torch.from_numpy(prompt).to(dev), torch.tensor([P], dtype=torch.int32, device=dev), ws)
    V = arch.vocab
    q_np = synth.gen_dirichlet_rows(78, K, V).reshape(1, K, V)
    u_np = synth.gen_uniforms(79, 0, 0, K + 1).reshape(1, K + 1)
    n_acc = torch.zeros(1, dtype=torch.int32, device=dev)
    nxt = torch.zeros(1, dtype=torch.int32, device=dev)
    p_dbg = torch.zeros(1, K + 1, V, device=dev)
    B.target_verify(model, kv, torch.from_numpy(rows_np).to(dev), K, torch.from_numpy(q_np).to(dev),
                    torch.from_numpy(u_np).to(dev), T, n_acc, nxt, 1, p_dbg, ws)
    logits = B.last_logits(model, 1, K + 1, ws).cpu().numpy()[0]
    p_gpu = p_dbg.cpu().numpy()[0]
    assert kv.status() == 0 and kv.lengths().tolist() == [P]
    # oracle: same weights, same tokens
    od.set_threads(16)
    om = od.Model(arch, ws_np)
    oc = om.new_cache(S)
    oc.feed(prompt[0], want_logits=False)
    ref = oc.feed(rows_np[0], advance=False)
    gu.assert_logits_close(logits, ref)
    p_ref = np.stack([osamp.softmax_t(ref[i], T) for i in range(K + 1)])
    assert np.abs(p_gpu - p_ref).max() <= gu.P_ATOL
    # decisions follow the rule on the GPU's own rows
    gu.check_decisions_on_own_rows(p_gpu, q_np[0], rows_np[0, 1:], u_np[0, :K], u_np[0, K],
                                   int(n_acc.cpu()[0]), int(nxt.cpu()[0]))
    # cache rows of the pass equal the oracle's up to one bf16 step
    cache = kv.cache_view().float().cpu().numpy()[:, 0, :, :, :P + K + 1]
    r = oc.kv[:, :, :, :P + K + 1]
    assert (np.abs(cache - r) <= gu.LOGIT_RTOL * np.abs(r) + gu.LOGIT_ATOL).all()


def test_7b_shape_pass_in_the_bench_configuration_properties():
    """The 7B Llama shape at full width and depth (32 layers, d 4096, 32 heads x 128, SwiGLU 11008, vocab
    32000), batch 1, context 2048, K = 4: the launch configuration of the verify sweep.  The oracle needs
    minutes for a pass of this size, so the pass is checked through properties that hold at any size:
    the five rows fed together give the logits and cache rows of the same rows fed one at a time (the
    claim that lets one verification pass replace K + 1 decode steps), the probabilities are the softmax
    of the logits (numpy, fp64), and the accept / resample decisions follow the oracle's rule on the
    pass's own rows."""
    import bench
    arch = synth.PRESETS["llama-7b"]["target"]
    K, T, ctx, S = 4, 1.0, 2048, 2048 + 64
    dev = "cuda"
    model = B.Model(arch, bench.random_weights_on_device(arch, 31, torch))   # bench.py's device-side N(0, 0.02) init
    V = arch.vocab
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    fill = torch.randn((arch.n_layers, 1, 2, arch.n_heads, S, arch.head_dim), generator=g, device=dev) * 0.5

    def fresh_kv():
        kv = B.KV(model, 1, S)
        kv.cache_view().copy_(fill)
        B.kv_commit(kv, torch.tensor([ctx], dtype=torch.int32, device=dev))
        assert kv.lengths().tolist() == [ctx]
        return kv

    rows_np = synth.gen_prompt(91, 1, K + 1, V)
    q_np = synth.gen_dirichlet_rows(92, K, V).reshape(1, K, V)
    u_np = synth.gen_uniforms(93, 0, 0, K + 1).reshape(1, K + 1)
    n_acc = torch.zeros(1, dtype=torch.int32, device=dev)
    nxt = torch.zeros(1, dtype=torch.int32, device=dev)
    p_dbg = torch.zeros(1, K + 1, V, device=dev)
    kv = fresh_kv()
    ws = model.new_workspace(1, K + 1, S)
    B.target_verify(model, kv, torch.from_numpy(rows_np).to(dev), K, torch.from_numpy(q_np).to(dev),
                    torch.from_numpy(u_np).to(dev), T, n_acc, nxt, 1, p_dbg, ws)
    together = B.last_logits(model, 1, K + 1, ws).cpu().numpy()[0]
    p_gpu = p_dbg.cpu().numpy()[0]
    assert kv.status() == 0
    cache_together = kv.cache_view().float().cpu().numpy()[:, 0, :, :, ctx:ctx + K + 1]
    assert np.abs(together).max() > 0.5                      # the comparison below is not about zeros
    # probabilities = softmax of the logits
    z = together.astype(np.float64) / T
    e = np.exp(z - z.max(axis=1, keepdims=True))
    assert np.abs(p_gpu - e / e.sum(axis=1, keepdims=True)).max() <= gu.P_ATOL
    # decisions follow the rule on the pass's own rows
    gu.check_decisions_on_own_rows(p_gpu, q_np[0], rows_np[0, 1:], u_np[0, :K], u_np[0, K],
                                   int(n_acc.cpu()[0]), int(nxt.cpu()[0]))
    # one row at a time
    kv1 = fresh_kv()
    ws1 = model.new_workspace(1, 1, S)
    one = torch.ones(1, dtype=torch.int32, device=dev)
    u1 = torch.full((1, 1), 0.5, device=dev)
    for i in range(K + 1):
        B.target_verify(model, kv1, torch.from_numpy(rows_np[:, i:i + 1].copy()).to(dev), 0, None, u1, T, n_acc, nxt, 1,
                        None, ws1)
        single = B.last_logits(model, 1, 1, ws1).cpu().numpy()[0, 0]
        B.kv_commit(kv1, one)
        gu.assert_logits_close(single, together[i])         # same math; fp32 reduction order and bf16 K/V flips only
    assert kv1.status() == 0 and kv1.lengths().tolist() == [ctx + K + 1]
    cache_single = kv1.cache_view().float().cpu().numpy()[:, 0, :, :, ctx:ctx + K + 1]
    tol = gu.LOGIT_RTOL * np.abs(cache_single) + gu.LOGIT_ATOL
    assert (np.abs(cache_together - cache_single) <= tol).all()
    assert (cache_together == cache_single).mean() > 0.8


def test_7b_shape_batch_of_eight_equals_single_sequences():
    """The batched configuration at full size: 8 independent sequences x (K + 1 = 5) rows = 40 rows in one pass of
    the 7B shape (the 40-row operand tiles and M = 128 MMAs, 256 (sequence, head) attention groups on 148 SMs),
    with ragged cache lengths.  Sequences are independent, so a sequence's logits, decisions and appended
    cache rows must be those of the same sequence run alone (the 8-row path checked above)."""
    import bench
    arch = synth.PRESETS["llama-7b"]["target"]
    K, T, S, Bn = 4, 1.0, 2048 + 64, 8
    lens = [2048, 1900, 2047, 1024, 2048, 129, 640, 2048]
    dev = "cuda"
    model = B.Model(arch, bench.random_weights_on_device(arch, 31, torch))
    V = arch.vocab
    g = torch.Generator(device=dev)
    kv = B.KV(model, Bn, S)
    view = kv.cache_view()                                   # [L, B, 2, H, S, Dh] bf16
    for b in range(Bn):
        g.manual_seed(100 + b)
        view[:, b].copy_(torch.randn((arch.n_layers, 2, arch.n_heads, S, arch.head_dim), generator=g, device=dev) * 0.5)
    B.kv_commit(kv, torch.tensor(lens, dtype=torch.int32, device=dev))
    assert kv.lengths().tolist() == lens
    rows_np = synth.gen_prompt(94, Bn, K + 1, V)
    q_np = synth.gen_dirichlet_rows(95, Bn * K, V).reshape(Bn, K, V)
    u_np = np.stack([synth.gen_uniforms(96, b, 0, K + 1) for b in range(Bn)])
    n_acc = torch.zeros(Bn, dtype=torch.int32, device=dev)
    nxt = torch.zeros(Bn, dtype=torch.int32, device=dev)
    p_dbg = torch.zeros(Bn, K + 1, V, device=dev)
    ws = model.new_workspace(Bn, K + 1, S)
    B.target_verify(model, kv, torch.from_numpy(rows_np).to(dev), K, torch.from_numpy(q_np).to(dev),
                    torch.from_numpy(u_np).to(dev), T, n_acc, nxt, 1, p_dbg, ws)
    batched = B.last_logits(model, Bn, K + 1, ws).cpu().numpy()
    assert kv.status() == 0 and kv.lengths().tolist() == lens
    p_gpu, a_gpu, y_gpu = p_dbg.cpu().numpy(), n_acc.cpu().numpy(), nxt.cpu().numpy()
    for b in range(Bn):
        gu.check_decisions_on_own_rows(p_gpu[b], q_np[b], rows_np[b, 1:], u_np[b, :K], u_np[b, K], int(a_gpu[b]), int(y_gpu[b]))
    for b in (1, 5, 7):                                       # sampled sequences, each alone on a cache of its own
        kv1 = B.KV(model, 1, S)
        kv1.cache_view()[:, 0].copy_(view[:, b])
        # (the batched pass appended its rows behind lens[b]; the single pass overwrites them with its own)
        B.kv_commit(kv1, torch.tensor([lens[b]], dtype=torch.int32, device=dev))
        assert kv1.lengths().tolist() == [lens[b]]          # (also refreshes the host-side bound the splits are planned from)
        ws1 = model.new_workspace(1, K + 1, S)
        B.target_verify(model, kv1, torch.from_numpy(rows_np[b:b + 1].copy()).to(dev), K,
                        torch.from_numpy(q_np[b:b + 1].copy()).to(dev), torch.from_numpy(u_np[b:b + 1].copy()).to(dev), T,
                        n_acc[:1], nxt[:1], 1, None, ws1)
        alone = B.last_logits(model, 1, K + 1, ws1).cpu().numpy()[0]
        assert kv1.status() == 0
        gu.assert_logits_close(batched[b], alone)
        n0 = lens[b]
        cb = view[:, b, :, :, n0:n0 + K + 1].float().cpu().numpy()
        c1 = kv1.cache_view()[:, 0, :, :, n0:n0 + K + 1].float().cpu().numpy()
        assert (np.abs(cb - c1) <= gu.LOGIT_RTOL * np.abs(c1) + gu.LOGIT_ATOL).all()
        assert (cb == c1).mean() > 0.8
