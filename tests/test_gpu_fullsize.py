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


@pytest.fixture(scope="module")
def llama7b():
    """The 7B Llama-shape target at full width and depth with bench.py's device-side N(0, 0.02) init, shared
    by the tests of this module; the oracle gets the same bf16 bit patterns, copied back as data."""
    import bench
    arch = synth.PRESETS["llama-7b"]["target"]
    model = B.Model(arch, bench.random_weights_on_device(arch, 31, torch))
    holder = {"arch": arch, "model": model, "host": None}

    def host_weights():
        if holder["host"] is None:
            holder["host"] = bench.weights_to_host(model.tensors, torch)
        return holder["host"]
    holder["host_weights"] = host_weights
    yield holder
    holder.clear()


def _seeded_fill(kv, seed, scale=0.5):
    """N(0, scale^2) values, rounded to bf16 on the device, as the cache contents; returns nothing (the
    host reads the very same bf16 values back through the cache view)."""
    g = torch.Generator(device="cuda")
    view = kv.cache_view()
    for b in range(view.shape[1]):
        g.manual_seed(seed + b)
        view[:, b].copy_(torch.randn(view[:, b].shape, generator=g, device="cuda") * scale)


def _oracle_rows(omodel, kv, b, n_ctx, rows, S):
    """The oracle's logits for `rows` fed behind n_ctx cached positions of sequence b, its cache seeded with
    the bf16 values the GPU cache holds; also returns the oracle cache."""
    oc = omodel.new_cache(S)
    oc.kv[...] = kv.cache_view()[:, b].float().cpu().numpy()
    oc.len = n_ctx
    return oc.feed(rows, advance=False), oc


def _check_pass_against_oracle(arch, model, omodel, kv, lens, seqs, rows_np, K, T, q_np, u_np, S):
    """One verification pass through the C ABI, compared with the oracle for the sequences in `seqs`:
    logits, probabilities, appended cache rows, and decisions by the oracle's rule on the pass's own rows."""
    dev = "cuda"
    Bn, V = rows_np.shape[0], arch.vocab
    oracle = {b: _oracle_rows(omodel, kv, b, lens[b], rows_np[b], S) for b in seqs}   # before the pass appends its rows
    n_acc = torch.zeros(Bn, dtype=torch.int32, device=dev)
    nxt = torch.zeros(Bn, dtype=torch.int32, device=dev)
    p_dbg = torch.zeros(Bn, K + 1, V, device=dev)
    ws = model.new_workspace(Bn, K + 1, S)
    B.target_verify(model, kv, torch.from_numpy(rows_np).to(dev), K, torch.from_numpy(q_np).to(dev),
                    torch.from_numpy(u_np).to(dev), T, n_acc, nxt, 1, p_dbg, ws)
    logits = B.last_logits(model, Bn, K + 1, ws).cpu().numpy()
    assert kv.status() == 0 and kv.lengths().tolist() == list(lens)
    p_gpu, a_gpu, y_gpu = p_dbg.cpu().numpy(), n_acc.cpu().numpy(), nxt.cpu().numpy()
    for b in range(Bn):
        gu.check_decisions_on_own_rows(p_gpu[b], q_np[b], rows_np[b, 1:], u_np[b, :K], u_np[b, K], int(a_gpu[b]), int(y_gpu[b]))
    for b in seqs:
        ref, oc = oracle[b]
        assert np.abs(ref).max() > 0.5
        gu.assert_logits_close(logits[b], ref)
        p_ref = np.stack([osamp.softmax_t(ref[i], T) for i in range(K + 1)])
        assert np.abs(p_gpu[b] - p_ref).max() <= gu.P_ATOL
        n0, n1 = lens[b], lens[b] + K + 1
        g = kv.cache_view()[:, b, :, :, n0:n1].float().cpu().numpy()
        r = oc.kv[:, :, :, n0:n1]
        assert (np.abs(g - r) <= gu.LOGIT_RTOL * np.abs(r) + gu.LOGIT_ATOL).all()
        assert (g == r).mean() > 0.8
    return logits


def test_7b_shape_pass_matches_the_oracle(llama7b):
    """The configuration the latency target is quoted on - 7B Llama shape, 32 layers, batch 1, 2048 cached
    positions, K = 4 - against the oracle on the same weights and the same seeded cache: the stream-K GEMMs at
    d_ff = 11008 (172 k-chunks), vocabulary 32000 and 32 layers of accumulated error are all inside."""
    arch, model = llama7b["arch"], llama7b["model"]
    od.set_threads(16)
    omodel = od.Model(arch, llama7b["host_weights"]())
    K, T, ctx, S = 4, 1.0, 2048, 2048 + 64
    V = arch.vocab
    kv = B.KV(model, 1, S)
    _seeded_fill(kv, 5)
    B.kv_commit(kv, torch.tensor([ctx], dtype=torch.int32, device="cuda"))
    assert kv.lengths().tolist() == [ctx]
    rows_np = synth.gen_prompt(91, 1, K + 1, V)
    q_np = synth.gen_dirichlet_rows(92, K, V).reshape(1, K, V)
    u_np = synth.gen_uniforms(93, 0, 0, K + 1).reshape(1, K + 1)
    _check_pass_against_oracle(arch, model, omodel, kv, [ctx], [0], rows_np, K, T, q_np, u_np, S)


def test_7b_shape_batch_of_eight_matches_the_oracle(llama7b):
    """The batched configuration: 8 sequences x 5 rows = 40 rows in one pass with ragged cache lengths (the
    40-row operand tiles, 256 (sequence, head) attention groups on 148 SMs); three of the sequences - a full
    one, a short one and one ending one position before a tile boundary - against the oracle."""
    arch, model = llama7b["arch"], llama7b["model"]
    od.set_threads(16)
    omodel = od.Model(arch, llama7b["host_weights"]())
    K, T, S, Bn = 4, 1.0, 2048 + 64, 8
    lens = [2048, 1900, 2047, 1024, 2048, 129, 640, 2048]
    V = arch.vocab
    kv = B.KV(model, Bn, S)
    _seeded_fill(kv, 100)
    B.kv_commit(kv, torch.tensor(lens, dtype=torch.int32, device="cuda"))
    assert kv.lengths().tolist() == lens
    rows_np = synth.gen_prompt(94, Bn, K + 1, V)
    q_np = synth.gen_dirichlet_rows(95, Bn * K, V).reshape(Bn, K, V)
    u_np = np.stack([synth.gen_uniforms(96, b, 0, K + 1) for b in range(Bn)])
    _check_pass_against_oracle(arch, model, omodel, kv, lens, [2, 5, 7], rows_np, K, T, q_np, u_np, S)


def test_7b_shape_many_row_prompt_pass_matches_the_oracle(llama7b):
    """The many-row prompt pass at the 7B shape, all 32 layers: three sequences with seeded caches of ragged
    lengths are continued by 70, 49 and 3 prompt tokens in one pass (210 rows: two 128-row GEMM tiles at
    d_ff = 11008 and 172 k-chunks, two 64-row attention tiles over hundreds of cached positions); the appended
    cache rows of two sequences against the oracle, then a verification pass on top of them."""
    arch, model = llama7b["arch"], llama7b["model"]
    od.set_threads(16)
    omodel = od.Model(arch, llama7b["host_weights"]())
    Bn, S, P = 3, 1024, 70
    lens0, n_new = [700, 321, 64], [70, 49, 3]
    V = arch.vocab
    kv = B.KV(model, Bn, S)
    _seeded_fill(kv, 300)
    B.kv_commit(kv, torch.tensor(lens0, dtype=torch.int32, device="cuda"))
    prompts = synth.gen_prompt(301, Bn, P, V)
    oracle = {}
    for b in (0, 1):
        oc = omodel.new_cache(S)
        oc.kv[...] = kv.cache_view()[:, b].float().cpu().numpy()
        oc.len = lens0[b]
        oc.feed(prompts[b, :n_new[b]], want_logits=False)
        oracle[b] = oc
    B.set_prefill_mode(2)
    try:
        nbytes = model.prefill_workspace_bytes(Bn, P)
        assert nbytes > 0
        B.kv_prefill(model, kv, torch.from_numpy(prompts).cuda(), torch.tensor(n_new, dtype=torch.int32, device="cuda"),
                     B.device_buffer(nbytes))
    finally:
        B.set_prefill_mode(0)
    lens1 = [a + b for a, b in zip(lens0, n_new)]
    assert kv.status() == 0 and kv.lengths().tolist() == lens1
    for b in (0, 1):
        g = kv.cache_view()[:, b, :, :, lens0[b]:lens1[b]].float().cpu().numpy()
        r = oracle[b].kv[:, :, :, lens0[b]:lens1[b]]
        # (70 rows x 32 layers: the relative term is taken against the row's largest entry - the error of a key or
        #  value row is a vector whose size goes with the row, and a row whose attention is nearly tied between two
        #  cached positions carries the roundings of the earlier layers' keys into every entry of the later ones)
        bad = np.argwhere(np.abs(g - r) > gu.LOGIT_RTOL * np.abs(r).max(axis=-1, keepdims=True) + gu.LOGIT_ATOL)
        assert bad.shape[0] == 0, (b, bad.shape[0], bad[:12].tolist(), [(float(g[tuple(i)]), float(r[tuple(i)])) for i in bad[:12]])
        assert (g == r).mean() > 0.5      # (most bf16 entries are the oracle's bit for bit even after 32 layers)
    K, T = 4, 1.0
    rows_np = synth.gen_prompt(302, Bn, K + 1, V)
    q_np = synth.gen_dirichlet_rows(303, Bn * K, V).reshape(Bn, K, V)
    u_np = np.stack([synth.gen_uniforms(304, b, 0, K + 1) for b in range(Bn)])
    _check_pass_against_oracle(arch, model, omodel, kv, lens1, [0], rows_np, K, T, q_np, u_np, S)


@pytest.mark.parametrize("ctx,M", [(8192, 5), (8192, 17), (16384, 5), (16384, 17)])
def test_7b_width_long_context_tensor_core_attention_matches_the_oracle(llama7b, ctx, M):
    """The long-context points of the verify sweep through target_verify with the default attention choice: at 5
    rows the warp-MMA items that carry hi and lo in one tile (hundreds of position blocks per warp), at 17 rows the
    tcgen05 form (2048 to 8192 positions per split, the K/V ring wrapping many times, two 16-row tiles); 2 to 4
    splits merged; first four layers of the 7B model at full width + final norm + LM head, against the oracle on
    the seeded cache."""
    arch4 = llama7b["arch"].replace(n_layers=4)
    model4 = llama7b["model"].share_prefix(4)
    od.set_threads(16)
    o_arch, o_ws = synth.prefix_draft(llama7b["arch"], llama7b["host_weights"](), 4)
    omodel = od.Model(o_arch, o_ws)
    K, T, S = M - 1, 1.0, ctx + 64
    V = arch4.vocab
    kv = B.KV(model4, 1, S)
    _seeded_fill(kv, 7 + ctx)
    B.kv_commit(kv, torch.tensor([ctx], dtype=torch.int32, device="cuda"))
    assert kv.lengths().tolist() == [ctx]
    rows_np = synth.gen_prompt(97, 1, M, V)
    q_np = synth.gen_dirichlet_rows(98, K, V).reshape(1, K, V)
    u_np = synth.gen_uniforms(99, 0, 0, M).reshape(1, M)
    _check_pass_against_oracle(arch4, model4, omodel, kv, [ctx], [0], rows_np, K, T, q_np, u_np, S)


def test_12b_width_pass_matches_the_oracle():
    """The 12B NeoX shape at full width (d 5120: rows wider than the 4096 columns a norm phase keeps in registers,
    40 heads of 128 with rotary on 32 of them, MLP 20480 = 320 k-chunks, vocabulary 50304), two layers, K = 5 at
    T = 1 on a seeded cache of 300 positions, against the oracle."""
    import bench
    arch = synth.PRESETS["neox-12b"]["target"].replace(n_layers=2)
    model = B.Model(arch, bench.random_weights_on_device(arch, 41, torch))
    od.set_threads(16)
    omodel = od.Model(arch, bench.weights_to_host(model.tensors, torch))
    K, T, ctx, S = 5, 1.0, 300, 320
    V = arch.vocab
    kv = B.KV(model, 1, S)
    _seeded_fill(kv, 12)
    B.kv_commit(kv, torch.tensor([ctx], dtype=torch.int32, device="cuda"))
    rows_np = synth.gen_prompt(121, 1, K + 1, V)
    q_np = synth.gen_dirichlet_rows(122, K, V).reshape(1, K, V)
    u_np = synth.gen_uniforms(123, 0, 0, K + 1).reshape(1, K + 1)
    _check_pass_against_oracle(arch, model, omodel, kv, [ctx], [0], rows_np, K, T, q_np, u_np, S)


def test_2p7b_width_greedy_pass_matches_the_oracle():
    """The 2.7B NeoX shape at full width (d 2560, 32 heads of 80, MLP 10240, vocabulary 50304), four layers,
    K = 8, greedy: 9 rows in one pass against the oracle; the greedy decisions are the oracle's unless the
    oracle's top-2 logit margin of the deciding row is inside the logit tolerance."""
    import bench
    arch = synth.PRESETS["neox-2.7b"]["target"].replace(n_layers=4)
    K, T, P, S = 8, 0.0, 40, 96
    model = B.Model(arch, bench.random_weights_on_device(arch, 21, torch))
    od.set_threads(16)
    omodel = od.Model(arch, bench.weights_to_host(model.tensors, torch))
    V = arch.vocab
    dev = "cuda"
    prompt = synth.gen_prompt(23, 1, P, V)
    kv = B.KV(model, 1, S)
    ws = model.new_workspace(1, K + 1, S)
    B.kv_prefill(model, kv, torch.from_numpy(prompt).to(dev), torch.tensor([P], dtype=torch.int32, device=dev),
                 model.new_workspace(1, 8, S))
    oc = omodel.new_cache(S)
    oc.feed(prompt[0], want_logits=False)
    # drafts: the oracle's own greedy continuation for the first rows (so that some are accepted), then others
    rows = [int(synth.gen_prompt(24, 1, 1, V)[0, 0])]
    probe = omodel.new_cache(S)
    probe.feed(prompt[0], want_logits=False)
    for i in range(K):
        nxt_tok = int(np.argmax(probe.feed([rows[-1]])[0]))
        rows.append(nxt_tok if i < 5 else (nxt_tok + 1) % V)
    rows_np = np.array([rows], np.int32)
    ref = oc.feed(rows_np[0], advance=False)
    q_np = np.zeros((1, K, V), np.float32)
    for i in range(K):
        q_np[0, i, rows[i + 1]] = 1.0           # greedy draft rows are one-hot at the draft token
    u_np = synth.gen_uniforms(25, 0, 0, K + 1).reshape(1, K + 1)
    n_acc = torch.zeros(1, dtype=torch.int32, device=dev)
    nxt = torch.zeros(1, dtype=torch.int32, device=dev)
    p_dbg = torch.zeros(1, K + 1, V, device=dev)
    B.target_verify(model, kv, torch.from_numpy(rows_np).to(dev), K, torch.from_numpy(q_np).to(dev),
                    torch.from_numpy(u_np).to(dev), T, n_acc, nxt, 1, p_dbg, ws)
    logits = B.last_logits(model, 1, K + 1, ws).cpu().numpy()[0]
    assert kv.status() == 0
    gu.assert_logits_close(logits, ref)
    p_gpu = p_dbg.cpu().numpy()[0]
    a_gpu, y_gpu = int(n_acc.cpu()[0]), int(nxt.cpu()[0])
    gu.check_decisions_on_own_rows(p_gpu, q_np[0], rows_np[0, 1:], u_np[0, :K], u_np[0, K], a_gpu, y_gpu)
    p_ref = [osamp.softmax_t(ref[i], T) for i in range(K + 1)]
    a_ref, y_ref = osamp.accept_resample(p_ref, list(q_np[0]), rows[1:], u_np[0, :K], u_np[0, K])
    if (a_gpu, y_gpu) != (a_ref, y_ref):
        top = np.sort(ref[min(a_gpu, a_ref)])[::-1]
        assert top[0] - top[1] <= 2 * (gu.LOGIT_ATOL + gu.LOGIT_RTOL * abs(top[0])), (a_gpu, y_gpu, a_ref, y_ref, top[:2])
    else:
        assert a_ref == 5                      # five drafts follow the argmax chain, the sixth does not
    g = kv.cache_view()[:, 0, :, :, P:P + K + 1].float().cpu().numpy()
    r = oc.kv[:, :, :, P:P + K + 1]
    assert (np.abs(g - r) <= gu.LOGIT_RTOL * np.abs(r) + gu.LOGIT_ATOL).all()


def test_2p7b_greedy_speculative_tokens_equal_greedy_autoregressive_tokens_on_the_gpu():
    """The third named workload at full size (32 layers, layer-skip draft = first four layers, K = 8,
    greedy): the speculative engine must emit the autoregressive engine's tokens.  Both run on the GPU; the
    two differ only in fp32 summation order (rows fed together or one by one), so a difference is accepted
    only where the top-2 margin of the autoregressive logits at that step is below 1e-3."""
    import bench
    from paper_2311_04951_b200 import engine
    cfg = bench.resolve("neox-2.7b")
    arch, K = cfg["target"], cfg["K"]
    target = B.Model(arch, bench.random_weights_on_device(arch, cfg["seeds"]["w"], torch, **bench.late_scaling(cfg)))
    draft = target.share_prefix(4)
    P, n_new, S = 48, 64, 48 + 64 + 2 * (K + 1) + 16
    prompts = synth.gen_prompt(cfg["seeds"]["prompt"], 1, P, arch.vocab)
    uni = lambda s, it: synth.gen_uniforms(cfg["seeds"]["u"], s, it, 2 * K + 1)
    sp = engine.Engine(target, draft, 1, S, K, 0.0, 128).generate(prompts, n_new, uni)
    # autoregressive, step by step, keeping the top-2 margin of every step
    ar = engine.Engine(target, None, 1, S, 0, 0.0, 128)
    ar.prefill(torch.from_numpy(prompts).cuda())
    u1 = torch.zeros(1, 1, device="cuda")
    margins, toks = [], []
    for _ in range(n_new):
        ar.ar_step(u1)
        top = torch.topk(B.last_logits(target, 1, 1, ar.ws_t)[0, 0], 2).values
        margins.append(float(top[0] - top[1]))
        toks.append(int(ar.next_tok.cpu()[0]))
    assert sp["status"] == 0 and ar.tkv.status() == 0
    got = sp["tokens"][0]
    flips = 0
    for i, (a, b) in enumerate(zip(got, toks)):
        if a != b:
            assert margins[i] <= 1e-3, (i, a, b, margins[i])
            flips += 1
            break                                # the sequences part ways behind an excused flip
    print(f"greedy 2.7B: {flips} margin-excused flip(s) in {n_new} tokens, {sp['iterations']} iterations")
    assert flips == 0 or i >= 8
    assert sp["iterations"] <= n_new


@pytest.mark.parametrize("which", ["neox-1.4b", "llama-7b-4-layers"])
def test_two_identical_passes_run_to_run(which, llama7b):
    """Run-to-run behaviour of a verification pass.  The stream-K GEMMs add their partial sums to the output
    with fp32 reductions in the order the CTAs arrive, so two identical passes may differ in the last bits;
    this test records whether they do and bounds the difference far below the logit tolerance.  Cache rows
    (bf16) of the two passes agree up to one rounding step in a few places."""
    import bench
    if which == "neox-1.4b":
        arch = synth.PRESETS["neox-1.4b"]["target"]
        model = B.Model(arch, bench.random_weights_on_device(arch, 11, torch))
    else:
        arch = llama7b["arch"].replace(n_layers=4)
        model = llama7b["model"].share_prefix(4)
    K, ctx, S = 5, 300, 384
    V = arch.vocab
    dev = "cuda"
    rows = torch.from_numpy(synth.gen_prompt(81, 1, K + 1, V)).to(dev)
    q = torch.from_numpy(synth.gen_dirichlet_rows(82, K, V)).to(dev).reshape(1, K, V)
    u = torch.from_numpy(synth.gen_uniforms(83, 0, 0, K + 1)).to(dev).reshape(1, K + 1)
    outs = []
    for _ in range(2):
        kv = B.KV(model, 1, S)
        _seeded_fill(kv, 9)
        B.kv_commit(kv, torch.tensor([ctx], dtype=torch.int32, device=dev))
        kv.lengths()
        ws = model.new_workspace(1, K + 1, S)
        n_acc = torch.zeros(1, dtype=torch.int32, device=dev)
        nxt = torch.zeros(1, dtype=torch.int32, device=dev)
        B.target_verify(model, kv, rows, K, q, u, 1.0, n_acc, nxt, 1, None, ws)
        outs.append((B.last_logits(model, 1, K + 1, ws).cpu().numpy(),
                     kv.cache_view()[:, 0, :, :, ctx:ctx + K + 1].float().cpu().numpy(), int(n_acc.cpu()[0]), int(nxt.cpu()[0])))
        assert kv.status() == 0
    (l0, c0, a0, y0), (l1, c1, a1, y1) = outs
    diff = float(np.abs(l0 - l1).max())
    print(f"{which}: logits bit-identical: {np.array_equal(l0, l1)}, max |difference| {diff:.3e}; "
          f"cache rows identical: {(c0 == c1).mean():.6f}")
    assert diff <= 1e-3
    assert (c0 == c1).mean() > 0.99
    assert (a0, y0) == (a1, y1) or diff > 0      # equal decisions unless the logits moved


def test_7b_shape_pass_in_the_bench_configuration_properties(llama7b):
    """The 7B Llama shape at full width and depth (32 layers, d 4096, 32 heads x 128, SwiGLU 11008, vocab
    32000), batch 1, context 2048, K = 4: the launch configuration of the verify sweep, checked through
    properties that hold at any size (the comparison with the oracle is the test above): the five rows fed together give the logits and cache rows of the same rows fed one at a time (the
    claim that lets one verification pass replace K + 1 decode steps), the probabilities are the softmax
    of the logits (numpy, fp64), and the accept / resample decisions follow the oracle's rule on the
    pass's own rows."""
    arch, model = llama7b["arch"], llama7b["model"]                         # bench.py's device-side N(0, 0.02) init
    K, T, ctx, S = 4, 1.0, 2048, 2048 + 64
    dev = "cuda"
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


def test_7b_shape_batch_of_eight_equals_single_sequences(llama7b):
    """The batched configuration at full size: 8 independent sequences x (K + 1 = 5) rows = 40 rows in one pass of
    the 7B shape (the 40-row operand tiles and M = 128 MMAs, 256 (sequence, head) attention groups on 148 SMs),
    with ragged cache lengths.  Sequences are independent, so a sequence's logits, decisions and appended
    cache rows must be those of the same sequence run alone (the 8-row path checked above)."""
    arch, model = llama7b["arch"], llama7b["model"]
    K, T, S, Bn = 4, 1.0, 2048 + 64, 8
    lens = [2048, 1900, 2047, 1024, 2048, 129, 640, 2048]
    dev = "cuda"
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
