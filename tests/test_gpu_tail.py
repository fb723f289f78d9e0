"""GPU parity of the vocabulary-wide tail (softmax, accept scan, residual resample, bonus draw)
on supplied logits, draft rows and uniforms, through the C ABI (verify_from_logits)."""
import numpy as np
import pytest
import torch

from oracle import sampling as osamp
from paper_2311_04951_b200 import binding as B, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def run_tail(logits, rows, q, u, T, want_p=True):
    Bn, M, V = logits.shape
    K = M - 1
    dev = "cuda"
    lg = torch.from_numpy(logits).to(dev)
    n_acc = torch.full((Bn,), -7, dtype=torch.int32, device=dev)
    nxt = torch.full((Bn,), -7, dtype=torch.int32, device=dev)
    p = torch.zeros(Bn, M, V, dtype=torch.float32, device=dev) if want_p else None
    scratch = torch.empty(B.verify_scratch_bytes(Bn, K), dtype=torch.uint8, device=dev)
    B.verify_from_logits(lg, K, torch.from_numpy(rows).to(dev), None if K == 0 else torch.from_numpy(q).to(dev),
                         torch.from_numpy(u).to(dev), T, n_acc, nxt, 1, p, scratch)
    torch.cuda.synchronize()
    return n_acc.cpu().numpy(), nxt.cpu().numpy(), (p.cpu().numpy() if want_p else None)


def make_case(seed, Bn, K, V, T, corr):
    """Logits ~ N(0, 1.5); draft rows either Dirichlet(0.1) (far from p) or a perturbed copy of p
    (acceptance non-trivial); draft tokens drawn from q."""
    logits = synth.gen_logits(seed, Bn * (K + 1), V, 1.5).reshape(Bn, K + 1, V)
    if corr:
        noise = synth.gen_logits(seed + 100, Bn * K, V, 0.7).reshape(Bn, K, V)
        ql = logits[:, :K] + noise
        q = np.stack([[osamp.softmax_t(ql[b, i], T if T > 0 else 1.0) for i in range(K)] for b in range(Bn)]) \
            if K else np.zeros((Bn, 0, V), np.float32)
    else:
        q = synth.gen_dirichlet_rows(seed + 1, Bn * K, V).reshape(Bn, K, V) if K else np.zeros((Bn, 0, V), np.float32)
    toks = synth.draw_tokens_from_rows(seed + 2, q.reshape(Bn * K, V)).reshape(Bn, K) if K else np.zeros((Bn, 0), np.int32)
    if T == 0 and K:  # greedy drafts propose one-hot rows
        hot = np.zeros_like(q)
        for b in range(Bn):
            for i in range(K):
                # half of the rows agree with the target argmax so that acceptance varies
                t = int(np.argmax(logits[b, i])) if (b + i) % 2 == 0 else int(toks[b, i])
                toks[b, i] = t
                hot[b, i, t] = 1
        q = hot
    rows = np.concatenate([np.zeros((Bn, 1), np.int32), toks.astype(np.int32)], axis=1)
    u = np.stack([synth.gen_uniforms(seed + 3, b, 0, K + 1) for b in range(Bn)])
    return logits, rows, q.astype(np.float32), u


@pytest.mark.parametrize("V", [1000, 32000, 50304])
@pytest.mark.parametrize("K,Bn", [(0, 1), (1, 2), (4, 1), (8, 3), (16, 1)])
@pytest.mark.parametrize("T,corr", [(1.0, False), (0.8, True), (0.0, True)])
def test_tail_matches_oracle(V, K, Bn, T, corr):
    logits, rows, q, u = make_case(1000 + V % 97 + K, Bn, K, V, T, corr)
    n_acc, nxt, p = run_tail(logits, rows, q, u, T)
    exact = 0
    for b in range(Bn):
        p_ref = np.stack([osamp.softmax_t(logits[b, i], T) for i in range(K + 1)])
        assert np.abs(p[b] - p_ref).max() <= gu.P_ATOL                      # layer A
        assert abs(p[b].sum(axis=1) - 1).max() < 1e-4
        exact += gu.check_decisions_on_own_rows(p[b], q[b], rows[b, 1:], u[b, :K], u[b, K], int(n_acc[b]), int(nxt[b]))
        # and against the oracle end to end, unless a decision is within tolerance of its threshold
        a_ref, y_ref = osamp.accept_resample(p_ref, q[b], rows[b, 1:], u[b, :K], u[b, K])
        if (a_ref, y_ref) != (int(n_acc[b]), int(nxt[b])):
            i = min(a_ref, int(n_acc[b]))
            if a_ref != int(n_acc[b]):
                x = rows[b, 1 + i]
                assert abs(float(p_ref[i, x]) - float(np.float32(u[b, i]) * q[b, i, x])) <= gu.P_ATOL + 4e-2 * p_ref[i, x]
    assert exact >= Bn - 1


def test_acceptance_varies_and_all_branches_are_hit():
    """Over many seeded cases every accepted count 0..K occurs (rejection at each row and the bonus
    branch), so the parity above covers all paths."""
    K, V, seen = 3, 2000, set()
    for seed in range(12):
        logits, rows, q, u = make_case(50 + seed, 4, K, V, 1.0, True)
        n_acc, nxt, _ = run_tail(logits, rows, q, u, 1.0, want_p=False)
        for b in range(4):
            p_ref = np.stack([osamp.softmax_t(logits[b, i], 1.0) for i in range(K + 1)])
            a_ref, y_ref = osamp.accept_resample(p_ref, q[b], rows[b, 1:], u[b, :K], u[b, K])
            seen.add(a_ref)
            if (a_ref, y_ref) != (int(n_acc[b]), int(nxt[b])):
                assert a_ref == int(n_acc[b])   # a token may differ only at a CDF step of near-equal sums
    assert seen == {0, 1, 2, 3}


def test_degenerate_rows():
    V, K = 512, 2
    logits = np.zeros((1, K + 1, V), np.float32)
    logits[0, :, 7] = 50.0                               # p is (numerically) one-hot at 7
    q = np.zeros((1, K, V), np.float32)
    q[0, 0, 7] = 1.0                                     # q == p -> accept
    q[0, 1, 9] = 1.0                                     # draft certain of a token the target excludes
    rows = np.array([[0, 7, 9]], np.int32)
    u = np.array([[0.5, 0.5, 0.3]], np.float32)
    n_acc, nxt, p = run_tail(logits, rows, q, u, 1.0)
    assert n_acc[0] == 1 and nxt[0] == 7                 # rejected at row 2, residual = p -> 7
    # q(x~) = 0 < p(x~): accepted even for u close to 1
    q2 = q.copy(); q2[0, 0] = 0; q2[0, 0, 3] = 1.0
    n_acc, nxt, _ = run_tail(logits, np.array([[0, 7, 7]], np.int32), q2, np.array([[0.999, 0.999, 0.1]], np.float32), 1.0)
    assert n_acc[0] == 2 and nxt[0] == 7
    # ties in greedy mode: lowest index wins
    lg = np.zeros((1, 1, V), np.float32); lg[0, 0, [5, 400]] = 3.0
    n_acc, nxt, p = run_tail(lg, np.zeros((1, 1), np.int32), np.zeros((1, 0, V), np.float32), np.array([[0.7]], np.float32), 0.0)
    assert nxt[0] == 5 and p[0, 0, 5] == 1.0 and p[0, 0].sum() == 1.0


def test_argument_errors_are_reported_on_the_host():
    dev = "cuda"
    lg = torch.zeros(1, 2, 128, device=dev)
    z = torch.zeros(4, dtype=torch.int32, device=dev)
    f = torch.zeros(256, device=dev)
    sc = torch.empty(B.verify_scratch_bytes(1, 1), dtype=torch.uint8, device=dev)
    with pytest.raises(B.SsdError) as e:
        B.verify_from_logits(lg, 1, z, None, f, 1.0, z, z, 1, None, sc)     # K > 0 without q
    assert e.value.code == -1
    with pytest.raises(B.SsdError) as e:
        B.verify_from_logits(lg, 1, z, f, f, 1.0, z, z, 1, None, sc[:8])    # scratch too small
    assert e.value.code == -3
    with pytest.raises(B.SsdError):
        B.verify_from_logits(lg, 1, z, f, f, -1.0, z, z, 1, None, sc)       # negative temperature


@pytest.mark.parametrize("V", [1000, 32000, 50304])
@pytest.mark.parametrize("top_k,top_p", [(50, 1.0), (0, 0.9), (40, 0.7), (1, 1.0), (0, 0.2), (100000, 0.999)])
def test_restricted_tail_matches_oracle(V, top_k, top_p):
    """top-k / top-p restriction inside the tail: the p rows the decisions use equal the oracle's restricted
    rows (same kept set unless a token sits at the nucleus boundary within rounding of the running sum), and
    the decisions follow the oracle's rule on those rows.  q is restricted the same way on the host side of
    the test, as a draft that runs under the same setting would deliver it."""
    T, K, Bn = 0.9, 4, 2
    logits, rows, q, u = make_case(2000 + V % 89 + top_k % 7, Bn, K, V, T, True)
    std = 3.0 if V > 1000 else 1.5          # peakier rows: a nucleus of tens, not thousands, of tokens
    logits = (logits * np.float32(std / 1.5)).astype(np.float32)
    q = np.stack([[osamp.filter_top_k_top_p(q[b, i], top_k, top_p) for i in range(K)] for b in range(Bn)])
    toks = synth.draw_tokens_from_rows(77, q.reshape(Bn * K, V)).reshape(Bn, K)
    rows[:, 1:] = toks
    B.set_sampling(top_k, top_p)
    try:
        n_acc, nxt, p = run_tail(logits, rows, q, u, T)
    finally:
        B.set_sampling(0, 1.0)
    for b in range(Bn):
        for i in range(K + 1):
            raw = osamp.softmax_t(logits[b, i], T)
            ref = osamp.filter_top_k_top_p(raw, top_k, top_p)
            got = p[b, i]
            same = (got > 0) == (ref > 0)
            if not same.all():
                # only tokens whose probability equals the threshold up to rounding of the running sums may differ
                thr = min(raw[got > 0].min(), raw[ref > 0].min())
                odd = raw[~same]
                assert (np.abs(odd - thr) <= 1e-6 * max(thr, 1e-30) + 1e-12).all() or \
                    abs(raw[got > 0].astype(np.float64).sum() - raw[ref > 0].astype(np.float64).sum()) <= 2e-6
            else:
                assert np.abs(got - ref).max() <= gu.P_ATOL
                assert abs(float(got.astype(np.float64).sum()) - 1.0) < 1e-5
        gu.check_decisions_on_own_rows(p[b], q[b], rows[b, 1:], u[b, :K], u[b, K], int(n_acc[b]), int(nxt[b]))
        assert p[b, int(n_acc[b])][int(nxt[b])] > 0       # the emitted token lies inside the restricted target
    if top_k == 1:
        assert ((p > 0).sum(axis=2) == 1).all()


def test_draft_and_verify_under_a_restriction_follow_the_oracle_loop():
    """Whole speculative iterations with top-k / top-p set (fp32 model, so the two sides agree to rounding):
    the draft's exported q rows, its tokens, the accepted counts and the target's tokens equal the oracle's
    loop run with the same restriction."""
    from oracle import decoder as od, spec as ospec
    from paper_2311_04951_b200 import engine
    arch = synth.gpt2_like(3, 128, 4, 256, 400, 160)
    ws = gu.scaled_weights(synth, arch, 21, 7.0)
    d_arch, d_ws = synth.prefix_draft(arch, ws, 1)
    tgt = B.Model(arch, B.upload_weights(arch, ws))
    K, T, n_new, top_k, top_p = 3, 0.9, 40, 12, 0.85
    prompt = synth.gen_prompt(22, 1, 12, arch.vocab)
    ref = ospec.speculative_generate(od.Model(arch, ws), od.Model(d_arch, d_ws), prompt[0], n_new, K, T,
                                     lambda it: synth.gen_uniforms(23, 0, it, 2 * K + 1), 160, keep_trace=True,
                                     top_k=top_k, top_p=top_p)
    B.set_sampling(top_k, top_p)
    try:
        eng = engine.Engine(tgt, tgt.share_prefix(1), 1, 160, K, T, 128)
        res = gu.lockstep(eng, synth, prompt[0], ref["iterations"], K, 23, ref["trace"])
    finally:
        B.set_sampling(0, 1.0)
    assert eng.tkv.status() == 0 and eng.dkv.status() == 0
    assert res["identical"] == res["iterations"] == ref["iterations"] and res["excused"] == 0
    assert max(int((t["q"][0] > 0).sum()) for t in ref["trace"]) <= top_k     # the restriction was active
    n_out = int(eng.out_count.cpu()[0])
    assert eng.out_tokens.cpu().numpy()[0, :n_out].tolist() == ref["all_tokens"][len(prompt[0]):]
