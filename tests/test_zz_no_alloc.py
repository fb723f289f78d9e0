"""The allocation-free variant of the verification tail (verify_from_logits_noalloc).

Some users of this library cannot allocate device memory around a call: a serving runtime that
owns a fixed arena and forbids cudaMalloc once it is up, a decode loop where an allocation would
stall the device, a binding that can forward pointers but not own buffers.  For them the library
keeps the small scratch of the tail kernels in a fixed array of its own.  This test calls that
entry point through the C ABI twice in a row (second call: other sizes and values, so leftovers of
the first would show) and requires exactly the outputs of the ordinary entry point; it also checks
that a request beyond the array's size is refused.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2311_04951_b200 import binding as B, synth

pytestmark = pytest.mark.gpu


def _case(seed, Bn, K, V):
    logits = synth.gen_logits(seed, Bn * (K + 1), V, 1.5).reshape(Bn, K + 1, V)
    q = synth.gen_dirichlet_rows(seed + 1, Bn * K, V).reshape(Bn, K, V)
    toks = synth.draw_tokens_from_rows(seed + 2, q.reshape(Bn * K, V)).reshape(Bn, K)
    # make some drafts likely to be accepted: point half of them at a token the target favours
    for b in range(Bn):
        for i in range(0, K, 2):
            t = int(np.argmax(logits[b, i]))
            toks[b, i] = t
            q[b, i] *= 0.5
            q[b, i, t] += 0.5
    rows = np.concatenate([np.zeros((Bn, 1), np.int32), toks.astype(np.int32)], axis=1)
    u = np.stack([synth.gen_uniforms(seed + 3, b, 0, K + 1) for b in range(Bn)])
    dev = "cuda"
    return [torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in (logits, rows, q.astype(np.float32), u)]


def _run(fn, logits, rows, q, u, K, T, with_scratch):
    Bn, M, V = logits.shape
    dev = "cuda"
    n_acc = torch.full((Bn,), -1, dtype=torch.int32, device=dev)
    nxt = torch.full((Bn,), -1, dtype=torch.int32, device=dev)
    p = torch.zeros(Bn, M, V, device=dev)
    if with_scratch:
        scratch = torch.empty(B.verify_scratch_bytes(Bn, K), dtype=torch.uint8, device=dev)
        fn(logits, K, rows, q, u, T, n_acc, nxt, 1, p, scratch)
    else:
        fn(logits, K, rows, q, u, T, n_acc, nxt, 1, p)
    torch.cuda.synchronize()
    return n_acc.cpu().numpy(), nxt.cpu().numpy(), p.cpu().numpy()


def test_noalloc_variant_equals_the_ordinary_entry_point_twice_in_a_row():
    for seed, Bn, K, V, T in ((7, 3, 4, 32000, 1.0), (8, 2, 7, 5000, 0.8)):
        logits, rows, q, u = _case(seed, Bn, K, V)
        ref = _run(B.verify_from_logits, logits, rows, q, u, K, T, True)
        got = _run(B.verify_from_logits_noalloc, logits, rows, q, u, K, T, False)
        assert np.array_equal(got[0], ref[0]) and np.array_equal(got[1], ref[1])
        assert np.abs(got[2] - ref[2]).max() <= 1e-4 and np.array_equal(got[2], ref[2])
        assert (ref[0] >= 0).all() and (ref[1] >= 0).all() and abs(ref[2].sum(axis=2) - 1).max() < 1e-4


def test_noalloc_variant_refuses_more_rows_than_its_array_holds():
    dev = "cuda"
    K, V = 1, 128
    Bn = B.NOALLOC_MAX_ROWS // (K + 1) + 1
    logits = torch.zeros(Bn, K + 1, V, device=dev)
    rows = torch.zeros(Bn, K + 1, dtype=torch.int32, device=dev)
    q = torch.full((Bn, K, V), 1.0 / V, device=dev)
    u = torch.zeros(Bn, K + 1, device=dev)
    out = torch.zeros(Bn, dtype=torch.int32, device=dev)
    with pytest.raises(B.SsdError) as e:
        B.verify_from_logits_noalloc(logits, K, rows, q, u, 1.0, out, out.clone(), 1, None)
    assert e.value.code == -3
