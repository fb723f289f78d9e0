"""GPU parity of the K-query causal attention over the cache at long context (split over CTAs
and merged), against the oracle's attention on a seeded random cache."""
import numpy as np
import pytest
import torch

from oracle import decoder as od
from paper_2311_04951_b200 import binding as B, synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,H,Dh,S,lens,rows", [
    (synth.DT_BF16, 4, 128, 4200, [4099, 37], 5),      # several splits, ragged tail, short neighbour
    (synth.DT_BF16, 3, 80, 1100, [1000], 9),           # head 80
    (synth.DT_BF16, 2, 64, 700, [0, 650, 64], 17),     # empty cache; exactly one tile; 17 rows
    (synth.DT_F32, 2, 64, 300, [255, 1], 2),
    (synth.DT_BF16, 2, 128, 16500, [16384], 5),        # longest context of the sweep
])
def test_attention_rows_match_oracle(dtype, H, Dh, S, lens, rows):
    d = H * Dh
    arch = synth.llama_like(1, d, H, 128, 128, dtype=dtype)
    model = B.Model(arch, B.upload_weights(arch, synth.gen_weights(arch, 1)))
    Bn = len(lens)
    kv = B.KV(model, Bn, S)
    fill = synth.gen_kv_fill(5, (1, Bn, 2, H, S, Dh), dtype)
    dev = "cuda"
    if dtype:
        kv.cache_view().copy_(torch.from_numpy(fill.view(np.int16)).to(dev).view(torch.bfloat16))
        fill_f = synth.bf16_bits_to_f32(fill)
    else:
        kv.cache_view().copy_(torch.from_numpy(fill).to(dev))
        fill_f = fill
    B.kv_commit(kv, torch.tensor(lens, dtype=torch.int32, device=dev))
    assert kv.lengths().tolist() == lens
    q = synth.gen_logits(6, Bn * rows, d, 1.0).reshape(Bn, rows, d)
    out = torch.zeros(Bn, rows, d, device=dev)
    B.attention_rows(model, kv, 0, torch.from_numpy(q).to(dev), rows, out, model.new_workspace(Bn, rows, S))
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert kv.status() == 0
    od.set_threads(8)
    for b in range(Bn):
        ref = od.attention_rows(q[b], fill_f[0, b], lens[b], rows)
        assert np.abs(got[b] - ref).max() <= 2e-4, (b, np.abs(got[b] - ref).max())


@pytest.mark.parametrize("mode", [2, 1])     # tensor-core items / warp-MMA items
@pytest.mark.parametrize("lens,M", [
    ([3000, 120], 20),      # 2 chunks per split, two 16-row tiles, rows of sequence 1 straddle position 128, empty splits
    ([1000, 0], 5),         # one chunk per split; an empty cache beside it
    ([255, 256], 3),        # rows start one before / exactly at a chunk boundary
])
def test_forward_over_a_long_seeded_cache_head_128(lens, M, mode):
    _forward_over_seeded_cache(synth.llama_like(2, 256, 2, 512, 512), lens, M, mode)


@pytest.mark.parametrize("mode", [2, 1])
def test_forward_many_heads_one_split_of_many_chunks(mode):
    """160 (sequence, head) pairs on 148 SMs: one split per pair, up to ten 128-position chunks each (the
    K/V ring wraps several times), some SMs run two items in a row, and lengths of 127 mod 128 put the rows
    of the pass into the last two chunks."""
    # weights x1.5: the same activation scale at d = 4096 as x6 gives at d = 256
    _forward_over_seeded_cache(synth.llama_like(1, 4096, 32, 512, 512), [1151, 127, 1152, 64, 300], 5, mode, scale=1.5)


@pytest.mark.parametrize("mode", [2, 1])
@pytest.mark.parametrize("lens,M", [([700, 90], 6), ([2100], 5), ([300, 1, 129], 2)])
def test_parallel_residual_out_projection_behind_the_attention_count(lens, M, mode):
    """Parallel-residual layers with few attention items: some CTAs run the attention items while the others
    run the MLP-out GEMM and then the out-projection, whose operand copies wait for the count of finished
    attention CTAs instead of a grid barrier.  Several layers (the count runs on from layer to layer),
    several splits per head (the last split to finish merges before its CTA signals), both attention forms."""
    _forward_over_seeded_cache(synth.neox_like(3, 256, 2, 512, 520), lens, M, mode)


@pytest.mark.parametrize("arch,lens,M", [
    (synth.llama_like(2, 256, 2, 512, 512), [3000, 120], 2),      # head 128: several splits per head, ragged lengths
    (synth.llama_like(2, 256, 2, 512, 512), [1000, 0], 1),        # one row; an empty cache beside it
    (synth.llama_like(2, 256, 2, 512, 512), [255, 7], 2),         # blocks that end inside a load; fewer positions than a block
    (synth.llama_like(2, 256, 4, 512, 512), [2100, 77, 0], 2),    # head 64: 8 lanes per position, 16 positions per block
    (synth.llama_like(2, 256, 4, 512, 512), [513, 64, 31], 1),
    (synth.neox_like(3, 256, 4, 512, 520), [700, 90], 2),         # parallel residual: the out-projection waits for the attention count
    (synth.llama_like(1, 4096, 32, 512, 512), [1151, 127, 1152, 64, 300], 2),   # 160 (sequence, head) items on 148 SMs
])
def test_one_and_two_row_passes_on_the_packed_mma_items(arch, lens, M):
    """Passes of one or two rows per sequence (draft steps, decode steps) on the warp-MMA items that carry hi and lo in
    one tile: blocks that end inside the range, empty caches, head 64 and head 128, splits and their merge."""
    _forward_over_seeded_cache(arch, lens, M, 3, scale=1.5 if arch.d_model == 4096 else 6.0)


@pytest.mark.parametrize("arch,lens,M", [
    (synth.llama_like(2, 256, 2, 512, 512), [3000, 120], 5),      # head 128: several splits per head, ragged lengths
    (synth.llama_like(2, 256, 2, 512, 512), [1000, 0], 8),        # a full tile of rows; an empty cache beside it
    (synth.llama_like(2, 256, 2, 512, 512), [255, 7], 3),         # blocks that end inside the range; fewer positions than a block
    (synth.llama_like(2, 256, 2, 512, 512), [16, 17, 15], 6),     # exactly one block / one more / one less
    (synth.llama_like(2, 256, 4, 512, 512), [2100, 77, 0], 5),    # head 64
    (synth.llama_like(2, 256, 4, 512, 512), [513, 64, 31], 4),
    (synth.neox_like(3, 256, 4, 512, 520), [700, 90], 6),         # parallel residual: the out-projection waits for the attention count
    (synth.llama_like(1, 4096, 32, 512, 512), [1151, 127, 1152, 64, 300], 5),   # 160 (sequence, head) items on 148 SMs
])
def test_passes_of_up_to_eight_rows_on_the_packed_mma_items(arch, lens, M):
    """Passes of three to eight rows per sequence take the warp-MMA items that carry the hi and lo parts of the
    queries and of the probabilities in one 16-row tile: per-warp position blocks through private copy rings, the
    rows of the pass as one more block, merge of the eight warps and of the splits."""
    _forward_over_seeded_cache(arch, lens, M, 3, scale=1.5 if arch.d_model == 4096 else 6.0)


def _forward_over_seeded_cache(arch, lens, M, mode, scale=6.0):
    """Whole verification pass (single forward kernel) of a head-128 model over a seeded cache:
    logits of all rows and the appended cache rows against the oracle.  Exercises the tensor-core
    attention (mode 2) and the warp-MMA attention (mode 1): splits of several chunks, the merge of
    splits, empty splits, more than 16 rows per sequence, and rows of the pass that cross a chunk
    boundary."""
    assert arch.head_dim in (64, 128)
    from tests import gpu_util as gu
    ws_np = gu.scaled_weights(synth, arch, 11, scale)
    model = B.Model(arch, B.upload_weights(arch, ws_np))
    omodel = od.Model(arch, ws_np)
    Bn, S = len(lens), max(lens) + 64
    kv = B.KV(model, Bn, S)
    fill = synth.gen_kv_fill(12, (arch.n_layers, Bn, 2, arch.n_heads, S, arch.head_dim), arch.dtype)
    fill_f = synth.bf16_bits_to_f32(fill) * np.float32(0.5)
    fill = synth.f32_to_bf16_bits(fill_f)            # halving is exact in bf16
    dev = "cuda"
    kv.cache_view().copy_(torch.from_numpy(fill.view(np.int16)).to(dev).view(torch.bfloat16))
    B.kv_commit(kv, torch.tensor(lens, dtype=torch.int32, device=dev))
    assert kv.lengths().tolist() == lens      # also refreshes the host-side bound the splits are planned from
    rows = synth.gen_prompt(13, Bn, M, arch.vocab)
    ws = model.new_workspace(Bn, M, S)
    V = arch.vocab
    K = M - 1
    n_acc = torch.zeros(Bn, dtype=torch.int32, device=dev)
    nxt = torch.zeros(Bn, dtype=torch.int32, device=dev)
    q = torch.full((Bn, max(K, 1), V), 1.0 / V, device=dev)
    u = torch.full((Bn, M), 0.5, device=dev)
    B.set_attention_mode(mode)
    try:
        B.target_verify(model, kv, torch.from_numpy(rows).to(dev), K, q if K else None, u, 1.0, n_acc, nxt, 1, None, ws)
        got = B.last_logits(model, Bn, M, ws).cpu().numpy()
    finally:
        B.set_attention_mode(0)
    assert kv.status() == 0
    cache = kv.cache_view().float().cpu().numpy()
    od.set_threads(8)
    for b in range(Bn):
        oc = omodel.new_cache(S)
        oc.kv[...] = fill_f[:, b]
        oc.len = lens[b]
        ref = oc.feed(rows[b], advance=False)
        gu.assert_logits_close(got[b], ref)
        n0, n1 = lens[b], lens[b] + M
        g, r = cache[:, b, :, :, n0:n1], oc.kv[:, :, :, n0:n1]
        assert (np.abs(g - r) <= gu.LOGIT_RTOL * np.abs(r) + gu.LOGIT_ATOL).all()
        assert np.array_equal(cache[:, b, :, :, :n0], fill_f[:, b, :, :, :n0])   # committed rows untouched
