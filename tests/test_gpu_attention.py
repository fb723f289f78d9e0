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
