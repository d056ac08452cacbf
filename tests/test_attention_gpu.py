"""GPU parity of the tensor-core window attention (sjd_attention through the C-ABI) against the
definition in fp64: softmax(q k^T / sqrt(d)) v over the cache rows each query may see."""
import numpy as np
import pytest
import torch

from paper_2410_01699_b200 import binding as B

pytestmark = pytest.mark.gpu


def _reference(q, kv, pos, window, n_kv_heads):
    m, h, hd = q.shape
    group = h // n_kv_heads
    out = np.zeros((m, h, hd))
    q64, kv64 = q.double().numpy(), kv.to(torch.float64).numpy()
    for r in range(m):
        b, p = r // window, int(pos[r])
        if p < 0:
            continue
        for head in range(h):
            k = kv64[b, 0, head // group, :p + 1]
            v = kv64[b, 1, head // group, :p + 1]
            s = k @ q64[r, head] / np.sqrt(hd)
            w = np.exp(s - s.max())
            out[r, head] = (w / w.sum()) @ v
    return out


@pytest.mark.parametrize("batch,window,prefix,heads,kv_heads,hd", [
    (1, 32, 100, 32, 32, 128),    # the 7B shape early in an image
    (1, 32, 1500, 4, 4, 128),     # long prefix: many tiles per split (few heads keep the fp64 check cheap)
    (2, 64, 300, 8, 2, 128),      # grouped-query heads, W = 64, two sequences
    (3, 16, 70, 8, 2, 64),        # head_dim 64
    (1, 5, 1, 4, 4, 64),          # first step after a one-token prompt: query k sees k + 1 rows
    (1, 24, 64, 4, 1, 128),       # window not a multiple of 16, one kv head
    (5, 16, 90, 32, 8, 64),       # 160 (head, sequence) pairs: one key range each, output written without a merge
    (10, 32, 130, 32, 32, 128),   # the same at the 7B head shape, W = 32
])
def test_attention_matches_definition(batch, window, prefix, heads, kv_heads, hd):
    g = torch.Generator().manual_seed(prefix + window)
    max_seq = prefix + window + 3
    q = torch.randn(batch * window, heads, hd, generator=g)
    kv = torch.randn(batch, 2, kv_heads, max_seq, hd, generator=g).to(torch.bfloat16)
    pos = (prefix - 1 + torch.arange(window, dtype=torch.int32)).repeat(batch)
    if window > 8:
        pos[-3:] = -1                       # inactive rows (a window shortened at the end of the image)
    out, status = B.sjd_attention(q.cuda(), kv.cuda(), pos.cuda(), window, kv_heads)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = _reference(q, kv, pos, window, kv_heads)
    err = np.abs(out.cpu().double().numpy() - ref).max()
    # q and the probabilities carry bf16 hi + lo parts (2^-17 relative), accumulation in fp32
    assert err <= 2e-4, f"max |err| {err:.3e}"
    assert torch.all(out[pos.cuda() < 0] == 0)


def test_attention_rejects_uncovered_shapes():
    assert B.lib().sjd_attention_workspace_bytes(1, 32, 8, 96) == 0
    assert B.lib().sjd_attention_workspace_bytes(1, 65, 8, 128) == 0
