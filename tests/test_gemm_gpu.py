"""GPU parity of the tensor-core weight-streaming GEMM (sjd_gemm through the C-ABI) against a plain
fp64 matrix product of the same bf16 weights and fp32 activations."""
import numpy as np
import pytest
import torch

from paper_2410_01699_b200 import binding as B

pytestmark = pytest.mark.gpu


def _case(m, n, k, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(m, k, generator=g, dtype=torch.float32)
    w = (torch.randn(n, k, generator=g, dtype=torch.float32) * 0.05).to(torch.bfloat16)
    ref = x.to(torch.float64).numpy() @ w.to(torch.float64).numpy().T      # the definition, fp64
    return x, w, ref


def _tolerance(x, w, k):
    # activations carry bf16 hi + lo (relative 2^-17 per element), products accumulate in fp32
    scale = float(np.sqrt(k) * x.abs().max() * w.to(torch.float32).abs().max())
    return 3e-5 * scale + 1e-6


@pytest.mark.parametrize("m,n,k", [
    (32, 128, 64),        # one tile, one k-block
    (32, 256, 4096),      # two tiles over all CTAs: every segment partial
    (32, 4096, 4096),     # the attention output projection of the 7B shape
    (32, 1024, 11008),    # long K (SwiGLU down projection), 172 k-blocks
    (17, 384, 512),       # ragged row count (padded to 32 columns of the MMA)
    (1, 128, 128),        # single row
    (64, 2048, 1024),     # W = 64
    (128, 512, 256),      # widest supported window batch
    (32, 65536, 512),     # 512 tiles (vocabulary-sized N)
    (112, 768, 1024),     # 112 rows in one slab: accumulators of 224 columns
    (128, 22016, 4096),   # four images x W = 32 on the gate|up projection: 172 tiles on 148 SMs
    (129, 256, 512),      # first row count cut into token slabs: two of 80 rows (the second holds 49)
    (256, 1024, 1024),    # two full slabs of 128 rows
    (300, 384, 640),      # three ragged slabs of 112 rows (the last holds 76)
    (512, 4096, 4096),    # 8 images x W = 64 on the attention output projection: 4 slabs x 32 tiles x K splits
    (1024, 256, 256),     # most rows covered: eight slabs
])
def test_gemm_matches_fp64_product(m, n, k):
    x, w, ref = _case(m, n, k, seed=m + n + k)
    out, status = B.sjd_gemm(x.cuda(), w.cuda())
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a device-side wait ran out"
    got = out.cpu().to(torch.float64).numpy()
    err = np.abs(got - ref).max()
    assert err <= _tolerance(x, w, k), f"max |err| {err:.3e}"


def test_gemm_wide_rows_do_not_mix():
    """Each token row of a many-row product depends on its own activations only: rows of a 512-row call
    equal the same rows computed in a call of their own slab size (catches a wrong slab offset)."""
    x, w, _ = _case(512, 512, 1024, seed=5)
    full, st = B.sjd_gemm(x.cuda(), w.cuda())
    part, _ = B.sjd_gemm(x[256:].contiguous().cuda(), w.cuda())
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert torch.equal(full[256:], part)


def test_gemm_accumulates_and_is_deterministic():
    x, w, ref = _case(32, 1024, 2048, seed=9)
    base = torch.full((32, 1024), 0.5, dtype=torch.float32, device="cuda")
    out, status = B.sjd_gemm(x.cuda(), w.cuda(), out=base.clone(), accumulate=True)
    out2, _ = B.sjd_gemm(x.cuda(), w.cuda(), out=base.clone(), accumulate=True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out, out2)
    assert np.abs(out.cpu().to(torch.float64).numpy() - (ref + 0.5)).max() <= _tolerance(x, w, 2048)


def test_gemm_rejects_uncovered_shapes():
    x = torch.zeros(8, 96, device="cuda")
    w = torch.zeros(128, 96, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.SJDError) as e:
        B.sjd_gemm(x, w)                      # K not a multiple of 64
    assert e.value.status == B.SJD_ERR_UNSUPPORTED
    assert B.lib().sjd_gemm_workspace_bytes(1025, 128, 64) == 0
