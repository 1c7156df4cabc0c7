"""The allocation-free GEMM entry point (dkv_op_gemm_static) against the
regular one (dkv_op_gemm), through the C ABI.

Who needs it: code that must issue a projection at a moment when it may not
allocate device memory (on a serving thread whose pool is fixed at start-up,
inside a process whose device memory belongs to another framework).
The entry point keeps the split-K partial sums in a fixed array inside the
library, so successive calls share that array and see each other's leftovers.
The test therefore makes two calls in a row with different shapes and checks
each result, and it must pass both as the first GPU work of a fresh process
and after every other test (this file is collected last)."""
import numpy as np
import pytest
import torch

from paper_2505_15781_b200 import binding as B

pytestmark = pytest.mark.gpu


def case(rows, n, k, dtype, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    tdt = torch.float16 if dtype == B.DKV_F16 else torch.bfloat16
    x = torch.randn(rows, k, generator=g).to(tdt).cuda()
    w = (torch.randn(n, k, generator=g) * 0.05).to(tdt).cuda()
    return x, w


def test_static_scratch_gemm_matches_workspace_gemm_on_two_calls_in_a_row():
    assert B.dkv_static_scratch_bytes() == 16 << 20
    # first call: large partials (3 splits of 130 x 4096 floats); second call: a smaller
    # problem that lands on top of the first call's leftovers
    for rows, n, k, splits, dtype, seed in [(130, 4096, 1024, 3, B.DKV_F16, 1), (17, 384, 512, 0, B.DKV_BF16, 2)]:
        x, w = case(rows, n, k, dtype, seed)
        ref = torch.empty(rows, n, dtype=torch.float32, device="cuda")
        got = torch.full((rows, n), float("nan"), dtype=torch.float32, device="cuda")
        workspace = B.dkv_op_gemm(x, w, ref, dtype, splits)
        torch.cuda.synchronize()
        # the entry point must not allocate: torch's allocator must not grow and the device's free memory
        # must not shrink across the call (every tensor of the test is alive on both sides of it)
        held, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        B.dkv_op_gemm_static(x, w, got, dtype, splits)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() <= held and torch.cuda.mem_get_info()[0] >= free_before
        del workspace
        exact = x.float().cpu().numpy().astype(np.float64) @ w.float().cpu().numpy().astype(np.float64).T
        # same tolerance as the GEMM parity tests: fp32 accumulation order only
        np.testing.assert_allclose(got.cpu().numpy(), ref.cpu().numpy(), atol=3e-6 * k ** 0.5 * 4, rtol=1e-5)
        np.testing.assert_allclose(got.cpu().numpy(), exact, atol=3e-6 * k ** 0.5 * 4, rtol=1e-5)


def test_static_scratch_gemm_rejects_what_does_not_fit():
    x, w = case(16, 128, 64, B.DKV_F16, 3)
    out = torch.empty(16, 128, dtype=torch.float32, device="cuda")
    big_x = torch.empty(1200, 64, dtype=torch.float16, device="cuda")
    big_w = torch.empty(4096, 64, dtype=torch.float16, device="cuda")
    big_out = torch.empty(1200, 4096, dtype=torch.float32, device="cuda")
    with pytest.raises(B.DkvError) as e:                       # one slab = 18.75 MiB > 16 MiB
        B.dkv_op_gemm_static(big_x, big_w, big_out, B.DKV_F16)
    assert e.value.status == -4
    with pytest.raises(B.DkvError) as e:                       # 9 slabs of 2 MiB do not fit
        B.dkv_op_gemm_static(torch.empty(128, 640, dtype=torch.float16, device="cuda"),
                             torch.empty(4096, 640, dtype=torch.float16, device="cuda"),
                             torch.empty(128, 4096, dtype=torch.float32, device="cuda"), B.DKV_F16, 9)
    assert e.value.status == -4
    with pytest.raises(B.DkvError) as e:
        B.dkv_op_gemm_static(x.float(), w.float(), out, B.DKV_F32)
    assert e.value.status == -6
    B.dkv_op_gemm_static(x, w, out, B.DKV_F16)                 # still usable afterwards
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()
