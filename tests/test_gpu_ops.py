"""Kernel-level parity through the C ABI: the projection GEMM (fp32 check
kernel and the tcgen05 kernel) and the attention kernels against the oracle's
plain definitions, plus the selection and the index kernels."""
import numpy as np
import pytest
import torch

from oracle import dkv_oracle as O
from paper_2505_15781_b200 import binding as B
from paper_2505_15781_b200 import synth

pytestmark = pytest.mark.gpu


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


@pytest.mark.parametrize("rows,n,k", [(1, 8, 8), (37, 200, 136), (64, 64, 64), (130, 1376, 256), (5, 1000, 688)])
def test_gemm_f32_check_kernel(rows, n, k):
    r = rng(rows * 7 + n)
    x = r.standard_normal((rows, k)).astype(np.float32)
    w = (r.standard_normal((n, k)) * 0.05).astype(np.float32)
    out = torch.empty(rows, n, dtype=torch.float32, device="cuda")
    B.dkv_op_gemm(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), out, B.DKV_F32)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    np.testing.assert_allclose(out.cpu().numpy(), ref, atol=2e-5 * np.sqrt(k))


# rows span every TMA box size, ragged tails in rows / n / k, several row tiles, and split-K
GEMM_BF16_CASES = [
    (1, 128, 64, 0), (2, 256, 256, 0), (16, 128, 128, 1), (17, 384, 512, 0), (33, 768, 256, 2),
    (64, 256, 688, 0), (100, 1376, 256, 0), (130, 1024, 1024, 3), (257, 512, 1024, 0), (300, 4096, 512, 0),
    (512, 1024, 4096, 0), (700, 256, 256, 1), (8, 12288, 4096, 0), (40, 4096, 12288, 0), (3, 1000, 72, 0),
]


@pytest.mark.parametrize("xdtype", ["f16", "bf16"])
@pytest.mark.parametrize("rows,n,k,splits", GEMM_BF16_CASES)
def test_gemm_tcgen05_bf16_weights(rows, n, k, splits, xdtype):
    """Both operands fp16 (the benchmark's mode) or both bf16."""
    r = rng(rows * 13 + n + k)
    tdt, code = (torch.float16, B.DKV_F16) if xdtype == "f16" else (torch.bfloat16, B.DKV_BF16)
    x = torch.from_numpy(r.standard_normal((rows, k)).astype(np.float32)).to(tdt).cuda()
    w = torch.from_numpy((r.standard_normal((n, k)) * 0.05).astype(np.float32)).to(tdt).cuda()
    out = torch.full((rows, n), float("nan"), dtype=torch.float32, device="cuda")
    B.dkv_op_gemm(x, w, out, code, splits)
    torch.cuda.synchronize()
    ref = x.float().cpu().numpy().astype(np.float64) @ w.float().cpu().numpy().astype(np.float64).T
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    # 16-bit products are exact in fp32; only the fp32 accumulation order differs
    np.testing.assert_allclose(got, ref, atol=3e-6 * k ** 0.5 * 4, rtol=1e-5)


def make_attention_case(seed, batch, n_rows, L, hq, hkv, dh, dtype):
    r = rng(seed)
    rows = [int(n_rows[b]) for b in range(batch)]
    R = batch * max(rows)          # the entry point wants batch * rows_per_seq_bound rows allocated
    q = r.standard_normal((R, hq, dh)).astype(np.float32)
    k = r.standard_normal((batch, hkv, L, dh)).astype(np.float32)
    v = r.standard_normal((batch, hkv, L, dh)).astype(np.float32)
    tq, tk, tv = (torch.from_numpy(a).to(dtype).cuda() for a in (q, k, v))
    row_off = np.concatenate([[0], np.cumsum(rows)]).astype(np.int32)
    return rows, tq, tk, tv, torch.from_numpy(row_off).cuda()


def oracle_attention(tq, tk, tv, rows, row_off):
    q = tq.float().cpu().numpy().astype(np.float64)
    k = tk.float().cpu().numpy().astype(np.float64)
    v = tv.float().cpu().numpy().astype(np.float64)
    out = np.zeros_like(q)
    valid = np.zeros(len(q), bool)
    for b, n in enumerate(rows):
        s = slice(int(row_off[b]), int(row_off[b]) + n)
        out[s] = O.attention(q[s], k[b].transpose(1, 0, 2), v[b].transpose(1, 0, 2))
        valid[s] = True
    return out, valid


@pytest.mark.parametrize("batch,n_rows,L,hq,hkv,dh", [
    (1, [5], 40, 4, 4, 64), (2, [3, 9], 130, 4, 2, 64), (1, [1], 64, 2, 1, 128), (2, [70, 2], 200, 4, 4, 128)])
def test_attention_f32_check_kernel(batch, n_rows, L, hq, hkv, dh):
    rows, tq, tk, tv, row_off = make_attention_case(1, batch, n_rows, L, hq, hkv, dh, torch.float32)
    o = torch.zeros_like(tq)
    B.dkv_op_attention(tq, tk, tv, o, row_off, batch, max(rows), L, hq, hkv, dh, B.DKV_F32)
    ref, valid = oracle_attention(tq, tk, tv, rows, row_off.cpu().numpy())
    np.testing.assert_allclose(o.cpu().numpy()[valid], ref[valid], atol=2e-5)
    assert (o.cpu().numpy()[~valid] == 0).all()


@pytest.mark.parametrize("batch,n_rows,L,hq,hkv,dh", [
    (1, [5], 40, 4, 4, 64), (2, [3, 9], 130, 4, 2, 64), (1, [1], 64, 2, 1, 128), (2, [70, 2], 200, 4, 4, 128),
    (1, [257], 512, 8, 8, 128), (4, [64, 64, 64, 64], 768, 7, 1, 128), (1, [6], 1152, 4, 4, 128),
    (1, [129], 63, 2, 2, 64)])
@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_attention_flash_kernel_16bit(batch, n_rows, L, hq, hkv, dh, dt):
    tdt, code, ulp = (torch.float16, B.DKV_F16, 2.0 ** -11) if dt == "f16" else (torch.bfloat16, B.DKV_BF16, 2.0 ** -8)
    rows, tq, tk, tv, row_off = make_attention_case(2, batch, n_rows, L, hq, hkv, dh, tdt)
    o = torch.zeros_like(tq)
    B.dkv_op_attention(tq, tk, tv, o, row_off, batch, max(rows), L, hq, hkv, dh, code)
    ref, valid = oracle_attention(tq, tk, tv, rows, row_off.cpu().numpy())
    got = o.float().cpu().numpy()
    # P and the output are rounded to the 16-bit type (half an ulp each); values are O(1)
    np.testing.assert_allclose(got[valid], ref[valid], atol=6 * ulp, rtol=6 * ulp)
    assert np.abs(got[valid] - ref[valid]).mean() < ulp
    assert (got[~valid] == 0).all()          # rows that belong to no sequence are left alone


def test_select_unmask_bit_exact_with_ties_and_nan():
    r = rng(5)
    batch, L, lo, hi = 3, 40, 8, 37
    for k in (1, 2, 5):
        conf = r.choice([0.1, 0.25, 0.25, 0.5, np.nan], size=(batch, L)).astype(np.float32)
        masked = r.integers(0, 2, size=(batch, L)).astype(np.uint8)
        masked[:, lo:lo + k] = 1
        pred = r.integers(0, 1000, size=(batch, L)).astype(np.int32)
        tokens = np.full((batch, L), 1023, np.int32)
        t_tok, t_m = torch.from_numpy(tokens).cuda(), torch.from_numpy(masked).cuda()
        chosen = torch.empty(batch, k, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.dkv_select_unmask(torch.from_numpy(conf).cuda(), torch.from_numpy(pred).cuda(), batch, L, lo, hi, k,
                            t_tok, t_m, chosen, status)
        got = chosen.cpu().numpy()
        for b in range(batch):
            exp = O.select_unmask(conf[b].astype(np.float64), masked[b], lo, hi, k)
            assert got[b].tolist() == exp
            m2 = masked[b].copy()
            m2[exp] = 0
            np.testing.assert_array_equal(t_m[b].cpu().numpy(), m2)
            assert (t_tok[b].cpu().numpy()[exp] == pred[b][exp]).all()
        assert status.item() == 0


def test_select_unmask_reports_too_few_candidates():
    conf = torch.zeros(1, 8, device="cuda")
    pred = torch.zeros(1, 8, dtype=torch.int32, device="cuda")
    tokens = torch.zeros(1, 8, dtype=torch.int32, device="cuda")
    masked = torch.zeros(1, 8, dtype=torch.uint8, device="cuda")
    masked[0, 3] = 1
    chosen = torch.empty(1, 2, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.dkv_select_unmask(conf, pred, 1, 8, 0, 8, 2, tokens, masked, chosen, status)
    assert chosen.cpu().tolist() == [[3, -1]] and status.item() & 2


def test_generator_is_identical_on_device():
    k1, k2 = synth.tensor_key(3, 5, 7)
    a = synth.hash_u16_torch(11, 200000, k1, k2, "cuda").cpu().numpy()
    np.testing.assert_array_equal(a, synth.hash_u16_numpy(11, 200000, k1, k2))
    w = synth.normal_tensor(0, 1, "wd", (96, 200), 0.02, "bfloat16", "cuda")
    assert torch.equal(w.cpu(), synth.normal_tensor(0, 1, "wd", (96, 200), 0.02, "bfloat16", "cpu"))


def test_stream_probe_runs_to_completion_and_checks_its_arguments():
    """The measurement kernel (a ring of bulk copies without arithmetic) moves every chunk, reports no
    wait that ran out, and the entry point refuses sizes the copy engine cannot take."""
    lib = B.load()
    streamed = torch.ones(64 << 20, dtype=torch.uint8, device="cuda")
    reread = torch.ones(1 << 20, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for ctas, chunk, rechunk, stages in ((148, 32 << 10, 18 << 10, 4), (3, 16, 0, 1), (96, 32 << 10, 9 << 10, 5)):
        B.dkv_op_stream_probe(streamed, reread if rechunk else None, ctas, chunk, rechunk, stages, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    args = (streamed.data_ptr(), streamed.numel(), reread.data_ptr(), reread.numel())
    assert lib.dkv_op_stream_probe(*args, 148, 24, 0, 4, None, None) == -2               # chunk not a multiple of 16
    assert lib.dkv_op_stream_probe(*args, 148, 64 << 10, 0, 4, None, None) == -4         # ring larger than shared memory
    assert lib.dkv_op_stream_probe(*args, 0, 1024, 0, 4, None, None) == -2
    assert lib.dkv_op_stream_probe(None, 1 << 20, None, 0, 8, 1024, 0, 4, None, None) == -1
    assert lib.dkv_op_stream_probe(args[0], args[1], None, 0, 8, 1024, 512, 4, None, None) == -1   # re-read buffer missing
