"""Unit parity of single operations against the CPU oracle (GPU required)."""
import numpy as np
import pytest
import torch

from oracle import wd_oracle as wo
from paper_2601_20332_b200 import binding as wd
from paper_2601_20332_b200 import build as wd_build

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def built():
    wd_build.build()
    assert wd.lib() is not None


def _ref_gemm(x, w):
    return x.double().cpu().numpy() @ w.double().cpu().numpy().T


GEMM_SHAPES = [  # rows, n, k  (ragged token counts, several tiles, ragged weight-row tail)
    (1, 128, 64), (7, 256, 128), (16, 128, 512), (34, 384, 1024), (35, 640, 4096), (68, 512, 2048),
    (130, 256, 1024), (256, 384, 512), (300, 256, 1024), (352, 512, 768), (700, 384, 512), (34, 200, 256),
    (10, 1000, 264), (512, 1000, 264), (1030, 256, 2048), (264, 130, 72),
    # wide weight matrices with every CTA pair getting two units: two accumulators per weight stage
    # (token super-tiles of 2 x 160 and 3 x 2 x 192 rows, ragged last weight tile)
    (300, 38016, 128), (1100, 16640, 192),
]


@pytest.mark.parametrize("rows,n,k", GEMM_SHAPES)
def test_gemm_tcgen05_vs_oracle(rows, n, k):
    g = torch.Generator(device=DEV).manual_seed(rows * 1000 + n + k)
    x = torch.randn(rows, k, device=DEV, generator=g).to(torch.bfloat16)
    w = (torch.randn(n, k, device=DEV, generator=g) * 0.05).to(torch.bfloat16)
    y = wd.op_gemm(x, w, wd.WD_GEMM_TCGEN05)
    assert wd.op_status() == 0
    ref = _ref_gemm(x, w)
    got = y.cpu().numpy().astype(np.float64)
    # bf16 inputs are exact on both sides; only the fp32 accumulation order differs
    err = np.abs(got - ref).max() / np.abs(ref).max()
    assert err < 2e-5, err
    # without scratch: single K slice straight into y
    y1 = wd.op_gemm(x, w, wd.WD_GEMM_TCGEN05, scratch=torch.empty(256, dtype=torch.uint8, device=DEV))
    assert np.abs(y1.cpu().numpy() - ref).max() / np.abs(ref).max() < 2e-5


@pytest.mark.parametrize("rows,n,k", [(1, 128, 128), (34, 384, 1024), (35, 640, 4096), (130, 200, 272), (300, 256, 1024),
                                      (700, 384, 512), (34, 1000, 144)])
def test_gemm_fp8_vs_oracle(rows, n, k):
    """Identical bf16 inputs on both sides, so the e4m3 codes and scales agree exactly and only the
    fp32 accumulation differs from the oracle's float64 product of the quantised operands."""
    g = torch.Generator(device=DEV).manual_seed(rows * 1000 + n + k)
    x = torch.randn(rows, k, device=DEV, generator=g).to(torch.bfloat16)
    w = (torch.randn(n, k, device=DEV, generator=g) * 0.05).to(torch.bfloat16)
    y = wd.op_gemm_fp8(x, w)
    assert wd.op_status() == 0
    ref = wo.fp8_matmul(x.float().cpu().numpy().astype(np.float64), w.float().cpu().numpy().astype(np.float64))
    got = y.cpu().numpy().astype(np.float64)
    assert np.abs(got - ref).max() <= 2e-5 * np.abs(ref).max()
    exact = x.double().cpu().numpy() @ w.double().cpu().numpy().T
    assert 5e-3 < np.linalg.norm(got - exact) / np.linalg.norm(exact) < 8e-2      # it really is an 8-bit product


@pytest.mark.parametrize("rows,n,k", [(1, 128, 256), (34, 384, 1024), (35, 640, 4096), (130, 200, 512), (300, 256, 1024),
                                      (700, 384, 768), (34, 1000, 256), (48, 12288, 4096)])
def test_gemm_nvfp4_vs_oracle(rows, n, k):
    """Identical bf16 inputs on both sides, so the e2m1 codes, the e4m3 block scales and the row scales agree
    exactly (both sides take every rounding decision in float32) and only the fp32 accumulation differs from
    the oracle's float64 sum over the blocks."""
    g = torch.Generator(device=DEV).manual_seed(rows * 1000 + n + k)
    x = torch.randn(rows, k, device=DEV, generator=g).to(torch.bfloat16)
    w = (torch.randn(n, k, device=DEV, generator=g) * 0.05).to(torch.bfloat16)
    y = wd.op_gemm_fp4(x, w)
    assert wd.op_status() == 0
    ref = wo.nvfp4_matmul(x.float().cpu().numpy().astype(np.float64), w.float().cpu().numpy().astype(np.float64))
    got = y.cpu().numpy().astype(np.float64)
    assert np.abs(got - ref).max() <= 2e-5 * np.abs(ref).max()
    exact = x.double().cpu().numpy() @ w.double().cpu().numpy().T
    assert 3e-2 < np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.25        # it really is a 4-bit product


def test_nvfp4_quantise_once_multiply_many_and_the_stored_format():
    """wd_op_nvfp4_quantize + wd_op_gemm_nvfp4 give the bits of wd_op_gemm_fp4, and the stored operand is the
    oracle's quantisation: codes two per byte (even element in the low nibble), e4m3 block scales, float row scales."""
    rows, n, k = 37, 300, 768
    g = torch.Generator(device=DEV).manual_seed(5)
    x = torch.randn(rows, k, device=DEV, generator=g).to(torch.bfloat16)
    x[3] = 0                                                    # an all-zero row: row scale 1, every code 0
    x[5, 32:48] = 0                                             # an all-zero block: block scale 0
    w = (torch.randn(n, k, device=DEV, generator=g) * 0.05).to(torch.bfloat16)
    xq, wq = wd.op_nvfp4_quantize(x), wd.op_nvfp4_quantize(w)
    y1 = wd.op_gemm_nvfp4(xq, wq, rows, n, k)
    y2 = wd.op_gemm_nvfp4(xq, wq, rows, n, k)
    assert torch.equal(y1, y2) and torch.equal(y1, wd.op_gemm_fp4(x, w)) and wd.op_status() == 0
    q, s, gr = wo.nvfp4_quant_rows(x.float().cpu().numpy().astype(np.float64))
    raw = xq.cpu().numpy()
    up = lambda v: (v + 255) // 256 * 256
    codes = raw[: rows * k // 2].reshape(rows, k // 2)
    sf = raw[up(rows * k // 2): up(rows * k // 2) + rows * k // 16].reshape(rows, k // 16)
    g_off = up(rows * k // 2) + up(rows * k // 16)
    gs = raw[g_off: g_off + 4 * rows].view(np.float32)
    grid = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
    val = lambda c: np.where(c & 8, -1.0, 1.0) * grid[c & 7]
    got = np.empty((rows, k))
    got[:, 0::2] = val(codes & 15)
    got[:, 1::2] = val(codes >> 4)
    np.testing.assert_array_equal(np.abs(got), np.abs(q))       # (-0 and +0 are the same element)
    np.testing.assert_array_equal(np.sign(got) * (got != 0), np.sign(q) * (q != 0))
    np.testing.assert_array_equal(torch.from_numpy(sf.copy()).view(torch.float8_e4m3fn).double().numpy(), s)
    np.testing.assert_array_equal(gs, gr)
    assert gs[3] == 1.0 and not codes[3].any() and sf[5, 2] == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("rows,n,k", [(1, 5, 3), (10, 70, 33), (34, 384, 256), (97, 130, 1000)])
def test_gemm_plain_vs_oracle(dtype, rows, n, k):
    g = torch.Generator(device=DEV).manual_seed(7)
    x = torch.randn(rows, k, device=DEV, generator=g).to(dtype)
    w = torch.randn(n, k, device=DEV, generator=g).to(dtype)
    y = wd.op_gemm(x, w, wd.WD_GEMM_PLAIN)
    ref = _ref_gemm(x, w)
    assert np.abs(y.cpu().numpy() - ref).max() / np.abs(ref).max() < 2e-5


def test_gemm_bad_arguments():
    x = torch.zeros(4, 64, device=DEV, dtype=torch.bfloat16)
    w = torch.zeros(128, 64, device=DEV, dtype=torch.bfloat16)
    y = torch.zeros(4, 128, device=DEV)
    L = wd.lib()
    assert L.wd_op_gemm(wd.WD_BF16, wd.WD_GEMM_TCGEN05, None, w.data_ptr(), y.data_ptr(), 4, 128, 64, None, 0, None) == wd.WD_ERR_NULL
    assert L.wd_op_gemm(wd.WD_BF16, wd.WD_GEMM_TCGEN05, x.data_ptr(), w.data_ptr(), y.data_ptr(), 0, 128, 64, None, 0, None) == wd.WD_ERR_BAD_PARAM
    assert L.wd_op_gemm(wd.WD_F32, wd.WD_GEMM_TCGEN05, x.data_ptr(), w.data_ptr(), y.data_ptr(), 4, 128, 64, None, 0, None) == wd.WD_ERR_BAD_PARAM
    # K must keep rows 16-byte aligned for TMA
    assert L.wd_op_gemm(wd.WD_BF16, wd.WD_GEMM_TCGEN05, x.data_ptr(), w.data_ptr(), y.data_ptr(), 4, 128, 60, None, 0, None) == wd.WD_ERR_BAD_PARAM


ATTN_CASES = [  # rows, n_vis, Hq, Hkv, dh, S
    (1, 1, 4, 4, 64, 8), (3, 5, 4, 2, 64, 16), (10, 56, 4, 4, 64, 96), (34, 352, 8, 8, 128, 512),
    (35, 333, 14, 2, 128, 400), (5, 1000, 7, 1, 128, 1024),
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("rows,nv,Hq,Hkv,dh,S", ATTN_CASES)
def test_attention_vs_oracle(dtype, rows, nv, Hq, Hkv, dh, S):
    g = torch.Generator(device=DEV).manual_seed(rows + nv)
    q = (torch.randn(rows, Hq, dh, device=DEV, generator=g) * 1.5).to(dtype)
    kc = torch.randn(Hkv, S, dh, device=DEV, generator=g).to(dtype)
    vc = torch.randn(Hkv, S, dh, device=DEV, generator=g).to(dtype)
    vis_np = np.sort(np.random.default_rng(nv).choice(S, size=nv, replace=False)).astype(np.int32)
    # poison what must not be read
    hidden = np.setdiff1d(np.arange(S), vis_np)
    if len(hidden):
        kc[:, torch.as_tensor(hidden, device=DEV)] = float("nan")
        vc[:, torch.as_tensor(hidden, device=DEV)] = float("nan")
    vis = torch.as_tensor(vis_np, device=DEV)
    out = wd.op_attention(q, kc, vc.transpose(1, 2).contiguous(), vis).float().cpu().numpy().astype(np.float64)
    K = kc.double().cpu().numpy().transpose(1, 0, 2)[vis_np]
    V = vc.double().cpu().numpy().transpose(1, 0, 2)[vis_np]
    ref, _ = wo.attention_rows(q.double().cpu().numpy(), K, V, Hq // Hkv)
    tol = 2e-2 if dtype == torch.bfloat16 else 1e-5
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() / np.abs(ref).max() < tol


# The tensor-core attention kernel alone: rows and visible lengths around the 128-wide tiles, MHA and a
# 7:1 query group, mild and large score magnitudes (q scale 8 puts the row maxima of different key tiles
# tens of units apart, so the running maximum moves and earlier tiles are rescaled), NaN in every cache
# row that must not be read, and key splits that leave CTAs of a cluster without a key tile.
ATTN_TC_CASES = [  # rows, n_vis, Hq, Hkv, S, q scale, max_vis (0 = n_vis)
    (1, 1, 1, 1, 8, 1.5, 0), (1, 127, 1, 1, 128, 8.0, 0), (127, 128, 1, 1, 136, 1.5, 0), (128, 129, 1, 1, 256, 8.0, 0),
    (129, 127, 7, 1, 128, 1.5, 0), (300, 1025, 1, 1, 1032, 8.0, 0), (34, 352, 8, 8, 512, 1.5, 0),
    (35, 3072, 7, 1, 3072, 8.0, 0), (129, 1025, 14, 2, 1040, 1.5, 0), (5, 3072, 1, 1, 3072, 1.5, 0),
    # max_vis > n_vis: the split is sized for 8 or 24 key tiles, this sequence has 1, 2 or 3
    (34, 129, 1, 1, 1024, 8.0, 1024), (1, 1, 7, 1, 3072, 1.5, 3072), (130, 300, 2, 2, 1024, 1.5, 1000),
    # grouped-query heads with few rows: 4 heads per tile (<= 32 rows, slots of 32), 2 heads per tile (<= 64 rows),
    # groups that leave the last tile with an empty slot (7 = 4 + 3, 3 = 2 + 1), 65 rows (no packing)
    (32, 700, 8, 2, 704, 8.0, 0), (33, 500, 8, 2, 512, 1.5, 0), (64, 260, 4, 2, 264, 8.0, 0), (65, 260, 4, 2, 264, 1.5, 0),
    (20, 129, 12, 4, 136, 8.0, 1024), (7, 1300, 28, 4, 1304, 1.5, 0),
]


@pytest.mark.parametrize("rows,nv,Hq,Hkv,S,qs,mv", ATTN_TC_CASES)
def test_attention_tc_kernel_vs_oracle(rows, nv, Hq, Hkv, S, qs, mv):
    dh = 128
    g = torch.Generator(device=DEV).manual_seed(rows * 7 + nv)
    q = (torch.randn(rows, Hq, dh, device=DEV, generator=g) * qs).to(torch.bfloat16)
    kc = torch.randn(Hkv, S, dh, device=DEV, generator=g).to(torch.bfloat16)
    vc = torch.randn(Hkv, S, dh, device=DEV, generator=g).to(torch.bfloat16)
    K = kc.double().cpu().numpy().transpose(1, 0, 2)[:nv]
    V = vc.double().cpu().numpy().transpose(1, 0, 2)[:nv]
    kc[:, nv:] = float("nan")                     # what must not be read as a value
    vc[:, nv:] = float("nan")
    out = wd.op_attention_tc(q, kc, vc.transpose(1, 2).contiguous(), nv, mv).float().cpu().numpy().astype(np.float64)
    assert wd.op_status() == 0
    ref, probs = wo.attention_rows(q.double().cpu().numpy(), K, V, Hq // Hkv)
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() / np.abs(ref).max() < 2e-2
    if qs >= 8 and nv > 128:
        assert probs.max() > 0.5                  # the large-scale cases really are peaked


@pytest.mark.parametrize("n,V,K", [(6, 20000, 256), (34, 126464, 128), (130, 5001, 64), (300, 4099, 64)])
def test_lm_head_epilogue_statistics_exact_ties(n, V, K):
    """The LM-head GEMM's epilogue (per-CTA running maximum / lowest argmax / sum of exponentials, merged
    by the selection kernel) on constructed ties: two identical LM-head rows in different 128-row tiles
    and different CTAs (the token must be the lower id), an all-zero hidden row (every logit 0: token 0,
    confidence 1 / V), and two identical hidden rows (equal confidence: the lower position ranks first).
    The rule itself is checked on the GPU's own logits, which the operation also returns."""
    g = torch.Generator(device=DEV).manual_seed(n + V)
    x = torch.randn(n, K, device=DEV, generator=g).to(torch.bfloat16)
    w = (torch.randn(V, K, device=DEV, generator=g) * 0.05).to(torch.bfloat16)
    lo, hi = 77, V - 130                                   # far apart: different tiles, different CTAs
    x[1] = 0                                               # all-zero hidden row
    x[4] = x[2]                                            # duplicated hidden row
    w[lo] = (x[2].float() * 0.25).to(torch.bfloat16)       # the largest logit of rows 2 and 4, twice
    w[hi] = w[lo]
    pos_np = (np.arange(n) * 3 + 5).astype(np.int32)
    k = min(4, n)
    got = wd.op_lm_unmask(x, w, torch.as_tensor(pos_np, device=DEV), k)
    assert wd.op_status() == 0
    logits = got["logits"].cpu().numpy()
    exact = x.double().cpu().numpy() @ w.double().cpu().numpy().T
    assert np.abs(logits - exact).max() <= 2e-5 * np.abs(exact).max()
    um = wo.oracle_unmask(logits, pos_np.tolist(), k)
    assert got["row_token"].tolist() == um["ids"].tolist()
    assert logits[2, lo] == logits[2, hi] == logits[2].max() and got["row_token"][2] == lo and got["row_token"][4] == lo
    assert got["row_token"][1] == 0
    np.testing.assert_allclose(got["row_conf"][1], 1.0 / V, rtol=1e-6)
    np.testing.assert_allclose(got["row_sumexp"], 1.0 / um["conf"], rtol=1e-7)
    assert got["row_sumexp"][2] == got["row_sumexp"][4]                  # identical rows: identical bits
    assert got["positions"] == um["positions"] and got["token_ids"] == um["token_ids"]
    i2, i4 = got["positions"].index(int(pos_np[2])), got["positions"].index(int(pos_np[4]))
    assert i4 == i2 + 1                                                  # rows 2 and 4 lead (their logit is huge), lower position first


@pytest.mark.parametrize("n,V,k", [(1, 2, 1), (8, 1024, 1), (32, 126464, 1), (64, 126464, 2), (5, 1000, 9), (7, 333, 0)])
def test_unmask_vs_oracle_bit_exact(n, V, k):
    g = torch.Generator(device=DEV).manual_seed(n * V)
    logits = torch.randn(n, V, device=DEV, generator=g) * 1.3
    pos_np = np.sort(np.random.default_rng(n).choice(4096, size=n, replace=False)).astype(np.int32)
    got = wd.op_unmask(logits, torch.as_tensor(pos_np, device=DEV), k)
    um = wo.oracle_unmask(logits.cpu().numpy(), pos_np.tolist(), k)
    assert got["row_token"].tolist() == um["ids"].tolist()
    np.testing.assert_allclose(got["row_conf"], um["conf"], rtol=2e-5)
    assert got["positions"] == um["positions"]
    assert got["token_ids"] == um["token_ids"]


def test_unmask_exact_ties():
    V = 777
    logits = torch.zeros(6, V, device=DEV)
    logits[1, [50, 400]] = 3.0                      # two equal maxima -> lowest index
    logits[4] = logits[1]                           # duplicated row -> equal confidence -> lowest position
    logits[2, 9] = 50.0
    pos = torch.tensor([3, 5, 8, 13, 21, 34], dtype=torch.int32, device=DEV)
    got = wd.op_unmask(logits, pos, 4)
    um = wo.oracle_unmask(logits.cpu().numpy(), pos.cpu().tolist(), 4)
    assert got["row_token"].tolist() == um["ids"].tolist() == [0, 50, 9, 0, 50, 0]
    assert got["positions"] == um["positions"] == [8, 5, 21, 3]
    assert got["row_conf"][1] == got["row_conf"][4]                     # identical rows give identical bits
    np.testing.assert_allclose(got["row_conf"][0], 1.0 / V, rtol=1e-6)  # all-equal logits: 1 / V
    assert abs(got["row_conf"][2] - 1.0) < 1e-6


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    """A device-side wait that nothing satisfies gives up after its iteration limit, the kernel
    returns normally with WD_ERR_DEVICE_TIMEOUT in the status word (no trap, no hang), the word is
    cleared by reading it, and the next operation on the same context works."""
    assert wd.op_status() == 0
    wd.debug_wait_expire()
    assert wd.op_status() == wd.WD_ERR_DEVICE_TIMEOUT
    assert wd.op_status() == 0
    g = torch.Generator(device=DEV).manual_seed(5)
    x = torch.randn(34, 256, device=DEV, generator=g).to(torch.bfloat16)
    w = (torch.randn(384, 256, device=DEV, generator=g) * 0.05).to(torch.bfloat16)
    y = wd.op_gemm(x, w, wd.WD_GEMM_TCGEN05)
    assert wd.op_status() == 0
    assert np.abs(y.cpu().numpy() - _ref_gemm(x, w)).max() / np.abs(_ref_gemm(x, w)).max() < 2e-5
