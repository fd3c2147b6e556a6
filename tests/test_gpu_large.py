"""The largest sizes: a gradient-shaped tensor with more than 2^32 elements (the stochastic-rounding counters pass
2^32, every offset needs 64 bits, the token count is not a multiple of 128) through the two-axis quantizer, and the
product with a small weight.  Checked on sampled rows / slabs that the oracle computes by itself."""
import numpy as np
import pytest
import torch

import oracle as orc
from util import check_gemm_bound

pytestmark = pytest.mark.gpu

ROWS, COLS = (1 << 20) + 160, 4096          # 4.295e9 elements; 1048736 = 8193 * 128 + 32


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


@pytest.fixture(scope="module")
def big(mx):
    free, _ = torch.cuda.mem_get_info()
    if free < 24 << 30:
        pytest.skip("needs 24 GB of free device memory")
    g = torch.Generator(device="cuda").manual_seed(20853)
    x = torch.empty((ROWS, COLS), dtype=torch.bfloat16, device="cuda")
    step = 1 << 16
    for r in range(0, ROWS, step):          # heavy-tailed small values, like a gradient
        n = min(step, ROWS - r)
        t = torch.randn((n, COLS), device="cuda", generator=g) * torch.exp(torch.randn((n, 1), device="cuda", generator=g))
        x[r:r + n] = (t * 1e-3).to(torch.bfloat16)
    seed = 0x5EED0000 + 77
    st = mx.new_status()
    q, qt = mx.quantize_2axis(x, (0, 1, seed, 3), (0, 1, seed, 5), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    yield x, q, qt, seed
    del x, q, qt
    torch.cuda.empty_cache()


def rows_of(t, idx, as_float=False):
    sel = t[torch.as_tensor(idx, device=t.device)]
    return (sel.float() if as_float else sel).cpu().numpy()


def test_rowwise_operand_beyond_2_to_32_elements(mx, big):
    x, q, qt, seed = big
    rng = np.random.default_rng(1)
    rows = sorted(set(rng.integers(0, ROWS, 12).tolist()) | {0, ROWS - 1, ROWS - 33, (1 << 20) - 1, 1 << 20})
    xs = rows_of(x, rows, as_float=True)
    p = rows_of(q.data, rows)
    s = rows_of(q.scales_linear(), rows)
    for k, r in enumerate(rows):
        pr, sr, _ = orc.quantize(np.ascontiguousarray(xs[k:k + 1]), rounding=1, seed=seed, stream_id=3, out_row0=int(r), out_ld=COLS)
        assert (s[k] == sr[0]).all(), "scales of row %d" % r
        assert (p[k] == pr[0]).all(), "codes of row %d" % r


def test_transposed_operand_beyond_2_to_32_elements(mx, big):
    x, q, qt, seed = big
    # 32-row groups x 32-column blocks; the last column block with late rows has output indices above 2^32
    for r0, c0 in [(0, 0), (ROWS - 32, COLS - 32), (1 << 20, COLS - 32), (524288, 2048), (ROWS - 160, 32)]:
        sub = x[r0:r0 + 32, c0:c0 + 32].float().cpu().numpy()
        ps, ss, _ = orc.quantize(np.ascontiguousarray(sub), transpose=True, rounding=1, seed=seed, stream_id=5,
                                 out_row0=int(c0), out_col0=int(r0), out_ld=ROWS)
        gp = qt.data[c0:c0 + 32, r0 // 2:r0 // 2 + 16].cpu().numpy()
        gs = qt.scales_linear()[c0:c0 + 32, r0 // 32].cpu().numpy()
        assert (gs == ss[:, 0]).all(), "scales at rows %d, cols %d" % (r0, c0)
        assert (gp == ps).all(), "codes at rows %d, cols %d" % (r0, c0)
    assert (COLS - 1) * ROWS + ROWS - 1 >= 1 << 32     # the last slab's output indices pass 2^32


def test_product_with_8194_row_tiles(mx, big):
    x, q, qt, seed = big
    n = 256
    g = torch.Generator(device="cuda").manual_seed(5)
    w = (torch.randn((n, COLS), device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    wq = mx.quantize(w)
    st = mx.new_status()
    y = mx.gemm(q, wq, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    rng = np.random.default_rng(2)
    rows = sorted(set(rng.integers(0, ROWS, 20).tolist()) | {0, 127, 128, ROWS - 1, ROWS - 32, ROWS - 33})
    pa, sa = rows_of(q.data, rows), rows_of(q.scales_linear(), rows)
    pb, sb = wq.data.cpu().numpy(), wq.scales_linear().cpu().numpy()
    dref, tref = orc.gemm(pa, sa, pb, sb)
    check_gemm_bound(rows_of(y, rows, as_float=True), dref, tref, True, "Y on sampled rows of 1048736")
