"""GPU parity of the diagnostics (Sec. 4.2 / App. A): the confidence histogram is integer work decided in FP32 on both
sides (bit-exact counts); the rate-of-change sums are FP32 partial sums added in FP64 in no fixed order, compared with
the FP64 oracle to 2e-6 relative (each thread adds at most a few hundred FP32 terms)."""
import numpy as np
import pytest
import torch

import oracle as orc
import workloads
from util import numpy_to_qmat, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


@pytest.mark.parametrize("n,k,bins,scale_mode", [(768, 192, 20, 0), (1536, 384, 64, 0), (333, 96, 7, 1), (4096, 1024, 20, 0)])
def test_confidence_histogram_matches_oracle(mx, n, k, bins, scale_mode):
    rng = np.random.default_rng(n + k + bins)
    w = workloads.round_to_bf16(rng.normal(0, 0.02, (n, k)).astype(np.float32))
    w[0, :32] = 0.0                      # an all-zero group
    w[1, 5] = np.inf                     # a group that is skipped
    w[2, 32:64] = 2.0 ** -130            # below the normal range
    ref = orc.quant_conf_hist(w, bins=bins, scale_mode=scale_mode)
    h = mx.quant_conf_hist(to_dev_bf16(w), bins=bins, scale_mode=scale_mode)
    torch.cuda.synchronize()
    assert (h.cpu().numpy().astype(np.uint64) == ref).all()
    assert int(h.sum().item()) == n * k - 32
    # counts are added: a second call doubles them
    mx.quant_conf_hist(to_dev_bf16(w), bins=bins, scale_mode=scale_mode, out=h)
    assert (h.cpu().numpy().astype(np.uint64) == 2 * ref).all()


def test_confidence_histogram_argument_errors(mx):
    w = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    for kw in (dict(bins=0), dict(bins=65), dict(scale_mode=7)):
        with pytest.raises(mx.MxError):
            mx.quant_conf_hist(w, **kw)
    with pytest.raises(mx.MxError):
        mx.quant_conf_hist(torch.zeros((4, 48), dtype=torch.bfloat16, device="cuda"))


@pytest.mark.parametrize("count", [1, 7, 4096 * 1024 + 5, 25216 * 384])
def test_change_sums_bf16(mx, count):
    rng = np.random.default_rng(count % 1013)
    prev = workloads.round_to_bf16(rng.normal(0, 0.02, count).astype(np.float32))
    cur = workloads.round_to_bf16((prev + rng.normal(0, 1e-3, count)).astype(np.float32))
    d2, p2 = orc.change_sums(cur, prev)
    out = mx.change_sums(to_dev_bf16(cur), to_dev_bf16(prev))
    got = out.cpu().numpy()
    assert abs(got[0] - d2) <= 2e-6 * d2 + 1e-300 and abs(got[1] - p2) <= 2e-6 * p2


def test_change_sums_quantized_weights(mx):
    rng = np.random.default_rng(9)
    w0 = workloads.round_to_bf16(rng.normal(0, 0.02, (768, 192)).astype(np.float32))
    w1 = workloads.round_to_bf16((w0 + rng.normal(0, 2e-3, w0.shape)).astype(np.float32))
    (p0, s0, _), (p1, s1, _) = orc.quantize(w0), orc.quantize(w1)
    d2, p2 = orc.change_sums(orc.dequantize(p1, s1), orc.dequantize(p0, s0))
    out = mx.change_sums(numpy_to_qmat(mx, p1, s1), numpy_to_qmat(mx, p0, s0))
    got = out.cpu().numpy()
    assert abs(got[0] - d2) <= 2e-6 * d2 and abs(got[1] - p2) <= 2e-6 * p2
    # the rate of change of one step (App. A.3)
    assert abs(np.sqrt(got[0] / got[1]) - np.sqrt(d2 / p2)) < 1e-6
