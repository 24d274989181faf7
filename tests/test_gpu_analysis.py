"""GPU parity of the analysis kernels against the CPU oracle: the channel magnitude scan bit for bit, the quantization
error sums within the rounding of a binary64 sum taken in another order (element counts exactly)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import synth

from parity_util import configs, np16

pytestmark = pytest.mark.gpu
TINY = synth.WORKLOADS["tiny"]


@pytest.mark.parametrize("batch,seq,hidden", [(1, 256, 512), (3, 77, 4096), (2, 5, 40), (1, 1, 8), (2, 300, 2056)])
def test_channel_scan(batch, seq, hidden):
    wl = TINY.scaled(batch=batch, seq=seq, hidden=hidden, channels=tuple(c % hidden for c in TINY.channels), seed=60 + seq)
    H = synth.make_hidden(wl, "cuda")
    if seq > 2:
        H[0, 1, 3] = float("nan")
        H[0, 2, 5] = float("-inf")
    assert np.array_equal(kv.channel_absmax(H).cpu().numpy(), oracle.channel_absmax(np16(H)))
    # padded rows and an odd channel count take the per-channel kernel
    big = torch.zeros((batch, seq + 2, hidden + 24), dtype=torch.float16, device="cuda")
    big[:, :seq, :hidden] = H
    view = big[:, :seq, 3:hidden - 2]
    if view.shape[2] > 0:
        assert np.array_equal(kv.channel_absmax(view).cpu().numpy(), oracle.channel_absmax(np16(view)))


def test_channel_scan_of_no_tokens_is_zero():
    H = torch.zeros((2, 0, 64), dtype=torch.float16, device="cuda")
    assert not kv.channel_absmax(H).cpu().numpy().any()


@pytest.mark.parametrize("bits,d,group,seq", [(2, 128, 128, 300), (3, 128, 64, 200), (4, 64, 32, 130), (2, 64, 16, 50), (4, 128, 256, 600)])
@pytest.mark.parametrize("per_channel", [True, False])
@pytest.mark.parametrize("exclude", [True, False])
def test_quantization_error_split(bits, d, group, seq, per_channel, exclude):
    wl = TINY.scaled(bits=bits, head_dim=d, group=group, n_q_heads=6, n_kv_heads=3, batch=2, seq=seq, topk=7, pfn_n=2, seed=7000 + bits + group)
    ocfg, gcfg = configs(wl)
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    sinks = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, sinks)
    bm, _, _ = oracle.predict_sinks(ocfg, np16(H))
    x = K if per_channel else V
    got = kv.quant_error(gcfg, x, sinks, per_channel, exclude).cpu().numpy()
    want = oracle.quant_error(ocfg, np16(x), bm, per_channel, exclude)
    assert got[1] == want[1] and got[3] == want[3]                       # element counts are exact
    assert np.allclose(got[[0, 2]], want[[0, 2]], rtol=1e-11, atol=0)   # binary64 sums in another order
    # strided input ([B, S, H, D] storage)
    xt = x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    got2 = kv.quant_error(gcfg, xt, sinks, per_channel, exclude).cpu().numpy()
    assert np.allclose(got2, want, rtol=1e-11, atol=0)
