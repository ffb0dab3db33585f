"""One-shot magnitude pruning on the GPU: masks bit-identical to the oracle's (both sides decide on fp64
sums of exact squares taken in the same order), and the pruned layer runs through pack + kernel."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from util import TOL_BF16, dev, floored_rel_err, host

pytestmark = pytest.mark.gpu


def to_u64(t):
    return t.cpu().numpy().view(np.uint64)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("geo", [
    dict(K=32, C=32, R=3, S=3, Mb=8, Nb=4, keep=3),
    dict(K=64, C=48, R=3, S=3, Mb=16, Nb=8, keep=0),
    dict(K=16, C=16, R=5, S=5, Mb=16, Nb=16, keep=25),
    dict(K=24, C=20, R=1, S=1, Mb=1, Nb=1, keep=1),
    dict(K=256, C=256, R=3, S=3, Mb=16, Nb=8, keep=3),            # the ResNet-50 stage-3 layer
])
def test_prune_bp_matches_oracle(geo, dtype):
    rng = inputs.rng_for(901)
    w = rng.standard_normal((geo["K"], geo["R"], geo["S"], geo["C"]), dtype=np.float32)
    w[: geo["Mb"], 0, 0, :] = 0.0                                   # an all-zero tap and exact ties with it
    if dtype == "bf16":
        w = inputs.bf16_representable(w)
    tm = npas.prune_bp_magnitude(dev(w, dtype), geo["Mb"], geo["Nb"], geo["keep"])
    assert np.array_equal(to_u64(tm), oracle.prune_bp(w, Mb=geo["Mb"], Nb=geo["Nb"], keep=geo["keep"]))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("geo", [
    dict(O=128, I=192, Bo=64, Bi=64, kr=16, kc=16),
    dict(O=40, I=48, Bo=8, Bi=16, kr=3, kc=5),
    dict(O=64, I=64, Bo=64, Bi=64, kr=64, kc=0),
    dict(O=2048, I=512, Bo=64, Bi=64, kr=16, kc=16),               # the 16x-pruned GEMM
])
def test_prune_bb_matches_oracle(geo, dtype):
    rng = inputs.rng_for(902)
    w = rng.standard_normal((geo["O"], geo["I"]), dtype=np.float32)
    if dtype == "bf16":
        w = inputs.bf16_representable(w)
    rk, ck = npas.prune_bb_magnitude(dev(w, dtype), geo["Bo"], geo["Bi"], geo["kr"], geo["kc"])
    rk0, ck0 = oracle.prune_bb(w, Bo=geo["Bo"], Bi=geo["Bi"], keep_rows=geo["kr"], keep_cols=geo["kc"])
    assert np.array_equal(to_u64(rk), rk0) and np.array_equal(to_u64(ck), ck0)


def test_pruned_layer_end_to_end():
    """dense weights -> magnitude masks -> blob -> convolution, against the oracle fed the oracle's masks."""
    c = inputs.config2()
    w = dev(c.w, "bf16")
    tm = npas.prune_bp_magnitude(w, c.Mb, c.Nb, 3)
    tm_host = to_u64(tm)
    assert np.array_equal(tm_host, oracle.prune_bp(c.w, Mb=c.Mb, Nb=c.Nb, keep=3))
    blob = npas.pack_bp(w, tm_host, c.Mb, c.Nb)
    ws = npas.workspace()
    y = npas.conv2d_bp(dev(c.x, "bf16"), blob, dev(c.bias), None, stride=1, pad=1, relu=True, ws=ws)
    npas.check_device_status(ws)
    ref = oracle.conv2d_bp(c.x, c.w, tm_host, Mb=c.Mb, Nb=c.Nb, stride=1, pad=1, bias=c.bias, relu=True)
    assert floored_rel_err(host(y), ref) < TOL_BF16


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("geo", [
    dict(K=32, C=32, R=3, S=3, Mb=8, Nb=4, rate=3.0),
    dict(K=64, C=48, R=3, S=3, Mb=16, Nb=8, rate=2.5),
    dict(K=16, C=16, R=5, S=5, Mb=16, Nb=16, rate=1.0),             # nothing pruned
    dict(K=24, C=20, R=1, S=1, Mb=1, Nb=1, rate=10.0),
    dict(K=256, C=256, R=3, S=3, Mb=16, Nb=8, rate=7.0),            # 4608 groups: several passes of the single CTA
    dict(K=512, C=512, R=3, S=3, Mb=16, Nb=16, rate=2.5),           # 9216 groups
])
def test_prune_bp_global_matches_oracle(geo, dtype):
    rng = inputs.rng_for(903)
    w = rng.standard_normal((geo["K"], geo["R"], geo["S"], geo["C"]), dtype=np.float32)
    w[: geo["Mb"], 0, 0, :] = 0.0                                   # all-zero groups: exact ties at the bottom
    if geo["K"] >= 2 * geo["Mb"]:
        w[geo["Mb"]:2 * geo["Mb"]] = w[:geo["Mb"]]                  # and exact ties between two filter blocks
    if dtype == "bf16":
        w = inputs.bf16_representable(w)
    G = (geo["K"] // geo["Mb"]) * (geo["C"] // geo["Nb"]) * geo["R"] * geo["S"]
    n_keep = int(np.floor(G / geo["rate"] + 0.5))
    tm = npas.prune_bp_magnitude_global(dev(w, dtype), geo["Mb"], geo["Nb"], rate=geo["rate"])
    ref = oracle.prune_bp_global(w, Mb=geo["Mb"], Nb=geo["Nb"], n_keep=n_keep)
    assert np.array_equal(to_u64(tm), ref)
    assert sum(bin(int(v)).count("1") for v in ref.ravel()) == n_keep


def test_prune_bp_global_extremes_and_all_ties():
    w = np.ones((8, 3, 3, 8), dtype=np.float32)                      # every group scores the same
    for n_keep in (0, 1, 10, 35, 36):
        tm = npas.prune_bp_magnitude_global(dev(w), 4, 4, n_keep=n_keep)
        assert np.array_equal(to_u64(tm), oracle.prune_bp_global(w, Mb=4, Nb=4, n_keep=n_keep))
    with pytest.raises(npas.NpasError) as e:
        npas.prune_bp_magnitude_global(dev(w), 4, 4, n_keep=37)
    assert e.value.code == 2


@pytest.mark.parametrize("rate,Mb,Nb", [(2.5, 16, 8), (7.0, 16, 16)])
def test_rate_pruned_layer_end_to_end(rate, Mb, Nb):
    """A layer pruned to 2.5x / 7x (blocks keep different numbers of taps) through pack + convolution."""
    c = inputs.conv_case(N=4, H=14, W=14, C=128, K=256, Mb=Mb, Nb=Nb, keep=0, dtype="bf16", seed=904)
    w = dev(c.w, "bf16")
    tm = to_u64(npas.prune_bp_magnitude_global(w, Mb, Nb, rate=rate))
    counts = [bin(int(v)).count("1") for v in tm.ravel()]
    assert len(set(counts)) > 2 and sum(counts) == int(np.floor(tm.size * 9 / rate + 0.5))
    blob = npas.pack_bp(w, tm, Mb, Nb)
    assert np.array_equal(blob.data.cpu().numpy(), oracle.pack_bp(c.w, tm, Mb, Nb, "bf16"))
    ws = npas.workspace()
    ref = oracle.conv2d_bp(c.x, c.w, tm, Mb=Mb, Nb=Nb, stride=1, pad=1, bias=c.bias, relu=True)
    paths = (0, 6, 7, 8) if Nb == 16 else (0, 6, 7)
    for path in paths:
        y = npas.conv2d_bp(dev(c.x, "bf16"), blob, dev(c.bias), None, stride=1, pad=1, relu=True, ws=ws, path=path)
        npas.check_device_status(ws)
        assert floored_rel_err(host(y), ref) < TOL_BF16, path
