"""Host-only checks of the kernel choice: the committed (case, path) table and the plan cache."""
import pytest

import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import binding as B
from dispatch_table import (CONV_AUTO, CONV_CASES, CONV_TAKES, LINEAR_AUTO, LINEAR_CASES, LINEAR_TAKES, UNSUPPORTED)


def _conv_query(kw, path, variant=0):
    R, S = kw.get("R", 3), kw.get("S", 3)
    keep = kw["keep"]
    max_taps = R * S if callable(keep) else min(keep, R * S)
    blob = B.BpBlob(None, B.BpDesc(kw["K"], kw["C"], R, S, kw["Mb"], kw["Nb"], B.BF16, B.BF16, max_taps))
    return npas.conv2d_bp_kernel((kw["N"], kw["H"], kw["W"], kw["C"]), blob, stride=kw.get("stride", 1),
                                 pad=kw.get("pad", 1), relu=True, bias=True, residual=True, path=path, variant=variant)


def _linear_query(kw, path, residual=False, variant=0):
    kc = kw["keep_cols"]
    blob = B.BbBlob(None, B.BbDesc(kw["O"], kw["I"], kw["Bo"], kw["Bi"], B.BF16, B.BF16, kw["Bi"] if callable(kc) else kc))
    return npas.linear_bb_kernel(kw["M"], blob, relu=True, bias=True, residual=residual, path=path, variant=variant)


@pytest.mark.parametrize("path", sorted(CONV_TAKES))
def test_conv_forced_paths_take_exactly_the_listed_cases(path):
    for i, kw in enumerate(CONV_CASES):
        if i in CONV_TAKES[path]:
            assert _conv_query(kw, path) == path, (i, path)
        else:
            with pytest.raises(npas.NpasError) as e:
                _conv_query(kw, path)
            assert e.value.code == UNSUPPORTED, (i, path)


def test_conv_automatic_choice():
    for i, kw in enumerate(CONV_CASES):
        assert _conv_query(kw, 0) == CONV_AUTO[i], i
        assert _conv_query(kw, 2) == CONV_AUTO[i], i          # every case has a tensor-core kernel


@pytest.mark.parametrize("path", sorted(LINEAR_TAKES))
def test_linear_forced_paths_take_exactly_the_listed_cases(path):
    for i, kw in enumerate(LINEAR_CASES):
        for residual in (False, True):
            if i in LINEAR_TAKES[path]:
                assert _linear_query(kw, path, residual) == path, (i, path)
            else:
                with pytest.raises(npas.NpasError) as e:
                    _linear_query(kw, path, residual)
                assert e.value.code == UNSUPPORTED, (i, path)


def test_linear_automatic_choice():
    for i, kw in enumerate(LINEAR_CASES):
        assert _linear_query(kw, 0) == LINEAR_AUTO[i], i


def test_sweep_shape_choices():
    """64x28x28x512 -> 512: kept pairs only where measured faster (up to 3 of 9 taps at 16x16 blocks, up to 4
    of 9 at 32x32), the CTA-pair dense-image kernel elsewhere, also for the block sizes below 16."""
    def q(Mb, Nb, taps):
        return _conv_query(dict(N=64, H=28, W=28, C=512, K=512, Mb=Mb, Nb=Nb, keep=taps), 0)
    assert [q(16, 16, t) for t in (1, 2, 3, 4, 5, 9)] == [8, 8, 8, 7, 7, 7]
    assert [q(32, 32, t) for t in (1, 2, 3, 4, 5, 9)] == [8, 8, 8, 8, 7, 7]
    assert [q(8, 8, t) for t in (1, 9)] == [7, 7] and [q(4, 4, t) for t in (1, 9)] == [7, 7]
    # the tile-shape variant of the pair kernel: only combinations the geometry allows
    kw = dict(N=64, H=28, W=28, C=512, K=512, Mb=16, Nb=16, keep=3)
    for nt, mt in ((128, 1), (128, 2), (256, 1), (256, 2)):
        assert _conv_query(kw, 7, nt | (mt << 16)) == 7
    with pytest.raises(npas.NpasError):
        _conv_query(kw, 7, 64 | (1 << 16))


def test_plan_cache_round_trip_and_rejects_garbage():
    c = npas.PlanCache()
    blob = B.BpBlob(None, B.BpDesc(512, 512, 3, 3, 16, 16, B.BF16, B.BF16, 3))
    k1 = c.conv_key((64, 28, 28, 512), blob, 1, 1, False, False, False)
    lb = B.BbBlob(None, B.BbDesc(2048, 512, 64, 64, B.BF16, B.BF16, 16))
    k2 = c.linear_key(3136, lb, True, True, False)
    assert k1 != c.conv_key((64, 28, 28, 512), B.BpBlob(None, B.BpDesc(512, 512, 3, 3, 16, 16, B.BF16, B.BF16, 1)), 1, 1,
                            False, False, False)                       # the mask statistic is part of the key
    c.put(k1, 7, 256 | (1 << 16), 155.25)
    c.put(k2, 6, 128, 11.5)
    text = c.to_json()
    d = npas.PlanCache.from_json(text)
    assert d.get(k1) == (7, 256 | (1 << 16)) and d.get(k2) == (6, 128) and d.get("conv:other") is None
    assert d.to_json() == text
    for bad in ('{"version": 2, "plans": {}}', '{"plans": []}', '{"version": 1, "plans": {"k": [1, 2]}}'):
        with pytest.raises(ValueError):
            npas.PlanCache.from_json(bad)
