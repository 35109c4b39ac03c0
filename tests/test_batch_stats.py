"""Batch reductions after the advantage call: zero-advantage share (Section 4.5),
advantage norm kept after cutting (Section 3.4), savings accounting (Table 1)."""
import os

import numpy as np
import pytest

import oracle
from paper_2605_05802_b200 import binding, build, workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _table1():
    rows = []
    for ln in open(os.path.join(GOLDEN, "table1_savings.txt")):
        if ln.strip() and not ln.startswith("#"):
            rows.append([float(x) for x in ln.split(";")])
    return rows


def test_savings_match_the_papers_table():
    build.build()
    lib = binding.load()
    rows = _table1()
    assert len(rows) == 6
    for _, cut, tp, safe, raw in rows:
        for fn in (oracle.savings_fraction, lambda *a: lib.sr_savings_fraction(*a)):
            assert round(100 * fn(int(cut), 100, 30, 10), 1) == raw
            assert round(100 * fn(int(tp), 100, 30, 10), 1) == safe
    # the formula, not a lookup: 17 * 20 / 3000
    assert oracle.savings_fraction(17, 100, 30, 10) == 17 * 20 / 3000


def test_dilution_gain_matches_the_papers_arithmetic():
    build.build()
    lib = binding.load()
    # Section 4.5: zero-advantage share 40 % -> 28 %, contributing share 0.60 -> 0.72, ratio 1.20
    for fn in (oracle.dilution_gain, lib.sr_dilution_gain):
        assert fn(0.40, 0.28) == pytest.approx(0.72 / 0.60, rel=1e-15)
        assert round(fn(0.40, 0.28), 2) == 1.20
        assert fn(0.3, 0.3) == 1.0


def test_batch_stats_oracle_against_numpy():
    s = W.streaming_gate(n_groups=4096)
    adv, zv = oracle.advantage(s.rewards, None, 1e-6)
    rng = np.random.default_rng(1)
    stop = (rng.random(4096) < 0.2).astype(np.uint8)
    counts, sumsq = oracle.batch_stats(adv, stop)
    a = adv.astype(np.float64)
    kept = stop == 0
    assert counts.tolist() == [int((a == 0).sum()), int((a[kept] == 0).sum()), int(kept.sum())]
    assert sumsq[0] == pytest.approx((a ** 2).sum(), rel=1e-12)
    assert sumsq[1] == pytest.approx((a[kept] ** 2).sum(), rel=1e-12)
    # zero-variance groups produce N zero advantages each (Section 2.1)
    assert counts[0] == 8 * int(zv.sum())
    # cutting only zero-variance groups loses no advantage norm (true positives are lossless)
    _, ss = oracle.batch_stats(adv, zv)
    assert ss[1] == ss[0]
    c_none, ss_none = oracle.batch_stats(adv, None)
    assert c_none[2] == 4096 and ss_none[1] == ss_none[0] and c_none[0] == c_none[1]


@pytest.mark.gpu
def test_batch_stats_gpu_matches_oracle():
    import torch
    import paper_2605_05802_b200 as sr
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(2)
    for G, N in ((1, 8), (777, 5), (65536, 8), (4096, 16)):
        r = rng.integers(0, 2, size=(G, N)).astype(np.float32)
        adv, _ = oracle.advantage(r, None, 1e-6)
        for stop in (None, (rng.random(G) < 0.3).astype(np.uint8)):
            want_c, want_s = oracle.batch_stats(adv, stop)
            counts = torch.full((3,), -1, dtype=torch.int64, device=dev)
            sumsq = torch.full((2,), -1.0, dtype=torch.float64, device=dev)
            sr.sr_batch_stats(torch.from_numpy(adv).to(dev), None if stop is None else torch.from_numpy(stop).to(dev),
                              counts=counts, sumsq=sumsq)
            torch.cuda.synchronize()
            assert counts.cpu().numpy().tolist() == want_c.tolist()
            # parallel fp64 accumulation: at most ~n * 2^-53 relative from the sequential sum
            assert np.allclose(sumsq.cpu().numpy(), want_s, rtol=1e-11, atol=0)
