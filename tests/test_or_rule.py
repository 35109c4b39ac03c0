"""Termination fraction tau_K and the OR-rule gate (Appendix B; Eq. 3)."""
import numpy as np
import pytest

import oracle
from paper_2605_05802_b200 import workloads as W


def test_tau_extremes_and_reduction_to_the_single_axis_gate():
    # tau_K = 0: nobody is done; tau_K = 1: all G are done (Appendix B)
    lens = np.array([[10] * 8, [4] * 8, [4] * 4 + [10] * 4], dtype=np.int32)
    mean = np.array([0.5, 0.5, 0.5])
    tau, stop = oracle.or_rule(mean, lens, None, 10, 0.12, 0.90)
    assert tau.tolist() == [0.0, 1.0, 0.5]
    assert stop.tolist() == [0, 1, 0]                      # only the tau clause can fire here
    # either clause suffices (logical OR), and >= is inclusive
    tau, stop = oracle.or_rule(np.array([0.05, 0.5, 0.5]), lens, None, 10, 0.12, 0.5)
    assert stop.tolist() == [1, 1, 1]
    # with tau_H above 1 the rule is Eq. 2 alone, strict in d_K
    w = W.agent_gate(K=15)
    _, _, mean, stop2 = oracle.gate(w.seqs, w.lens, w.K, 0.5)
    _, stop_or = oracle.or_rule(mean, w.lens, None, w.K, 0.5, 1.5)
    assert np.array_equal(stop_or, stop2)
    _, stop_eq = oracle.or_rule(np.array([0.12]), lens[:1], None, 10, 0.12, 1.5)
    assert stop_eq[0] == 0
    # the OR rule can only add cuts
    _, stop_or = oracle.or_rule(mean, w.lens, None, w.K, 0.5, 0.5)
    assert (stop_or >= stop2).all() and stop_or.sum() > stop2.sum()


def test_tau_counts_explicit_done_flags():
    rng = np.random.default_rng(0)
    done = (rng.random((50, 8)) < 0.4).astype(np.uint8)
    tau, stop = oracle.or_rule(np.ones(50), None, done, 10, 0.12, 0.75)
    assert np.array_equal(tau, done.sum(axis=1) / 8.0)     # eighths are exact in binary
    assert np.array_equal(stop, (done.sum(axis=1) >= 6).astype(np.uint8))
    # 7 of 8 finished is 0.875: below a 0.90 bar, at a 0.875 bar
    d = np.array([[1] * 7 + [0]], dtype=np.uint8)
    assert oracle.or_rule(np.ones(1), None, d, 10, 0.12, 0.90)[1][0] == 0
    assert oracle.or_rule(np.ones(1), None, d, 10, 0.12, 0.875)[1][0] == 1


@pytest.mark.gpu
def test_or_rule_gpu_matches_oracle():
    import torch
    import paper_2605_05802_b200 as sr
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(5)
    for N in (1, 3, 8, 16, 32):
        G = 1000
        lens = rng.integers(0, 31, size=(G, N)).astype(np.int32)
        done = (rng.random((G, N)) < 0.5).astype(np.uint8)
        mean = rng.random(G)
        for use_done in (False, True):
            for tau_h in (0.5, 0.9, 1.5):
                want_tau, want_stop = oracle.or_rule(mean, lens, done if use_done else None, 15, 0.12, tau_h)
                tau = torch.empty(G, dtype=torch.float64, device=dev)
                stop = torch.empty(G, dtype=torch.uint8, device=dev)
                sr.sr_gate_or_rule(torch.from_numpy(mean).to(dev), torch.from_numpy(lens).to(dev),
                                   torch.from_numpy(done).to(dev) if use_done else None, N, 15, 0.12, tau_h,
                                   tau=tau, stop=stop)
                torch.cuda.synchronize()
                assert np.array_equal(tau.cpu().numpy().view(np.uint64), want_tau.view(np.uint64))
                assert np.array_equal(stop.cpu().numpy(), want_stop)
