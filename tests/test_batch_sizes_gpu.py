"""The batch-level kernels at the size their timings are quoted on (4 194 304 groups of 8,
plus a ragged tail): advantages, OR rule, batch statistics and the kept-group list against
the oracle on the whole batch."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu

G = 64 * 65536 + 3
N = 8


def test_batch_level_kernels_on_four_million_groups():
    import torch
    import paper_2605_05802_b200 as sr
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(41)
    rewards = (rng.random((G, N)) < 0.15).astype(np.float32)              # success / failure: about a quarter of the groups flat
    rewards[::5] = rng.random((len(rewards[::5]), N), dtype=np.float32)
    lens = rng.integers(0, 31, size=(G, N)).astype(np.int32)
    mean = rng.random(G) * 0.3

    # gate mask from the OR rule (Eq. 3), bit-exact tau
    want_tau, want_stop = oracle.or_rule(mean, lens, None, 15, 0.12, 0.9)
    tau = torch.empty(G, dtype=torch.float64, device=dev)
    stop = torch.empty(G, dtype=torch.uint8, device=dev)
    sr.sr_gate_or_rule(torch.from_numpy(mean).to(dev), torch.from_numpy(lens).to(dev), None, N, 15, 0.12, 0.9,
                       tau=tau, stop=stop)
    assert np.array_equal(tau.cpu().numpy().view(np.uint64), want_tau.view(np.uint64))
    assert np.array_equal(stop.cpu().numpy(), want_stop)
    assert 0 < want_stop.sum() < G

    # advantages with the cut groups dropped (Eq. 1): 1e-6 relative, zeros and flags exact
    want_adv, want_zv = oracle.advantage(rewards, want_stop, 1e-6)
    adv = torch.empty((G, N), dtype=torch.float32, device=dev)
    zv = torch.empty(G, dtype=torch.uint8, device=dev)
    sr.sr_grpo_advantage(torch.from_numpy(rewards).to(dev), stop, 1e-6, adv=adv, zero_var=zv)
    got_adv = adv.cpu().numpy()
    assert np.array_equal(zv.cpu().numpy(), want_zv)
    zero = want_adv == 0
    assert np.array_equal(got_adv == 0, zero) and not np.signbit(got_adv[zero]).any()
    assert np.all(np.abs(got_adv[~zero] - want_adv[~zero]) <= 1e-6 * np.abs(want_adv[~zero]))

    # batch statistics over advantages computed without a drop mask
    full_adv, _ = oracle.advantage(rewards, None, 1e-6)
    want_c, want_s = oracle.batch_stats(full_adv, want_stop)
    counts = torch.empty(3, dtype=torch.int64, device=dev)
    sumsq = torch.empty(2, dtype=torch.float64, device=dev)
    sr.sr_batch_stats(torch.from_numpy(full_adv).to(dev), stop, counts=counts, sumsq=sumsq)
    assert counts.cpu().numpy().tolist() == want_c.tolist()
    # squares are exact in fp64 and all terms are positive, so any summation order lies within
    # n * 2^-53 relative of the true sum; the oracle adds the 33.5 M terms one after the
    # other, the kernel in a tree, hence twice that between the two
    assert np.allclose(sumsq.cpu().numpy(), want_s, rtol=2 * G * N * 2.0 ** -53, atol=0)

    # the groups that stay in the batch: not cut and not flat
    want_idx = oracle.kept_groups(want_stop, want_zv)
    index = torch.full((G,), -1, dtype=torch.int32, device=dev)
    count = torch.full((1,), -1, dtype=torch.int32, device=dev)
    ws = torch.empty(sr.sr_kept_groups_workspace_bytes(G), dtype=torch.uint8, device=dev)
    sr.sr_kept_groups(stop, zv, index=index, count=count, workspace=ws)
    n = int(count.item())
    assert n == len(want_idx) and 0 < n < G
    assert np.array_equal(index.cpu().numpy()[:n], want_idx)
