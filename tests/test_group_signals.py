"""The other action-only divergence signals of Appendix B (unique-prefix ratio,
unique-action ratio, action entropy, action-bigram Jaccard)."""
import numpy as np
import pytest
from scipy.stats import entropy as scipy_entropy

import oracle
from paper_2605_05802_b200 import workloads as W


def _by_sets(seqs, lens, K):
    """The same four signals written with Python sets, tuples and scipy's entropy."""
    G, N, _ = seqs.shape
    out = np.zeros((4, G))
    for g in range(G):
        L = [K if lens is None else int(lens[g, i]) for i in range(N)]
        pre = [tuple(int(x) for x in seqs[g, i, :min(max(L[i], 0), K)]) for i in range(N)]
        out[0, g] = len(set(pre)) / N
        keys = [("act", int(seqs[g, i, K - 1])) if (L[i] >= K and K >= 1) else ("none",) for i in range(N)]
        out[1, g] = len(set(keys)) / N
        _, counts = np.unique([hash(k) for k in keys], return_counts=True)
        out[2, g] = scipy_entropy(counts / N) / np.log(N)
        tot = 0.0
        for i in range(N):
            for j in range(i + 1, N):
                A = set(zip(pre[i], pre[i][1:]))
                B = set(zip(pre[j], pre[j][1:]))
                tot += (1 - len(A & B) / len(A | B)) if (A | B) else 0.0
        out[3, g] = tot / (N * (N - 1) // 2)
    return out


def test_signal_extremes_from_the_appendix():
    # identical trajectories: the ratios sit at their minimum 1/G, entropy and Jaccard at 0
    seqs = np.tile(np.array([3, 1, 4, 1, 5, 9, 2, 6], dtype=np.int32), (1, 8, 1))
    upr, uar, ent, jac = oracle.group_signals(seqs, None, 8)
    assert (upr[0], uar[0], ent[0], jac[0]) == (1 / 8, 1 / 8, 0.0, 0.0)
    # every trajectory different, no shared action: everything at its maximum 1
    seqs = np.arange(64, dtype=np.int32).reshape(1, 8, 8)
    upr, uar, ent, jac = oracle.group_signals(seqs, None, 8)
    assert upr[0] == 1.0 and uar[0] == 1.0 and jac[0] == 1.0 and ent[0] == pytest.approx(1.0, abs=1e-15)
    # same prefixes except the last action: prefixes all distinct, bigram sets share 6 of 8
    seqs = np.tile(np.arange(8, dtype=np.int32), (1, 4, 1))
    seqs[0, :, 7] = [100, 101, 102, 103]
    upr, uar, ent, jac = oracle.group_signals(seqs, None, 8)
    assert upr[0] == 1.0 and uar[0] == 1.0
    assert jac[0] == pytest.approx(1 - 6 / 8, abs=1e-15)
    # repeated bigrams count once (sets): 1,2,1,2,1,2 has the two bigrams (1,2),(2,1)
    seqs = np.zeros((1, 2, 8), dtype=np.int32)
    seqs[0, 0, :6] = [1, 2, 1, 2, 1, 2]
    seqs[0, 1, :6] = [1, 2, 7, 7, 7, 7]
    lens = np.array([[6, 6]], dtype=np.int32)
    _, _, _, jac = oracle.group_signals(seqs, lens, 8)
    assert jac[0] == pytest.approx(1 - 1 / 4, abs=1e-15)       # A={12,21} B={12,27,77}: 1 of 4


def test_signals_match_the_set_formulation():
    rng = np.random.default_rng(4)
    for vocab in (2, 4, 50):
        seqs = rng.integers(0, vocab, size=(60, 6, 12)).astype(np.int32)
        lens = rng.integers(0, 13, size=(60, 6)).astype(np.int32)
        for K in (1, 5, 12):
            got = np.array(oracle.group_signals(seqs, lens, K))
            want = _by_sets(seqs, lens, K)
            assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
            assert np.allclose(got[2], want[2], rtol=0, atol=1e-12)
            assert np.allclose(got[3], want[3], rtol=0, atol=1e-12)
    w = W.agent_gate(K=15)
    got = np.array(oracle.group_signals(w.seqs[:64], w.lens[:64], 15))
    want = _by_sets(w.seqs[:64], w.lens[:64], 15)
    assert np.allclose(got, want, rtol=0, atol=1e-12)
    assert ((got >= 0) & (got <= 1 + 1e-15)).all()


def test_unique_prefix_ratio_agrees_with_zero_edit_distances():
    # two prefixes are the same trajectory exactly when their edit distance is 0
    w = W.large_group_gate(n_groups=200)
    pd, _, _, _ = oracle.gate(w.seqs, w.lens, w.K, 0.12)
    upr = oracle.group_signals(w.seqs, w.lens, w.K)[0]
    N = w.N
    for g in range(200):
        dup = np.zeros(N, dtype=bool)
        p = 0
        for i in range(N):
            for j in range(i + 1, N):
                if pd[g, p] == 0:
                    dup[j] = True
                p += 1
        assert upr[g] == (N - dup.sum()) / N


@pytest.mark.gpu
def test_group_signals_gpu_matches_oracle():
    import torch
    import paper_2605_05802_b200 as sr
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(9)
    cases = [(W.tiny_gate().seqs, W.tiny_gate().lens, 10), (W.agent_gate().seqs, W.agent_gate().lens, 15),
             (W.agent_gate().seqs, W.agent_gate().lens, 30), (W.large_group_gate(n_groups=512).seqs, None, 30)]
    for N in (2, 5, 32):
        cases.append((rng.integers(0, 3, size=(40, N, 32)).astype(np.int32),
                      rng.integers(0, 33, size=(40, N)).astype(np.int32), 32))
        cases.append((rng.integers(0, 3, size=(40, N, 32)).astype(np.int32),
                      rng.integers(0, 33, size=(40, N)).astype(np.int32), 1))
    for seqs, lens, K in cases:
        G = seqs.shape[0]
        want = oracle.group_signals(seqs, lens, K)
        outs = [torch.full((G,), -1.0, dtype=torch.float64, device=dev) for _ in range(4)]
        sr.sr_group_signals(torch.from_numpy(seqs).to(dev), None if lens is None else torch.from_numpy(lens).to(dev), K,
                            unique_prefix_ratio=outs[0], unique_action_ratio=outs[1], action_entropy=outs[2],
                            bigram_jaccard_mean=outs[3])
        torch.cuda.synchronize()
        got = [o.cpu().numpy() for o in outs]
        for k in (0, 1, 3):            # ratios and the Jaccard mean: bit for bit
            assert np.array_equal(got[k].view(np.uint64), want[k].view(np.uint64)), (k, K)
        # entropy: device log vs host log, a few ulp per term
        assert np.allclose(got[2], want[2], rtol=0, atol=1e-13)


@pytest.mark.gpu
def test_group_signals_on_65536_groups_of_16():
    """The batch the kernel's timing is quoted on: first and last groups and a seeded sample
    against the oracle (bit for bit but for the entropy's logarithms)."""
    import torch
    import paper_2605_05802_b200 as sr
    dev = torch.device("cuda:0")
    w = W.large_group_gate(n_groups=65536)
    G = w.seqs.shape[0]
    outs = [torch.full((G,), -1.0, dtype=torch.float64, device=dev) for _ in range(4)]
    sr.sr_group_signals(torch.from_numpy(w.seqs).to(dev), torch.from_numpy(w.lens).to(dev), w.K,
                        unique_prefix_ratio=outs[0], unique_action_ratio=outs[1], action_entropy=outs[2],
                        bigram_jaccard_mean=outs[3])
    torch.cuda.synchronize()
    rng = np.random.default_rng(17)
    pick = np.unique(np.concatenate([np.arange(32), np.arange(G - 32, G), rng.integers(0, G, size=700)]))
    want = oracle.group_signals(w.seqs[pick], w.lens[pick], w.K)
    got = [o.cpu().numpy()[pick] for o in outs]
    for k in (0, 1, 3):
        assert np.array_equal(got[k].view(np.uint64), want[k].view(np.uint64)), k
    assert np.allclose(got[2], want[2], rtol=0, atol=1e-13)
    assert all((o.cpu().numpy() >= 0).all() for o in outs)        # every group was written
