"""sr_gate_decide: the exact stop mask from lower bounds where they suffice."""
import numpy as np
import pytest

import oracle
from paper_2605_05802_b200 import workloads as W


def test_absent_symbol_bound_never_exceeds_the_distance():
    rng = np.random.default_rng(3)
    for _ in range(400):
        v = int(rng.integers(2, 12))
        a = rng.integers(0, v, size=int(rng.integers(0, 40)))
        b = rng.integers(0, v, size=int(rng.integers(0, 40)))
        d = oracle.levenshtein(a, b)
        assert oracle.absent_lower_bound(a, b) <= d
        assert oracle.absent_lower_bound(b, a) <= d
    assert oracle.absent_lower_bound([1, 2, 3], [7, 8, 9]) == 3 == oracle.levenshtein([1, 2, 3], [7, 8, 9])
    assert oracle.absent_lower_bound([1, 2, 3], [3, 2, 1]) == 0


def test_a_pair_beyond_its_budget_settles_the_group():
    """The reasoning behind capped bands, checked on the definition alone: with every
    other pair at a LOWER bound of its distance, pair p can keep d_K below d_L only while
    d_p <= L_p (P d_L - sum of the other bounded terms).  So whenever some true distance
    exceeds that budget, the oracle's gate must say "continue"."""
    rng = np.random.default_rng(17)
    seen = 0
    for trial in range(300):
        N = int(rng.integers(2, 6))
        P = N * (N - 1) // 2
        K = 24
        vocab = int(rng.integers(2, 5))
        seqs = rng.integers(0, vocab, size=(1, N, K)).astype(np.int32)
        lens = rng.integers(1, K + 1, size=(1, N)).astype(np.int32)
        thr = float(rng.uniform(0.05, 0.9))
        pd, _, _, stop = oracle.gate(seqs, lens, K, thr)
        rows = [seqs[0, i, :lens[0, i]] for i in range(N)]
        pairs = [(i, j) for i in range(N) for j in range(i + 1, N)]
        lb = [oracle.absent_lower_bound(rows[i], rows[j]) for i, j in pairs]
        longer = [max(len(rows[i]), len(rows[j])) for i, j in pairs]
        terms = [b / L for b, L in zip(lb, longer)]
        for p in range(P):
            budget = longer[p] * (P * thr - (sum(terms) - terms[p]))
            if pd[0, p] > budget + 1e-9:
                assert stop[0] == 0, (trial, p)
                seen += 1
    assert seen > 50


def _run_decide(w, thr, norm_mode=0):
    import torch
    import paper_2605_05802_b200 as sr
    dev = torch.device("cuda:0")
    G, N, stride = w.seqs.shape
    P = N * (N - 1) // 2
    seqs = torch.from_numpy(w.seqs).to(dev)
    lens = torch.from_numpy(w.lens).to(dev)
    pd = torch.full((G, P), -1, dtype=torch.int32, device=dev)
    ps = torch.full((G,), -1, dtype=torch.int32, device=dev)
    mean = torch.full((G,), -1.0, dtype=torch.float64, device=dev)
    stop = torch.full((G,), 9, dtype=torch.uint8, device=dev)
    exact = torch.full((G,), 9, dtype=torch.uint8, device=dev)
    wsb = sr.sr_gate_workspace_bytes(G, N, stride, w.K)
    ws = torch.empty(max(wsb, 1), dtype=torch.uint8, device=dev) if wsb else None
    sr.sr_gate_decide(seqs, lens, w.K, thr, norm_mode, pair_dist=pd, pair_sum=ps, mean=mean, stop=stop,
                      exact=exact, workspace=ws)
    torch.cuda.synchronize()
    return [t.cpu().numpy() for t in (pd, ps, mean, stop, exact)]


@pytest.mark.gpu
@pytest.mark.parametrize("thr", [0.05, 0.12, 0.3, 0.6, 0.95])
def test_decide_mask_is_exact_and_bounds_are_bounds(thr):
    cases = [W.token_gate(n_groups=48), W.token_gate(seed=8, n_groups=20, min_len=33, max_len=200, N=5),
             W.agent_gate(K=30)]
    rng = np.random.default_rng(2)
    few = W.token_gate(seed=9, n_groups=16, min_len=40, max_len=120, vocab=6)     # heavy repeats
    cases.append(few)
    for w in cases:
        opd, ops, omean, ostop = oracle.gate(w.seqs, w.lens, w.K, thr, w.norm_mode, threads=8)
        pd, ps, mean, stop, exact = _run_decide(w, thr, w.norm_mode)
        assert np.array_equal(stop, ostop), w.name                       # the mask, always
        assert set(np.unique(exact)) <= {0, 1}
        ex = exact == 1
        assert np.array_equal(pd[ex], opd[ex]) and np.array_equal(ps[ex], ops[ex])
        assert np.array_equal(mean[ex].view(np.uint64), omean[ex].view(np.uint64))
        lo = ~ex                                                          # settled by bounds or caps
        assert (stop[lo] == 0).all()
        assert (pd[lo] <= opd[lo]).all() and (pd[lo] >= 0).all()
        assert (ps[lo] == pd[lo].sum(axis=1)).all()
        assert (mean[lo] <= omean[lo]).all() and (mean[lo] >= thr).all()
        if w.K <= 32:
            assert ex.all()


@pytest.mark.gpu
def test_decide_skips_work_on_the_token_workload():
    w = W.token_gate(n_groups=128)
    *_, exact = _run_decide(w, 0.12)
    assert exact.mean() < 0.5          # at the paper's threshold most token-level groups are dismissed early


@pytest.mark.gpu
@pytest.mark.parametrize("thr", [0.2, 0.3, 0.5])
def test_decide_computes_open_groups_in_capped_bands(thr):
    """Converged token-level groups (10 % substitutions) lie near these thresholds, so the
    lower bounds cannot dismiss them: their pairs run in bands cut to what the threshold
    still allows.  The mask stays exact, exact groups carry exact values, the others lower
    bounds; and a fair share of the batch is decided either way."""
    w = W.token_gate(seed=13, n_groups=96)
    opd, ops, omean, ostop = oracle.gate(w.seqs, w.lens, w.K, thr, w.norm_mode, threads=8)
    pd, ps, mean, stop, exact = _run_decide(w, thr, w.norm_mode)
    assert np.array_equal(stop, ostop)
    ex = exact == 1
    assert np.array_equal(pd[ex], opd[ex]) and np.array_equal(ps[ex], ops[ex])
    assert np.array_equal(mean[ex].view(np.uint64), omean[ex].view(np.uint64))
    lo = ~ex
    assert (stop[lo] == 0).all() and (pd[lo] <= opd[lo]).all() and (pd[lo] >= 0).all()
    assert (ps[lo] == pd[lo].sum(axis=1)).all()
    assert (mean[lo] <= omean[lo]).all() and (mean[lo] >= thr).all()
    assert stop[ex].sum() == ostop.sum()                  # every cut group was computed exactly


@pytest.mark.gpu
def test_decide_large_groups_and_raw_distances():
    """Groups of 32 rollouts (496 pairs: the finish pass takes its one-thread-per-group path)
    and the raw-distance normalisation, at thresholds that leave groups open."""
    big = W.token_gate(seed=21, n_groups=6, min_len=40, max_len=130, N=32)
    for thr in (0.15, 0.4, 0.8):
        opd, ops, omean, ostop = oracle.gate(big.seqs, big.lens, big.K, thr, big.norm_mode, threads=8)
        pd, ps, mean, stop, exact = _run_decide(big, thr, big.norm_mode)
        assert np.array_equal(stop, ostop)
        ex = exact == 1
        assert np.array_equal(pd[ex], opd[ex]) and np.array_equal(mean[ex].view(np.uint64), omean[ex].view(np.uint64))
        assert (pd[~ex] <= opd[~ex]).all() and (stop[~ex] == 0).all()
    w = W.token_gate(seed=22, n_groups=40, min_len=60, max_len=400)
    for thr in (30.0, 120.0, 300.0):                                    # thresholds on the raw mean distance
        opd, ops, omean, ostop = oracle.gate(w.seqs, w.lens, w.K, thr, 1, threads=8)
        pd, ps, mean, stop, exact = _run_decide(w, thr, 1)
        assert np.array_equal(stop, ostop)
        ex = exact == 1
        assert np.array_equal(pd[ex], opd[ex]) and np.array_equal(ps[ex], ops[ex])
        assert np.array_equal(mean[ex].view(np.uint64), omean[ex].view(np.uint64))
        assert (pd[~ex] <= opd[~ex]).all() and (stop[~ex] == 0).all() and (mean[~ex] >= thr).all()
    assert 0 < ostop.sum() < 40
