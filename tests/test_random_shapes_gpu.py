"""Seeded sweep over group sizes, prefix limits, strides, length mixes and symbol structure:
every output of sr_gate is compared with the oracle element by element, and the mask of
sr_gate_decide with the oracle's mask (exact groups: every value).  The cases are drawn
from a fixed seed, so a failure names a reproducible (case, shape)."""
import numpy as np
import pytest

import oracle
from helpers import assert_gate_matches, gate_gpu


def _draw_group_batch(rng, G, N, K, stride, vocab, kind):
    """Rollouts of one group are edits of a common base (kind 0), independent (kind 1),
    copies with different lengths (kind 2: containment, distance = length difference) or a
    mix of the three per group (kind 3)."""
    seqs = np.zeros((G, N, stride), dtype=np.int32)
    lens = np.zeros((G, N), dtype=np.int32)
    for g in range(G):
        k = kind if kind < 3 else int(rng.integers(0, 3))
        base = rng.integers(0, vocab, size=stride)
        lo = int(rng.integers(0, K + 1))
        for i in range(N):
            L = int(rng.integers(min(lo, K), K + 1)) if rng.random() < 0.9 else int(rng.integers(0, 3))
            if k == 0:
                row = base.copy()
                edits = rng.random(stride) < rng.choice([0.02, 0.1, 0.4])
                row[edits] = rng.integers(0, vocab, size=int(edits.sum()))
                if rng.random() < 0.3:                    # an insertion near the front shifts the rest
                    at = int(rng.integers(0, max(1, stride // 4)))
                    row = np.concatenate([row[:at], rng.integers(0, vocab, size=1), row[at:-1]])
            elif k == 1:
                row = rng.integers(0, vocab, size=stride)
            else:
                row = base.copy()
            seqs[g, i, :L] = row[:L]
            lens[g, i] = L
    return seqs, lens


CASES = []
_rng = np.random.default_rng(20260511)
for _case in range(36):
    N = int(_rng.choice([2, 3, 4, 5, 8, 8, 11, 16, 32]))
    K = int(_rng.choice([1, 7, 16, 17, 31, 32, 33, 40, 64, 65, 100, 255, 256, 257, 500, 1000, 1024]))
    stride = (K + int(_rng.integers(0, 9)) + 3) // 4 * 4          # the boundary wants a multiple of 4
    G = int(_rng.choice([1, 2, 5, 17, 33])) if K > 256 or N > 16 else int(_rng.choice([1, 3, 19, 64, 150]))
    vocab = int(_rng.choice([2, 3, 17, 300, 100000]))
    kind = int(_rng.integers(0, 4))
    norm = int(_rng.integers(0, 2))
    CASES.append((_case, G, N, K, stride, vocab, kind, norm))


@pytest.mark.gpu
@pytest.mark.parametrize("case,G,N,K,stride,vocab,kind,norm", CASES)
def test_gate_on_drawn_shapes(case, G, N, K, stride, vocab, kind, norm):
    rng = np.random.default_rng(1000 + case)
    seqs, lens = _draw_group_batch(rng, G, N, K, stride, vocab, kind)
    want = oracle.gate(seqs, lens, K, 0.12, norm, threads=8)
    # a threshold among the batch's own d_K values, so that both answers occur and some
    # groups sit exactly on it (strict comparison)
    thr = float(np.median(want[2])) if G > 1 else float(want[2][0])
    want = oracle.gate(seqs, lens, K, thr, norm, threads=8)
    got = gate_gpu(seqs, lens, K, thr, norm)
    assert_gate_matches(got, want, f"case {case}: G={G} N={N} K={K} stride={stride} vocab={vocab} kind={kind}")


@pytest.mark.gpu
@pytest.mark.parametrize("case,G,N,K,stride,vocab,kind,norm", [c for c in CASES if c[3] > 32])
def test_decide_on_drawn_shapes(case, G, N, K, stride, vocab, kind, norm):
    import torch
    import paper_2605_05802_b200 as sr
    rng = np.random.default_rng(1000 + case)
    seqs, lens = _draw_group_batch(rng, G, N, K, stride, vocab, kind)
    opd, ops, omean, _ = oracle.gate(seqs, lens, K, 0.12, norm, threads=8)
    for thr in sorted({float(np.median(omean)), float(np.quantile(omean, 0.9)) * 1.01, 0.5 * float(omean.max()) + 1e-3}):
        _, _, _, ostop = oracle.gate(seqs, lens, K, thr, norm, threads=8)
        dev = torch.device("cuda:0")
        P = N * (N - 1) // 2
        pd = torch.full((G, P), -1, dtype=torch.int32, device=dev)
        ps = torch.full((G,), -1, dtype=torch.int32, device=dev)
        mean = torch.full((G,), -1.0, dtype=torch.float64, device=dev)
        stop = torch.full((G,), 9, dtype=torch.uint8, device=dev)
        exact = torch.full((G,), 9, dtype=torch.uint8, device=dev)
        ws = torch.empty(max(sr.sr_gate_workspace_bytes(G, N, stride, K), 1), dtype=torch.uint8, device=dev)
        sr.sr_gate_decide(torch.from_numpy(seqs).to(dev), torch.from_numpy(lens).to(dev), K, thr, norm,
                          pair_dist=pd, pair_sum=ps, mean=mean, stop=stop, exact=exact, workspace=ws)
        torch.cuda.synchronize()
        pd, ps, mean, stop, exact = [t.cpu().numpy() for t in (pd, ps, mean, stop, exact)]
        tag = f"case {case} thr={thr}: G={G} N={N} K={K} vocab={vocab} kind={kind} norm={norm}"
        assert np.array_equal(stop, ostop), tag
        assert set(np.unique(exact)) <= {0, 1}, tag
        ex = exact == 1
        assert np.array_equal(pd[ex], opd[ex]) and np.array_equal(ps[ex], ops[ex]), tag
        assert np.array_equal(mean[ex].view(np.uint64), omean[ex].view(np.uint64)), tag
        lo = ~ex
        assert (stop[lo] == 0).all() and (pd[lo] >= 0).all() and (pd[lo] <= opd[lo]).all(), tag
        assert (mean[lo] <= omean[lo]).all() and (mean[lo] >= thr).all(), tag


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(12))
def test_single_word_and_incremental_on_drawn_shapes(seed):
    """Any N in 2..32 and K in 0..32 for the single-word kernels (symbol ids over the whole
    int32 range); any group size, step limit and termination pattern -- early stops, pauses
    -- for the incremental gate, which must equal the recomputation after every step."""
    from helpers import IncrementalGate
    from paper_2605_05802_b200.binding import SR_NO_ACTION
    rng = np.random.default_rng(500 + seed)
    N = int(rng.integers(2, 33))
    K = int(rng.integers(0, 33))
    stride = max(4, (K + int(rng.integers(0, 9)) + 3) // 4 * 4)
    G = int(rng.choice([1, 2, 17, 100, 513, 3000]))
    vocab = int(rng.choice([1, 2, 3, 17, 300, 2 ** 31 - 1]))
    kind, norm = int(rng.integers(0, 4)), int(rng.integers(0, 2))
    seqs, lens = _draw_group_batch(rng, G, N, K, stride, vocab, kind)
    if seed % 4 == 3:
        seqs = seqs - (2 ** 31 - 1) // 2                   # negative ids are legal too
    want = oracle.gate(seqs, lens, K, 0.12, norm, threads=8)
    thr = float(np.quantile(want[2], rng.random()))
    want = oracle.gate(seqs, lens, K, thr, norm, threads=8)
    assert_gate_matches(gate_gpu(seqs, lens, K, thr, norm), want,
                        f"seed {seed}: N={N} K={K} G={G} vocab={vocab} kind={kind} norm={norm}")

    N = int(rng.choice([2, 3, 5, 8, 8, 13, 16, 32]))
    steps = int(rng.integers(1, 33))
    G = int(rng.choice([1, 7, 64, 700]))
    vocab = int(rng.choice([2, 5, 40, 100000]))
    norm, thr = int(rng.integers(0, 2)), float(rng.random() * 0.5)
    inc = IncrementalGate(G, N, steps)
    base = rng.integers(0, vocab, size=(G, 1, steps))
    own = rng.integers(0, vocab, size=(G, N, steps))
    acts = np.where(rng.random((G, N, steps)) < rng.choice([0.05, 0.3, 1.0]), own, base).astype(np.int32)
    stop_at = rng.integers(0, steps + 1, size=(G, N)) if seed % 2 else np.full((G, N), steps)
    hist = np.zeros((G, N, 32), dtype=np.int32)
    hl = np.zeros((G, N), dtype=np.int32)
    for t in range(steps):
        act = np.where(t < stop_at, acts[:, :, t], SR_NO_ACTION).astype(np.int32)
        if seed % 3 == 0:                                  # pauses: a rollout skips a step and resumes
            act = np.where(rng.random((G, N)) < 0.3, SR_NO_ACTION, act).astype(np.int32)
        gi, ni = np.nonzero(act != SR_NO_ACTION)
        hist[gi, ni, hl[gi, ni]] = act[gi, ni]
        hl[gi, ni] += 1
        want = oracle.gate(hist, hl, steps, thr, norm, threads=8)
        assert_gate_matches(inc.step(act, thr, norm), want, f"seed {seed}: incremental N={N} steps={steps} G={G} t={t}")
