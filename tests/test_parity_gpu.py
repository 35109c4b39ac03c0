"""CUDA path vs CPU oracle, element by element, through the C ABI.

Integer outputs (pair distances, pair sums, stop masks) and the fp64 d_K must be
bit-identical; fp32 advantages must agree to 1e-6 relative (exact zeros exactly)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_05802_b200 as sr
from paper_2605_05802_b200 import workloads as W

from helpers import IncrementalGate, advantage_gpu, assert_gate_matches, gate_gpu

pytestmark = pytest.mark.gpu


def _check_workload(w, thresholds=None):
    for thr in (thresholds or [w.threshold]):
        want = oracle.gate(w.seqs, w.lens, w.K, thr, w.norm_mode, threads=8)
        got = gate_gpu(w.seqs, w.lens, w.K, thr, w.norm_mode)
        assert_gate_matches(got, want, f"{w.name} thr={thr}")
    return want


def test_c1_tiny_both_threshold_readings():
    want = _check_workload(W.tiny_gate(raw_threshold=True))
    assert 0 < want[3].sum() < 16
    _check_workload(W.tiny_gate(raw_threshold=False))


def test_c2_agent_ragged_lengths():
    _check_workload(W.agent_gate(K=15), [0.12, 0.5])
    _check_workload(W.agent_gate(K=30), [0.12, 0.5])
    w = W.agent_gate(K=15)
    got = gate_gpu(w.seqs, w.lens, w.K, 0.5, want_pair_dist=False)      # optional output omitted
    want = oracle.gate(w.seqs, w.lens, w.K, 0.5)
    assert_gate_matches(got, want, "C2 no pair_dist")


def test_c3_large_group_n16():
    want = _check_workload(W.large_group_gate(), [0.12, 0.09])
    assert 0 < want[3].sum() < 4096


@pytest.mark.parametrize("make", ["agent_x128", "large_x16"])
def test_single_word_batches_of_65536_groups(make):
    """The single-word kernels on the batch sizes the benchmark's side measurements time
    (65 536 groups: many groups per CTA, a ragged last CTA): every output of the first and
    the last groups and of a seeded sample in between, against the oracle."""
    w = W.agent_gate(K=15, n_groups=65536) if make == "agent_x128" else W.large_group_gate(n_groups=65536)
    got = gate_gpu(w.seqs, w.lens, w.K, 0.12, w.norm_mode)
    rng = np.random.default_rng(7)
    G = w.seqs.shape[0]
    pick = np.unique(np.concatenate([np.arange(40), np.arange(G - 40, G), rng.integers(0, G, size=600)]))
    want = oracle.gate(w.seqs[pick], w.lens[pick], w.K, 0.12, w.norm_mode, threads=8)
    assert_gate_matches(tuple(x[pick] for x in got), want, f"{make}: sampled groups")
    assert 0 < got[3].sum() < G


def test_c4_token_level_small_slice_every_element():
    w = W.token_gate(n_groups=24)
    _check_workload(w, [0.12, 0.6])


def test_c4_token_level_full_size():
    w = W.token_gate()
    want = oracle.gate(w.seqs, w.lens, w.K, 0.5, w.norm_mode, threads=8)
    got = gate_gpu(w.seqs, w.lens, w.K, 0.5, w.norm_mode)
    assert_gate_matches(got, want, "C4 full")
    assert 0 < want[3].sum() < 1024


def test_multiword_repeated_symbols_and_ragged_tails():
    rng = np.random.default_rng(17)
    for vocab, lo, hi, stride in [(3, 33, 200, 200), (40, 1, 130, 132), (1000, 90, 700, 704),
                                  (7, 1000, 1024, 1024), (100000, 33, 65, 68)]:
        G, N = 6, 5
        seqs = rng.integers(0, vocab, size=(G, N, stride)).astype(np.int32)
        lens = rng.integers(lo, hi + 1, size=(G, N)).astype(np.int32)
        lens[0, 0] = 0
        lens[1, :] = hi
        want = oracle.gate(seqs, lens, stride, 0.5, threads=8)
        got = gate_gpu(seqs, lens, stride, 0.5)
        assert_gate_matches(got, want, f"multi vocab={vocab}")
        K = (lo + hi) // 2                         # prefix truncation inside the multi-word path
        if K > 32:
            want = oracle.gate(seqs, lens, K, 0.5, threads=8)
            got = gate_gpu(seqs, lens, K, 0.5)
            assert_gate_matches(got, want, f"multi vocab={vocab} K={K}")


def test_multiword_maximum_sizes_and_degenerate_groups():
    rng = np.random.default_rng(23)
    # the largest group the ABI accepts at the longest prefix, ragged
    seqs = rng.integers(0, 50000, size=(2, 32, 1024)).astype(np.int32)
    seqs[1] = seqs[1, 0]                                   # second group: 32 identical rollouts ...
    lens = rng.integers(900, 1025, size=(2, 32)).astype(np.int32)
    lens[1] = 1024                                         # ... of full length: d_K = 0
    lens[0, 5] = 0
    lens[0, 6] = 1
    want = oracle.gate(seqs, lens, 1024, 0.12, threads=8)
    got = gate_gpu(seqs, lens, 1024, 0.12)
    assert_gate_matches(got, want, "N=32 K=1024")
    assert want[2][1] == 0.0 and want[3][1] == 1
    # K just above the single-word limit, one group, every length 0, one symbol repeated
    for K, stride in ((33, 36), (64, 64)):
        seqs = rng.integers(0, 4, size=(1, 4, stride)).astype(np.int32)
        for lens in (np.zeros((1, 4), dtype=np.int32), np.full((1, 4), K, dtype=np.int32),
                     np.array([[K, 0, 1, K - 1]], dtype=np.int32)):
            want = oracle.gate(seqs, lens, K, 0.5)
            got = gate_gpu(seqs, lens, K, 0.5)
            assert_gate_matches(got, want, f"K={K} lens={lens.tolist()}")
    seqs = np.full((3, 3, 256), 7, dtype=np.int32)         # a single symbol: the longest chains
    lens = np.array([[256, 200, 33], [256, 256, 256], [40, 0, 255]], dtype=np.int32)
    want = oracle.gate(seqs, lens, 256, 0.3)
    got = gate_gpu(seqs, lens, 256, 0.3)
    assert_gate_matches(got, want, "one symbol")


def test_multiword_null_lengths_raw_norm_and_negative_lengths():
    """The multi-word path with lens = NULL (every prefix has K symbols), with the raw-distance
    normalisation, and with negative lengths (treated as 0 and flagged)."""
    rng = np.random.default_rng(41)
    G, N, stride = 7, 6, 104
    seqs = rng.integers(0, 30, size=(G, N, stride)).astype(np.int32)
    for K in (100, 33):
        full = np.full((G, N), K, dtype=np.int32)
        want = oracle.gate(seqs, full, K, 0.8)
        got = gate_gpu(seqs, None, K, 0.8)
        assert_gate_matches(got, want, f"lens=NULL K={K}")
    lens = rng.integers(40, 101, size=(G, N)).astype(np.int32)
    want = oracle.gate(seqs, lens, 100, 70.0, sr.SR_NORM_NONE)
    got = gate_gpu(seqs, lens, 100, 70.0, sr.SR_NORM_NONE)
    assert_gate_matches(got, want, "raw distances")
    assert 0 < want[3].sum() < G
    lens[2, 3] = -5
    lens[4, 0] = -1
    status = []
    want = oracle.gate(seqs, np.maximum(lens, 0), 100, 0.8)
    got = gate_gpu(seqs, lens, 100, 0.8, status=status)
    assert_gate_matches(got, want, "negative lengths")
    assert status[0] & sr.SR_STATUS_NEG_LEN


@pytest.mark.parametrize("n_groups", [1, 8, 40, 100, 130])
def test_multiword_small_batches(n_groups):
    """Small token-level batches: the multi-word path spreads a pair over more lanes (up to a
    whole warp) when there are too few pairs to fill the machine; same outputs at every size."""
    w = W.token_gate(seed=11, n_groups=n_groups, min_len=40, max_len=1024)
    want = oracle.gate(w.seqs, w.lens, w.K, 0.4, w.norm_mode, threads=8)
    got = gate_gpu(w.seqs, w.lens, w.K, 0.4, w.norm_mode)
    assert_gate_matches(got, want, f"{n_groups} groups")


def test_multiword_shared_prefixes():
    """Rollouts that agree on their first symbols: the multi-word path leaves the common
    prefix of a pair out of the recurrence, so every prefix length around its 4-symbol
    and 128-position steps, whole-prefix containment and repeats on both sides of the
    cut are compared with the oracle."""
    rng = np.random.default_rng(31)
    stride = 512
    heads = [0, 1, 3, 4, 5, 31, 32, 33, 127, 128, 129, 255, 256, 257, 300, 511]
    G, N = len(heads), 6
    for vocab in (5, 300, 100000):                         # small vocabularies: long occurrence chains
        base = rng.integers(0, vocab, size=(G, 1, stride))
        own = rng.integers(0, vocab, size=(G, N, stride))
        pos = np.arange(stride).reshape(1, 1, stride)
        head = np.array(heads).reshape(G, 1, 1)
        seqs = np.where(pos < head, base, own).astype(np.int32)
        # force a mismatch right after the head so that the common prefix is exactly `head`
        for g, h in enumerate(heads):
            if h < stride:
                seqs[g, :, h] = vocab + np.arange(N)
        lens = rng.integers(40, stride + 1, size=(G, N)).astype(np.int32)
        lens[:, 0] = stride
        lens[3, 1] = 2                                     # shorter than the shared head: a pure prefix
        lens[9, 2] = 128
        lens[12, 3] = 256
        lens[15, 4] = 511
        want = oracle.gate(seqs, lens, stride, 0.5, threads=8)
        got = gate_gpu(seqs, lens, stride, 0.5)
        assert_gate_matches(got, want, f"shared heads vocab={vocab}")
    # identical rollouts of different lengths (every pair: one prefix contains the other),
    # and rollouts that differ only in their last symbol
    seqs = np.tile(rng.integers(0, 9, size=(1, 1, 400)), (2, 5, 1)).astype(np.int32)
    seqs[1, :, 399] = np.arange(5) + 100
    lens = np.array([[400, 399, 250, 33, 0], [400, 400, 400, 400, 400]], dtype=np.int32)
    want = oracle.gate(seqs, lens, 400, 0.01)
    got = gate_gpu(seqs, lens, 400, 0.01)
    assert_gate_matches(got, want, "contained prefixes")
    assert want[0][1].max() == 1                           # second group: one substitution per pair


def _edited_group(rng, base, N, subs, indels, vocab):
    """N rollouts derived from `base`: `subs` substitutions each, then `indels` single-symbol
    insertions or deletions at random places (lengths end up different)."""
    rows = []
    for _ in range(N):
        r = list(base)
        for p in rng.choice(len(r), size=min(subs, len(r)), replace=False):
            r[p] = int(rng.integers(0, vocab))
        for _ in range(indels):
            p = int(rng.integers(0, len(r)))
            if rng.random() < 0.5 and len(r) > 40:
                del r[p]
            else:
                r.insert(p, int(rng.integers(0, vocab)))
        rows.append(r)
    return rows


@pytest.mark.parametrize("vocab", [4, 50000])
def test_multiword_banded_pairs(vocab):
    """Pairs whose mismatch count bounds their distance well below their length run the
    banded recurrence.  Bands of every shape (few to a few hundred diagonals), lengths
    from two blocks to the maximum, equal and unequal lengths, edits bunched at the ends
    or spread out, rollouts that differ in nothing but their last symbol, and a small
    vocabulary whose repeats make the mismatch count loose and the occurrence chains long:
    every distance is compared with the oracle."""
    rng = np.random.default_rng(77 + vocab)
    stride = 1024
    groups = []
    for L in (70, 130, 300, 640, 1000, 1024):
        for subs, indels in ((1, 0), (3, 2), (L // 16, 0), (L // 8, 3), (L // 5, 8), (L // 3, 20)):
            base = rng.integers(0, vocab, size=min(L, stride - 24)).tolist()
            groups.append(_edited_group(rng, base, 5, subs, indels, vocab))
    # edits bunched at the start / at the end of otherwise identical rollouts
    base = rng.integers(0, vocab, size=900).tolist()
    front = [[int(rng.integers(0, vocab)) for _ in range(k)] + base[k:] for k in (1, 5, 37, 64, 100)]
    back = [base[:900 - k] + [int(rng.integers(0, vocab)) for _ in range(k)] for k in (1, 5, 37, 64, 100)]
    grown = [base[:900 - k] for k in (0, 1, 31, 32, 200)]                   # prefixes of one another
    shifted = [base[k:] + base[:k] for k in (0, 1, 2, 3, 40)]                # rotations: loose bound
    groups += [front, back, grown, shifted]
    G, N = len(groups), 5
    seqs = np.zeros((G, N, stride), dtype=np.int32)
    lens = np.zeros((G, N), dtype=np.int32)
    for g, rows in enumerate(groups):
        for i, r in enumerate(rows):
            r = r[:stride]
            seqs[g, i, :len(r)] = r
            lens[g, i] = len(r)
    want = oracle.gate(seqs, lens, stride, 0.1, threads=8)
    got = gate_gpu(seqs, lens, stride, 0.1)
    assert_gate_matches(got, want, f"banded pairs vocab={vocab}")
    assert 0 < want[3].sum() < G


def test_multiword_banded_full_size_converged_groups():
    """The benchmark's recipe with every group converged (10 % substitutions): all long
    equal-length pairs take the banded path, at the size the benchmark runs."""
    w = W.token_gate(seed=5, n_groups=256)
    seqs = w.seqs.copy()
    conv = W.token_gate(seed=6, n_groups=256)
    seqs[1::2] = conv.seqs[0::2][:128]                     # odd groups converged as well
    lens = w.lens.copy()
    lens[1::2] = conv.lens[0::2][:128]
    want = oracle.gate(seqs, lens, w.K, 0.25, threads=16)
    got = gate_gpu(seqs, lens, w.K, 0.25)
    assert_gate_matches(got, want, "converged token groups")


@pytest.mark.parametrize("N", [2, 3, 7, 8, 16, 32])
def test_group_sizes(N):
    rng = np.random.default_rng(N)
    for stride, K in [(32, 30), (32, 32), (8, 5), (160, 150)]:
        G = 11
        seqs = rng.integers(0, 6, size=(G, N, stride)).astype(np.int32)
        lens = rng.integers(0, stride + 1, size=(G, N)).astype(np.int32)
        want = oracle.gate(seqs, lens, K, 0.4, threads=8)
        got = gate_gpu(seqs, lens, K, 0.4)
        assert_gate_matches(got, want, f"N={N} K={K}")


def test_single_word_edges():
    rng = np.random.default_rng(1)
    # K = 0, K = 1, K = 31, K = 32 (top bit of the word), lens NULL, extreme IDs
    for K in (0, 1, 31, 32):
        seqs = rng.integers(0, 3, size=(9, 8, 32)).astype(np.int32)
        seqs[0] = np.iinfo(np.int32).max
        seqs[1, ::2] = np.iinfo(np.int32).min
        seqs[2] = -1
        for lens in (None, rng.integers(0, 33, size=(9, 8)).astype(np.int32)):
            want = oracle.gate(seqs, lens, K, 0.3)
            got = gate_gpu(seqs, lens, K, 0.3)
            assert_gate_matches(got, want, f"K={K}")
    # identical group -> d_K = 0 exactly; disjoint equal-length group -> d_K = 1 exactly
    seqs = np.zeros((2, 8, 32), dtype=np.int32)
    seqs[0] = np.arange(32)
    seqs[1] = np.arange(8 * 32).reshape(8, 32)
    _, _, mean, stop = gate_gpu(seqs, None, 30, 0.12)
    assert mean.tolist() == [0.0, 1.0] and stop.tolist() == [1, 0]


def test_threshold_is_strict_and_modes():
    seqs = np.zeros((1, 2, 4), dtype=np.int32)
    seqs[0, 0] = [1, 2, 3, 4]
    seqs[0, 1] = [1, 2, 3, 5]
    _, _, mean, stop = gate_gpu(seqs, None, 4, 0.25)
    assert mean[0] == 0.25 and stop[0] == 0
    _, _, _, stop = gate_gpu(seqs, None, 4, np.nextafter(0.25, 1.0))
    assert stop[0] == 1
    _, ps, mean, _ = gate_gpu(seqs, None, 4, 0.25, sr.SR_NORM_NONE)
    assert ps[0] == 1 and mean[0] == 1.0


def test_negative_lengths_are_clamped_and_flagged():
    rng = np.random.default_rng(6)
    for stride in (32, 96):
        seqs = rng.integers(0, 4, size=(5, 4, stride)).astype(np.int32)
        lens = rng.integers(1, stride, size=(5, 4)).astype(np.int32)
        lens[2, 1] = -5
        st = []
        got = gate_gpu(seqs, lens, stride, 0.3, status=st)
        want = oracle.gate(seqs, np.maximum(lens, 0), stride, 0.3)
        assert_gate_matches(got, want, "neg len")
        assert st[0] & sr.SR_STATUS_NEG_LEN


def test_host_buffer_entry_point():
    w = W.agent_gate(K=15)
    for wl in (w, W.token_gate(n_groups=72)):
        G, N, stride = wl.seqs.shape
        P = N * (N - 1) // 2
        h_seqs = torch.from_numpy(wl.seqs).pin_memory()
        h_lens = torch.from_numpy(wl.lens).pin_memory()
        pd = torch.empty((G, P), dtype=torch.int32).pin_memory()
        ps = torch.empty((G,), dtype=torch.int32).pin_memory()
        mean = torch.empty((G,), dtype=torch.float64).pin_memory()
        stop = torch.empty((G,), dtype=torch.uint8).pin_memory()
        arena = torch.empty(sr.sr_gate_host_arena_bytes(G, N, stride, wl.K), dtype=torch.uint8, device="cuda:0")
        want = oracle.gate(wl.seqs, wl.lens, wl.K, 0.5, threads=8)
        for cs in (None, torch.cuda.Stream()):          # one stream, then copies overlapped in chunks
            for t in (pd, ps, mean, stop):
                t.zero_()
            sr.sr_gate_host(h_seqs, h_lens, wl.K, 0.5, pair_dist=pd, pair_sum=ps, mean=mean, stop=stop,
                            arena=arena, copy_stream=cs)
            torch.cuda.synchronize()
            assert_gate_matches((pd.numpy(), ps.numpy(), mean.numpy(), stop.numpy()), want, "host " + wl.name)


# ------------------------------------------------------------------ incremental
def _check_stream(s, G=None):
    actions = s.actions if G is None else s.actions[:, :G]
    inc = IncrementalGate(actions.shape[1], actions.shape[2], max_steps=actions.shape[0])
    for t, opd, ops, omean, ostop in oracle.gate_stream(actions, s.threshold, s.norm_mode, threads=8):
        got = inc.step(actions[t - 1], s.threshold, s.norm_mode)
        assert_gate_matches(got, (opd, ops, omean, ostop), f"{s.name} step {t}")
    assert int(inc.status.item()) == 0
    return inc


def test_packed_host_entry_point():
    """Packed (ragged) host input: same outputs as the oracle on the padded batch, on the
    single-word and the multi-word path, with empty rows and rows longer than K, in one
    piece and in pieces on a copy stream, on one arena."""
    dev = torch.device("cuda:0")
    cs = torch.cuda.Stream(device=dev)
    cases = [(W.agent_gate(K=15), 15), (W.token_gate(n_groups=72), 1024), (W.token_gate(n_groups=72), 500)]
    for w, K in cases:
        lens = w.lens.copy()
        lens[0, 0] = 0
        G, N, stride = w.seqs.shape
        P = N * (N - 1) // 2
        want = oracle.gate(w.seqs, lens, K, 0.3, w.norm_mode, threads=8)
        symbols, row_start = W.pack_rows(w.seqs, lens)
        h_sym = torch.from_numpy(symbols).pin_memory()
        h_rs = torch.from_numpy(row_start).pin_memory()
        arena = torch.empty(sr.sr_gate_host_packed_arena_bytes(G, N, stride, K), dtype=torch.uint8, device=dev)
        for copy_stream in (None, cs, cs):
            pd = torch.full((G, P), -7, dtype=torch.int32).pin_memory()
            ps = torch.full((G,), -7, dtype=torch.int32).pin_memory()
            mean = torch.full((G,), -7.0, dtype=torch.float64).pin_memory()
            stop = torch.full((G,), 9, dtype=torch.uint8).pin_memory()
            st = torch.zeros(1, dtype=torch.int32).pin_memory()
            sr.sr_gate_host_packed(h_sym, h_rs, N, stride, K, 0.3, w.norm_mode, pair_dist=pd, pair_sum=ps,
                                   mean=mean, stop=stop, status=st, arena=arena, copy_stream=copy_stream)
            torch.cuda.synchronize()
            assert_gate_matches((pd.numpy(), ps.numpy(), mean.numpy(), stop.numpy()), want,
                                f"packed {w.name} K={K} copy stream {copy_stream is not None}")
            assert int(st.item()) == 0


def test_c5_incremental_equals_recompute_every_step():
    _check_stream(W.streaming_gate(n_groups=2048))


def test_c5_incremental_ragged_termination():
    _check_stream(W.streaming_gate(n_groups=1024, ragged=True))


def test_incremental_full_size_every_step():
    """The benchmark's own size (65 536 groups), compared with a recomputation from
    scratch after every one of the 30 steps."""
    s = W.streaming_gate()
    inc = IncrementalGate(s.n_groups, s.N, max_steps=s.steps)
    threads = min(16, oracle.max_threads())
    for t in range(s.steps):
        got = inc.step(s.actions[t], s.threshold, s.norm_mode)
        seqs, lens = W.stream_prefix(s.actions, t + 1)
        want = oracle.gate(seqs, lens, 32, s.threshold, s.norm_mode, threads=threads)
        assert_gate_matches(got, want, f"C5 full step {t + 1}")


def test_incremental_other_group_sizes_overflow_and_snapshot():
    rng = np.random.default_rng(12)
    for N in (2, 5, 16):
        G, steps = 37, 32
        actions = rng.integers(0, 4, size=(steps, G, N)).astype(np.int32)
        actions[rng.random(actions.shape) < 0.2] = sr.SR_NO_ACTION
        inc = IncrementalGate(G, N, max_steps=32)
        snap = None
        for t, opd, ops, omean, ostop in oracle.gate_stream(actions, 0.4, 0):
            got = inc.step(actions[t - 1], 0.4)
            assert_gate_matches(got, (opd, ops, omean, ostop), f"N={N} step {t}")
            if t == 15:
                snap = inc.state.clone()
        # restore the snapshot into a fresh buffer and replay: identical results
        inc2 = IncrementalGate(G, N, max_steps=32)
        inc2.state.copy_(snap)
        for t in range(15, steps):
            got2 = inc2.step(actions[t], 0.4)
        assert_gate_matches(got2, got, "snapshot replay")
    # a 33rd action is ignored and flagged
    inc = IncrementalGate(3, 4, max_steps=4)
    a = np.ones((3, 4), dtype=np.int32)
    for _ in range(4):
        before = inc.step(a, 0.4)
    after = inc.step(a, 0.4)
    assert_gate_matches(after, before, "overflow ignored")
    assert int(inc.status.item()) & sr.SR_STATUS_STEP_OVERFLOW
    # state formatted for other sizes is refused
    inc.status.zero_()
    bad = torch.from_numpy(np.ones((2, 4), dtype=np.int32)).cuda()
    sr.sr_gate_step_incremental(inc.state, bad, 0.4, stop=inc.stop[:2], status=inc.status)
    torch.cuda.synchronize()
    assert int(inc.status.item()) & sr.SR_STATUS_BAD_STATE


# -------------------------------------------------------------------- advantages
def _check_adv(rewards, drop=None, eps=1e-6):
    adv, zv = advantage_gpu(rewards, drop, eps)
    oadv, ozv = oracle.advantage(rewards, drop, eps)
    assert np.array_equal(zv, ozv)
    zero = oadv == 0
    assert np.array_equal(adv == 0, zero) and not np.signbit(adv[zero]).any()
    nan = np.isnan(oadv)
    assert np.array_equal(np.isnan(adv), nan)
    ok = ~zero & ~nan
    assert np.all(np.abs(adv[ok] - oadv[ok]) <= 1e-6 * np.abs(oadv[ok]))
    return adv, zv


def test_advantages_on_every_config():
    for w in (W.tiny_gate(), W.agent_gate(), W.large_group_gate(), W.token_gate(n_groups=1024)):
        _, zv = _check_adv(w.rewards)
    s = W.streaming_gate()
    _, zv = _check_adv(s.rewards)
    assert 0 < zv.sum() < s.n_groups
    drop = (np.arange(s.n_groups) % 3 == 0).astype(np.uint8)
    adv, _ = _check_adv(s.rewards, drop)
    assert (adv[drop == 1] == 0).all()


def test_advantage_edges():
    rng = np.random.default_rng(3)
    for N in (2, 3, 5, 8, 16, 31, 32):
        r = rng.random((257, N)).astype(np.float32)
        r[0] = 0.3
        r[1] = -0.0
        r[1, 0] = 0.0
        r[2, 0] = np.nan
        r[3] = np.float32(1e30)
        r[4, : N // 2] = 1.0
        r[4, N // 2:] = 0.0
        for eps in (1e-6, 0.0):
            _check_adv(r, None, eps)


def test_binding_refuses_short_or_misplaced_buffers():
    """An output that cannot hold what the call writes, or a host tensor where the library
    expects device memory, is refused by the binding before anything is launched."""
    dev = torch.device("cuda:0")
    w = W.agent_gate(K=15)
    seqs, lens = torch.from_numpy(w.seqs).to(dev), torch.from_numpy(w.lens).to(dev)
    G, N, _ = seqs.shape
    stop = torch.zeros(G, dtype=torch.uint8, device=dev)
    with pytest.raises(ValueError, match="stop holds"):
        sr.sr_gate(seqs, lens, w.K, 0.12, stop=stop[: G - 1])
    with pytest.raises(ValueError, match="pair_dist holds"):
        sr.sr_gate(seqs, lens, w.K, 0.12, stop=stop, pair_dist=torch.zeros((G, 27), dtype=torch.int32, device=dev))
    with pytest.raises(ValueError, match="lens holds"):
        sr.sr_gate(seqs, lens[:-1], w.K, 0.12, stop=stop)
    with pytest.raises(ValueError, match="CUDA tensor"):
        sr.sr_gate(seqs, lens.cpu(), w.K, 0.12, stop=stop)
    with pytest.raises(ValueError, match="host tensor"):
        sr.sr_gate_host(seqs, None, w.K, 0.12, stop=stop.cpu(), arena=torch.empty(1 << 20, dtype=torch.uint8, device=dev))
    rewards = torch.rand((G, N), device=dev)
    with pytest.raises(ValueError, match="adv holds"):
        sr.sr_grpo_advantage(rewards, None, 1e-6, adv=torch.empty((G, N - 1), device=dev))
    sr.sr_gate(seqs, lens, w.K, 0.12, stop=stop)                       # and the well-formed call still runs
    torch.cuda.synchronize()
    assert np.array_equal(stop.cpu().numpy(), oracle.gate(w.seqs, w.lens, w.K, 0.12)[3])
