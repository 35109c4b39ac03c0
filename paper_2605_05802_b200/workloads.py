"""Seeded synthetic inputs for the Selective Rollout gate.

This module only *draws inputs* (action / token ID sequences, prefix lengths,
rewards).  It contains none of the method's arithmetic: no edit distance, no
normalisation, no thresholding, no advantages.  Both the CPU oracle and the
CUDA path consume the arrays produced here, so that the two are compared on
identical inputs without sharing any computational code.

The five workloads stand in for the paper's ALFWorld rollouts (Section 3.1:
G = 8 rollouts per group, horizon T_max = 30, gate step K in {10, 15}, about
40 % zero-variance groups), which are not available offline.  All randomness
comes from ``numpy.random.Generator(PCG64(seed))``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

SR_NORM_MAXLEN = 0
SR_NORM_NONE = 1
SR_NO_ACTION = -(2 ** 31)


@dataclass
class GateWorkload:
    """One batch of GRPO groups handed to the gate.

    seqs     int32 [n_groups, N, stride]  action (or token) IDs, zero padded
    lens     int32 [n_groups, N]          actions emitted so far per rollout
    K        gate step; the effective prefix of rollout i is min(lens_i, K)
    rewards  float32 [n_groups, N]        terminal rewards (advantage input)
    """

    name: str
    seqs: np.ndarray
    lens: np.ndarray
    K: int
    threshold: float
    norm_mode: int
    rewards: np.ndarray
    extra: Dict[str, object] = field(default_factory=dict)

    @property
    def n_groups(self) -> int:
        return int(self.seqs.shape[0])

    @property
    def N(self) -> int:
        return int(self.seqs.shape[1])

    @property
    def stride(self) -> int:
        return int(self.seqs.shape[2])


@dataclass
class StreamWorkload:
    """Streaming input: one new action per rollout per environment step.

    actions  int32 [steps, n_groups, N]; SR_NO_ACTION where a rollout has
             already terminated.
    """

    name: str
    actions: np.ndarray
    threshold: float
    norm_mode: int
    rewards: np.ndarray

    @property
    def steps(self) -> int:
        return int(self.actions.shape[0])

    @property
    def n_groups(self) -> int:
        return int(self.actions.shape[1])

    @property
    def N(self) -> int:
        return int(self.actions.shape[2])


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def mutated_rollouts(rng: np.random.Generator, n_groups: int, N: int, vocab: int,
                     out_len: int, p: np.ndarray, stride: int) -> np.ndarray:
    """Rollouts of a group as noisy copies of one per-group base sequence.

    Each rollout walks its group's base; at every position, with probability
    p[g], one of {substitute, insert, delete} (chosen uniformly) is applied,
    otherwise the base symbol is emitted.  The first ``out_len`` emitted
    symbols form the rollout.  Returns int32 [n_groups, N, stride].
    """
    base_len = 4 * out_len + 8
    base = rng.integers(0, vocab, size=(n_groups, base_len), dtype=np.int64)
    seqs = np.zeros((n_groups, N, stride), dtype=np.int32)
    ptr = np.zeros((n_groups, N), dtype=np.int64)
    cnt = np.zeros((n_groups, N), dtype=np.int64)
    pg = np.broadcast_to(np.asarray(p, dtype=np.float64).reshape(n_groups, 1), (n_groups, N))
    gi = np.broadcast_to(np.arange(n_groups).reshape(n_groups, 1), (n_groups, N))
    ni = np.broadcast_to(np.arange(N).reshape(1, N), (n_groups, N))
    for _ in range(8 * out_len + 64):
        live = cnt < out_len
        if not live.any():
            break
        u = rng.random((n_groups, N))
        op = rng.integers(0, 3, size=(n_groups, N))
        rnd = rng.integers(0, vocab, size=(n_groups, N), dtype=np.int64)
        mutate = u < pg
        cur = base[gi, np.minimum(ptr, base_len - 1)]
        sub = mutate & (op == 0)
        ins = mutate & (op == 1)
        dele = mutate & (op == 2)
        emit = live & ~dele
        sym = np.where(sub | ins, rnd, cur)
        g_e, n_e = gi[emit], ni[emit]
        seqs[g_e, n_e, cnt[emit]] = sym[emit].astype(np.int32)
        cnt = cnt + emit.astype(np.int64)
        ptr = ptr + (live & ~ins).astype(np.int64)
    assert (cnt >= out_len).all()
    return seqs


def _equal_or_iid_rewards(rng: np.random.Generator, n_groups: int, N: int,
                          equal: np.ndarray) -> np.ndarray:
    """Binary rewards: groups flagged in ``equal`` get one shared Bernoulli(0.5)
    draw, the others independent Bernoulli(0.5) draws."""
    shared = rng.integers(0, 2, size=(n_groups, 1))
    iid = rng.integers(0, 2, size=(n_groups, N))
    r = np.where(equal.reshape(n_groups, 1), shared, iid)
    return r.astype(np.float32)


def tiny_gate(seed: int = 0, raw_threshold: bool = True) -> GateWorkload:
    """16 groups x N=8, vocab 64, every prefix length 10; groups 0-7 mutate with
    probability 0.05 (converged), groups 8-15 with 0.6 (divergent).  With
    ``raw_threshold`` the gate thresholds the un-normalised mean distance at 2.0,
    otherwise the normalised mean at 0.2."""
    rng = _rng(seed)
    n_groups, N, K = 16, 8, 10
    p = np.where(np.arange(n_groups) < 8, 0.05, 0.6)
    seqs = mutated_rollouts(rng, n_groups, N, 64, K, p, 32)
    lens = np.full((n_groups, N), K, dtype=np.int32)
    rewards = rng.integers(0, 2, size=(n_groups, N)).astype(np.float32)
    if raw_threshold:
        return GateWorkload("C1-tiny", seqs, lens, K, 2.0, SR_NORM_NONE, rewards)
    return GateWorkload("C1-tiny-normalised", seqs, lens, K, 0.2, SR_NORM_MAXLEN, rewards)


def agent_gate(seed: int = 1, K: int = 15, n_groups: int = 512) -> GateWorkload:
    """512 groups x N=8, vocab 4096, rollout lengths uniform on 1..30, gate at
    step K; 40 % of groups converged (mutation 0.02, all rewards equal) and 60 %
    divergent (mutation 0.5, iid Bernoulli rewards)."""
    rng = _rng(seed)
    N, T = 8, 30
    converged = rng.random(n_groups) < 0.4
    p = np.where(converged, 0.02, 0.5)
    seqs = mutated_rollouts(rng, n_groups, N, 4096, T, p, 32)
    lens = rng.integers(1, T + 1, size=(n_groups, N)).astype(np.int32)
    mask = np.arange(32).reshape(1, 1, 32) < lens[:, :, None]
    seqs = np.where(mask, seqs, 0).astype(np.int32)
    rewards = _equal_or_iid_rewards(rng, n_groups, N, converged)
    return GateWorkload(f"C2-agent-K{K}", seqs, lens, K, 0.12, SR_NORM_MAXLEN, rewards)


def large_group_gate(seed: int = 2, n_groups: int = 4096, threshold: float = 0.12) -> GateWorkload:
    """4096 groups x N=16 (120 pairs), vocab 4096, every prefix length 30,
    per-group mutation probability from Beta(0.5, 2); rewards all-equal with
    probability 1 - p_g, else iid Bernoulli(0.5)."""
    rng = _rng(seed)
    N, K = 16, 30
    p = rng.beta(0.5, 2.0, size=n_groups)
    seqs = mutated_rollouts(rng, n_groups, N, 4096, K, p, 32)
    lens = np.full((n_groups, N), K, dtype=np.int32)
    equal = rng.random(n_groups) < (1.0 - p)
    rewards = _equal_or_iid_rewards(rng, n_groups, N, equal)
    return GateWorkload("C3-large-group", seqs, lens, K, threshold, SR_NORM_MAXLEN, rewards,
                        {"mutation_p": p})


def token_gate(seed: int = 3, n_groups: int = 1024, min_len: int = 256, max_len: int = 1024,
               N: int = 8, vocab: int = 151936, shared_head: bool = True) -> GateWorkload:
    """Token-level prefixes: lengths uniform on min_len..max_len.  Even groups
    are converged (one base, every rollout substitutes an independent random
    10 % of positions); odd groups share a random-length head then diverge
    (``shared_head=False``: they diverge from the first token, a variant used to
    time the kernels on inputs without common prefixes)."""
    rng = _rng(seed)
    stride = (max_len + 3) // 4 * 4
    lens = rng.integers(min_len, max_len + 1, size=(n_groups, N)).astype(np.int32)
    base = rng.integers(0, vocab, size=(n_groups, 1, stride), dtype=np.int64)
    own = rng.integers(0, vocab, size=(n_groups, N, stride), dtype=np.int64)
    sub = rng.random((n_groups, N, stride)) < 0.10
    conv = np.where(sub, own, base)
    head = (rng.random(n_groups) * (lens.min(axis=1) + 1)).astype(np.int64)
    if not shared_head:
        head[:] = 0
    pos = np.arange(stride).reshape(1, 1, stride)
    div = np.where(pos < head.reshape(n_groups, 1, 1), base, own)
    is_conv = (np.arange(n_groups) % 2 == 0).reshape(n_groups, 1, 1)
    seqs = np.where(is_conv, conv, div)
    seqs = np.where(pos < lens[:, :, None], seqs, 0).astype(np.int32)
    rewards = rng.random((n_groups, N), dtype=np.float32)
    return GateWorkload("C4-token", seqs, lens, max_len, 0.12, SR_NORM_MAXLEN, rewards)


def streaming_gate(seed: int = 4, n_groups: int = 65536, steps: int = 30, N: int = 8,
                   ragged: bool = False) -> StreamWorkload:
    """One new action per rollout per step.  Each group has a 64-symbol base and
    each rollout a base pointer: with probability 1 - p_g the rollout emits
    base[ptr] and advances, otherwise uniformly one of {random symbol & advance,
    random symbol & stay, base[ptr+1] & advance by two}.  p_g ~ Beta(0.5, 2).
    With ``ragged`` every rollout terminates after U{10..steps} actions and
    emits SR_NO_ACTION from then on."""
    rng = _rng(seed)
    vocab, base_len = 4096, 2 * steps + 8
    p = rng.beta(0.5, 2.0, size=n_groups)
    base = rng.integers(0, vocab, size=(n_groups, base_len), dtype=np.int64)
    ptr = np.zeros((n_groups, N), dtype=np.int64)
    gi = np.broadcast_to(np.arange(n_groups).reshape(n_groups, 1), (n_groups, N))
    actions = np.empty((steps, n_groups, N), dtype=np.int32)
    stop_at = (rng.integers(10, steps + 1, size=(n_groups, N)) if ragged
               else np.full((n_groups, N), steps))
    for t in range(steps):
        u = rng.random((n_groups, N))
        op = rng.integers(0, 3, size=(n_groups, N))
        rnd = rng.integers(0, vocab, size=(n_groups, N), dtype=np.int64)
        mutate = u < p.reshape(n_groups, 1)
        skip = mutate & (op == 2)
        cur = base[gi, np.minimum(ptr + skip, base_len - 1)]
        sym = np.where(mutate & (op < 2), rnd, cur)
        adv = np.where(mutate & (op == 1), 0, np.where(skip, 2, 1))
        ptr = ptr + adv
        actions[t] = np.where(t < stop_at, sym, SR_NO_ACTION).astype(np.int32)
    equal = rng.random(n_groups) < (1.0 - p)
    rewards = _equal_or_iid_rewards(rng, n_groups, N, equal)
    return StreamWorkload("C5-stream" + ("-ragged" if ragged else ""), actions, 0.12,
                          SR_NORM_MAXLEN, rewards)


def stream_prefix(actions: np.ndarray, upto: int, stride: int = 32):
    """Replay the first ``upto`` steps of a stream into (seqs, lens) arrays: a
    rollout's sequence is its non-SR_NO_ACTION entries in step order."""
    steps, n_groups, N = actions.shape
    seqs = np.zeros((n_groups, N, stride), dtype=np.int32)
    lens = np.zeros((n_groups, N), dtype=np.int32)
    gi = np.broadcast_to(np.arange(n_groups).reshape(n_groups, 1), (n_groups, N))
    ni = np.broadcast_to(np.arange(N).reshape(1, N), (n_groups, N))
    for t in range(upto):
        a = actions[t]
        act = a != SR_NO_ACTION
        seqs[gi[act], ni[act], lens[act]] = a[act]
        lens = lens + act.astype(np.int32)
    return seqs, lens


def dp_cells(lens: np.ndarray, K: int) -> int:
    """Number of cells of the textbook DP matrices the gate's definition covers:
    the sum over unordered rollout pairs of m_i * m_j with m = min(len, K).
    Used only to express throughput; not part of the method."""
    m = np.minimum(np.maximum(lens.astype(np.int64), 0), K)
    s1 = m.sum(axis=1)
    s2 = (m * m).sum(axis=1)
    return int(((s1 * s1 - s2) // 2).sum())


def _band_units(rows: np.ndarray, cols: np.ndarray, ub: np.ndarray) -> np.ndarray:
    """(column, 32-row block) units inside the band of a rows x cols matrix whose
    distance is at most ub: diagonals d = row - column with |d| + |(rows - cols) - d| <= ub
    (at least two diagonals).  Vectorised over pairs; loops over the columns."""
    D = rows - cols
    e = np.maximum((ub - np.abs(D)) // 2, 0)
    dlo = np.minimum(D, 0) - e
    dhi = np.maximum(D, 0) + e
    dhi = np.where(dhi == dlo, dhi + 1, dhi)
    total = np.zeros_like(rows)
    for c in range(int(cols.max(initial=0))):
        lo = np.maximum(c + dlo, 0)
        hi = np.minimum(c + dhi, rows - 1)
        ok = (c < cols) & (hi >= lo)
        total += np.where(ok, hi // 32 - lo // 32 + 1, 0)
    return total


def word_columns(lens: np.ndarray, K: int, seqs: np.ndarray = None, band: bool = False) -> int:
    """Work units of the bit-vector method: the sum over unordered pairs of
    (text columns) x (32-row blocks of the pattern), taking for every pair the
    cheaper of the two orientations.  Used only to express roofline fractions.
    With ``seqs`` the common prefix of every pair, rounded down to a multiple of
    four symbols, is left out (nothing at all if one prefix contains the other):
    the multi-word kernels never run those rows and columns.  With ``band`` a pair
    also counts no more than the units inside the band that its mismatch count
    implies (differing positions after the common prefix + length difference is an
    upper bound of the distance; an optimal alignment stays within the diagonals
    that bound allows), again in the cheaper orientation."""
    m = np.minimum(np.maximum(lens.astype(np.int64), 0), K)
    total = 0
    N = lens.shape[1]
    pos = None if seqs is None else np.arange(seqs.shape[2]).reshape(1, -1)
    for i in range(N):
        for j in range(i + 1, N):
            a, b = m[:, i], m[:, j]
            if seqs is not None:
                lo = np.minimum(a, b)
                differs = (seqs[:, i, :] != seqs[:, j, :]) | (pos >= lo.reshape(-1, 1))
                first = np.where(differs.any(axis=1), np.argmax(differs, axis=1), lo)
                cut = np.where(first >= lo, np.maximum(a, b), first & ~3)
                ra, rb = np.maximum(a - cut, 0), np.maximum(b - cut, 0)
            else:
                ra, rb = a, b
            units = np.minimum(ra * ((rb + 31) // 32), rb * ((ra + 31) // 32))
            if band and seqs is not None:
                lo = np.minimum(a, b)
                mism = ((seqs[:, i, :] != seqs[:, j, :]) & (pos < lo.reshape(-1, 1))).sum(axis=1)
                ub = mism + np.abs(a - b)
                live = (ra > 0) & (rb > 0)
                banded = np.minimum(_band_units(np.where(live, ra, 0), np.where(live, rb, 0), ub),
                                    _band_units(np.where(live, rb, 0), np.where(live, ra, 0), ub))
                units = np.where(live, np.minimum(units, banded), units)
            total += int(units.sum())
    return total


def pack_rows(seqs: np.ndarray, lens: np.ndarray):
    """Packed (ragged) form of a padded batch: the first len symbols of every row back to
    back, and the int64 offsets at which the rows begin (rows + 1 entries)."""
    G, N, stride = seqs.shape
    n = np.clip(lens.reshape(-1).astype(np.int64), 0, stride)
    row_start = np.zeros(G * N + 1, dtype=np.int64)
    np.cumsum(n, out=row_start[1:])
    keep = np.arange(stride).reshape(1, stride) < n.reshape(-1, 1)
    symbols = np.ascontiguousarray(seqs.reshape(G * N, stride)[keep], dtype=np.int32)
    return symbols, row_start


def all_gate_configs() -> List[GateWorkload]:
    return [tiny_gate(), tiny_gate(raw_threshold=False), agent_gate(K=15), agent_gate(K=30),
            large_group_gate(), token_gate()]
