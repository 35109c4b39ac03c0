"""CPU oracle for the Selective Rollout gate -- TEST INFRASTRUCTURE ONLY.

Python face of ``sr_oracle.c`` (textbook O(mn) Levenshtein DP, ordered fp64
mean, strict threshold, fp64 mean/std advantages).  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library and its binding never do, and this package never imports them.

Section 3.2 and Appendix B of the paper define d_K, Eq. 2 the gate, Eq. 1 the
advantages and Section 2.1 the zero-variance case.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from fractions import Fraction
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sr_oracle.c")
_LIB = os.path.join(_HERE, "_sr_oracle.so")

NORM_MAXLEN = 0
NORM_NONE = 1
NO_ACTION = -(2 ** 31)

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fused multiply-add contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC",
                               "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        lib.sro_levenshtein.restype = ctypes.c_int32
        lib.sro_levenshtein.argtypes = [i32p, ctypes.c_int32, i32p, ctypes.c_int32]
        lib.sro_gate.restype = None
        lib.sro_gate.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                 ctypes.c_int32, ctypes.c_int32, ctypes.c_double, ctypes.c_int32,
                                 ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                 ctypes.c_int32]
        lib.sro_advantage.restype = None
        lib.sro_advantage.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                                      ctypes.c_int32, ctypes.c_float, ctypes.c_void_p,
                                      ctypes.c_void_p]
        lib.sro_or_rule.restype = None
        lib.sro_or_rule.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                                    ctypes.c_int32, ctypes.c_int32, ctypes.c_double, ctypes.c_double,
                                    ctypes.c_void_p, ctypes.c_void_p]
        lib.sro_batch_stats.restype = None
        lib.sro_batch_stats.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                        ctypes.c_void_p, ctypes.c_void_p]
        lib.sro_savings_fraction.restype = ctypes.c_double
        lib.sro_savings_fraction.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32]
        lib.sro_dilution_gain.restype = ctypes.c_double
        lib.sro_dilution_gain.argtypes = [ctypes.c_double, ctypes.c_double]
        lib.sro_group_signals.restype = None
        lib.sro_group_signals.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                          ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_void_p]
        lib.sro_kept_groups.restype = ctypes.c_int32
        lib.sro_kept_groups.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p]
        lib.sro_max_threads.restype = ctypes.c_int32
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().sro_max_threads())


def levenshtein(a, b) -> int:
    """Unit-cost edit distance between two integer sequences (Section 3.2)."""
    a = np.ascontiguousarray(np.asarray(a, dtype=np.int32).reshape(-1))
    b = np.ascontiguousarray(np.asarray(b, dtype=np.int32).reshape(-1))
    i32p = ctypes.POINTER(ctypes.c_int32)
    return int(_load().sro_levenshtein(a.ctypes.data_as(i32p), a.size, b.ctypes.data_as(i32p), b.size))


def gate(seqs: np.ndarray, lens: Optional[np.ndarray], K: int, threshold: float,
         norm_mode: int = NORM_MAXLEN, threads: int = 1):
    """d_K and the stop mask for every group.

    Returns (pair_dist int32 [G, P], pair_sum int32 [G], mean float64 [G],
    stop uint8 [G]) with pairs ordered (0,1),(0,2),...,(N-2,N-1).
    """
    seqs = np.ascontiguousarray(seqs, dtype=np.int32)
    G, N, stride = seqs.shape
    assert N >= 2 and 0 <= K <= stride
    P = N * (N - 1) // 2
    lp = None
    if lens is not None:
        lens = np.ascontiguousarray(lens, dtype=np.int32)
        assert lens.shape == (G, N)
        lp = lens.ctypes.data
    pair_dist = np.zeros((G, P), dtype=np.int32)
    pair_sum = np.zeros(G, dtype=np.int32)
    mean = np.zeros(G, dtype=np.float64)
    stop = np.zeros(G, dtype=np.uint8)
    _load().sro_gate(seqs.ctypes.data, lp, G, N, stride, K, float(threshold), int(norm_mode),
                     pair_dist.ctypes.data, pair_sum.ctypes.data, mean.ctypes.data,
                     stop.ctypes.data, int(threads))
    return pair_dist, pair_sum, mean, stop


def advantage(rewards: np.ndarray, drop_mask: Optional[np.ndarray] = None, eps: float = 1e-6
              ) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 1 advantages (fp32) and the zero-variance flag per group."""
    rewards = np.ascontiguousarray(rewards, dtype=np.float32)
    G, N = rewards.shape
    dp = None
    if drop_mask is not None:
        drop_mask = np.ascontiguousarray(drop_mask, dtype=np.uint8)
        dp = drop_mask.ctypes.data
    adv = np.zeros((G, N), dtype=np.float32)
    zv = np.zeros(G, dtype=np.uint8)
    _load().sro_advantage(rewards.ctypes.data, dp, G, N, float(np.float32(eps)), adv.ctypes.data,
                          zv.ctypes.data)
    return adv, zv


def or_rule(mean: np.ndarray, lens: Optional[np.ndarray], done: Optional[np.ndarray], K: int,
            threshold: float, tau_high: float):
    """tau_K (fraction of finished rollouts) and the OR-rule mask of Eq. 3.
    Returns (tau float64 [G], stop uint8 [G])."""
    mean = np.ascontiguousarray(mean, dtype=np.float64)
    G = mean.shape[0]
    lp = dp = None
    if done is not None:
        done = np.ascontiguousarray(done, dtype=np.uint8)
        N = done.shape[1]
        dp = done.ctypes.data
    if lens is not None:
        lens = np.ascontiguousarray(lens, dtype=np.int32)
        N = lens.shape[1]
        lp = lens.ctypes.data
    tau = np.zeros(G, dtype=np.float64)
    stop = np.zeros(G, dtype=np.uint8)
    _load().sro_or_rule(mean.ctypes.data, lp, dp, G, N, int(K), float(threshold), float(tau_high),
                        tau.ctypes.data, stop.ctypes.data)
    return tau, stop


def absent_lower_bound(a, b) -> int:
    """max(|len a - len b|, symbols of b that occur nowhere in a): a lower bound of the
    edit distance (every such symbol must be deleted or substituted)."""
    a = [int(x) for x in a]
    b = [int(x) for x in b]
    present = set(a)
    return max(abs(len(a) - len(b)), sum(1 for x in b if x not in present))


def group_signals(seqs: np.ndarray, lens: Optional[np.ndarray], K: int):
    """(unique_prefix_ratio, unique_action_ratio, action_entropy, bigram_jaccard_mean),
    float64 [G] each (Appendix B)."""
    seqs = np.ascontiguousarray(seqs, dtype=np.int32)
    G, N, stride = seqs.shape
    lp = None
    if lens is not None:
        lens = np.ascontiguousarray(lens, dtype=np.int32)
        lp = lens.ctypes.data
    outs = [np.zeros(G, dtype=np.float64) for _ in range(4)]
    _load().sro_group_signals(seqs.ctypes.data, lp, G, N, stride, int(K), *[o.ctypes.data for o in outs])
    return tuple(outs)


def batch_stats(adv: np.ndarray, stop: Optional[np.ndarray]):
    """(counts int64 [3], sumsq float64 [2]): zero advantages over all / kept groups,
    kept groups; squared advantage norm over all / kept groups."""
    adv = np.ascontiguousarray(adv, dtype=np.float32)
    G, N = adv.shape
    sp = None
    if stop is not None:
        stop = np.ascontiguousarray(stop, dtype=np.uint8)
        sp = stop.ctypes.data
    counts = np.zeros(3, dtype=np.int64)
    sumsq = np.zeros(2, dtype=np.float64)
    _load().sro_batch_stats(adv.ctypes.data, sp, G, N, counts.ctypes.data, sumsq.ctypes.data)
    return counts, sumsq


def kept_groups(stop: Optional[np.ndarray], zero_var: Optional[np.ndarray] = None,
                n_groups: Optional[int] = None) -> np.ndarray:
    """Ascending indices (int32) of the groups that stay in the batch: not cut
    (Appendix C.1) and, when ``zero_var`` is given, not zero-variance either."""
    sp = zp = None
    if stop is not None:
        stop = np.ascontiguousarray(stop, dtype=np.uint8)
        sp, n_groups = stop.ctypes.data, stop.shape[0]
    if zero_var is not None:
        zero_var = np.ascontiguousarray(zero_var, dtype=np.uint8)
        zp, n_groups = zero_var.ctypes.data, zero_var.shape[0]
    index = np.zeros(max(int(n_groups), 1), dtype=np.int32)
    kept = int(_load().sro_kept_groups(sp, zp, int(n_groups), index.ctypes.data))
    return index[:kept].copy()


def savings_fraction(cut: int, n_groups: int, T_max: int, K: int) -> float:
    return float(_load().sro_savings_fraction(cut, n_groups, T_max, K))


def dilution_gain(before: float, after: float) -> float:
    return float(_load().sro_dilution_gain(before, after))


def replay(actions: np.ndarray, upto: int, stride: int = 32):
    """Sequences and lengths after the first ``upto`` steps of an action stream
    (int32 [steps, G, N], NO_ACTION where a rollout did not act)."""
    steps, G, N = actions.shape
    seqs = np.zeros((G, N, stride), dtype=np.int32)
    lens = np.zeros((G, N), dtype=np.int32)
    for t in range(upto):
        a = actions[t]
        act = a != NO_ACTION
        g_idx, n_idx = np.nonzero(act)
        seqs[g_idx, n_idx, lens[g_idx, n_idx]] = a[g_idx, n_idx]
        lens[g_idx, n_idx] += 1
    return seqs, lens


def gate_stream(actions: np.ndarray, threshold: float, norm_mode: int = NORM_MAXLEN,
                threads: int = 1, steps: Optional[int] = None):
    """Gate evaluated after every step of a stream, each time recomputed from
    scratch on the prefixes emitted so far (no incremental state).  Yields
    (step, pair_dist, pair_sum, mean, stop)."""
    total = actions.shape[0] if steps is None else steps
    for t in range(1, total + 1):
        seqs, lens = replay(actions, t)
        yield (t,) + gate(seqs, lens, seqs.shape[2], threshold, norm_mode, threads)


def exact_mask(pair_dist: np.ndarray, lens: np.ndarray, K: int, threshold: float,
               norm_mode: int = NORM_MAXLEN) -> np.ndarray:
    """Stop mask evaluated in exact rational arithmetic (diagnostic for groups
    whose fp64 mean lies within rounding of the threshold)."""
    G, P = pair_dist.shape
    N = lens.shape[1]
    thr = Fraction(float(threshold))
    out = np.zeros(G, dtype=np.uint8)
    m = np.minimum(np.maximum(lens, 0), K)
    for g in range(G):
        s = Fraction(0)
        p = 0
        for i in range(N):
            for j in range(i + 1, N):
                d = int(pair_dist[g, p])
                if norm_mode == NORM_NONE:
                    s += d
                else:
                    longer = int(max(m[g, i], m[g, j]))
                    if longer > 0:
                        s += Fraction(d, longer)
                p += 1
        out[g] = 1 if s / P < thr else 0
    return out
