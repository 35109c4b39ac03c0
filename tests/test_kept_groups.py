"""Kept-group index list: the groups the trainer still sees after the gate (Appendix C.1)
and, optionally, after the zero-variance filter (Section 2.1, dynamic-sampling baseline)."""
import numpy as np
import pytest

import oracle


def _flags(rng, n, p):
    f = (rng.random(n) < p).astype(np.uint8)
    # any non-zero byte means "set"
    f[f == 1] = rng.integers(1, 256, size=int(f.sum()), dtype=np.uint8)
    return f


# ------------------------------------------------------------------ oracle pins (CPU)
def test_oracle_against_flatnonzero():
    rng = np.random.default_rng(11)
    for n in (0, 1, 5, 4097, 70001):
        stop = _flags(rng, n, 0.3)
        zv = _flags(rng, n, 0.4)
        assert np.array_equal(oracle.kept_groups(stop, None, n), np.flatnonzero(stop == 0))
        assert np.array_equal(oracle.kept_groups(None, zv, n), np.flatnonzero(zv == 0))
        assert np.array_equal(oracle.kept_groups(stop, zv, n), np.flatnonzero((stop == 0) & (zv == 0)))


def test_oracle_closed_forms():
    n = 1000
    zeros, ones = np.zeros(n, np.uint8), np.ones(n, np.uint8)
    assert np.array_equal(oracle.kept_groups(zeros), np.arange(n))            # nothing cut: identity
    assert oracle.kept_groups(ones).size == 0                                 # everything cut
    assert np.array_equal(oracle.kept_groups(None, None, n), np.arange(n))
    alt = (np.arange(n) % 2).astype(np.uint8)
    assert np.array_equal(oracle.kept_groups(alt), np.arange(0, n, 2))
    kept = oracle.kept_groups(alt, 1 - alt)                                   # the filters are AND-ed
    assert kept.size == 0
    # ascending and without repeats, whatever the flags
    rng = np.random.default_rng(5)
    k = oracle.kept_groups(_flags(rng, 5000, 0.5), _flags(rng, 5000, 0.5))
    assert np.all(np.diff(k) > 0)


def test_oracle_matches_the_gate_and_advantage_flags():
    """Feeding the oracle's own stop mask and zero-variance flags: the kept list is exactly
    the set of groups whose advantages are not all forced to zero."""
    from paper_2605_05802_b200 import workloads as W
    w = W.agent_gate(K=15)
    _, _, _, stop = oracle.gate(w.seqs, w.lens, w.K, w.threshold)
    adv, zv = oracle.advantage(w.rewards, stop)
    kept = oracle.kept_groups(stop, zv)
    nonzero = np.flatnonzero(np.any(adv != 0.0, axis=1))
    assert np.array_equal(kept, nonzero)


# ------------------------------------------------------------------------ GPU parity
def _run_gpu(stop, zv, n, offset=0):
    import torch
    import paper_2605_05802_b200 as sr
    dev = torch.device("cuda:0")

    def put(a):
        if a is None:
            return None
        buf = torch.zeros(n + offset + 16, dtype=torch.uint8, device=dev)
        buf[offset:offset + n] = torch.from_numpy(a).to(dev)
        return buf[offset:offset + n]

    d_stop, d_zv = put(stop), put(zv)
    index = torch.full((max(n, 1) + 64,), -7, dtype=torch.int32, device=dev)
    count = torch.full((1,), -7, dtype=torch.int32, device=dev)
    ws = torch.empty(sr.sr_kept_groups_workspace_bytes(n), dtype=torch.uint8, device=dev)
    sr.sr_kept_groups(d_stop, d_zv, index=index, count=count, workspace=ws, n_groups=n)
    torch.cuda.synchronize()
    c = int(count.item())
    out = index.cpu().numpy()
    assert np.all(out[c:] == -7), "wrote past the end of the list"
    return out[:c]


@pytest.mark.gpu
@pytest.mark.parametrize("n", [0, 1, 15, 16, 17, 777, 4096, 4097, 65536, 4194304 + 5])
def test_gpu_matches_oracle(n):
    rng = np.random.default_rng(n + 1)
    stop, zv = _flags(rng, n, 0.2), _flags(rng, n, 0.4)
    for s, z in ((stop, None), (None, zv), (stop, zv), (None, None)):
        assert np.array_equal(_run_gpu(s, z, n), oracle.kept_groups(s, z, n))


@pytest.mark.gpu
def test_gpu_unaligned_flags_and_extremes():
    rng = np.random.default_rng(3)
    n = 10007
    stop, zv = _flags(rng, n, 0.5), _flags(rng, n, 0.5)
    for off in (1, 3, 8):
        assert np.array_equal(_run_gpu(stop, zv, n, offset=off), oracle.kept_groups(stop, zv))
    assert _run_gpu(np.ones(n, np.uint8), None, n).size == 0
    assert np.array_equal(_run_gpu(np.zeros(n, np.uint8), None, n), np.arange(n))


def test_boundary_errors():
    import paper_2605_05802_b200 as sr
    lib = sr.load()
    assert lib.sr_kept_groups(None, None, -1, None, None, None, 0, None) == sr.SR_ERR_BAD_N
    assert lib.sr_kept_groups(None, None, 4, None, None, None, 0, None) == sr.SR_ERR_NULL
    assert lib.sr_kept_groups(None, None, 4, 256, 256, None, 0, None) == sr.SR_ERR_WORKSPACE
    assert lib.sr_kept_groups(None, None, 4, 256, 256, 256, 8, None) == sr.SR_ERR_WORKSPACE
    assert sr.sr_kept_groups_workspace_bytes(-1) == 0
    assert sr.sr_kept_groups_workspace_bytes(1) >= 4
    assert sr.sr_kept_groups_workspace_bytes(4096 * 100 + 1) >= 101 * 4
