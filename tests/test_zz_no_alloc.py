"""sr_gate_noalloc: the gate for callers that are not allowed to allocate device
memory (a rollout worker living inside an inference engine or trainer that has
already claimed the GPU's memory).  Its scratch is a fixed array inside the
library, so this file checks that it (a) refuses problems that do not fit, on the
host, and (b) gives exactly sr_gate's results, call after call, although every call
reuses the same array with the previous call's leftovers in it.

Collected last on purpose: a run that stops at the first failure has then already
run every other test."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle

import paper_2605_05802_b200 as sr
from paper_2605_05802_b200 import binding, build, workloads as W


def test_noalloc_refuses_what_does_not_fit_before_touching_the_gpu():
    build.build()
    lib = binding.load()
    limit = lib.sr_gate_noalloc_limit_bytes()
    assert limit == 16 << 20
    fake = 1 << 20                       # never dereferenced: the call is refused on the host
    assert lib.sr_gate_workspace_bytes(1024, 8, 1024, 1024) > limit
    rc = lib.sr_gate_noalloc(fake, None, 1024, 8, 1024, 1024, 0.12, 0, None, None, None, fake, None, None)
    assert rc == binding.SR_ERR_SCRATCH_LIMIT
    assert b"scratch" in lib.sr_strerror(rc)
    assert lib.sr_gate_noalloc(fake, None, 4, 1, 64, 64, 0.12, 0, None, None, None, fake, None, None) == binding.SR_ERR_BAD_N
    assert lib.sr_gate_noalloc(fake, None, 4, 8, 64, 65, 0.12, 0, None, None, None, fake, None, None) == binding.SR_ERR_BAD_K
    # an invalid call reports its own error even when the problem would not fit either
    assert lib.sr_gate_noalloc(fake, None, 1024, 8, 1024, 1024, 0.12, 7, None, None, None, fake, None, None) == binding.SR_ERR_BAD_MODE
    assert lib.sr_gate_noalloc(None, None, 1024, 8, 1024, 1024, 0.12, 0, None, None, None, fake, None, None) == binding.SR_ERR_NULL
    assert lib.sr_gate_noalloc(fake + 4, None, 1024, 8, 1024, 1024, 0.12, 0, None, None, None, fake, None, None) == binding.SR_ERR_ALIGN


def _run(fn, w, thr, **extra):
    dev = torch.device("cuda:0")
    G, N, stride = w.seqs.shape
    P = N * (N - 1) // 2
    seqs = torch.from_numpy(w.seqs).to(dev)
    lens = torch.from_numpy(w.lens).to(dev)
    pd = torch.full((G, P), -1, dtype=torch.int32, device=dev)
    ps = torch.full((G,), -1, dtype=torch.int32, device=dev)
    mean = torch.full((G,), -1.0, dtype=torch.float64, device=dev)
    stop = torch.full((G,), 7, dtype=torch.uint8, device=dev)
    fn(seqs, lens, w.K, thr, w.norm_mode, pair_dist=pd, pair_sum=ps, mean=mean, stop=stop, **extra)
    torch.cuda.synchronize()
    return [t.cpu().numpy() for t in (pd, ps, mean, stop)]


@pytest.mark.gpu
def test_noalloc_matches_sr_gate_on_consecutive_calls():
    dev = torch.device("cuda:0")
    # two different multi-word problems back to back, then the first again: the shared
    # array still holds the other problem's match streams and counters each time
    big = W.token_gate(seed=11, n_groups=48, min_len=200, max_len=1024)
    small = W.token_gate(seed=12, n_groups=9, min_len=33, max_len=150, N=5)
    assert sr.sr_gate_workspace_bytes(48, 8, 1024, 1024) <= sr.sr_gate_noalloc_limit_bytes()
    for w in (big, small, big, big):
        G, N, stride = w.seqs.shape
        ws = torch.empty(sr.sr_gate_workspace_bytes(G, N, stride, w.K), dtype=torch.uint8, device=dev)
        want = _run(sr.sr_gate, w, 0.5, workspace=ws)
        got = _run(sr.sr_gate_noalloc, w, 0.5)
        for a, b in zip(got, want):                 # integers and the fp64 d_K bit for bit
            assert a.dtype == b.dtype and np.array_equal(a.view(np.uint8), b.view(np.uint8))
        for a, b in zip(got, oracle.gate(w.seqs, w.lens, w.K, 0.5, w.norm_mode)):   # and the definition itself
            assert np.array_equal(a.view(np.uint8), b.view(np.uint8))
        assert 0 < want[3].sum() < G
    # the single-word path needs no scratch and is served as well
    w1 = W.agent_gate(K=15)
    for a, b in zip(_run(sr.sr_gate_noalloc, w1, 0.5), _run(sr.sr_gate, w1, 0.5)):
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8))


_FIRST_CALL = """
import sys
sys.path.insert(0, {root!r})
import numpy as np, torch
import oracle
import paper_2605_05802_b200 as sr
from paper_2605_05802_b200 import workloads as W
w = W.token_gate(seed=21, n_groups=6, min_len=40, max_len=260, N=4)
dev = torch.device("cuda:0")
seqs, lens = torch.from_numpy(w.seqs).to(dev), torch.from_numpy(w.lens).to(dev)
G, N, stride = w.seqs.shape
pd = torch.empty((G, N * (N - 1) // 2), dtype=torch.int32, device=dev)
stop = torch.empty(G, dtype=torch.uint8, device=dev)
mean = torch.empty(G, dtype=torch.float64, device=dev)
# the very first library call of this process is the entry point under test
sr.sr_gate_noalloc(seqs, lens, w.K, 0.5, w.norm_mode, pair_dist=pd, mean=mean, stop=stop)
torch.cuda.synchronize()
opd, _, omean, ostop = oracle.gate(w.seqs, w.lens, w.K, 0.5, w.norm_mode)
assert np.array_equal(pd.cpu().numpy(), opd)
assert np.array_equal(mean.cpu().numpy().view(np.uint64), omean.view(np.uint64))
assert np.array_equal(stop.cpu().numpy(), ostop)
print("first-call ok")
"""


@pytest.mark.gpu
def test_first_call_of_a_fresh_process_sets_the_scratch_up():
    """The documented set-up happens inside the first call on a device: check it in a
    process that has made no other library call before."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", _FIRST_CALL.format(root=root)], capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0 and "first-call ok" in out.stdout, out.stdout + out.stderr
