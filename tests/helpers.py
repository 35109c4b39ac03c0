"""Run the CUDA path through the binding on numpy inputs (GPU tests only)."""
import numpy as np
import torch

import paper_2605_05802_b200 as sr

GUARD = 256          # bytes of canary on either side of every buffer a kernel writes
CANARY = 0xA5


class Guarded:
    """Device buffers with canary bytes before and after them.  compute-sanitizer is not
    available on the test machines, so every output, workspace and state buffer the GPU
    tests hand to the library sits between two 256-byte guard regions that must still
    hold the canary after the call: a write past either end of a buffer fails the test."""

    def __init__(self, dev):
        self.dev = dev
        self.bufs = []

    def alloc(self, shape, dtype, fill=None):
        shape = tuple(int(x) for x in (shape if isinstance(shape, (tuple, list)) else (shape,)))
        nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        padded = (nbytes + 255) // 256 * 256
        raw = torch.full((GUARD + padded + GUARD,), CANARY, dtype=torch.uint8, device=self.dev)
        view = raw[GUARD:GUARD + nbytes].view(dtype).reshape(shape)
        if fill is not None:
            view.fill_(fill)
        self.bufs.append((raw, nbytes))
        return view

    def check(self, tag=""):
        torch.cuda.synchronize()
        for k, (raw, nbytes) in enumerate(self.bufs):
            head = raw[:GUARD]
            tail = raw[GUARD + nbytes:]
            assert bool((head == CANARY).all()), f"{tag}: buffer {k}: write before its start"
            assert bool((tail == CANARY).all()), f"{tag}: buffer {k}: write past its end"


def gate_gpu(seqs, lens, K, threshold, norm_mode=0, want_pair_dist=True, status=None):
    dev = torch.device("cuda:0")
    d_seqs = torch.from_numpy(np.ascontiguousarray(seqs, dtype=np.int32)).to(dev)
    d_lens = None if lens is None else torch.from_numpy(np.ascontiguousarray(lens, dtype=np.int32)).to(dev)
    G, N, stride = d_seqs.shape
    P = N * (N - 1) // 2
    guard = Guarded(dev)
    pd = guard.alloc((G, P), torch.int32, -7) if want_pair_dist else None
    ps = guard.alloc((G,), torch.int32, -7)
    mean = guard.alloc((G,), torch.float64, -7.0)
    stop = guard.alloc((G,), torch.uint8, 9)
    st = guard.alloc((1,), torch.int32, 0)
    wsb = sr.sr_gate_workspace_bytes(G, N, stride, K)
    ws = guard.alloc((wsb,), torch.uint8) if wsb else None
    sr.sr_gate(d_seqs, d_lens, K, threshold, norm_mode, pair_dist=pd, pair_sum=ps, mean=mean,
               stop=stop, status=st, workspace=ws)
    guard.check(f"sr_gate G={G} N={N} K={K}")
    if status is not None:
        status.append(int(st.item()))
    return (None if pd is None else pd.cpu().numpy(), ps.cpu().numpy(), mean.cpu().numpy(),
            stop.cpu().numpy())


def assert_gate_matches(got, want, tag=""):
    pd, ps, mean, stop = got
    opd, ops, omean, ostop = want
    if pd is not None:
        assert np.array_equal(pd, opd), f"{tag}: pair distances differ at {np.argwhere(pd != opd)[:5]}"
    assert np.array_equal(ps, ops), f"{tag}: pair sums differ"
    assert np.array_equal(mean.view(np.uint64), omean.view(np.uint64)), f"{tag}: d_K not bit-identical"
    assert np.array_equal(stop, ostop), f"{tag}: stop masks differ"


def advantage_gpu(rewards, drop=None, eps=1e-6):
    dev = torch.device("cuda:0")
    r = torch.from_numpy(np.ascontiguousarray(rewards, dtype=np.float32)).to(dev)
    d = None if drop is None else torch.from_numpy(np.ascontiguousarray(drop, dtype=np.uint8)).to(dev)
    guard = Guarded(dev)
    adv = guard.alloc(tuple(r.shape), torch.float32, 77.0)
    zv = guard.alloc((r.shape[0],), torch.uint8, 9)
    sr.sr_grpo_advantage(r, d, eps, adv=adv, zero_var=zv)
    guard.check("sr_grpo_advantage")
    return adv.cpu().numpy(), zv.cpu().numpy()


class IncrementalGate:
    def __init__(self, G, N, max_steps=30):
        self.dev = torch.device("cuda:0")
        self.G, self.N, self.P = G, N, N * (N - 1) // 2
        nbytes = sr.sr_incr_state_bytes(G, N, max_steps)
        self.guard = Guarded(self.dev)
        self.state = self.guard.alloc((nbytes,), torch.uint8)
        sr.sr_incr_init(self.state, G, N, max_steps)
        self.pd = self.guard.alloc((G, self.P), torch.int32, -7)
        self.ps = self.guard.alloc((G,), torch.int32, -7)
        self.mean = self.guard.alloc((G,), torch.float64, -7.0)
        self.stop = self.guard.alloc((G,), torch.uint8, 9)
        self.status = self.guard.alloc((1,), torch.int32, 0)

    def step(self, actions, threshold, norm_mode=0):
        a = torch.from_numpy(np.ascontiguousarray(actions, dtype=np.int32)).to(self.dev)
        sr.sr_gate_step_incremental(self.state, a, threshold, norm_mode, pair_dist=self.pd,
                                    pair_sum=self.ps, mean=self.mean, stop=self.stop,
                                    status=self.status)
        self.guard.check("sr_gate_step_incremental")
        return (self.pd.cpu().numpy(), self.ps.cpu().numpy(), self.mean.cpu().numpy(),
                self.stop.cpu().numpy())
