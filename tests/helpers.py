"""Run the CUDA path through the binding on numpy inputs (GPU tests only)."""
import numpy as np
import torch

import paper_2605_05802_b200 as sr


def gate_gpu(seqs, lens, K, threshold, norm_mode=0, want_pair_dist=True, status=None):
    dev = torch.device("cuda:0")
    d_seqs = torch.from_numpy(np.ascontiguousarray(seqs, dtype=np.int32)).to(dev)
    d_lens = None if lens is None else torch.from_numpy(np.ascontiguousarray(lens, dtype=np.int32)).to(dev)
    G, N, stride = d_seqs.shape
    P = N * (N - 1) // 2
    pd = torch.full((G, P), -7, dtype=torch.int32, device=dev) if want_pair_dist else None
    ps = torch.full((G,), -7, dtype=torch.int32, device=dev)
    mean = torch.full((G,), -7.0, dtype=torch.float64, device=dev)
    stop = torch.full((G,), 9, dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    wsb = sr.sr_gate_workspace_bytes(G, N, stride, K)
    ws = torch.empty(max(wsb, 1), dtype=torch.uint8, device=dev) if wsb else None
    sr.sr_gate(d_seqs, d_lens, K, threshold, norm_mode, pair_dist=pd, pair_sum=ps, mean=mean,
               stop=stop, status=st, workspace=ws)
    torch.cuda.synchronize()
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
    adv = torch.full_like(r, 77.0)
    zv = torch.full((r.shape[0],), 9, dtype=torch.uint8, device=dev)
    sr.sr_grpo_advantage(r, d, eps, adv=adv, zero_var=zv)
    torch.cuda.synchronize()
    return adv.cpu().numpy(), zv.cpu().numpy()


class IncrementalGate:
    def __init__(self, G, N, max_steps=30):
        self.dev = torch.device("cuda:0")
        self.G, self.N, self.P = G, N, N * (N - 1) // 2
        nbytes = sr.sr_incr_state_bytes(G, N, max_steps)
        self.state = torch.empty(nbytes, dtype=torch.uint8, device=self.dev)
        sr.sr_incr_init(self.state, G, N, max_steps)
        self.pd = torch.empty((G, self.P), dtype=torch.int32, device=self.dev)
        self.ps = torch.empty((G,), dtype=torch.int32, device=self.dev)
        self.mean = torch.empty((G,), dtype=torch.float64, device=self.dev)
        self.stop = torch.empty((G,), dtype=torch.uint8, device=self.dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.dev)

    def step(self, actions, threshold, norm_mode=0):
        a = torch.from_numpy(np.ascontiguousarray(actions, dtype=np.int32)).to(self.dev)
        sr.sr_gate_step_incremental(self.state, a, threshold, norm_mode, pair_dist=self.pd,
                                    pair_sum=self.ps, mean=self.mean, stop=self.stop,
                                    status=self.status)
        torch.cuda.synchronize()
        return (self.pd.cpu().numpy(), self.ps.cpu().numpy(), self.mean.cpu().numpy(),
                self.stop.cpu().numpy())
