"""Thin ctypes binding of the sr_gate C ABI (include/sr_gate.h, include/sr_probe.h).

Argument marshalling only: every step of the path runs in the CUDA library.
PyTorch tensors are used as device (or pinned host) memory and for streams.  There
is no CPU fallback: if the shared library is missing or fails to load, every call
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsr_gate.so")

SR_OK = 0
SR_ERR_NULL, SR_ERR_BAD_N, SR_ERR_BAD_K, SR_ERR_ALIGN = -1, -2, -3, -4
SR_ERR_STATE_SIZE, SR_ERR_WORKSPACE, SR_ERR_CUDA, SR_ERR_BAD_MODE = -5, -6, -7, -8
SR_ERR_SCRATCH_LIMIT = -9
SR_ERR_BAD_OFFSETS = -10
SR_NORM_MAXLEN, SR_NORM_NONE = 0, 1
SR_NO_ACTION = -(2 ** 31)
SR_STATUS_NEG_LEN, SR_STATUS_STEP_OVERFLOW, SR_STATUS_BAD_STATE = 1, 2, 4
SR_MAX_N, SR_MAX_K, SR_MAX_INCR_STEPS = 32, 1024, 32
SR_PROBE_LOGIC, SR_PROBE_ADD, SR_PROBE_MIX = 0, 1, 2

_vp, _i32, _f64, _f32, _sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_double, ctypes.c_float, ctypes.c_size_t

_SIGNATURES = {
    "sr_version": (ctypes.c_int, []),
    "sr_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "sr_last_cuda_error": (ctypes.c_char_p, []),
    "sr_gate": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _f64, _i32, _vp, _vp, _vp, _vp, _vp,
                               _vp, _sz, _vp]),
    "sr_gate_noalloc": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _f64, _i32, _vp, _vp, _vp, _vp,
                                       _vp, _vp]),
    "sr_gate_noalloc_limit_bytes": (_sz, []),
    "sr_gate_decide": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _f64, _i32, _vp, _vp, _vp, _vp, _vp,
                                      _vp, _vp, _sz, _vp]),
    "sr_gate_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32]),
    "sr_gate_host": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _f64, _i32, _vp, _vp, _vp, _vp,
                                    _vp, _vp, _sz, _vp, _vp]),
    "sr_gate_host_arena_bytes": (_sz, [_i32, _i32, _i32, _i32]),
    "sr_gate_host_packed": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _f64, _i32, _vp, _vp, _vp, _vp,
                                           _vp, _vp, _sz, _vp, _vp]),
    "sr_gate_host_packed_arena_bytes": (_sz, [_i32, _i32, _i32, _i32]),
    "sr_incr_state_bytes": (_sz, [_i32, _i32, _i32]),
    "sr_incr_init": (ctypes.c_int, [_vp, _sz, _i32, _i32, _i32, _vp]),
    "sr_gate_step_incremental": (ctypes.c_int, [_vp, _sz, _vp, _i32, _i32, _f64, _i32, _vp, _vp, _vp,
                                                _vp, _vp, _vp]),
    "sr_gate_or_rule": (ctypes.c_int, [_vp, _vp, _vp, _i32, _i32, _i32, _f64, _f64, _vp, _vp, _vp]),
    "sr_group_signals": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "sr_batch_stats": (ctypes.c_int, [_vp, _vp, _i32, _i32, _vp, _vp, _vp]),
    "sr_kept_groups": (ctypes.c_int, [_vp, _vp, _i32, _vp, _vp, _vp, _sz, _vp]),
    "sr_kept_groups_workspace_bytes": (_sz, [_i32]),
    "sr_savings_fraction": (ctypes.c_double, [ctypes.c_int64, ctypes.c_int64, _i32, _i32]),
    "sr_dilution_gain": (ctypes.c_double, [_f64, _f64]),
    "sr_grpo_advantage": (ctypes.c_int, [_vp, _vp, _i32, _i32, _f32, _vp, _vp, _vp]),
    "sr_gate_stages": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _f64, _i32, _vp, _vp, _vp, _vp,
                                      _vp, _vp, _sz, _vp, _vp]),
    "sr_probe_int32": (ctypes.c_int, [_i32, _i32, _i32, _i32, _vp, _vp]),
    "sr_probe_int32_ops": (ctypes.c_uint64, [_i32, _i32, _i32]),
}

_lib = None


class SrError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(what)


def load() -> ctypes.CDLL:
    """Load libsr_gate.so (built in-tree by ``python -m paper_2605_05802_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise SrError(SR_ERR_CUDA, f"{LIB_PATH} is missing: build it with "
                                       "`python -m paper_2605_05802_b200.build`; there is no fallback path")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _check(rc: int) -> None:
    if rc != SR_OK:
        lib = load()
        msg = lib.sr_strerror(rc).decode()
        if rc == SR_ERR_CUDA:
            msg += ": " + lib.sr_last_cuda_error().decode()
        raise SrError(rc, f"sr_gate error {rc}: {msg}")


def _ptr(t: Optional[torch.Tensor], dtype: Optional[torch.dtype] = None, *, need: Optional[int] = None,
         host: bool = False, name: str = "tensor") -> Optional[int]:
    """Address of a caller-owned buffer.  The library dereferences it on the device (on the
    host for ``host=True``), so a tensor that lives on the wrong side, has another element
    type, is not contiguous or holds fewer than ``need`` elements is refused here instead of
    faulting there."""
    if t is None:
        return None
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if t.is_cuda == host:
        raise ValueError(f"{name} must be a {'host' if host else 'CUDA'} tensor")
    if need is not None and t.numel() < need:
        raise ValueError(f"{name} holds {t.numel()} elements, the call writes or reads {need}")
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def sr_version() -> int:
    return int(load().sr_version())


def sr_strerror(code: int) -> str:
    return load().sr_strerror(code).decode()


def sr_gate_workspace_bytes(n_groups: int, N: int, stride: int, K: int) -> int:
    return int(load().sr_gate_workspace_bytes(n_groups, N, stride, K))


def sr_gate(seqs: torch.Tensor, lens: Optional[torch.Tensor], K: int, threshold: float,
            norm_mode: int = SR_NORM_MAXLEN, *, pair_dist: Optional[torch.Tensor] = None,
            pair_sum: Optional[torch.Tensor] = None, mean: Optional[torch.Tensor] = None,
            stop: torch.Tensor = None, status: Optional[torch.Tensor] = None,
            workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    """seqs int32 [G, N, stride] on the device; outputs are preallocated tensors."""
    G, N, stride = seqs.shape
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().sr_gate(_ptr(seqs, torch.int32), _ptr(lens, torch.int32, need=G * N, name="lens"), G, N, stride, K,
                          float(threshold), norm_mode, _ptr(pair_dist, torch.int32, need=G * (N * (N - 1) // 2), name="pair_dist"),
                          _ptr(pair_sum, torch.int32, need=G, name="pair_sum"), _ptr(mean, torch.float64, need=G, name="mean"),
                          _ptr(stop, torch.uint8, need=G, name="stop"), _ptr(status, torch.int32, need=1, name="status"), _ptr(workspace),
                          ws_bytes, _stream(stream)))


def sr_gate_noalloc_limit_bytes() -> int:
    return int(load().sr_gate_noalloc_limit_bytes())


def sr_gate_noalloc(seqs: torch.Tensor, lens: Optional[torch.Tensor], K: int, threshold: float,
                    norm_mode: int = SR_NORM_MAXLEN, *, pair_dist=None, pair_sum=None, mean=None,
                    stop=None, status=None, stream=None) -> None:
    """sr_gate without a workspace argument, for code that may not allocate on the
    device (it runs inside a process whose GPU memory is already spoken for).  The
    scratch is a fixed array inside the library; problems whose scratch need exceeds
    sr_gate_noalloc_limit_bytes() are refused with SR_ERR_SCRATCH_LIMIT.  Calls that
    may overlap on the device must be serialised by the caller."""
    G, N, stride = seqs.shape
    _check(load().sr_gate_noalloc(_ptr(seqs, torch.int32), _ptr(lens, torch.int32, need=G * N, name="lens"), G, N, stride, K,
                                  float(threshold), norm_mode, _ptr(pair_dist, torch.int32, need=G * (N * (N - 1) // 2), name="pair_dist"),
                                  _ptr(pair_sum, torch.int32, need=G, name="pair_sum"), _ptr(mean, torch.float64, need=G, name="mean"),
                                  _ptr(stop, torch.uint8, need=G, name="stop"), _ptr(status, torch.int32, need=1, name="status"),
                                  _stream(stream)))


def sr_gate_decide(seqs: torch.Tensor, lens: Optional[torch.Tensor], K: int, threshold: float,
                   norm_mode: int = SR_NORM_MAXLEN, *, pair_dist=None, pair_sum=None, mean=None,
                   stop=None, exact=None, status=None, workspace=None, stream=None) -> None:
    """Same stop mask as sr_gate; groups that a lower bound of d_K already dismisses are
    not computed (exact[g] = 0 marks them, their other outputs are lower bounds)."""
    G, N, stride = seqs.shape
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().sr_gate_decide(_ptr(seqs, torch.int32), _ptr(lens, torch.int32, need=G * N, name="lens"), G, N, stride, K,
                                 float(threshold), norm_mode, _ptr(pair_dist, torch.int32, need=G * (N * (N - 1) // 2), name="pair_dist"),
                                 _ptr(pair_sum, torch.int32, need=G, name="pair_sum"), _ptr(mean, torch.float64, need=G, name="mean"),
                                 _ptr(stop, torch.uint8, need=G, name="stop"), _ptr(exact, torch.uint8, need=G, name="exact"),
                                 _ptr(status, torch.int32, need=1, name="status"), _ptr(workspace), ws_bytes, _stream(stream)))


def sr_gate_stages(seqs, lens, K, threshold, norm_mode=SR_NORM_MAXLEN, *, pair_dist=None, pair_sum=None,
                   mean=None, stop=None, status=None, workspace=None, stream=None, events=None) -> None:
    """sr_gate that also records five torch.cuda.Event (created with
    enable_timing=True and recorded once beforehand) at the pipeline's stage boundaries."""
    G, N, stride = seqs.shape
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    handles = (ctypes.c_void_p * 5)(*[e.cuda_event for e in events])
    _check(load().sr_gate_stages(_ptr(seqs, torch.int32), _ptr(lens, torch.int32, need=G * N, name="lens"), G, N, stride, K,
                                 float(threshold), norm_mode, _ptr(pair_dist, torch.int32, need=G * (N * (N - 1) // 2), name="pair_dist"),
                                 _ptr(pair_sum, torch.int32, need=G, name="pair_sum"), _ptr(mean, torch.float64, need=G, name="mean"),
                                 _ptr(stop, torch.uint8, need=G, name="stop"), _ptr(status, torch.int32, need=1, name="status"), _ptr(workspace),
                                 ws_bytes, _stream(stream), handles))


def sr_gate_host_arena_bytes(n_groups: int, N: int, stride: int, K: int) -> int:
    return int(load().sr_gate_host_arena_bytes(n_groups, N, stride, K))


def sr_gate_host(seqs: torch.Tensor, lens: Optional[torch.Tensor], K: int, threshold: float,
                 norm_mode: int = SR_NORM_MAXLEN, *, pair_dist=None, pair_sum=None, mean=None,
                 stop=None, status=None, arena: torch.Tensor = None, stream=None,
                 copy_stream: Optional[torch.cuda.Stream] = None) -> None:
    """Same as sr_gate with HOST tensors (ideally pinned) for inputs and outputs and
    a device ``arena``; the caller synchronises the stream before reading outputs."""
    for t in (seqs, lens, pair_dist, pair_sum, mean, stop, status):
        if t is not None and t.is_cuda:
            raise ValueError("sr_gate_host takes host tensors")
    G, N, stride = seqs.shape
    _check(load().sr_gate_host(_ptr(seqs, torch.int32, host=True, name="seqs"), _ptr(lens, torch.int32, need=G * N, host=True, name="lens"), G, N, stride, K,
                               float(threshold), norm_mode, _ptr(pair_dist, torch.int32, need=G * (N * (N - 1) // 2), host=True, name="pair_dist"),
                               _ptr(pair_sum, torch.int32, need=G, host=True, name="pair_sum"), _ptr(mean, torch.float64, need=G, host=True, name="mean"),
                               _ptr(stop, torch.uint8, need=G, host=True, name="stop"), _ptr(status, torch.int32, need=1, host=True, name="status"), _ptr(arena),
                               arena.numel() * arena.element_size(), _stream(stream),
                               None if copy_stream is None else copy_stream.cuda_stream))


def sr_gate_host_packed_arena_bytes(n_groups: int, N: int, stride: int, K: int) -> int:
    return int(load().sr_gate_host_packed_arena_bytes(n_groups, N, stride, K))


def sr_gate_host_packed(symbols: torch.Tensor, row_start: torch.Tensor, N: int, stride: int, K: int,
                        threshold: float, norm_mode: int = SR_NORM_MAXLEN, *, pair_dist=None,
                        pair_sum=None, mean=None, stop=None, status=None, arena: torch.Tensor = None,
                        stream=None, copy_stream: Optional[torch.cuda.Stream] = None) -> None:
    """sr_gate_host on packed HOST input: ``symbols`` (int32) holds the prefixes of all rows
    back to back, ``row_start`` (int64, rows + 1 entries, first 0) where each begins."""
    for t in (symbols, row_start, pair_dist, pair_sum, mean, stop, status):
        if t is not None and t.is_cuda:
            raise ValueError("sr_gate_host_packed takes host tensors")
    rows = row_start.numel() - 1
    if rows < 0 or rows % N:
        raise ValueError("row_start needs n_groups * N + 1 entries")
    G = rows // N
    _check(load().sr_gate_host_packed(_ptr(symbols, torch.int32, host=True, name="symbols"), _ptr(row_start, torch.int64, host=True, name="row_start"),
                                      rows // N, N, stride, K, float(threshold), norm_mode,
                                      _ptr(pair_dist, torch.int32, need=G * (N * (N - 1) // 2), host=True, name="pair_dist"), _ptr(pair_sum, torch.int32, need=G, host=True, name="pair_sum"),
                                      _ptr(mean, torch.float64, need=G, host=True, name="mean"), _ptr(stop, torch.uint8, need=G, host=True, name="stop"),
                                      _ptr(status, torch.int32, need=1, host=True, name="status"), _ptr(arena),
                                      arena.numel() * arena.element_size(), _stream(stream),
                                      None if copy_stream is None else copy_stream.cuda_stream))


def sr_incr_state_bytes(n_groups: int, N: int, max_steps: int) -> int:
    return int(load().sr_incr_state_bytes(n_groups, N, max_steps))


def sr_incr_init(state: torch.Tensor, n_groups: int, N: int, max_steps: int, stream=None) -> None:
    _check(load().sr_incr_init(_ptr(state), state.numel() * state.element_size(), n_groups, N,
                               max_steps, _stream(stream)))


def sr_gate_step_incremental(state: torch.Tensor, new_actions: torch.Tensor, threshold: float,
                             norm_mode: int = SR_NORM_MAXLEN, *, pair_dist=None, pair_sum=None,
                             mean=None, stop=None, status=None, stream=None) -> None:
    G, N = new_actions.shape
    _check(load().sr_gate_step_incremental(
        _ptr(state), state.numel() * state.element_size(), _ptr(new_actions, torch.int32, name="new_actions"), G, N,
        float(threshold), norm_mode, _ptr(pair_dist, torch.int32, need=G * (N * (N - 1) // 2), name="pair_dist"), _ptr(pair_sum, torch.int32, need=G, name="pair_sum"),
        _ptr(mean, torch.float64, need=G, name="mean"), _ptr(stop, torch.uint8, need=G, name="stop"), _ptr(status, torch.int32, need=1, name="status"),
        _stream(stream)))


def sr_gate_or_rule(mean: torch.Tensor, lens: Optional[torch.Tensor], done: Optional[torch.Tensor],
                    N: int, K: int, threshold: float, tau_high: float, *, tau: Optional[torch.Tensor] = None,
                    stop: torch.Tensor = None, stream=None) -> None:
    G = mean.shape[0]
    _check(load().sr_gate_or_rule(_ptr(mean, torch.float64), _ptr(lens, torch.int32, need=G * N, name="lens"),
                                  _ptr(done, torch.uint8, need=G * N, name="done"), mean.shape[0], N, K, float(threshold),
                                  float(tau_high), _ptr(tau, torch.float64, need=G, name="tau"), _ptr(stop, torch.uint8, need=G, name="stop"),
                                  _stream(stream)))


def sr_group_signals(seqs: torch.Tensor, lens: Optional[torch.Tensor], K: int, *,
                     unique_prefix_ratio=None, unique_action_ratio=None, action_entropy=None,
                     bigram_jaccard_mean=None, stream=None) -> None:
    G, N, stride = seqs.shape
    _check(load().sr_group_signals(_ptr(seqs, torch.int32), _ptr(lens, torch.int32, need=G * N, name="lens"), G, N, stride, K,
                                   _ptr(unique_prefix_ratio, torch.float64, need=G, name="unique_prefix_ratio"),
                                   _ptr(unique_action_ratio, torch.float64, need=G, name="unique_action_ratio"),
                                   _ptr(action_entropy, torch.float64, need=G, name="action_entropy"),
                                   _ptr(bigram_jaccard_mean, torch.float64, need=G, name="bigram_jaccard_mean"), _stream(stream)))


def sr_batch_stats(adv: torch.Tensor, stop: Optional[torch.Tensor], *, counts: torch.Tensor,
                   sumsq: torch.Tensor, stream=None) -> None:
    """counts: int64 [3] device tensor, sumsq: float64 [2] device tensor (see sr_gate.h)."""
    G, N = adv.shape
    _check(load().sr_batch_stats(_ptr(adv, torch.float32), _ptr(stop, torch.uint8, need=G, name="stop"), G, N,
                                 _ptr(counts, torch.int64, need=3, name="counts"), _ptr(sumsq, torch.float64, need=2, name="sumsq"), _stream(stream)))


def sr_kept_groups_workspace_bytes(n_groups: int) -> int:
    return int(load().sr_kept_groups_workspace_bytes(n_groups))


def sr_kept_groups(stop: Optional[torch.Tensor], zero_var: Optional[torch.Tensor], *, index: torch.Tensor,
                   count: torch.Tensor, workspace: Optional[torch.Tensor], n_groups: Optional[int] = None,
                   stream=None) -> None:
    """index int32 [n_groups], count int32 [1] (device): ascending indices of the groups
    with stop == 0 (and zero_var == 0 when given)."""
    if n_groups is None:
        n_groups = (stop if stop is not None else zero_var if zero_var is not None else index).shape[0]
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().sr_kept_groups(_ptr(stop, torch.uint8, need=n_groups, name="stop"), _ptr(zero_var, torch.uint8, need=n_groups, name="zero_var"), n_groups,
                                 _ptr(index, torch.int32, need=n_groups, name="index"), _ptr(count, torch.int32, need=1, name="count"), _ptr(workspace),
                                 ws_bytes, _stream(stream)))


def sr_savings_fraction(cut: int, n_groups: int, T_max: int, K: int) -> float:
    return float(load().sr_savings_fraction(cut, n_groups, T_max, K))


def sr_dilution_gain(before: float, after: float) -> float:
    return float(load().sr_dilution_gain(before, after))


def sr_grpo_advantage(rewards: torch.Tensor, drop_mask: Optional[torch.Tensor], eps: float, *,
                      adv: torch.Tensor, zero_var: Optional[torch.Tensor] = None, stream=None) -> None:
    G, N = rewards.shape
    _check(load().sr_grpo_advantage(_ptr(rewards, torch.float32), _ptr(drop_mask, torch.uint8, need=G, name="drop_mask"), G, N,
                                    float(eps), _ptr(adv, torch.float32, need=G * N, name="adv"), _ptr(zero_var, torch.uint8, need=G, name="zero_var"),
                                    _stream(stream)))


def sr_probe_int32(variant: int, iters: int, blocks: int, threads: int, sink: torch.Tensor,
                   stream=None) -> None:
    _check(load().sr_probe_int32(variant, iters, blocks, threads, _ptr(sink), _stream(stream)))


def sr_probe_int32_ops(iters: int, blocks: int, threads: int) -> int:
    return int(load().sr_probe_int32_ops(iters, blocks, threads))


def shard_groups(n_groups: int, world_size: int, rank: int):
    """Contiguous range of groups owned by ``rank``: groups are independent (each
    rollout worker applies the gate to its own groups, Appendix C.1), so sharding
    needs no exchange."""
    base, extra = divmod(n_groups, world_size)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)
