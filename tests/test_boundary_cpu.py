"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the headers declare, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

import paper_2605_05802_b200 as sr
from paper_2605_05802_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        text = open(os.path.join(inc, f)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(sr_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert {"sr_gate", "sr_gate_step_incremental", "sr_grpo_advantage", "sr_incr_init",
            "sr_gate_host", "sr_probe_int32"} <= names
    for n in names:
        assert hasattr(lib, n), n
    assert names == set(binding._SIGNATURES), names ^ set(binding._SIGNATURES)
    assert lib.sr_version() == 100


def test_strerror_is_total(lib):
    codes = {v for k, v in vars(binding).items() if k.startswith("SR_ERR_")} | {binding.SR_OK}
    header = open(os.path.join(ROOT, "include", "sr_gate.h")).read()
    declared = {int(m) for m in re.findall(r"#define SR_ERR_[A-Z_]+ \((-\d+)\)", header)} | {0}
    assert codes == declared                      # the binding knows every code the header defines
    fallback = lib.sr_strerror(-99)
    assert b"unknown" in fallback
    for code in codes:
        text = lib.sr_strerror(code)
        assert text and text != fallback, code


def test_noalloc_limit_is_the_header_constant(lib):
    header = open(os.path.join(ROOT, "include", "sr_gate.h")).read()
    m = re.search(r"#define SR_NOALLOC_SCRATCH_BYTES \((\d+)u << (\d+)\)", header)
    assert m and lib.sr_gate_noalloc_limit_bytes() == int(m.group(1)) << int(m.group(2))


def test_gate_rejects_bad_arguments_before_any_launch(lib):
    fake = 1 << 20          # never dereferenced: every call below fails validation
    def gate(seqs=fake, lens=None, G=4, N=8, stride=32, K=10, thr=0.12, mode=0, stop=fake,
             ws=None, wsb=0):
        return lib.sr_gate(seqs, lens, G, N, stride, K, thr, mode, None, None, None, stop, None,
                           ws, wsb, None)
    assert gate(N=1) == binding.SR_ERR_BAD_N
    assert gate(N=33) == binding.SR_ERR_BAD_N
    assert gate(G=-1) == binding.SR_ERR_BAD_N
    assert gate(K=-1) == binding.SR_ERR_BAD_K
    assert gate(K=33) == binding.SR_ERR_BAD_K            # K > stride
    assert gate(stride=2048, K=1025) == binding.SR_ERR_BAD_K
    assert gate(mode=2) == binding.SR_ERR_BAD_MODE
    assert gate(seqs=None) == binding.SR_ERR_NULL
    assert gate(stop=None) == binding.SR_ERR_NULL
    assert gate(stride=30, K=10) == binding.SR_ERR_ALIGN
    assert gate(seqs=fake + 4) == binding.SR_ERR_ALIGN
    # multi-word path needs a workspace
    assert gate(stride=64, K=64) == binding.SR_ERR_WORKSPACE
    assert gate(stride=64, K=64, ws=fake, wsb=16) == binding.SR_ERR_WORKSPACE
    assert gate(stride=64, K=64, ws=fake + 8, wsb=1 << 30) == binding.SR_ERR_WORKSPACE
    dec = lib.sr_gate_decide
    assert dec(fake, None, 4, 8, 64, 64, 0.12, 0, None, None, None, fake, None, None, None, 0, None) == binding.SR_ERR_WORKSPACE
    assert dec(fake, None, 4, 1, 64, 64, 0.12, 0, None, None, None, fake, None, None, None, 0, None) == binding.SR_ERR_BAD_N
    assert dec(None, None, 0, 8, 64, 64, 0.12, 0, None, None, None, None, None, None, None, 0, None) == binding.SR_OK
    # an empty batch is a valid no-op on either path
    assert gate(G=0, seqs=None, stop=None) == binding.SR_OK
    assert gate(G=0, seqs=None, stop=None, stride=64, K=64) == binding.SR_OK


def test_workspace_and_state_sizes(lib):
    assert lib.sr_gate_workspace_bytes(1024, 8, 32, 30) == 0
    w = lib.sr_gate_workspace_bytes(1024, 8, 1024, 1024)
    assert w > 1024 * 28 * 1024 * 2 and w % 256 == 0
    assert lib.sr_gate_workspace_bytes(1024, 1, 1024, 1024) == 0
    assert lib.sr_gate_host_arena_bytes(16, 8, 32, 10) >= 16 * 8 * 32 * 4
    s = lib.sr_incr_state_bytes(65536, 8, 30)
    assert s >= 65536 * (8 * 4 + 8 * 32 * 4 + 28 * 16) and s % 256 == 0
    assert lib.sr_incr_state_bytes(10, 8, 33) == 0
    assert lib.sr_incr_state_bytes(10, 1, 30) == 0


def test_incremental_and_advantage_reject_bad_arguments(lib):
    fake = 1 << 20
    assert lib.sr_incr_init(None, 1 << 20, 4, 8, 30, None) == binding.SR_ERR_NULL
    assert lib.sr_incr_init(fake, 1 << 20, 4, 8, 0, None) == binding.SR_ERR_BAD_K
    assert lib.sr_incr_init(fake, 1 << 20, 4, 8, 33, None) == binding.SR_ERR_BAD_K
    assert lib.sr_incr_init(fake, 1 << 20, 4, 40, 30, None) == binding.SR_ERR_BAD_N
    assert lib.sr_incr_init(fake, 16, 4, 8, 30, None) == binding.SR_ERR_STATE_SIZE
    step = lib.sr_gate_step_incremental
    assert step(None, 1 << 20, fake, 4, 8, 0.12, 0, None, None, None, fake, None, None) == binding.SR_ERR_NULL
    assert step(fake, 1 << 20, None, 4, 8, 0.12, 0, None, None, None, fake, None, None) == binding.SR_ERR_NULL
    assert step(fake, 1 << 20, fake, 4, 8, 0.12, 7, None, None, None, fake, None, None) == binding.SR_ERR_BAD_MODE
    assert step(fake, 16, fake, 4, 8, 0.12, 0, None, None, None, fake, None, None) == binding.SR_ERR_STATE_SIZE
    orr = lib.sr_gate_or_rule
    assert orr(None, fake, None, 4, 8, 10, 0.12, 0.9, None, fake, None) == binding.SR_ERR_NULL
    assert orr(fake, None, None, 4, 8, 10, 0.12, 0.9, None, fake, None) == binding.SR_ERR_NULL
    assert orr(fake, fake, None, 4, 33, 10, 0.12, 0.9, None, fake, None) == binding.SR_ERR_BAD_N
    assert orr(None, None, None, 0, 8, 10, 0.12, 0.9, None, None, None) == binding.SR_OK
    gs = lib.sr_group_signals
    assert gs(None, None, 4, 8, 32, 10, fake, None, None, None, None) == binding.SR_ERR_NULL
    assert gs(fake, None, 4, 8, 64, 33, fake, None, None, None, None) == binding.SR_ERR_BAD_K
    assert gs(fake, None, 4, 1, 32, 10, fake, None, None, None, None) == binding.SR_ERR_BAD_N
    assert gs(fake + 4, None, 4, 8, 32, 10, fake, None, None, None, None) == binding.SR_ERR_ALIGN
    bs = lib.sr_batch_stats
    assert bs(fake, None, 4, 8, None, fake, None) == binding.SR_ERR_NULL
    assert bs(None, None, 4, 8, fake, fake, None) == binding.SR_ERR_NULL
    assert bs(fake, None, 4, 0, fake, fake, None) == binding.SR_ERR_BAD_N
    adv = lib.sr_grpo_advantage
    assert adv(None, None, 4, 8, 1e-6, fake, None, None) == binding.SR_ERR_NULL
    assert adv(fake, None, 4, 1, 1e-6, fake, None, None) == binding.SR_ERR_BAD_N
    assert adv(None, None, 0, 8, 1e-6, None, None, None) == binding.SR_OK
    assert lib.sr_probe_int32(0, 1, 1, 32, None, None) == binding.SR_ERR_NULL
    assert lib.sr_probe_int32_ops(10, 4, 128) == 10 * 16 * 8 * 4 * 128


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libsr_gate.so")
    with pytest.raises(binding.SrError):
        binding.sr_version()


def test_shard_groups_partitions_exactly():
    for G in (0, 1, 7, 512, 65536):
        for W in (1, 2, 3, 8):
            spans = [sr.shard_groups(G, W, r) for r in range(W)]
            assert spans[0][0] == 0 and spans[-1][1] == G
            for (a, b), (c, d) in zip(spans, spans[1:]):
                assert b == c
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1


def test_work_accounting_leaves_out_common_prefixes():
    """word_columns (the roofline's unit count) with and without the pairs' common prefixes."""
    import numpy as np
    from paper_2605_05802_b200 import workloads as W
    seqs = np.zeros((4, 2, 128), dtype=np.int32)
    seqs[:, 0, :] = np.arange(128)
    seqs[:, 1, :] = np.arange(128)
    seqs[0, 1, 0] = -1            # differ at once: nothing removed
    seqs[1, 1, 5] = -1            # common prefix 5 -> 4 symbols removed on both sides
    seqs[2, 1, 100] = -1          # common prefix 100 (a multiple of 4)
    lens = np.array([[128, 100], [128, 100], [128, 128], [128, 64]], dtype=np.int32)   # last: contained
    full = [min(100 * 4, 128 * 4), min(100 * 4, 128 * 4), 128 * 4, min(64 * 4, 128 * 2)]
    assert W.word_columns(lens, 128) == sum(full)
    cut = [full[0], min(96 * 4, 124 * 3), 28 * 1, 0]
    assert W.word_columns(lens, 128, seqs) == sum(cut)


def test_packed_host_entry_rejects_bad_offsets_before_any_launch(lib):
    import numpy as np
    sym = np.zeros(64, dtype=np.int32)
    stop = np.zeros(1, dtype=np.uint8)
    fn = lib.sr_gate_host_packed

    def call(row_start, stride=32, K=30, n_groups=1, N=2):
        rs = np.asarray(row_start, dtype=np.int64)
        return fn(sym.ctypes.data, rs.ctypes.data, n_groups, N, stride, K, 0.5, 0, None, None, None,
                  stop.ctypes.data, None, None, 0, None, None)

    assert call([1, 5, 9]) == binding.SR_ERR_BAD_OFFSETS          # does not begin at 0
    assert call([0, 9, 5]) == binding.SR_ERR_BAD_OFFSETS          # decreases
    assert call([0, 40, 65]) == binding.SR_ERR_BAD_OFFSETS        # more symbols than rows x stride
    assert call([0, 5, 9], stride=30) == binding.SR_ERR_BAD_K     # stride not a multiple of 4
    assert call([0, 5, 9], K=33) == binding.SR_ERR_BAD_K          # K > stride
    assert call([0, 5, 9]) == binding.SR_ERR_WORKSPACE            # well-formed, but no arena
    assert call([0], n_groups=0) == binding.SR_OK
    assert lib.sr_gate_host_packed_arena_bytes(4, 8, 64, 64) > lib.sr_gate_host_arena_bytes(4, 8, 64, 64)


def test_headers_are_plain_c_and_a_c_program_links(lib, tmp_path):
    """The boundary is a C ABI: both headers compile as C11 with warnings as errors, and a C
    program linked against the library reaches the entry points that need no GPU."""
    import shutil
    import subprocess
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        pytest.skip("no C compiler")
    src = tmp_path / "use_sr_gate.c"
    src.write_text(
        '#include <stdio.h>\n#include <string.h>\n#include "sr_gate.h"\n#include "sr_probe.h"\n'
        "int main(void) {\n"
        "    if (sr_version() != 100) return 1;\n"
        "    if (strlen(sr_strerror(SR_ERR_BAD_N)) == 0) return 2;\n"
        "    /* K <= 32 needs no workspace; the multi-word pipeline says how much it wants */\n"
        "    if (sr_gate_workspace_bytes(4, 8, 32, 30) != 0) return 3;\n"
        "    if (sr_gate_workspace_bytes(4, 8, 1024, 1024) == 0) return 4;\n"
        "    /* argument checks come before any CUDA call: N = 1 is refused on a machine without a GPU too */\n"
        "    if (sr_gate((const int32_t*)0, (const int32_t*)0, 1, 1, 4, 4, 0.12, SR_NORM_MAXLEN, 0, 0, 0,\n"
        "                (uint8_t*)0, 0, 0, 0, 0) >= 0) return 5;\n"
        '    printf("ok %d\\n", sr_version());\n'
        "    return 0;\n}\n")
    exe = tmp_path / "use_sr_gate"
    libdir = os.path.dirname(binding.LIB_PATH)
    subprocess.run([cc, "-std=c11", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                    str(src), "-o", str(exe), "-L", libdir, "-lsr_gate", f"-Wl,-rpath,{libdir}"],
                   check=True, capture_output=True, text=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True, timeout=120)
    assert out.stdout.strip() == "ok 100"


def test_binding_refuses_tensors_on_the_wrong_side(lib):
    """The device entry points dereference their pointers on the GPU: a host tensor handed to
    them (or a device-style call with the wrong element type) is refused by the binding."""
    import torch
    seqs = torch.zeros((2, 8, 16), dtype=torch.int32)
    stop = torch.zeros(2, dtype=torch.uint8)
    with pytest.raises(ValueError, match="CUDA tensor"):
        sr.sr_gate(seqs, None, 15, 0.12, stop=stop)
    with pytest.raises(TypeError, match="int32"):
        sr.sr_gate(seqs.to(torch.int64), None, 15, 0.12, stop=stop)
    with pytest.raises(ValueError, match="CUDA tensor"):
        sr.sr_grpo_advantage(torch.zeros((2, 8)), None, 1e-6, adv=torch.zeros((2, 8)))
    with pytest.raises(ValueError, match="contiguous"):
        sr.sr_gate(seqs.transpose(0, 1), None, 15, 0.12, stop=stop)
