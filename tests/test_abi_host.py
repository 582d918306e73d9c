"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
its host-only helpers agree with the oracle and the golden tables, and argument problems are
reported as status codes before anything touches a GPU."""
import ctypes
import os
import re

import pytest

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return sd.load_library()


def test_header_symbols_are_exported(lib):
    with open(os.path.join(ROOT, "include", "sparsed.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(sparsed_[a-z_]+)\s*\(", text))
    assert declared == set(binding.EXPORTED_SYMBOLS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_struct_layouts_match_header():
    assert ctypes.sizeof(binding.Shape) == 5 * 4 + 4 + 12 * 8 + 8   # ints, pad, strides, float + pad
    assert ctypes.sizeof(binding.SelectParams) == 24
    assert ctypes.sizeof(binding.Pattern) == 48


def test_schedule_helper_matches_golden_table_and_oracle(lib):
    with open(os.path.join(ROOT, "tests", "golden", "schedule_table.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    for T, skip, s, n_full, n_sparse in rows:
        T, skip, s = int(T), float(skip), int(s)
        assert sd.sparsed_switch_step(T, skip) == s
        modes = [sd.sparsed_schedule_mode(t, T, skip) for t in range(1, T + 1)]
        assert modes == [orc.schedule_mode(t, T, skip) for t in range(1, T + 1)]
        assert modes.count(sd.MODE_SPARSE) == int(n_sparse)
    assert sd.sparsed_schedule_mode(0, 10, 0.2) == -1
    assert sd.sparsed_schedule_mode(11, 10, 0.2) == -1
    assert sd.sparsed_switch_step(0, 0.2) == -1 and sd.sparsed_switch_step(10, 1.5) == -1


def test_kept_per_row_matches_golden_table():
    with open(os.path.join(ROOT, "tests", "golden", "kept_blocks_table.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    for n, rho, kept in rows:
        n, rho, kept = int(n), float(rho), int(kept)
        assert sd.sparsed_kept_per_row(sd.make_params(128, rho, 0), n * 128) == (0, kept)
        assert sd.sparsed_kept_per_row(sd.make_params(64, rho, n * 64), n * 64) == (kept, 0)
    assert sd.sparsed_kept_per_row(sd.make_params(128, 0.2, 4096), 8192) == (7, 7)
    assert sd.sparsed_kept_per_row(sd.make_params(128, 0.1, 16384), 32768) == (13, 13)
    assert sd.sparsed_kept_per_row(sd.make_params(128, 0.35, 0, rounding=1), 1280) == (0, 3)
    assert sd.sparsed_kept_per_row(sd.make_params(32, 0.5, 352), 1024) == (6, 11)   # the short-context setting


def test_argument_errors_are_status_codes(lib):
    with pytest.raises(sd.SparsedError) as e:
        sd.sparsed_kept_per_row(sd.make_params(16, 0.3, 0), 1024)
    assert e.value.status == 2                       # block size 16 unsupported
    with pytest.raises(sd.SparsedError) as e:
        sd.sparsed_kept_per_row(sd.make_params(128, 0.3, 0), 1000)
    assert e.value.status == 3                       # seq_len not a multiple of block_size
    with pytest.raises(sd.SparsedError) as e:
        sd.sparsed_kept_per_row(sd.make_params(128, 0.3, 100), 1024)
    assert e.value.status == 3                       # prefill_len not a multiple of block_size
    with pytest.raises(sd.SparsedError) as e:
        sd.sparsed_kept_per_row(sd.make_params(128, 0.0, 0), 1024)
    assert e.value.status == 1
    shape = binding.Shape(1, 3, 2, 1024, 128)        # heads_q % heads_kv != 0
    assert lib.sparsed_attn_full(ctypes.byref(shape), 16, 16, 16, 16, None, 16, 256, None) == 1
    shape = binding.Shape(1, 2, 2, 1024, 64)         # head_dim 64
    assert lib.sparsed_attn_full(ctypes.byref(shape), 16, 16, 16, 16, None, 16, 256, None) == 2
    shape = binding.Shape(1, 2, 2, 1024, 128)
    assert lib.sparsed_attn_full(ctypes.byref(shape), None, 16, 16, 16, None, 16, 256, None) == 1
    assert lib.sparsed_attn_full(ctypes.byref(shape), 8, 16, 16, 16, None, 16, 256, None) == 3   # misaligned q
    assert lib.sparsed_attn_full(ctypes.byref(shape), 16, 16, 16, 16, None, 16, 8, None) == 4    # workspace
    shape.q_strides[2] = 132                          # token stride not a multiple of 8
    shape.q_strides[1] = 132 * 1024; shape.q_strides[0] = 132 * 2048
    assert lib.sparsed_attn_full(ctypes.byref(shape), 16, 16, 16, 16, None, 16, 256, None) == 3
    assert sd.sparsed_workspace_bytes(sd.OP_ATTN_FULL) == 256
    n = sd.sparsed_workspace_bytes(sd.OP_SELECT_PATTERN, binding.Shape(1, 2, 2, 1024, 128), sd.make_params(64, 0.3))
    assert n >= 256 + 2 * 16 * 16 * 4 + 2 * 1024 * 4
    assert binding.status_string(5) == "pattern invalid or too small"


def test_misaligned_side_buffers_are_refused_before_any_launch(lib):
    """fp32 side buffers (LSE, tile statistics, scores, workspace) are read with 16-byte loads and the
    CSR arrays as int32: a pointer offset by 4 (or 2) bytes must come back as an alignment error from
    the host-side checks, with nothing launched (there is no GPU here to launch on)."""
    shape = binding.Shape(1, 2, 2, 1024, 128)
    params = sd.make_params(128, 0.25, 0)
    ok, off = 4096, 4096 + 4
    pat = binding.Pattern(ok, ok, 1 << 20, 0, 0, 0, 0, 0)
    byref = ctypes.byref
    assert lib.sparsed_attn_full(byref(shape), ok, ok, ok, ok, off, ok, 256, None) == 3             # lse
    assert lib.sparsed_attn_full(byref(shape), ok, ok, ok, ok, None, off, 256, None) == 3            # ws
    assert lib.sparsed_attn_full_stats(byref(shape), 128, ok, ok, ok, ok, ok, off, ok, 256, None) == 3    # tile stats
    assert lib.sparsed_select_from_stats(byref(shape), byref(params), off, ok, byref(pat), None, ok, 256, None) == 3
    assert lib.sparsed_select_from_stats(byref(shape), byref(params), ok, off, byref(pat), None, ok, 256, None) == 3
    assert lib.sparsed_select_from_stats(byref(shape), byref(params), ok, ok, byref(pat), off, ok, 256, None) == 3
    assert lib.sparsed_select_from_stats(byref(shape), byref(params), ok, ok, byref(pat), None, off, 256, None) == 3
    assert lib.sparsed_select_from_scores(byref(params), off, 1, 2, 8, byref(pat), ok, 256, None) == 3
    assert lib.sparsed_select_from_scores(byref(params), ok, 1, 2, 8, byref(pat), off, 256, None) == 3
    big = 1 << 24
    assert lib.sparsed_select_pattern(byref(shape), byref(params), ok, ok, off, byref(pat), None, ok, big, None) == 3
    assert lib.sparsed_select_pattern(byref(shape), byref(params), ok, ok, None, byref(pat), off, ok, big, None) == 3
    assert lib.sparsed_select_pattern(byref(shape), byref(params), ok, ok, None, byref(pat), None, off, big, None) == 3
    assert lib.sparsed_select_pattern_pooled_qk(byref(shape), byref(params), ok, ok, byref(pat), off, ok, big, None) == 3
    assert lib.sparsed_select_pattern_pooled_qk(byref(shape), byref(params), ok, ok, byref(pat), None, off, big, None) == 3
    bad_pat = binding.Pattern(ok + 2, ok, 1 << 20, 0, 128, 8, 1, 2)
    assert lib.sparsed_attn_sparse(byref(shape), byref(bad_pat), ok, ok, ok, ok, ok, 256, None) == 3
    assert lib.sparsed_select_from_stats(byref(shape), byref(params), ok, ok, byref(bad_pat), None, ok, 256, None) == 3
    assert lib.sparsed_workspace_init(off, 256, None) == 3
    assert lib.sparsed_pattern_validate(byref(binding.Pattern(ok, ok + 2, 16, 16, 128, 8, 1, 2)), ok, 256, None) == 3


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding._build, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library()
