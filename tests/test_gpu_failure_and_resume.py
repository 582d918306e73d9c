"""Failure detection without a GPU fault (a bounded wait that nothing satisfies runs out and is reported
through the status word, after which the context keeps working) and resuming from a saved pattern."""
import pytest
import torch

import paper_2509_24014_b200 as sd
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import gpu_select, gpu_sparse

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_bounded_wait_reports_and_context_stays_usable():
    ws = sd.new_workspace(256, DEV)
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    sd.sparsed_selftest_wait_timeout(ws)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (1, 99)
    st = sd.load_library().sparsed_last_device_status(ws.data_ptr(), None, None, None)
    assert st == 8 and sd.binding.status_string(st) == "device-side wait ran out"
    sd.sparsed_workspace_init(ws)
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    # the context is intact: a real call still works and leaves the status clean
    cfg = syn.AttnConfig("f", 1, 2, 2, 256, 128, 128, 0.5, 0, seed=91)
    q, k, v = syn.make_qkv(cfg, DEV)
    o = torch.empty_like(q)
    sd.sparsed_attn_full(q, k, v, o, None, ws)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0) and torch.isfinite(o.float()).all()


def test_resume_sparse_phase_from_saved_pattern(tmp_path):
    cfg = syn.AttnConfig("r", 1, 4, 2, 1024, 128, 128, 0.3, 512, seed=92)
    q, k, v = syn.make_qkv(cfg, DEV)
    pat, row_ptr, col_idx, _ = gpu_select(q, k, 128, 0.3, 512)
    o1 = gpu_sparse(q, k, v, pat)
    path = str(tmp_path / "pattern.npz")
    sd.save_pattern(path, pat, row_ptr, col_idx, keep_ratio=0.3, prefill_len=512, switch_step=12)
    pat2, rp2, ci2, meta = sd.load_pattern(path, DEV)
    assert meta == {"keep_ratio": 0.3, "prefill_len": 512, "switch_step": 12}
    assert torch.equal(rp2, row_ptr) and torch.equal(ci2, col_idx[: pat.nnz]) and pat2.num_blocks == pat.num_blocks
    assert sd.sparsed_pattern_validate(pat2, sd.new_workspace(256, DEV))
    assert torch.equal(gpu_sparse(q, k, v, pat2), o1)


@pytest.mark.parametrize("bs", [128, 32])
def test_row_pointers_outside_the_column_array_are_not_followed(bs):
    """A corrupt row_ptr (pointing past col_idx, or backwards) must not make the sparse kernel read out
    of bounds: the affected query blocks come back as zeros, the status word reads code 3, every other
    query block is computed as usual, and the context stays usable."""
    cfg = syn.AttnConfig("g", 1, 2, 2, 1024, 128, bs, 0.3, 0, seed=93)
    q, k, v = syn.make_qkv(cfg, DEV)
    pat, row_ptr, col_idx, _ = gpu_select(q, k, bs, 0.3, 0)
    good = gpu_sparse(q, k, v, pat)
    nb = 1024 // bs
    group = 128 // bs                                   # query blocks that share a 128-row tile
    bad_rp = row_ptr.clone()
    victim = 3 * group                                  # first query block of the fourth query tile of head 0
    bad_rp[victim + group] = 10 ** 9                    # its tile's list would end a billion entries in
    bad = sd.pattern_from_csr(bad_rp, col_idx, bs, nb, 1, 2)
    o = torch.full_like(q, float("nan"))
    ws = sd.new_workspace(256, DEV)
    sd.sparsed_attn_sparse(q, k, v, o, bad, ws)
    torch.cuda.synchronize()
    code, where = sd.sparsed_last_device_status(ws)
    assert (code, where) == (3, 2)
    rows = slice(victim * bs, (victim + group) * bs)
    assert torch.all(o[0, 0, rows] == 0)
    keep = torch.ones(1024, dtype=torch.bool, device=DEV)
    keep[rows] = False
    nxt = slice((victim + group) * bs, (victim + 2 * group) * bs)   # the next tile starts at the corrupt entry too
    keep[nxt] = False
    assert torch.equal(o[0, 0, keep], good[0, 0, keep]) and torch.equal(o[0, 1], good[0, 1])
    sd.sparsed_workspace_init(ws)
    assert torch.equal(gpu_sparse(q, k, v, pat), good)
