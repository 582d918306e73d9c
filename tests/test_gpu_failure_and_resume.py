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
