"""Sliding-window and sink+window comparison patterns (the paper's baselines, in block form) built
on the device, checked against a direct construction, and run through the block-sparse kernel."""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import check_outputs, gpu_sparse, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda"


def direct_window_lists(nb, sink, window):
    half = (window - 1) // 2
    return [sorted(set(range(min(sink, nb))) | set(range(max(0, i - half), min(nb - 1, i + half) + 1)))
            for i in range(nb)]


@pytest.mark.parametrize("nb,sink,window,bs", [(16, 0, 5, 64), (16, 2, 3, 128), (300, 30, 151, 128), (5, 9, 1, 64),
                                               (64, 6, 33, 128)])
def test_window_pattern_matches_direct_construction(nb, sink, window, bs):
    B, H = 2, 3
    pat, row_ptr, col_idx = sd.sparsed_build_window_pattern(B, H, nb, bs, sink, window, DEV)
    torch.cuda.synchronize()
    lists = direct_window_lists(nb, sink, window)
    rp = np.cumsum([0] + [len(x) for x in lists] * (B * H)).astype(np.int32)
    ci = np.concatenate(lists * (B * H)).astype(np.int32)
    assert pat.nnz == len(ci) and pat.num_blocks == nb and pat.batch == B and pat.heads_q == H
    np.testing.assert_array_equal(row_ptr.cpu().numpy(), rp)
    np.testing.assert_array_equal(col_idx.cpu().numpy()[: len(ci)], ci)
    assert sd.sparsed_pattern_validate(pat, sd.new_workspace(256, DEV))


def test_streaming_pattern_through_sparse_kernel():
    cfg = syn.AttnConfig("w", 1, 4, 2, 2048, 128, 128, 0.3, 0, seed=41)
    q, k, v = syn.make_qkv(cfg, DEV)
    nb = cfg.num_blocks
    pat, row_ptr, col_idx = sd.sparsed_build_window_pattern(1, 4, nb, 128, 2, 9, DEV)   # 10 % sink, window l/2
    o = gpu_sparse(q, k, v, pat)
    ref = orc.attn_sparse(to_f64(q), to_f64(k), to_f64(v), row_ptr.cpu().numpy(), col_idx.cpu().numpy(), 128)
    check_outputs(o, ref, "sink+window")


def test_sparse_kernel_empty_rows_give_zeros():
    cfg = syn.AttnConfig("e", 1, 2, 2, 512, 128, 128, 0.5, 0, seed=42)
    q, k, v = syn.make_qkv(cfg, DEV)
    lists = [[0, 2], [], [1], [], [3], [0, 1, 2, 3], [], [2]]
    rp = torch.tensor(np.cumsum([0] + [len(x) for x in lists]), dtype=torch.int32, device=DEV)
    ci = torch.tensor([j for x in lists for j in x], dtype=torch.int32, device=DEV)
    pat = sd.pattern_from_csr(rp, ci, 128, 4, 1, 2)
    assert not sd.sparsed_pattern_validate(pat, sd.new_workspace(256, DEV))   # the validator flags empty rows
    o = gpu_sparse(q, k, v, pat)
    qd, kd, vd = to_f64(q), to_f64(k), to_f64(v)
    for r, kept in enumerate(lists):
        h, ib = divmod(r, 4)
        got = to_f64(o[0, h, ib * 128:(ib + 1) * 128])
        if kept:
            ref = orc.head_sparse_rows(qd[0, h], kd[0, h], vd[0, h], ib, kept, 128)
            assert np.abs(got - ref).max() <= 2e-2
        else:
            assert np.all(got == 0.0)
