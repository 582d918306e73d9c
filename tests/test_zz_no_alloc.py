"""The allocation-free selection entry point (sparsed_select_pattern_static).

Some hosts of this library cannot call cudaMalloc when they need a pattern: a serving process
that handed all device memory to its own pool at start-up, or a request path where allocation
is banned because it stalls the device. For them the library carries a fixed scratch array of
its own. This test calls that entry point through the C ABI several times in a row, with different
shapes, with and without a caller-supplied LSE, and once with 32-token blocks (the case in which
the pooled scores and the LSE rows really live in the library's array and are read back from it),
and checks each result against the regular entry point (same kernels, so the block lists must be
identical) and against the CPU oracle's selection, and that oversized requests are refused.
Collected last on purpose: a failure here must not hide any other test.
"""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn
from paper_2509_24014_b200.binding import STATIC_SCRATCH_BYTES
from tests.parity_util import to_f64
from tests.test_gpu_parity_configs import check_row_list

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _regular(q, k, params, kept, lse):
    B, Hq, L, _ = q.shape
    nb = L // params.block_size
    pat, row_ptr, col_idx = sd.new_pattern(B, Hq, nb, kept, DEV)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_SELECT_PATTERN, sd.make_shape(q, k), params), DEV)
    sd.sparsed_select_pattern(q, k, params, pat, ws, lse=lse)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    return pat, row_ptr, col_idx


def _static(q, k, params, kept, lse):
    B, Hq, L, _ = q.shape
    nb = L // params.block_size
    pat, row_ptr, col_idx = sd.new_pattern(B, Hq, nb, kept, DEV)
    row_ptr.fill_(-1)
    col_idx.fill_(-1)
    sd.sparsed_select_pattern_static(q, k, params, pat, lse=lse)
    torch.cuda.synchronize()
    return pat, row_ptr, col_idx


def test_static_scratch_selection_matches_regular_entry_point_twice():
    calls = [
        # (config, use the LSE of a full-attention pass?)
        (syn.AttnConfig("a", 1, 4, 2, 2048, 128, 128, 0.25, 1024, seed=21), False),
        (syn.AttnConfig("b", 1, 2, 2, 1024, 128, 64, 0.3, 0, seed=22), True),
        # 32-token blocks are never ranked inside the scoring kernel: A' and the LSE rows go through the
        # static array (over what the two calls above left there) and the ranking kernel reads A' back
        (syn.AttnConfig("c", 1, 2, 2, 1024, 128, 32, 0.5, 512, seed=23), False),
        (syn.AttnConfig("a", 1, 4, 2, 2048, 128, 128, 0.25, 1024, seed=21), False),
    ]
    for cfg, with_lse in calls:
        q, k, v = syn.make_qkv(cfg, DEV)
        params = sd.make_params(cfg.block_size, cfg.keep_ratio, cfg.prefill_len)
        kept = sum(sd.sparsed_kept_per_row(params, cfg.seq_len))
        lse = None
        if with_lse:
            o = torch.empty_like(q)
            lse = torch.empty(q.shape[:3], dtype=torch.float32, device=DEV)
            ws = sd.new_workspace(256, DEV)
            sd.sparsed_attn_full(q, k, v, o, lse, ws)
        pat_r, rp_r, ci_r = _regular(q, k, params, kept, lse)
        pat_s, rp_s, ci_s = _static(q, k, params, kept, lse)
        assert pat_s.nnz == pat_r.nnz and pat_s.num_blocks == pat_r.num_blocks
        assert torch.equal(rp_s, rp_r)
        assert torch.equal(ci_s, ci_r)
        ws = sd.new_workspace(256, DEV)
        assert sd.sparsed_pattern_validate(pat_s, ws)
        # and against the oracle's own fp64 scores and ranking: list lengths and order exact, every block
        # clearly above / below the boundary in / out, rows with a clear boundary identical
        a_ref = orc.pooled_scores(to_f64(q), to_f64(k), cfg.block_size)
        rp, ci = rp_s.cpu().numpy(), ci_s.cpu().numpy()
        nb, pb = cfg.num_blocks, cfg.prefill_len // cfg.block_size
        n_exact = 0
        for h in range(cfg.heads_q):
            for ib in range(nb):
                r = h * nb + ib
                n_exact += check_row_list(ci[rp[r]:rp[r + 1]], a_ref[0, h, ib], pb, cfg.keep_ratio)
        assert n_exact > 0     # rows whose boundary gap is wider than the score tolerance matched exactly


def test_static_scratch_rejects_requests_beyond_its_size():
    # 32 heads x 16384 tokens: scores (2 MiB) + LSE rows (2 MiB) fit; 32 heads x 65536 do not.
    big = syn.AttnConfig("big", 1, 32, 32, 65536, 128, 128, 0.1, 0)
    params = sd.make_params(big.block_size, big.keep_ratio, 0)
    shape = sd.Shape(1, 32, 32, big.seq_len, 128)
    assert sd.sparsed_workspace_bytes(sd.OP_SELECT_PATTERN, shape, params) > STATIC_SCRATCH_BYTES
    q = torch.zeros(16, dtype=torch.bfloat16, device=DEV)  # never read: the size check comes first
    pat, _, _ = sd.new_pattern(1, 1, 1, 1, DEV)
    with pytest.raises(sd.SparsedError) as e:
        sd.load_library()  # make sure the error below is the library's, not a missing build
        st = sd.binding.load_library().sparsed_select_pattern_static(
            shape, params, q.data_ptr(), q.data_ptr(), None, pat, None)
        if st != 0:
            raise sd.SparsedError(st, "sparsed_select_pattern_static")
    assert e.value.status == 4
