"""The switch step without a second Q K^T pass: sparsed_attn_full_stats + sparsed_select_from_stats
against the oracle (scores within tolerance, selection logic bit-exact on the scores it produced,
full-attention output unchanged) and against the two-pass sparsed_select_pattern."""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import check_outputs, gpu_full, gpu_select, to_f64
from tests.test_gpu_parity_configs import SCORE_ATOL, SCORE_RTOL, check_row_list

pytestmark = pytest.mark.gpu
DEV = "cuda"


def gpu_switch_step(q, k, v, block_size, keep_ratio, prefill_len):
    B, Hq, L, _ = q.shape
    nb = L // block_size
    o = torch.empty_like(q)
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=q.device)
    stats = sd.new_tile_stats(q, block_size)
    stats.fill_(float("nan"))
    ws = sd.new_workspace(256, q.device)
    sd.sparsed_attn_full_stats(q, k, v, o, lse, stats, ws, block_size)
    params = sd.make_params(block_size, keep_ratio, prefill_len)
    kp, kg = sd.sparsed_kept_per_row(params, L)
    pat, row_ptr, col_idx = sd.new_pattern(B, Hq, nb, kp + kg, q.device)
    scores = torch.full((B, Hq, nb, nb), float("nan"), dtype=torch.float32, device=q.device)
    sd.sparsed_select_from_stats(q, k, params, lse, stats, pat, ws, scores_out=scores)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    return o, lse, pat, row_ptr, col_idx, scores


@pytest.mark.parametrize("name,L,Hq,Hkv,bs,rho,p", [("c1", 1024, 2, 2, 64, 0.3, 0), ("mid", 2048, 4, 2, 128, 0.25, 1024),
                                                    ("odd64", 448, 2, 1, 64, 0.4, 128)])
def test_switch_step_from_stats_matches_oracle(name, L, Hq, Hkv, bs, rho, p):
    cfg = syn.CONFIGS["c1"] if name == "c1" else syn.AttnConfig(name, 1, Hq, Hkv, L, 128, bs, rho, p, seed=31)
    q, k, v = syn.make_qkv(cfg, DEV)
    qd, kd, vd = to_f64(q), to_f64(k), to_f64(v)
    o, lse, pat, row_ptr, col_idx, scores = gpu_switch_step(q, k, v, bs, rho, p)
    o_plain, lse_plain = gpu_full(q, k, v)
    assert torch.equal(o, o_plain) and torch.equal(lse, lse_plain)      # recording statistics changes nothing
    check_outputs(o, orc.attn_full(qd, kd, vd)[0], name)
    a_ref = orc.pooled_scores(qd, kd, bs)
    a_gpu = scores.cpu().numpy()
    np.testing.assert_allclose(a_gpu, a_ref, rtol=SCORE_RTOL, atol=SCORE_ATOL)
    np.testing.assert_allclose(a_gpu.astype(np.float64).sum(-1), 1.0 / bs, rtol=2e-5)
    rp, ci = orc.select_blocks(a_gpu, bs, p, rho)                        # bit-exact on its own scores
    np.testing.assert_array_equal(row_ptr.cpu().numpy(), rp)
    np.testing.assert_array_equal(col_idx.cpu().numpy(), ci)
    nb, pb = L // bs, p // bs
    for h in range(Hq):
        for ib in range(nb):
            r = h * nb + ib
            check_row_list(ci[rp[r]:rp[r + 1]], a_ref[0, h, ib], pb, rho)
    # the two-pass path agrees within the score tolerance
    _, _, _, scores2 = gpu_select(q, k, bs, rho, p, lse=lse)
    np.testing.assert_allclose(a_gpu, scores2.cpu().numpy(), rtol=2 * SCORE_RTOL, atol=2 * SCORE_ATOL)


def test_switch_step_from_stats_config3_sampled():
    cfg = syn.CONFIGS["c3"]
    q, k, v = syn.make_qkv(cfg, DEV)
    bs, nb = cfg.block_size, cfg.num_blocks
    o, lse, pat, row_ptr, col_idx, scores = gpu_switch_step(q, k, v, bs, cfg.keep_ratio, cfg.prefill_len)
    rp, ci = row_ptr.cpu().numpy(), col_idx.cpu().numpy()
    assert pat.nnz == 28 * 128 * 20 and sd.sparsed_pattern_validate(pat, sd.new_workspace(256, DEV))
    group = cfg.heads_q // cfg.heads_kv
    for h in (0, 9, 27):
        qh, kh = to_f64(q[0, h]), to_f64(k[0, h // group])
        for ib in (0, 63, nb - 1):
            a_ref = orc.head_pooled_row(qh, kh, ib, bs)
            a_gpu = scores[0, h, ib].cpu().numpy()
            np.testing.assert_allclose(a_gpu, a_ref, rtol=SCORE_RTOL, atol=SCORE_ATOL)
            r = h * nb + ib
            assert list(ci[rp[r]:rp[r + 1]]) == orc.select_row(a_gpu, 0, cfg.keep_ratio)
            check_row_list(ci[rp[r]:rp[r + 1]], a_ref, 0, cfg.keep_ratio)
