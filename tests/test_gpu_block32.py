"""The paper's short-context setting (block_size 32, keep ratio 50 %): selection and block-sparse
attention against the oracle, including an odd number of kept blocks per row (a half-filled tile)."""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import check_outputs, gpu_full, gpu_select, gpu_sparse, to_f64
from tests.test_gpu_parity_configs import SCORE_ATOL, SCORE_RTOL, check_row_list

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("L,Hq,Hkv,rho,p", [(1024, 2, 2, 0.5, 0), (1024, 4, 2, 0.5, 352), (416, 2, 1, 0.3, 96),
                                            (4096, 2, 2, 0.5, 2048)])
def test_block32_select_and_sparse(L, Hq, Hkv, rho, p):
    bs = 32
    cfg = syn.AttnConfig("s32", 1, Hq, Hkv, L, 128, bs, rho, p, seed=61,
                         fixed_heads=(("band", "64"), ("sink+stripes", "16", "3")) * (Hq // 2))
    q, k, v = syn.make_qkv(cfg, DEV)
    qd, kd, vd = to_f64(q), to_f64(k), to_f64(v)
    o, lse = gpu_full(q, k, v)
    for use_lse in (lse, None):
        pat, row_ptr, col_idx, scores = gpu_select(q, k, bs, rho, p, lse=use_lse)
        a_ref = orc.pooled_scores(qd, kd, bs)
        a_gpu = scores.cpu().numpy()
        np.testing.assert_allclose(a_gpu, a_ref, rtol=SCORE_RTOL, atol=SCORE_ATOL)
        rp, ci = orc.select_blocks(a_gpu, bs, p, rho)
        np.testing.assert_array_equal(row_ptr.cpu().numpy(), rp)
        np.testing.assert_array_equal(col_idx.cpu().numpy(), ci)
    nb, pb = L // bs, p // bs
    for h in range(Hq):
        for ib in range(nb):
            r = h * nb + ib
            check_row_list(ci[rp[r]:rp[r + 1]], a_ref[0, h, ib], pb, rho)
    o_sp = gpu_sparse(q, k, v, pat)
    check_outputs(o_sp, orc.attn_sparse(qd, kd, vd, rp, ci, bs), "block 32 sparse")
    with pytest.raises(sd.SparsedError) as e:   # the statistics path is per 64 keys
        sd.sparsed_select_from_stats(q, k, sd.make_params(bs, rho, p), lse, sd.new_tile_stats(q), pat,
                                     sd.new_workspace(256, DEV))
    assert e.value.status == 2


def test_block32_ragged_user_lists():
    L, bs = 512, 32
    cfg = syn.AttnConfig("u32", 1, 2, 2, L, 128, bs, 0.5, 0, seed=62)
    q, k, v = syn.make_qkv(cfg, DEV)
    nb = L // bs
    lists = [sorted(np.random.default_rng(r).choice(nb, size=(r % 5) + 1, replace=False).tolist()) for r in range(2 * nb)]
    rp = np.cumsum([0] + [len(x) for x in lists]).astype(np.int32)
    ci = np.concatenate(lists).astype(np.int32)
    rp_d, ci_d = torch.from_numpy(rp).to(DEV), torch.from_numpy(ci).to(DEV)
    o = gpu_sparse(q, k, v, sd.pattern_from_csr(rp_d, ci_d, bs, nb, 1, 2))
    check_outputs(o, orc.attn_sparse(to_f64(q), to_f64(k), to_f64(v), rp, ci, bs), "block 32 user lists")
