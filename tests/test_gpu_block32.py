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
    # the switch step's own statistics (one per 32 keys here) give the same pattern without a second pass
    from tests.test_gpu_parity_configs import gpu_switch_step_from_stats
    o2, lse2, pat2, rp2, ci2, scores2 = gpu_switch_step_from_stats(q, k, v, bs, rho, p)
    assert torch.equal(o2, o) and torch.equal(lse2, lse)
    a2 = scores2.cpu().numpy()
    np.testing.assert_allclose(a2, a_ref, rtol=SCORE_RTOL, atol=SCORE_ATOL)
    np.testing.assert_allclose(a2.astype(np.float64).sum(-1), 1.0 / bs, rtol=2e-5)
    rp_o, ci_o = orc.select_blocks(a2, bs, p, rho)
    np.testing.assert_array_equal(rp2.cpu().numpy(), rp_o)
    np.testing.assert_array_equal(ci2.cpu().numpy(), ci_o)
    for h in range(Hq):
        for ib in range(nb):
            r = h * nb + ib
            check_row_list(ci_o[rp_o[r]:rp_o[r + 1]], a_ref[0, h, ib], pb, rho)


@pytest.mark.parametrize("bs,L,Hq,Hkv", [(32, 544, 2, 1), (64, 576, 3, 3), (32, 4096, 2, 2), (64, 2048, 4, 2)])
def test_small_blocks_share_a_query_tile_with_lists_of_their_own(bs, L, Hq, Hkv):
    """Four (two) neighbouring 32-key (64-key) query blocks share one 128-row tile and walk the union of
    their lists: lists that overlap fully, partly and not at all, empty lists next to full ones, a last
    tile with fewer query blocks than a full one, two batch entries."""
    B = 2
    cfg = syn.AttnConfig("pack", B, Hq, Hkv, L, 128, bs, 0.5, 0, seed=63 + bs, plant_norm=5.0)
    q, k, v = syn.make_qkv(cfg, DEV)
    nb = L // bs
    rng = np.random.default_rng(bs)
    lists = []
    for r in range(B * Hq * nb):
        kind = r % 7
        if kind == 0:
            lst = []                                         # empty row: zeros
        elif kind == 1:
            lst = list(range(nb))                            # everything
        elif kind == 2:
            lst = [int(rng.integers(0, nb))]                 # a single block
        elif kind == 3:
            lst = sorted(rng.choice(nb, size=min(nb, 5), replace=False).tolist())
        elif kind == 4:
            lst = list(range(0, nb, 2))                      # even blocks: disjoint from the next kind
        elif kind == 5:
            lst = list(range(1, nb, 2))
        else:
            lst = sorted(rng.choice(nb, size=max(1, nb // 3), replace=False).tolist())
        lists.append(lst)
    rp = np.cumsum([0] + [len(x) for x in lists]).astype(np.int32)
    ci = np.concatenate([np.asarray(x, dtype=np.int32) for x in lists]).astype(np.int32)
    rp_d, ci_d = torch.from_numpy(rp).to(DEV), torch.from_numpy(ci).to(DEV)
    o = gpu_sparse(q, k, v, sd.pattern_from_csr(rp_d, ci_d, bs, nb, B, Hq))
    with np.errstate(invalid="ignore"):                     # the oracle divides 0 by 0 on an empty row
        ref = orc.attn_sparse(to_f64(q), to_f64(k), to_f64(v), rp, ci, bs)
    got = to_f64(o)
    for r, lst in enumerate(lists):
        b, rem = divmod(r, Hq * nb)
        h, ib = divmod(rem, nb)
        rows = slice(ib * bs, (ib + 1) * bs)
        if not lst:
            assert np.all(got[b, h, rows] == 0.0), f"empty row {r} must give zeros"
            ref[b, h, rows] = 0.0
    check_outputs(o, ref, f"packed block {bs}")


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
