"""Further GPU-vs-oracle cases: a non-default softmax scale through every entry point, batch > 1 on the
statistics path, logits that keep outgrowing the running maximum inside the sparse kernel, and the batched
long-context settings."""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import check_outputs, to_f64
from tests.test_gpu_parity_configs import SCORE_ATOL, SCORE_RTOL

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_custom_scale_and_batch_two_through_all_entry_points():
    cfg = syn.AttnConfig("s", 2, 4, 2, 768, 128, 128, 0.4, 256, seed=81)
    q, k, v = syn.make_qkv(cfg, DEV)
    scale = 0.11
    scale32 = float(np.float32(scale))
    qd, kd, vd = to_f64(q), to_f64(k), to_f64(v)
    B, Hq, L, _ = q.shape
    nb = L // 128
    ws = sd.new_workspace(1 << 22, DEV)
    o = torch.empty_like(q)
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=DEV)
    stats = sd.new_tile_stats(q, 128)
    sd.sparsed_attn_full_stats(q, k, v, o, lse, stats, ws, 128, softmax_scale=scale)
    o_ref, lse_ref = orc.attn_full(qd, kd, vd, scale=scale32)
    check_outputs(o, o_ref, "scaled full")
    np.testing.assert_allclose(to_f64(lse), lse_ref, atol=3e-5, rtol=3e-6)
    params = sd.make_params(128, 0.4, 256)
    kp, kg = sd.sparsed_kept_per_row(params, L)
    a_ref = orc.pooled_scores(qd, kd, 128, scale=scale32)
    results = []
    for path in ("stats", "two_pass", "two_pass_own_lse"):
        pat, rp_t, ci_t = sd.new_pattern(B, Hq, nb, kp + kg, DEV)
        scores = torch.empty(B, Hq, nb, nb, dtype=torch.float32, device=DEV)
        if path == "stats":
            sd.sparsed_select_from_stats(q, k, params, lse, stats, pat, ws, scores_out=scores)
        else:
            sd.sparsed_select_pattern(q, k, params, pat, ws, lse=lse if path == "two_pass" else None,
                                      scores_out=scores, softmax_scale=scale)
        torch.cuda.synchronize()
        np.testing.assert_allclose(scores.cpu().numpy(), a_ref, rtol=SCORE_RTOL, atol=SCORE_ATOL)
        rp, ci = orc.select_blocks(scores.cpu().numpy(), 128, 256, 0.4)
        np.testing.assert_array_equal(ci_t.cpu().numpy(), ci)
        np.testing.assert_array_equal(rp_t.cpu().numpy(), rp)
        results.append((pat, rp, ci, rp_t, ci_t))
    pat, rp, ci, _, _ = results[0]
    o_sp = torch.empty_like(q)
    sd.sparsed_attn_sparse(q, k, v, o_sp, pat, ws, softmax_scale=scale)
    torch.cuda.synchronize()
    check_outputs(o_sp, orc.attn_sparse(qd, kd, vd, rp, ci, 128, scale=scale32), "scaled sparse")
    assert sd.sparsed_last_device_status(ws) == (0, 0)


@pytest.mark.parametrize("bs", [64, 128])
def test_sparse_kernel_with_growing_maxima(bs):
    # keys sorted so that each query's logits keep rising along its kept list: exercises the rescale path
    cfg = syn.AttnConfig("g", 1, 2, 2, 1024, 128, bs, 1.0, 0, seed=82)
    q, k, v = syn.make_qkv(cfg, DEV)
    q = (q.float() * 30).to(torch.bfloat16)
    order = torch.argsort(k[0, 0].float() @ q[0, 0].float().mean(0))
    k = k[:, :, order].contiguous()
    v = v[:, :, order].contiguous()
    nb = 1024 // bs
    lists = [list(range(r % 3, nb, 2 + r % 2)) for r in range(2 * nb)]
    rp = np.cumsum([0] + [len(x) for x in lists]).astype(np.int32)
    ci = np.concatenate(lists).astype(np.int32)
    rp_d, ci_d = torch.from_numpy(rp).to(DEV), torch.from_numpy(ci).to(DEV)
    o = torch.empty_like(q)
    ws = sd.new_workspace(256, DEV)
    sd.sparsed_attn_sparse(q, k, v, o, sd.pattern_from_csr(rp_d, ci_d, bs, nb, 1, 2), ws)
    torch.cuda.synchronize()
    ref = orc.attn_sparse(to_f64(q), to_f64(k), to_f64(v), rp, ci, bs)
    d = np.abs(to_f64(o) - ref)
    assert d.max() <= 2e-2 * max(1.0, np.abs(ref).max()) and d.mean() <= 2e-3
    assert np.linalg.norm(d) / np.linalg.norm(ref) <= 1e-2
    assert sd.sparsed_last_device_status(ws) == (0, 0)


@pytest.mark.parametrize("batch,seq_len,gen_len", [(16, 4096, 128), (8, 8192, 128)])
def test_batched_long_context_settings(batch, seq_len, gen_len):
    """The batched long-context evaluation settings (Table 3: batch 16 at 4k and batch 8 at 8k, block 128,
    rho = 0.3): the switch step's fused path on the whole batch, the oracle on rows sampled over every
    batch index."""
    bs, rho = 128, 0.3
    prefill = seq_len - gen_len
    cfg = syn.AttnConfig("batched", batch, 8, 4, seq_len, 128, bs, rho, prefill, seed=300 + batch)
    q, k, v = syn.make_qkv(cfg, DEV)
    B, Hq, L, _ = q.shape
    nb, pb, group = L // bs, prefill // bs, 2
    ws = sd.new_workspace(1 << 22, DEV)
    o = torch.empty_like(q)
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=DEV)
    stats = sd.new_tile_stats(q, bs)
    sd.sparsed_attn_full_stats(q, k, v, o, lse, stats, ws, bs)
    params = sd.make_params(bs, rho, prefill)
    kp, kg = sd.sparsed_kept_per_row(params, L)
    assert (kp, kg) == (orc.kept_per_region(pb, rho), orc.kept_per_region(nb - pb, rho))
    pat, rp_t, ci_t = sd.new_pattern(B, Hq, nb, kp + kg, DEV)
    scores = torch.empty(B, Hq, nb, nb, dtype=torch.float32, device=DEV)
    sd.sparsed_select_from_stats(q, k, params, lse, stats, pat, ws, scores_out=scores)
    o_sp = torch.empty_like(q)
    sd.sparsed_attn_sparse(q, k, v, o_sp, pat, ws)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    assert pat.nnz == B * Hq * nb * (kp + kg)
    rp, ci = rp_t.cpu().numpy(), ci_t.cpu().numpy()
    # the selection is bit-exact on the GPU's own scores for every row of every batch element
    rp_ref, ci_ref = orc.select_blocks(scores.cpu().numpy(), bs, prefill, rho)
    np.testing.assert_array_equal(rp, rp_ref)
    np.testing.assert_array_equal(ci, ci_ref)
    rng = np.random.default_rng(batch)
    for b in range(B):
        h = int(rng.integers(Hq))
        ib = int(rng.choice([0, pb - 1, pb, nb - 1, int(rng.integers(nb))]))
        qh, kh, vh = to_f64(q[b, h]), to_f64(k[b, h // group]), to_f64(v[b, h // group])
        rows = slice(ib * bs, (ib + 1) * bs)
        o_ref, lse_ref = orc.head_full_rows(qh, kh, vh, rows)
        check_outputs(o[b, h, rows], o_ref, f"batched full b{b} h{h} ib{ib}")
        np.testing.assert_allclose(to_f64(lse[b, h, rows]), lse_ref, atol=3e-5, rtol=3e-6)
        np.testing.assert_allclose(scores[b, h, ib].cpu().numpy(), orc.head_pooled_row(qh, kh, ib, bs),
                                   rtol=SCORE_RTOL, atol=SCORE_ATOL)
        r = (b * Hq + h) * nb + ib
        kept = ci[rp[r]:rp[r + 1]]
        check_outputs(o_sp[b, h, rows], orc.head_sparse_rows(qh, kh, vh, ib, kept, bs),
                      f"batched sparse b{b} h{h} ib{ib}")


def test_token_major_layout_through_every_entry_point():
    """Q, K, V and O as [batch, token, head, dim] (what a fused QKV projection writes), passed by strides:
    full + statistics, both selections, the block-mean estimate and sparse attention."""
    B, L, Hq, Hkv, bs, rho, prefill = 2, 640, 4, 2, 64, 0.3, 128
    cfg = syn.AttnConfig("tm", B, Hq, Hkv, L, 128, bs, rho, prefill, seed=123)
    qc, kc, vc = syn.make_qkv(cfg, DEV)
    q = qc.transpose(1, 2).contiguous().transpose(1, 2)     # same values, token-major memory
    k = kc.transpose(1, 2).contiguous().transpose(1, 2)
    v = vc.transpose(1, 2).contiguous().transpose(1, 2)
    assert not q.is_contiguous() and q.stride(2) == Hq * 128
    o = torch.empty(B, L, Hq, 128, dtype=torch.bfloat16, device=DEV).transpose(1, 2)
    nb = L // bs
    ws = sd.new_workspace(1 << 22, DEV)
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=DEV)
    stats = sd.new_tile_stats(q, bs)
    sd.sparsed_attn_full_stats(q, k, v, o, lse, stats, ws, bs)
    qd, kd, vd = to_f64(q), to_f64(k), to_f64(v)
    o_ref, lse_ref = orc.attn_full(qd, kd, vd)
    check_outputs(o, o_ref, "token-major full")
    np.testing.assert_allclose(to_f64(lse), lse_ref, atol=3e-5, rtol=3e-6)
    params = sd.make_params(bs, rho, prefill)
    kp, kg = sd.sparsed_kept_per_row(params, L)
    a_ref = orc.pooled_scores(qd, kd, bs)
    lists = []
    for path in ("stats", "two_pass"):
        pat, rp_t, ci_t = sd.new_pattern(B, Hq, nb, kp + kg, DEV)
        scores = torch.empty(B, Hq, nb, nb, dtype=torch.float32, device=DEV)
        if path == "stats":
            sd.sparsed_select_from_stats(q, k, params, lse, stats, pat, ws, scores_out=scores)
        else:
            sd.sparsed_select_pattern(q, k, params, pat, ws, scores_out=scores)
        torch.cuda.synchronize()
        np.testing.assert_allclose(scores.cpu().numpy(), a_ref, rtol=SCORE_RTOL, atol=SCORE_ATOL)
        rp, ci = orc.select_blocks(scores.cpu().numpy(), bs, prefill, rho)
        np.testing.assert_array_equal(ci_t.cpu().numpy(), ci)
        lists.append((pat, rp, ci, rp_t, ci_t))
    pat_e, rp_e, ci_e = sd.new_pattern(B, Hq, nb, kp + kg, DEV)
    est = torch.empty(B, Hq, nb, nb, dtype=torch.float32, device=DEV)
    ws_e = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_SELECT_POOLED_QK, sd.make_shape(q, k), params), DEV)
    sd.sparsed_select_pattern_pooled_qk(q, k, params, pat_e, ws_e, scores_out=est)
    torch.cuda.synchronize()
    np.testing.assert_allclose(est.cpu().numpy(), orc.pooled_qk_scores(qd, kd, bs), rtol=5e-5, atol=1e-12)
    pat, rp, ci, _, _ = lists[0]
    o_sp = torch.empty(B, L, Hq, 128, dtype=torch.bfloat16, device=DEV).transpose(1, 2)
    sd.sparsed_attn_sparse(q, k, v, o_sp, pat, ws)
    torch.cuda.synchronize()
    check_outputs(o_sp, orc.attn_sparse(qd, kd, vd, rp, ci, bs), "token-major sparse")
    assert sd.sparsed_last_device_status(ws) == (0, 0)


def test_ctas_that_run_through_several_query_tiles_match_one_tile_per_cta():
    """Block-sparse launches with more query tiles than CTAs fit on the device let every CTA roll on into
    further tiles (ring slots, S buffers and barrier phases carry over). 768 query tiles with ragged
    user-built lists, single empty ones and runs of them among them, must give bitwise what the same heads give when launched one
    head at a time (64 tiles each: one tile per CTA), and agree with the oracle on sampled rows."""
    B, Hq, Hkv, L, bs = 1, 12, 4, 8192, 128
    cfg = syn.AttnConfig("roll", B, Hq, Hkv, L, 128, bs, 0.1, 0, seed=404, plant_norm=6.0)
    q, k, v = syn.make_qkv(cfg, DEV)
    nb = L // bs
    rng = np.random.default_rng(404)
    lists = []
    for r in range(Hq * nb):
        # every fifth list is empty, and so is a run of six neighbouring ones in every head
        n = int(rng.integers(0, 7)) if (r % 5 and not 40 <= r % 64 < 46) else 0
        lists.append(sorted(rng.choice(nb, size=n, replace=False).tolist()))
    rp = np.cumsum([0] + [len(x) for x in lists]).astype(np.int32)
    ci = np.concatenate([np.asarray(x, dtype=np.int32) for x in lists] + [np.zeros(1, np.int32)]).astype(np.int32)
    rp_d, ci_d = torch.from_numpy(rp).to(DEV), torch.from_numpy(ci).to(DEV)
    ws = sd.new_workspace(256, DEV)
    o_all = torch.full_like(q, float("nan"))
    sd.sparsed_attn_sparse(q, k, v, o_all, sd.pattern_from_csr(rp_d, ci_d, bs, nb, B, Hq), ws)
    o_one = torch.full_like(q, float("nan"))
    group = Hq // Hkv
    for h in range(Hq):
        rp_h = (rp_d[h * nb:(h + 1) * nb + 1]).contiguous()   # absolute offsets into the shared col_idx
        pat_h = sd.pattern_from_csr(rp_h, ci_d, bs, nb, 1, 1)
        sd.sparsed_attn_sparse(q[:, h:h + 1], k[:, h // group:h // group + 1], v[:, h // group:h // group + 1],
                               o_one[:, h:h + 1], pat_h, ws)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    assert torch.equal(o_all, o_one)
    for h, ib in ((0, 0), (3, 17), (7, 63), (11, 40), (5, 5), (2, 43), (9, 46)):
        r = h * nb + ib
        rows = slice(ib * bs, (ib + 1) * bs)
        if not lists[r]:
            assert torch.all(o_all[0, h, rows] == 0)
        else:
            ref = orc.head_sparse_rows(to_f64(q[0, h]), to_f64(k[0, h // group]), to_f64(v[0, h // group]), ib,
                                       lists[r], bs)
            check_outputs(o_all[0, h, rows], ref, f"rolled-on tile h{h} ib{ib}")
